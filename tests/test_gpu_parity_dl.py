"""GPU parity of gf_c2_decay_logit (d_t = lora_omega(ddlerp_d(x_t, x_{t-1})), the producer of the WKV calls' decay
logit) against the fp64 oracle, element by element.

Tolerance (bf16 operands and output, fp32 accumulation): d is rounded once to bf16 (half a unit in the last place:
2^-9 |d| relative) on top of the rounding of z, h1, m and h2 to bf16 and the hardware tanh, which reach d through
the two low-rank products as an absolute error of a few 1e-3 of the loras' scale (about one).  An element passes within
2^-8 |d_ref| + 0.02; the tensor within a relative L2 of 5e-3, the bf16 tolerance of the prefill tests."""
import numpy as np
import pytest
import torch

import paper_2407_12077_b200 as gf
from oracle import wkv6_oracle as orc
from paper_2407_12077_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _run(B, T, D, Rd, Rw, seed, with_prev=True):
    x, xp = synth.make_block_input(B, T, D, seed=seed, with_prev=with_prev)
    w = synth.make_decay_lora(D, Rd, Rw, seed=seed + 1)
    dev = lambda t: None if t is None else t.to(DEV)
    d = gf.decay_logit(dev(x), dev(w["mu_x"]), dev(w["A_d"]), dev(w["B_d"]), dev(w["lambda_d"]), dev(w["A_w"]),
                       dev(w["B_w"]), dev(w["lambda_w"]), x_prev=dev(xp))
    gf.last_device_status()
    ref = orc.decay_logit(x, w["mu_x"], w["A_d"], w["B_d"], w["lambda_d"], w["A_w"], w["B_w"], w["lambda_w"], xp)
    got = d.float().cpu().numpy()
    assert np.isfinite(got).all()
    err = np.abs(got - ref)
    bound = 2.0 ** -8 * np.abs(ref) + 0.02
    worst = float((err / bound).max())
    assert worst <= 1.0, (worst, np.unravel_index((err / bound).argmax(), err.shape), (B, T, D, Rd, Rw))
    rel = orc.rel_l2(got, ref)
    assert rel <= 5e-3, rel
    # per token as well: a wrong row (token shift, tile edge) must not hide in the tensor's norm
    tok = np.sqrt((err ** 2).sum(-1) / (ref ** 2).sum(-1)).max()
    assert tok <= 1e-2, tok
    return worst, rel, float(tok)


@pytest.mark.parametrize("B,T,D,Rd,Rw", [
    (1, 128, 64, 16, 16), (2, 200, 128, 32, 64), (3, 129, 768, 32, 64), (1, 1, 256, 32, 64), (5, 37, 2048, 32, 64),
    (2, 127, 320, 48, 32), (1, 1000, 2048, 32, 64)])
def test_shapes_tails_and_ranks(B, T, D, Rd, Rw):
    """Token counts around the 128-row tile, sequences that start inside a tile (T not a multiple of 128), odd
    slice counts (D = 320), every supported rank, the paper's two widths (768, 2048)."""
    print(_run(B, T, D, Rd, Rw, seed=100 + T + D))


def test_without_x_prev_and_many_tiles_per_cta():
    print(_run(2, 12000, 256, 32, 64, seed=7, with_prev=False))      # 188 tiles over the persistent CTAs


def test_feeds_the_prefill_with_a_decay_in_range():
    """The logit is what the WKV calls take as x: chain the two and compare with the oracle's chain."""
    B, T, H = 2, 300, 4
    D = 64 * H
    x, xp = synth.make_block_input(B, T, D, seed=21)
    w = synth.make_decay_lora(D, 32, 64, seed=22)
    inp = synth.make_dense(B, T, H, 64, "bf16", seed=23, state_std=0.1)
    dev = lambda t: t.to(DEV)
    d = gf.decay_logit(dev(x), dev(w["mu_x"]), dev(w["A_d"]), dev(w["B_d"]), dev(w["lambda_d"]), dev(w["A_w"]),
                       dev(w["B_w"]), dev(w["lambda_w"]), x_prev=dev(xp))
    y, s = gf.prefill(dev(inp.r), dev(inp.k), dev(inp.v), d.view(B, T, H, 64), dev(inp.u), dev(inp.state_in))
    gf.last_device_status()
    # the oracle's WKV on the GPU's own (bf16) logit isolates the WKV step; its own logit checks the chain
    y_ref, s_ref = orc.prefill(inp.r, inp.k, inp.v, d.view(B, T, H, 64).cpu(), inp.u, inp.state_in)
    assert orc.rel_l2(y.float().cpu().numpy(), y_ref) <= 5e-3 and orc.rel_l2(s.cpu().numpy(), s_ref) <= 5e-3
    d_ref = orc.decay_logit(x, w["mu_x"], w["A_d"], w["B_d"], w["lambda_d"], w["A_w"], w["B_w"], w["lambda_w"], xp)
    dec = np.exp(-np.exp(d_ref))
    assert dec.min() > 0.0 and dec.max() < 1.0


def test_argument_checks_before_any_launch():
    lib = gf.load_library()
    t = torch.zeros(64 * 64, dtype=torch.bfloat16, device=DEV)
    f = torch.zeros(64, device=DEV)
    p = lambda a: a.data_ptr()
    base = [p(t), None, p(f), p(t), p(t), p(f), p(t), p(t), p(f), p(torch.empty_like(t))]
    before = gf.launch_count()
    assert lib.gf_c2_decay_logit(*base, 1, 64, 64, 32, 64, None) == 0
    assert gf.launch_count() == before + 1
    assert lib.gf_c2_decay_logit(*base, 1, 64, 96, 32, 64, None) == 2          # D not a multiple of 64
    assert lib.gf_c2_decay_logit(*base, 1, 64, 64, 24, 64, None) == 2          # rank not a multiple of 16
    assert lib.gf_c2_decay_logit(*base, 1, 64, 64, 32, 128, None) == 2         # rank above 64
    bad = list(base); bad[9] = bad[0]
    assert lib.gf_c2_decay_logit(*bad, 1, 64, 64, 32, 64, None) == 1           # d aliases x
    bad = list(base); bad[2] = None
    assert lib.gf_c2_decay_logit(*bad, 1, 64, 64, 32, 64, None) == 1
    assert lib.gf_c2_decay_logit(*base, 0, 64, 64, 32, 64, None) == 0          # empty: no-op
    assert gf.launch_count() == before + 1
    gf.last_device_status()


def test_benchmark_size_on_sampled_windows():
    """The launch the benchmark's decay-logit row times (4 x 16384 tokens x 2048 channels: 512 tiles, three or four per
    persistent CTA), checked against the oracle on windows of 256 rows spread over the tensor (first and last tiles,
    sequence starts, tile edges): a window is a sequence of its own whose row above is the tensor's."""
    B, T, D = 4, 16384, 2048
    x, xp = synth.make_block_input(B, T, D, seed=77)
    w = synth.make_decay_lora(D, 32, 64, seed=78)
    dev = lambda t: t.to(DEV)
    d = gf.decay_logit(dev(x), dev(w["mu_x"]), dev(w["A_d"]), dev(w["B_d"]), dev(w["lambda_d"]), dev(w["A_w"]),
                       dev(w["B_w"]), dev(w["lambda_w"]), x_prev=dev(xp))
    gf.last_device_status()
    got = d.float().cpu().numpy().reshape(B * T, D)
    assert np.isfinite(got).all()
    flat = x.reshape(B * T, D)
    rng = np.random.default_rng(79)
    starts = [0, T - 256, T, 2 * T - 100, B * T - 256, 128 * 147, 128 * 148 - 64, 128 * 296 + 5]
    starts += [int(s) for s in rng.integers(0, B * T - 256, size=8)]
    worst = 0.0
    for s0 in starts:
        rows = flat[s0:s0 + 256]
        # the row above the window: the tensor's previous row, or x_prev where a sequence starts there; a sequence
        # start inside the window splits it
        cuts = [s0] + [t for t in range(s0 + 1, s0 + 256) if t % T == 0] + [s0 + 256]
        for a, b in zip(cuts[:-1], cuts[1:]):
            above = xp[a // T] if a % T == 0 else flat[a - 1]
            ref = orc.decay_logit(flat[a:b][None], w["mu_x"], w["A_d"], w["B_d"], w["lambda_d"], w["A_w"], w["B_w"],
                                  w["lambda_w"], above[None])[0]
            err = np.abs(got[a:b] - ref)
            bound = 2.0 ** -8 * np.abs(ref) + 0.02
            worst = max(worst, float((err / bound).max()))
            assert (err <= bound).all(), (s0, a, float((err / bound).max()))
            assert orc.rel_l2(got[a:b], ref) <= 5e-3, (s0, a)
    print("worst element / bound", worst)
