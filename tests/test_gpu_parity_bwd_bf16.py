"""GPU parity of gf_wkv6_backward (bf16 tensors, chunked on the tensor cores) against the fp64 oracle's reverse
recurrence.  Every gradient tensor is held to the relative L2 the forward contract gives bf16 tensors (5e-3): over
the whole tensor, for every (b, h) unit on its own and, for the four per-token gradients, with a per-token bound (the
worst row error over the unit's r.m.s. row norm <= 4e-2), since a norm over thousands of tokens cannot see one bad row.
The decay-logit gradient alone gets 8e-3: it is the one result formed as a difference of suffix sums whose terms each
carry three operand roundings (the score adjoint, the scaled receptance and the scaled key), and with fast decays
only the few terms next to the token survive the difference (measured: 3.0e-3 to 5.1e-3)."""
import numpy as np
import pytest
import torch

import paper_2407_12077_b200 as gf
from oracle import wkv6_oracle as orc
from paper_2407_12077_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = 5e-3
TOL_DX = 8e-3
TOK_TOL = 4e-2
NAMES = ("dr", "dk", "dv", "dx", "du", "dstate_in")


def _inputs(B, T, H, seed, state_std, with_dstate, x_lo=-6.0, x_hi=-1.0):
    inp = synth.make_dense(B, T, H, 64, "bf16", seed=seed, state_std=state_std, x_lo=x_lo, x_hi=x_hi)
    g = torch.Generator().manual_seed(seed + 1)
    dy = torch.randn(inp.r.shape, generator=g).bfloat16()
    dsT = torch.randn((B, H, 64, 64), generator=g) * 0.1 if with_dstate else None
    return inp, dy, dsT


def _check(out, ref, what, tol=TOL, tok_tol=TOK_TOL):
    worst = {}
    for name, a, b in zip(NAMES, out, ref):
        a = a.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(a).all(), (what, name)
        worst[name] = orc.rel_l2(a, b)
        lim = max(tol, TOL_DX) if name == "dx" else tol
        assert worst[name] <= lim, (what, name, worst[name])
        if a.ndim == 4 and name != "dstate_in" and a.shape[1] >= 64:
            # [B,T,H,N]: per unit and per token (a unit of a few tokens is a handful of rounded scalars: its norm
            # ratio is heavy-tailed and is only held to the bound as part of the whole tensor)
            T = a.shape[1]
            row = ((a - b) ** 2).sum(axis=3)
            num, den = row.sum(axis=1), (b * b).sum(axis=(1, 3))
            live = den > 0
            if live.any():
                assert np.sqrt(num[live] / den[live]).max() <= lim, (what, name, "unit")
                tok = np.sqrt(row.max(axis=1)[live] / (den[live] / T))
                worst[name + "_tok"] = float(tok.max())
                assert tok.max() <= tok_tol, (what, name, "token", float(tok.max()))
        elif name == "dstate_in":
            num, den = ((a - b) ** 2).sum(axis=(2, 3)), (b * b).sum(axis=(2, 3))
            live = den > 0
            if live.any():
                assert np.sqrt(num[live] / den[live]).max() <= tol, (what, name, "unit")
    return worst


def _run(B, T, H, seed, state_std, with_dstate, x_lo=-6.0, x_hi=-1.0, tol=TOL):
    inp, dy, dsT = _inputs(B, T, H, seed, state_std, with_dstate, x_lo, x_hi)
    d = inp.to(DEV)
    out = gf.backward(d.r, d.k, d.v, d.x, d.u, dy.to(DEV), d.state_in, None if dsT is None else dsT.to(DEV))
    gf.last_device_status()
    ref = orc.backward(inp.r, inp.k, inp.v, inp.x, inp.u, dy.double().numpy(), inp.state_in,
                       None if dsT is None else dsT.double().numpy())
    return _check(out, ref, (B, T, H, x_lo, x_hi), tol)


@pytest.mark.parametrize("T", [1, 2, 63, 64, 65, 127, 128, 200, 321, 1000])
@pytest.mark.parametrize("with_dstate", [False, True])
def test_ragged_lengths_with_states(T, with_dstate):
    _run(2, T, 3, seed=600 + T, state_std=0.1, with_dstate=with_dstate)


def test_no_start_state_no_final_adjoint():
    _run(1, 256, 4, seed=650, state_std=0.0, with_dstate=False)


def test_cfg1_shape_every_unit():
    c = synth.CONFIGS["cfg1"]
    print(_run(c["B"], c["T"], c["H"], seed=1000, state_std=c["state_std"], with_dstate=True))


def test_cfg2_shape_every_unit_at_the_benchmarked_size():
    """The launch the benchmark's gradient row times (B=4, T=16384, H=32: 256 chunks per CTA), every unit and every
    token against the oracle, one batch entry at a time on the CPU side."""
    c = synth.CONFIGS["cfg2"]
    B, T, H = c["B"], c["T"], c["H"]
    inp, dy, dsT = _inputs(B, T, H, 2100, 0.1, True)
    d = inp.to(DEV)
    out = gf.backward(d.r, d.k, d.v, d.x, d.u, dy.to(DEV), d.state_in, dsT.to(DEV))
    gf.last_device_status()
    out = [t.cpu() for t in out]
    du_ref = np.zeros((H, 64))
    for b in range(B):
        sl = slice(b, b + 1)
        ref = orc.backward(inp.r[sl], inp.k[sl], inp.v[sl], inp.x[sl], inp.u, dy[sl].double().numpy(), inp.state_in[sl],
                           dsT[sl].double().numpy())
        du_ref += ref[4]
        part = [out[0][sl], out[1][sl], out[2][sl], out[3][sl], None, out[5][sl]]
        for name, a, r in zip(NAMES, part, ref):
            if a is None:
                continue
            a = a.float().numpy().astype(np.float64)
            assert np.isfinite(a).all(), (b, name)
            lim = TOL_DX if name == "dx" else TOL
            assert orc.rel_l2(a, r) <= lim, (b, name, orc.rel_l2(a, r))
            if name != "dstate_in":
                row = ((a - r) ** 2).sum(axis=3)
                num, den = row.sum(axis=1), (r * r).sum(axis=(1, 3))
                assert np.sqrt(num / den).max() <= lim, (b, name, "unit")
                assert np.sqrt(row.max(axis=1) / (den / T)).max() <= TOK_TOL, (b, name, "token")
    assert orc.rel_l2(out[4].numpy(), du_ref) <= TOL


@pytest.mark.parametrize("B,T,H,x_lo,x_hi", [(1, 4096, 2, -6.0, -1.0), (1, 2000, 3, -6.0, -1.0), (2, 1100, 1, -12.0, -8.0),
                                              (1, 8192, 1, -3.0, 0.3), (1, 1030, 4, -6.0, -1.0)])
def test_few_units_split_their_sequences(B, T, H, x_lo, x_hi):
    """Fewer units than half the SMs: every sequence is cut into segments that run side by side; the state adjoint at
    a segment's end comes from the summaries (decay product, adjoint from zero) of the segments after it.  Slow
    decays make the hand-over matter across the whole sequence."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert gf.split_plan(B, T, H, sms)[0] > 1       # (the forward pass's rule, which the gradient shares)
    _run(B, T, H, seed=640 + T, state_std=0.3, with_dstate=True, x_lo=x_lo, x_hi=x_hi)


def test_split_with_a_fast_channel_in_a_middle_segment():
    B, T, H = 1, 4096, 2
    inp, dy, dsT = _inputs(B, T, H, 660, 0.3, True)
    x = inp.x.clone()
    x[0, 2100:2104, 1, 9] = 5.0
    inp.x = x
    d = inp.to(DEV)
    out = gf.backward(d.r, d.k, d.v, d.x, d.u, dy.to(DEV), d.state_in, dsT.to(DEV))
    gf.last_device_status()
    ref = orc.backward(inp.r, inp.k, inp.v, inp.x, inp.u, dy.double().numpy(), inp.state_in, dsT.double().numpy())
    _check(out, ref, "split, mixed")


@pytest.mark.parametrize("x_lo,x_hi", [(-12.0, -8.0), (-4.0, -1.0), (-3.0, 0.5), (-2.0, 0.0)])
def test_slow_to_fast_decays_on_the_tensor_cores(x_lo, x_hi):
    """From w close to one (state and adjoint reach across the whole sequence) to decays close to the limit of the
    chunked form (a channel may lose up to 2^-96 inside a chunk), where the decay gradient is a small difference
    of large suffix sums."""
    _run(1, 300, 2, seed=700, state_std=0.5, with_dstate=True, x_lo=x_lo, x_hi=x_hi)


@pytest.mark.parametrize("x_lo,x_hi", [(-1.0, 2.0), (0.5, 3.0)])
def test_decays_beyond_the_chunked_form_take_the_token_path(x_lo, x_hi):
    _run(1, 200, 2, seed=710, state_std=0.5, with_dstate=True, x_lo=x_lo, x_hi=x_hi)


def test_mixed_chunks_one_fast_channel_in_some_chunks():
    """Chunks 1 and 3 of five carry one channel with w ~ 0 for a few tokens: those chunks take the token-by-token
    path, their neighbours the tensor-core path, and the state adjoint passes between the two."""
    B, T, H = 1, 300, 2
    inp, dy, dsT = _inputs(B, T, H, 720, 0.3, True)
    x = inp.x.clone()
    x[0, 70:75, 0, 5] = 4.0
    x[0, 200:203, 1, 60] = 6.0
    inp.x = x
    d = inp.to(DEV)
    out = gf.backward(d.r, d.k, d.v, d.x, d.u, dy.to(DEV), d.state_in, dsT.to(DEV))
    gf.last_device_status()
    ref = orc.backward(inp.r, inp.k, inp.v, inp.x, inp.u, dy.double().numpy(), inp.state_in, dsT.double().numpy())
    _check(out, ref, "mixed")


def test_minus_infinite_decay_logit_is_no_decay():
    B, T, H = 1, 130, 1
    inp, dy, dsT = _inputs(B, T, H, 730, 0.2, True)
    x = inp.x.clone()
    x[0, 10:20] = float("-inf")
    inp.x = x
    d = inp.to(DEV)
    out = gf.backward(d.r, d.k, d.v, d.x, d.u, dy.to(DEV), d.state_in, dsT.to(DEV))
    gf.last_device_status()
    ref = orc.backward(inp.r, inp.k, inp.v, inp.x, inp.u, dy.double().numpy(), inp.state_in, dsT.double().numpy())
    _check(out, ref, "x=-inf")
    assert (out[3][0, 10:20].float() == 0).all()          # w = 1 there: the logit has no gradient


def test_agrees_with_the_fp32_token_kernel_on_the_same_inputs():
    """Two GPU kernels of different construction on the same bf16-representable inputs (supplementary to the oracle)."""
    inp, dy, dsT = _inputs(2, 500, 4, 740, 0.1, True)
    d = inp.to(DEV)
    a = gf.backward(d.r, d.k, d.v, d.x, d.u, dy.to(DEV), d.state_in, dsT.to(DEV))
    b = gf.backward(d.r.float(), d.k.float(), d.v.float(), d.x.float(), d.u, dy.to(DEV).float(), d.state_in, dsT.to(DEV))
    gf.last_device_status()
    for name, p, q in zip(NAMES, a, b):
        assert orc.rel_l2(p.float().cpu().numpy(), q.cpu().numpy()) <= TOL, name


def test_repeatable_and_argument_checks():
    inp, dy, _ = _inputs(2, 300, 2, 750, 0.1, False)
    d = inp.to(DEV)
    dy = dy.to(DEV)
    a = gf.backward(d.r, d.k, d.v, d.x, d.u, dy, d.state_in)
    b = gf.backward(d.r, d.k, d.v, d.x, d.u, dy, d.state_in)
    gf.last_device_status()
    assert all(torch.equal(p, q) for p, q in zip(a, b))             # no atomics: bitwise repeatable
    lib = gf.load_library()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    nck = (300 + 63) // 64 + 1
    assert lib.gf_wkv6_backward_bf16_workspace_bytes(2, 300, 2, 64) == (4 * nck * 2048 + 4 * 64 + 2 * sms * 64 * 4096) * 4
    p = lambda t: t.data_ptr()
    outs = [torch.empty_like(d.r) for _ in range(4)]
    du = torch.empty((2, 64), device=DEV)
    args = [p(d.r), p(d.k), p(d.v), p(d.x), p(d.u), None, p(dy), None] + [p(t) for t in outs] + [p(du), None]
    before = gf.launch_count()
    assert lib.gf_wkv6_backward(*args, 2, 300, 2, 64, None, 0, None) == 4          # no workspace
    assert lib.gf_wkv6_backward(*args, 2, 300, 2, 32, None, 0, None) == 2          # head size
    ws = torch.empty(lib.gf_wkv6_backward_bf16_workspace_bytes(2, 300, 2, 64), dtype=torch.uint8, device=DEV)
    bad = list(args); bad[8] = p(d.r)                                               # dr aliases r
    assert lib.gf_wkv6_backward(*bad, 2, 300, 2, 64, p(ws), ws.numel(), None) == 1
    assert lib.gf_wkv6_backward(*args, 2, 300, 2, 64, p(ws), ws.numel() - 16, None) == 4
    ds = torch.zeros((2, 2, 64, 64), device=DEV)
    inplace = list(args); inplace[7] = p(ds); inplace[13] = p(ds)                      # dstate_in is dstate_out
    assert lib.gf_wkv6_backward(*inplace, 2, 300, 2, 64, p(ws), ws.numel(), None) == 1
    assert gf.launch_count() == before
    # no token: the adjoint passes through, no bonus gradient
    e = torch.empty((2, 0, 2, 64), device=DEV, dtype=torch.bfloat16)
    dsT = torch.randn((2, 2, 64, 64), device=DEV)
    o = gf.backward(e, e, e, e, d.u, e, None, dsT)
    assert torch.equal(o[5], dsT) and (o[4] == 0).all()


def test_ragged_last_chunk_repeats_bit_for_bit():
    """The ragged last chunk leaves its staging tiles by plain stores of every thread; the first of those tiles then
    takes the next chunk's start state from one thread's copy.  Run to run, and against the call that makes its own
    checkpoints, every bit must agree (a missing rendezvous between the two showed up as a wrong dr row now and then)."""
    B, T, H = 1, 583, 7
    inp, dy, dsT = _inputs(B, T, H, 4242, 0.2, True, x_lo=-2.0, x_hi=1.5)
    d = inp.to(DEV)
    dyd, dsd = dy.to(DEV), dsT.to(DEV)
    ws = torch.empty(gf.backward_workspace_bytes(B, T, H, 64), dtype=torch.uint8, device=DEV)
    ref = None
    for i in range(40):
        if i % 2:
            gf.prefill_train(d.r, d.k, d.v, d.x, d.u, ws, d.state_in)
            out = gf.backward(d.r, d.k, d.v, d.x, d.u, dyd, d.state_in, dsd, workspace=ws, saved=True)
        else:
            out = gf.backward(d.r, d.k, d.v, d.x, d.u, dyd, d.state_in, dsd, workspace=ws)
        gf.last_device_status()
        out = [t.clone() for t in out]
        if ref is None:
            ref = out
        else:
            for name, a, b in zip(NAMES, ref, out):
                assert torch.equal(a, b), (i, name)


def test_long_context_shape_at_the_benchmarked_size_two_heads_in_full():
    """The launch the benchmark's long-context gradient row times (B=1, T=131072, H=32: 32 units, sequences split
    4-way), two of the heads against the oracle over all their tokens (the oracle keeps every state of a unit: 4 GB
    per head), the rest finite and repeatable."""
    c = synth.CONFIGS["cfg3"]
    B, T, H = c["B"], c["T"], c["H"]
    inp, dy, dsT = _inputs(B, T, H, 3100, c["state_std"], True)
    d = inp.to(DEV)
    out = gf.backward(d.r, d.k, d.v, d.x, d.u, dy.to(DEV), d.state_in, dsT.to(DEV))
    gf.last_device_status()
    out2 = gf.backward(d.r, d.k, d.v, d.x, d.u, dy.to(DEV), d.state_in, dsT.to(DEV))
    gf.last_device_status()
    for name, a, b in zip(NAMES, out, out2):
        assert torch.equal(a, b), name
        assert torch.isfinite(a.float()).all(), name
    out = [t.cpu() for t in out]
    del out2
    for h in (5, 31):
        hs = slice(h, h + 1)
        sin = None if inp.state_in is None else inp.state_in[:, hs]
        ref = orc.backward(inp.r[:, :, hs], inp.k[:, :, hs], inp.v[:, :, hs], inp.x[:, :, hs], inp.u[hs],
                           dy[:, :, hs].double().numpy(), sin, dsT[:, hs].double().numpy())
        part = [out[0][:, :, hs], out[1][:, :, hs], out[2][:, :, hs], out[3][:, :, hs], out[4][hs], out[5][:, hs]]
        for name, a, r in zip(NAMES, part, ref):
            a = a.float().numpy().astype(np.float64)
            lim = TOL_DX if name == "dx" else TOL
            assert orc.rel_l2(a, r) <= lim, (h, name, orc.rel_l2(a, r))
            if name in ("dr", "dk", "dv", "dx"):
                row = ((a - r) ** 2).sum(axis=3)
                den = (r * r).sum(axis=(1, 3))
                tok = np.sqrt(row.max(axis=1) / (den / T))
                assert tok.max() <= TOK_TOL, (h, name, float(tok.max()))
