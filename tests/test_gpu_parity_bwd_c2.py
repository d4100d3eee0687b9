"""GPU parity of gf_wkv6_backward_c2 (gradient of the Finch-C2 form, bf16, chunked on the tensor cores) against the
fp64 oracle's reverse recurrence of that form; tolerances as for gf_wkv6_backward (5e-3 per tensor and unit, 8e-3
for the decay-logit gradient, 4e-2 per token row)."""
import numpy as np
import pytest
import torch

import paper_2407_12077_b200 as gf
from oracle import wkv6_oracle as orc
from paper_2407_12077_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL, TOL_DX, TOK_TOL = 5e-3, 8e-3, 4e-2
NAMES = ("dr", "dk", "dv", "dx", "dstate_in")


def _inputs(B, T, H, seed, state_std, with_dstate, x_lo=-6.0, x_hi=-1.0):
    inp = synth.make_dense(B, T, H, 64, "bf16", seed=seed, state_std=state_std, x_lo=x_lo, x_hi=x_hi)
    g = torch.Generator().manual_seed(seed + 1)
    dy = torch.randn(inp.r.shape, generator=g).bfloat16()
    dsT = torch.randn((B, H, 64, 64), generator=g) * 0.1 if with_dstate else None
    return inp, dy, dsT


def _check(out, ref, what):
    worst = {}
    for name, a, b in zip(NAMES, out, ref):
        a = a.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(a).all(), (what, name)
        lim = TOL_DX if name == "dx" else TOL
        worst[name] = orc.rel_l2(a, b)
        assert worst[name] <= lim, (what, name, worst[name])
        if name != "dstate_in" and a.shape[1] >= 64:
            T = a.shape[1]
            row = ((a - b) ** 2).sum(axis=3)
            num, den = row.sum(axis=1), (b * b).sum(axis=(1, 3))
            assert np.sqrt(num / den).max() <= lim, (what, name, "unit")
            assert np.sqrt(row.max(axis=1) / (den / T)).max() <= TOK_TOL, (what, name, "token")
    return worst


def _run(B, T, H, seed, state_std, with_dstate, x_lo=-6.0, x_hi=-1.0):
    inp, dy, dsT = _inputs(B, T, H, seed, state_std, with_dstate, x_lo, x_hi)
    d = inp.to(DEV)
    out = gf.backward_c2(d.r, d.k, d.v, d.x, dy.to(DEV), d.state_in, None if dsT is None else dsT.to(DEV))
    gf.last_device_status()
    ref = orc.backward_c2(inp.r, inp.k, inp.v, inp.x, dy.double().numpy(), inp.state_in,
                          None if dsT is None else dsT.double().numpy())
    return _check(out, ref, (B, T, H, x_lo, x_hi))


@pytest.mark.parametrize("T", [1, 2, 63, 64, 65, 128, 200, 321, 1000])
@pytest.mark.parametrize("with_dstate", [False, True])
def test_ragged_lengths_with_states(T, with_dstate):
    _run(2, T, 3, seed=800 + T, state_std=0.1, with_dstate=with_dstate)


def test_few_units_split_their_sequences():
    _run(1, 4096, 2, seed=850, state_std=0.3, with_dstate=True)
    _run(1, 2000, 3, seed=851, state_std=0.3, with_dstate=True, x_lo=-12.0, x_hi=-8.0)


def test_cfg1_shape_every_unit():
    c = synth.CONFIGS["cfg1"]
    print(_run(c["B"], c["T"], c["H"], seed=1100, state_std=c["state_std"], with_dstate=True))


@pytest.mark.parametrize("x_lo,x_hi", [(-12.0, -8.0), (-4.0, -1.0), (-3.0, 0.5)])
def test_slow_to_fast_decays_on_the_tensor_cores(x_lo, x_hi):
    """Slow decays make the key factor 1 - w tiny (6e-6 at x = -12): it is formed from the series of -expm1 there."""
    _run(1, 300, 2, seed=900, state_std=0.5, with_dstate=True, x_lo=x_lo, x_hi=x_hi)


@pytest.mark.parametrize("x_lo,x_hi", [(-1.0, 2.0), (0.5, 3.0)])
def test_decays_beyond_the_chunked_form_take_the_token_path(x_lo, x_hi):
    _run(1, 200, 2, seed=910, state_std=0.5, with_dstate=True, x_lo=x_lo, x_hi=x_hi)


def test_chains_with_the_forward_call_as_a_directional_derivative():
    """<dy, y> + <dS_T, S_T> of gf_wkv6_prefill_c2 moves by <grad, delta> under a small change of v (linear in v, so the
    finite difference is exact up to the kernels' own rounding): the two kernels describe the same function."""
    B, T, H = 1, 256, 2
    inp, dy, dsT = _inputs(B, T, H, 920, 0.2, True)
    d = inp.to(DEV)
    dyd, dsd = dy.to(DEV), dsT.to(DEV)
    grads = gf.backward_c2(d.r, d.k, d.v, d.x, dyd, d.state_in, dsd)
    g = torch.Generator().manual_seed(921)
    dv_dir = torch.randn(inp.v.shape, generator=g).bfloat16().to(DEV)
    y0, s0 = gf.prefill_c2(d.r, d.k, d.v, d.x, None, d.state_in)
    y1, s1 = gf.prefill_c2(d.r, d.k, dv_dir, d.x, None, torch.zeros_like(d.state_in))      # linear in v: the response to dv alone
    gf.last_device_status()
    lhs = (y1.float() * dyd.float()).sum().item() + (s1 * dsd).sum().item()
    rhs = (grads[2].float() * dv_dir.float()).sum().item()
    assert abs(lhs - rhs) <= 2e-2 * max(abs(lhs), abs(rhs)), (lhs, rhs)


def test_repeatable_and_argument_checks():
    inp, dy, _ = _inputs(2, 300, 2, 930, 0.1, False)
    d = inp.to(DEV)
    dy = dy.to(DEV)
    a = gf.backward_c2(d.r, d.k, d.v, d.x, dy, d.state_in)
    b = gf.backward_c2(d.r, d.k, d.v, d.x, dy, d.state_in)
    gf.last_device_status()
    assert all(torch.equal(p, q) for p, q in zip(a, b))
    lib = gf.load_library()
    p = lambda t: t.data_ptr()
    outs = [torch.empty_like(d.r) for _ in range(4)]
    args = [p(d.r), p(d.k), p(d.v), p(d.x), None, p(dy), None] + [p(t) for t in outs] + [None]
    before = gf.launch_count()
    assert lib.gf_wkv6_backward_c2(*args, 2, 300, 2, 64, None, 0, None) == 4          # no workspace
    assert lib.gf_wkv6_backward_c2(*args, 2, 300, 2, 32, None, 0, None) == 2          # head size
    assert gf.launch_count() == before
