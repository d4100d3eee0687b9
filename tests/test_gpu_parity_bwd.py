"""GPU parity of gf_wkv6_backward_f32 (the gradient of the recurrence) against the fp64 oracle's reverse
recurrence, per output tensor at the fp32 tolerance of the contract (relative L2 <= 1e-4)."""
import numpy as np
import pytest
import torch

import paper_2407_12077_b200 as gf
from oracle import wkv6_oracle as orc
from paper_2407_12077_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = 1e-4
NAMES = ("dr", "dk", "dv", "dx", "du", "dstate_in")


def _run(B, T, H, seed, state_std, with_dstate, x_lo=-6.0, x_hi=-1.0):
    inp = synth.make_dense(B, T, H, 64, "f32", seed=seed, state_std=state_std, x_lo=x_lo, x_hi=x_hi)
    g = torch.Generator().manual_seed(seed + 1)
    dy = torch.randn(inp.r.shape, generator=g)
    dsT = torch.randn((B, H, 64, 64), generator=g) * 0.1 if with_dstate else None
    d = inp.to(DEV)
    out = gf.backward(d.r, d.k, d.v, d.x, d.u, dy.to(DEV), d.state_in, None if dsT is None else dsT.to(DEV))
    gf.last_device_status()
    ref = orc.backward(inp.r, inp.k, inp.v, inp.x, inp.u, dy.double().numpy(), inp.state_in,
                       None if dsT is None else dsT.double().numpy())
    worst = {}
    for name, a, b in zip(NAMES, out, ref):
        a = a.cpu().numpy()
        assert np.isfinite(a).all(), name
        worst[name] = orc.rel_l2(a, b)
        assert worst[name] <= TOL, (name, worst[name], (B, T, H))
    # element by element as well, against the size of the tensor's typical entry
    for name, a, b in zip(NAMES, out, ref):
        scale = np.sqrt(np.mean(b * b))
        assert np.abs(a.cpu().numpy() - b).max() <= 2e-3 * scale, name
    return worst


def test_cfg0_shape():
    c = synth.CONFIGS["cfg0"]
    print(_run(c["B"], c["T"], c["H"], seed=0, state_std=0.0, with_dstate=False))


@pytest.mark.parametrize("T", [1, 2, 63, 64, 65, 128, 200, 321])
@pytest.mark.parametrize("with_dstate", [False, True])
def test_ragged_lengths_with_states(T, with_dstate):
    _run(2, T, 3, seed=300 + T, state_std=0.1, with_dstate=with_dstate)


@pytest.mark.parametrize("x_lo,x_hi", [(-12.0, -8.0), (-1.0, 2.0)])
def test_slow_and_fast_decays(x_lo, x_hi):
    """w close to one (the adjoint and the state both reach across the whole sequence) and w close to zero."""
    _run(1, 300, 2, seed=400, state_std=0.5, with_dstate=True, x_lo=x_lo, x_hi=x_hi)


def test_repeatable_and_argument_checks():
    inp = synth.make_dense(2, 100, 2, 64, "f32", seed=500, state_std=0.1).to(DEV)
    dy = torch.randn(inp.r.shape, device=DEV)
    a = gf.backward(inp.r, inp.k, inp.v, inp.x, inp.u, dy, inp.state_in)
    b = gf.backward(inp.r, inp.k, inp.v, inp.x, inp.u, dy, inp.state_in)
    gf.last_device_status()
    assert all(torch.equal(p, q) for p, q in zip(a, b))             # no atomics: bitwise repeatable
    lib = gf.load_library()
    assert lib.gf_wkv6_backward_workspace_bytes(2, 100, 2, 64) == 2 * 2 * (2 * 4096 + 64 * 4096 + 64) * 4
    p = lambda t: t.data_ptr()
    outs = [torch.empty_like(inp.r) for _ in range(4)]
    du = torch.empty((2, 64), device=DEV)
    args = [p(inp.r), p(inp.k), p(inp.v), p(inp.x), p(inp.u), None, p(dy), None] + [p(t) for t in outs] + [p(du), None]
    before = gf.launch_count()
    assert lib.gf_wkv6_backward_f32(*args, 2, 100, 2, 64, None, 0, None) == 4          # no workspace
    assert lib.gf_wkv6_backward_f32(*args, 2, 100, 2, 32, None, 0, None) == 2          # head size
    bad = list(args); bad[8] = p(inp.r)                                               # dr aliases r
    ws = torch.empty(lib.gf_wkv6_backward_workspace_bytes(2, 100, 2, 64), dtype=torch.uint8, device=DEV)
    assert lib.gf_wkv6_backward_f32(*bad, 2, 100, 2, 64, p(ws), ws.numel(), None) == 1
    assert gf.launch_count() == before
