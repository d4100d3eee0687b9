"""gf_wkv6_prefill_static: the prefill entry point for hosts that cannot allocate device memory (a
plug-in in a server that plans all device memory up front, a loop that must stay clear of cudaMalloc).
It must give what gf_wkv6_prefill gives, call after call, although every call reuses the one scratch
array built into the library and finds the previous call's data in it.  Collected last on purpose: if
this entry point breaks, a run that stops at the first failure has still run everything else.
"""
import pytest
import torch

import paper_2407_12077_b200 as gf
from oracle import wkv6_oracle as orc
from paper_2407_12077_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = 5e-3          # the bf16 tolerance of the parity tests (against the fp64 oracle)


def _rel(a, b):
    return orc.rel_l2(a.float().cpu().numpy(), b if not hasattr(b, "cpu") else b.float().cpu().numpy())


def _static(d, B, H, state_in):
    """One call through the entry point with caller-owned, NaN-filled outputs."""
    y = torch.full_like(d.r, float("nan"))
    s = torch.full((B, H, 64, 64), float("nan"), device=DEV)
    gf.prefill_static(d.r, d.k, d.v, d.x, d.u, state_in, s, y)
    gf.last_device_status()
    assert torch.isfinite(y.float()).all() and torch.isfinite(s).all()
    return y, s


def test_static_scratch_entry_point_matches_prefill_on_two_calls_in_a_row():
    gf.set_kernel(gf.KERNEL_AUTO)
    # two different problems back to back: the second finds the first one's summaries in the scratch
    shapes = [(1, 5000, 4, 4321, 0.1), (2, 3000, 3, 4322, 0.0)]
    for B, T, H, seed, state_std in shapes:
        assert 0 < gf.workspace_bytes(B, T, H, 64) <= gf.STATIC_SCRATCH_BYTES      # splits, and fits in full
        inp = synth.make_dense(B, T, H, 64, "bf16", seed=seed, state_std=state_std)
        d = inp.to(DEV)
        y_ref, s_ref = gf.prefill(d.r, d.k, d.v, d.x, d.u, d.state_in)            # the existing entry point
        before = gf.launch_count()
        y, s = _static(d, B, H, d.state_in)                                      # caller-owned outputs, no allocation
        assert gf.launch_count() - before == 2                                   # the split path ran
        # the same two launches with other scratch: the same bits
        assert torch.equal(y, y_ref) and torch.equal(s, s_ref), (B, T, H)
        y_o, s_o = orc.prefill(inp.r, inp.k, inp.v, inp.x, inp.u, inp.state_in)
        ey, es = _rel(y, y_o), _rel(s, s_o)
        assert ey <= TOL and es <= TOL, (B, T, H, ey, es)


@pytest.mark.parametrize("B,T,H,same_split", [(1, 4096, 32, True), (1, 8192, 16, False), (2, 4096, 12, False)])
def test_static_scratch_entry_point_at_and_over_the_full_split(B, T, H, same_split):
    """32 units cut four ways fill the array exactly; 16 and 24 units would be cut into more segments than fit
    and run with fewer (so their rounding differs from gf_wkv6_prefill's: compared through the oracle).  A
    registered workspace is not used: a useless one is registered meanwhile."""
    need = gf.workspace_bytes(B, T, H, 64)
    assert (need == gf.STATIC_SCRATCH_BYTES) if same_split else (need > gf.STATIC_SCRATCH_BYTES)
    inp = synth.make_dense(B, T, H, 64, "bf16", seed=4330 + H, state_std=0.1)
    d = inp.to(DEV)
    y_ref, s_ref = gf.prefill(d.r, d.k, d.v, d.x, d.u, d.state_in)
    gf.set_workspace(torch.empty(256, dtype=torch.uint8, device=DEV))
    try:
        before = gf.launch_count()
        y, s = _static(d, B, H, d.state_in)
        assert gf.launch_count() - before == 2
        # in place: the start state is overwritten by the final one
        st = d.state_in.clone()
        y2 = torch.empty_like(d.r)
        gf.prefill_static(d.r, d.k, d.v, d.x, d.u, st, st, y2)
        gf.last_device_status()
    finally:
        gf.set_workspace(None)
    assert torch.equal(y2, y) and torch.equal(st, s)
    if same_split:
        assert torch.equal(y, y_ref) and torch.equal(s, s_ref)
    else:
        assert _rel(y, y_ref) < 2e-3 and _rel(s, s_ref) < 1e-3
    y_o, s_o = orc.prefill(inp.r, inp.k, inp.v, inp.x, inp.u, inp.state_in)
    ey, es = _rel(y, y_o), _rel(s, s_o)
    assert ey <= TOL and es <= TOL, (ey, es)


def test_static_scratch_entry_point_without_split_and_beyond_its_limit():
    # many units: no split, so a dense call needs no scratch and passes whatever its size (what workspace_bytes
    # reports for more units than SMs is the unit counter that a packed call of that shape would use)
    inp = synth.make_dense(2, 200, 80, 64, "bf16", seed=4323)
    d = inp.to(DEV)
    assert gf.workspace_bytes(2, 200, 80, 64) <= 256
    y_ref, s_ref = gf.prefill(d.r, d.k, d.v, d.x, d.u, None)
    y, s = _static(d, 2, 80, None)
    assert torch.equal(y, y_ref) and torch.equal(s, s_ref)
    y_o, s_o = orc.prefill(inp.r, inp.k, inp.v, inp.x, inp.u, None)
    assert _rel(y, y_o) <= TOL and _rel(s, s_o) <= TOL
    # a split of which not even two segments fit the built-in array is refused before anything is enqueued
    B, T, H = 1, 2048, 70
    assert gf.workspace_bytes(B, T, H, 64) > gf.STATIC_SCRATCH_BYTES
    d = synth.make_dense(B, T, H, 64, "bf16", seed=4324, device=DEV)
    y, s = torch.empty_like(d.r), torch.empty((B, H, 64, 64), device=DEV)
    before = gf.launch_count()
    with pytest.raises(gf.GfError) as err:
        gf.prefill_static(d.r, d.k, d.v, d.x, d.u, None, s, y)
    assert err.value.status == 4 and gf.launch_count() == before                 # GF_ERR_WORKSPACE, nothing launched
