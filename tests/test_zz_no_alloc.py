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
TOL = 5e-3          # the bf16 tolerance of the parity tests


def _rel(a, b):
    return orc.rel_l2(a.float().cpu().numpy(), b.float().cpu().numpy())


def test_static_scratch_entry_point_matches_prefill_on_two_calls_in_a_row():
    gf.set_kernel(gf.KERNEL_AUTO)
    # two different problems back to back: the second finds the first one's summaries in the scratch
    shapes = [(1, 5000, 4, 4321, 0.1), (2, 3000, 3, 4322, 0.0)]
    for B, T, H, seed, state_std in shapes:
        assert 0 < gf.workspace_bytes(B, T, H, 64) <= gf.STATIC_SCRATCH_BYTES      # splits, and fits
        d = synth.make_dense(B, T, H, 64, "bf16", seed=seed, state_std=state_std, device=DEV)
        y_ref, s_ref = gf.prefill(d.r, d.k, d.v, d.x, d.u, d.state_in)            # the existing entry point
        y = torch.full_like(d.r, float("nan"))
        s = torch.full((B, H, 64, 64), float("nan"), device=DEV)
        before = gf.launch_count()
        gf.prefill_static(d.r, d.k, d.v, d.x, d.u, d.state_in, s, y)              # caller-owned outputs, no allocation
        gf.last_device_status()
        assert gf.launch_count() - before == 2                                   # the split path ran
        assert torch.isfinite(y.float()).all() and torch.isfinite(s).all()
        ey, es = _rel(y, y_ref), _rel(s, s_ref)
        assert ey <= TOL and es <= TOL, (B, T, H, ey, es)


def test_static_scratch_entry_point_without_split_and_beyond_its_limit():
    # many units: no split, so a dense call needs no scratch and passes whatever its size (what workspace_bytes
    # reports for more units than SMs is the unit counter that a packed call of that shape would use)
    d = synth.make_dense(2, 200, 80, 64, "bf16", seed=4323, device=DEV)
    assert gf.workspace_bytes(2, 200, 80, 64) <= 256
    y_ref, s_ref = gf.prefill(d.r, d.k, d.v, d.x, d.u, None)
    y, s = torch.empty_like(d.r), torch.empty((2, 80, 64, 64), device=DEV)
    gf.prefill_static(d.r, d.k, d.v, d.x, d.u, None, s, y)
    gf.last_device_status()
    assert _rel(y, y_ref) <= TOL and _rel(s, s_ref) <= TOL
    # a split that wants more than the built-in array is refused before anything is enqueued
    B, T, H = 1, 4096, 18
    assert gf.workspace_bytes(B, T, H, 64) > gf.STATIC_SCRATCH_BYTES
    d = synth.make_dense(B, T, H, 64, "bf16", seed=4324, device=DEV)
    y, s = torch.empty_like(d.r), torch.empty((B, H, 64, 64), device=DEV)
    before = gf.launch_count()
    with pytest.raises(gf.GfError) as err:
        gf.prefill_static(d.r, d.k, d.v, d.x, d.u, None, s, y)
    assert err.value.status == 4 and gf.launch_count() == before                 # GF_ERR_WORKSPACE, nothing launched
