"""The bounded device-side waits: a wait that runs out must surface as GF_ERR_TIMEOUT at the next status query,
once, and leave the context and the library fully usable.  Nothing here hangs or faults: the wait that runs out
belongs to a one-warp kernel made for the purpose, and its limit is two milliseconds."""
import time

import pytest
import torch

import paper_2407_12077_b200 as gf
from paper_2407_12077_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
GF_ERR_TIMEOUT = 5


def test_wait_that_runs_out_is_reported_once_and_harms_nothing():
    gf.set_kernel(gf.KERNEL_AUTO)
    d = synth.make_dense(2, 700, 6, 64, "bf16", seed=8800, state_std=0.1, device=DEV)
    y0, s0 = gf.prefill(d.r, d.k, d.v, d.x, d.u, d.state_in)
    gf.last_device_status()                                          # healthy so far
    t0 = time.perf_counter()
    gf.selftest_wait_timeout(2000)                                   # a barrier nobody arrives on, 2 ms limit
    with pytest.raises(gf.GfError) as err:
        gf.last_device_status()
    waited = time.perf_counter() - t0
    assert err.value.status == GF_ERR_TIMEOUT
    assert 0.0015 <= waited < 1.0, waited                            # it did wait, and it did give up
    gf.last_device_status()                                          # reported once: clear again
    y1, s1 = gf.prefill(d.r, d.k, d.v, d.x, d.u, d.state_in)
    gf.last_device_status()
    assert torch.equal(y0, y1) and torch.equal(s0, s1)


def test_wait_limit_setting_round_trip_and_argument_checks():
    gf.set_wait_limit(500000)                                        # half a second: far above any healthy wait
    try:
        d = synth.make_dense(1, 5000, 4, 64, "bf16", seed=8801, device=DEV)          # a call that splits
        y0, s0 = gf.prefill(d.r, d.k, d.v, d.x, d.u, None)
        gf.last_device_status()
    finally:
        gf.set_wait_limit(0)
    y1, s1 = gf.prefill(d.r, d.k, d.v, d.x, d.u, None)
    gf.last_device_status()
    assert torch.equal(y0, y1) and torch.equal(s0, s1)
    for bad in (0, 2000000):
        with pytest.raises(gf.GfError) as err:
            gf.selftest_wait_timeout(bad)
        assert err.value.status == 1                                 # GF_ERR_INVALID_ARG, nothing enqueued
    gf.last_device_status()
