"""The training step's pair: gf_wkv6_prefill_train leaves the chunk-start states in the gradient's workspace and
gf_wkv6_backward_saved takes them from there.  Both are bit-identical to the calls they shadow (same kernels, same
inputs); against the oracle those are checked in test_gpu_parity*.py, and once more here end to end."""
import numpy as np
import pytest
import torch

import paper_2407_12077_b200 as gf
from oracle import wkv6_oracle as orc
from paper_2407_12077_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("B,T,H", [(2, 300, 3), (1, 64, 1), (4, 1000, 8), (1, 37, 2), (1, 4096, 2)])   # (the last: the gradient splits)
@pytest.mark.parametrize("c2", [False, True])
def test_pair_is_bit_identical_to_the_separate_calls(B, T, H, c2):
    inp = synth.make_dense(B, T, H, 64, "bf16", seed=40 + T, state_std=0.1).to(DEV)
    g = torch.Generator(device=DEV).manual_seed(T)
    dy = torch.randn(inp.r.shape, generator=g, device=DEV).bfloat16()
    u2 = torch.randn(inp.r.shape, generator=g, device=DEV).bfloat16() if c2 else None
    dsT = torch.randn((B, H, 64, 64), generator=g, device=DEV) * 0.1
    ws = torch.empty(gf.backward_workspace_bytes(B, T, H, 64), dtype=torch.uint8, device=DEV)
    y, s = gf.prefill_train(inp.r, inp.k, inp.v, inp.x, inp.u, ws, inp.state_in, c2=c2, u2=u2)
    if c2:
        y0, s0 = gf.prefill_c2(inp.r, inp.k, inp.v, inp.x, u2, inp.state_in)
        ga = gf.backward_c2(inp.r, inp.k, inp.v, inp.x, dy, inp.state_in, dsT, workspace=ws, saved=True)
        gb = gf.backward_c2(inp.r, inp.k, inp.v, inp.x, dy, inp.state_in, dsT)
    else:
        y0, s0 = gf.prefill(inp.r, inp.k, inp.v, inp.x, inp.u, inp.state_in)
        ga = gf.backward(inp.r, inp.k, inp.v, inp.x, inp.u, dy, inp.state_in, dsT, workspace=ws, saved=True)
        gb = gf.backward(inp.r, inp.k, inp.v, inp.x, inp.u, dy, inp.state_in, dsT)
    gf.last_device_status()
    assert torch.equal(y, y0) and torch.equal(s, s0)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    if gf.split_plan(B, T, H, sms)[0] == 1:
        assert all(torch.equal(p, q) for p, q in zip(ga, gb))
    else:
        # a split gradient call makes its own checkpoints segment by segment (folded summaries): the states agree with
        # the forward pass's to fp32 rounding, the gradients to a bf16 ulp here and there
        for p, q in zip(ga, gb):
            assert orc.rel_l2(p.float().cpu().numpy(), q.float().cpu().numpy()) <= 2e-3


def test_pair_against_the_oracle_with_mixed_chunks():
    """One fast channel sends some chunks down the token-by-token path in both passes."""
    B, T, H = 1, 300, 2
    inp = synth.make_dense(B, T, H, 64, "bf16", seed=77, state_std=0.3)
    x = inp.x.clone()
    x[0, 70:75, 0, 5] = 4.0
    inp.x = x
    g = torch.Generator().manual_seed(78)
    dy = torch.randn(inp.r.shape, generator=g).bfloat16()
    d = inp.to(DEV)
    ws = torch.empty(gf.backward_workspace_bytes(B, T, H, 64), dtype=torch.uint8, device=DEV)
    y, s = gf.prefill_train(d.r, d.k, d.v, d.x, d.u, ws, d.state_in)
    grads = gf.backward(d.r, d.k, d.v, d.x, d.u, dy.to(DEV), d.state_in, None, workspace=ws, saved=True)
    gf.last_device_status()
    y_ref, s_ref = orc.prefill(inp.r, inp.k, inp.v, inp.x, inp.u, inp.state_in)
    assert orc.rel_l2(y.float().cpu().numpy(), y_ref) <= 5e-3 and orc.rel_l2(s.cpu().numpy(), s_ref) <= 5e-3
    ref = orc.backward(inp.r, inp.k, inp.v, inp.x, inp.u, dy.double().numpy(), inp.state_in, None)
    for name, a, b in zip(("dr", "dk", "dv", "dx", "du", "ds0"), grads, ref):
        assert orc.rel_l2(a.float().cpu().numpy(), b) <= (8e-3 if name == "dx" else 5e-3), name


def test_argument_checks():
    inp = synth.make_dense(1, 100, 2, 64, "bf16", seed=1).to(DEV)
    lib = gf.load_library()
    p = lambda t: t.data_ptr()
    y = torch.empty_like(inp.r)
    before = gf.launch_count()
    args = [p(inp.r), p(inp.k), p(inp.v), p(inp.x), p(inp.u), None, None, p(y)]
    assert lib.gf_wkv6_prefill_train(*args, 1, 100, 2, 64, None, 0, None) == 4          # no workspace
    assert lib.gf_wkv6_prefill_train(*args, 1, 100, 2, 32, None, 0, None) == 2          # head size
    assert gf.launch_count() == before


@pytest.mark.parametrize("lens", [(300, 64, 0, 37, 129), (1,), (4096, 100), (65, 65, 65, 1000)])
@pytest.mark.parametrize("c2", [False, True])
def test_packed_pair_is_bit_identical_to_the_separate_packed_calls(lens, c2):
    """gf_wkv6_prefill_varlen_train + gf_wkv6_backward_varlen_saved: same kernels on the same inputs as the packed
    prefill (unsplit) and the packed gradient, the checkpoints in the packed layout written by the forward pass."""
    H = 3
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32)
    inp = synth.make_varlen(cu, H, 64, "bf16", seed=90 + sum(lens), state_std=0.1).to(DEV)
    S, total, mx = len(lens), int(sum(lens)), max(lens)
    g = torch.Generator(device=DEV).manual_seed(total)
    dy = torch.randn(inp.r.shape, generator=g, device=DEV).bfloat16()
    u2 = torch.randn(inp.r.shape, generator=g, device=DEV).bfloat16() if c2 else None
    dsT = torch.randn((S, H, 64, 64), generator=g, device=DEV) * 0.1
    ws = torch.empty(gf.backward_varlen_workspace_bytes(S, total, H, 64), dtype=torch.uint8, device=DEV)
    y, s = gf.prefill_varlen_train(inp.r, inp.k, inp.v, inp.x, inp.u, inp.cu_seqlens, mx, ws, inp.state_in, c2=c2, u2=u2)
    ga = gf.backward_varlen(inp.r, inp.k, inp.v, inp.x, inp.u, dy, inp.cu_seqlens, mx, inp.state_in, dsT, workspace=ws, c2=c2, saved=True)
    gb = gf.backward_varlen(inp.r, inp.k, inp.v, inp.x, inp.u, dy, inp.cu_seqlens, mx, inp.state_in, dsT, c2=c2)
    if c2:
        y0, s0 = gf.prefill_varlen_c2(inp.r, inp.k, inp.v, inp.x, u2, inp.cu_seqlens, mx, inp.state_in, split=False)
    else:
        y0, s0 = gf.prefill_varlen(inp.r, inp.k, inp.v, inp.x, inp.u, inp.cu_seqlens, mx, inp.state_in, split=False)
    gf.last_device_status()
    assert torch.equal(y, y0) and torch.equal(s, s0)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    split = 2 * S * H <= sms and (mx + 63) // 64 >= 16      # (the gradient call's own checkpoint pass then runs in segments)
    for p, q in zip(ga, gb):
        if p is None and q is None:
            continue
        if split:
            assert orc.rel_l2(p.float().cpu().numpy(), q.float().cpu().numpy()) <= 2e-3
        else:
            assert torch.equal(p, q)
    # and once against the oracle
    dyn = dy.float().cpu().numpy().astype(np.float64)
    c = inp.to("cpu")
    if c2:
        ref = orc.backward_c2_varlen(c.r, c.k, c.v, c.x, dyn, cu, c.state_in, dsT.cpu().numpy().astype(np.float64))
        got = [ga[0], ga[1], ga[2], ga[3], ga[5]]
    else:
        ref = orc.backward_varlen(c.r, c.k, c.v, c.x, c.u, dyn, cu, c.state_in, dsT.cpu().numpy().astype(np.float64))
        got = list(ga)
    for i, (p, q) in enumerate(zip(got, ref)):
        assert orc.rel_l2(p.float().cpu().numpy(), q) <= (8e-3 if i == 3 else 5e-3), i


@pytest.mark.parametrize("c2", [False, True])
def test_pair_at_the_benchmarked_size(c2):
    """The two launches the benchmark's training rows time (B=4, T=16384, H=32): the forward pass equals the plain
    prefill and the gradient from its saved states equals the gradient call that makes its own, bit for bit."""
    c = synth.CONFIGS["cfg2"]
    B, T, H = c["B"], c["T"], c["H"]
    inp = synth.make_dense(B, T, H, 64, "bf16", seed=2200, state_std=0.1).to(DEV)
    g = torch.Generator(device=DEV).manual_seed(2201)
    dy = torch.randn(inp.r.shape, generator=g, device=DEV).bfloat16()
    u2 = torch.randn(inp.r.shape, generator=g, device=DEV).bfloat16() if c2 else None
    dsT = torch.randn((B, H, 64, 64), generator=g, device=DEV) * 0.1
    ws = torch.empty(gf.backward_workspace_bytes(B, T, H, 64), dtype=torch.uint8, device=DEV)
    y, s = gf.prefill_train(inp.r, inp.k, inp.v, inp.x, inp.u, ws, inp.state_in, c2=c2, u2=u2)
    if c2:
        y0, s0 = gf.prefill_c2(inp.r, inp.k, inp.v, inp.x, u2, inp.state_in)
        ga = gf.backward_c2(inp.r, inp.k, inp.v, inp.x, dy, inp.state_in, dsT, workspace=ws, saved=True)
        gb = gf.backward_c2(inp.r, inp.k, inp.v, inp.x, dy, inp.state_in, dsT)
    else:
        y0, s0 = gf.prefill(inp.r, inp.k, inp.v, inp.x, inp.u, inp.state_in)
        ga = gf.backward(inp.r, inp.k, inp.v, inp.x, inp.u, dy, inp.state_in, dsT, workspace=ws, saved=True)
        gb = gf.backward(inp.r, inp.k, inp.v, inp.x, inp.u, dy, inp.state_in, dsT)
    gf.last_device_status()
    assert torch.equal(y, y0) and torch.equal(s, s0)
    assert all(torch.equal(p, q) for p, q in zip(ga, gb))
