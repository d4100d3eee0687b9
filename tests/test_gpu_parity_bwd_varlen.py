"""Parity of gf_wkv6_backward_varlen / gf_wkv6_backward_varlen_c2 (gradient of the packed variable-length prefill, bf16
tensors) against the fp64 oracle, through the C ABI.  Tolerances as for the dense gradient (same arithmetic per unit)."""
import numpy as np
import pytest
import torch

from paper_2407_12077_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 5e-3
TOL_DX = 8e-3
GF_ERR_INVALID_ARG, GF_ERR_UNSUPPORTED, GF_ERR_WORKSPACE = 1, 2, 4      # gf_status_t of include/gf_wkv6.h


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    d = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / d) if d > 0 else float(np.linalg.norm(a))


def make(lens, H, seed, x_range=(-6.0, -1.0), with_state=True):
    """Packed inputs from the prefill's generator, plus seeded output gradients."""
    total, S = int(sum(lens)), len(lens)
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32)
    inp = synth.make_varlen(cu, H, 64, "bf16", seed=seed, state_std=0.3 if with_state else 0.0,
                            x_lo=x_range[0], x_hi=x_range[1])
    g = torch.Generator().manual_seed(seed + 4242)
    dy = torch.randn(total, H, 64, generator=g).to(torch.bfloat16)
    dsT = torch.randn(S, H, 64, 64, generator=g) * 0.1
    return inp.r, inp.k, inp.v, inp.x, inp.u, dy, inp.state_in, dsT, cu


def run_gpu(case, c2=False, dstate=True):
    import paper_2407_12077_b200 as gf
    r, k, v, x, u, dy, s0, dsT, cu = case
    dev = lambda t: None if t is None else t.cuda()
    lens = np.diff(cu.numpy())
    out = gf.backward_varlen(dev(r), dev(k), dev(v), dev(x), dev(u), dev(dy), dev(cu), int(lens.max()) if len(lens) else 0,
                             dev(s0), dev(dsT) if dstate else None, c2=c2)
    torch.cuda.synchronize()
    gf.last_device_status()
    return [None if t is None else t.float().cpu().numpy() for t in out]


def run_oracle(case, c2=False, dstate=True):
    from oracle import wkv6_oracle as orc
    r, k, v, x, u, dy, s0, dsT, cu = case
    dsT = dsT.numpy().astype(np.float64) if dstate else None
    dyn = dy.float().numpy().astype(np.float64)
    if c2:
        dr, dk, dv, dx, ds0 = orc.backward_c2_varlen(r, k, v, x, dyn, cu, s0, dsT)
        return [dr, dk, dv, dx, None, ds0]
    return list(orc.backward_varlen(r, k, v, x, u, dyn, cu, s0, dsT))


def check(got, ref, cu, c2=False, tol=TOL, tol_dx=TOL_DX, what=""):
    names = ("dr", "dk", "dv", "dx")
    lens = np.diff(np.asarray(cu))
    for i, n in enumerate(names):
        lim = tol_dx if n == "dx" else tol
        e = rel_l2(got[i], ref[i])
        assert e <= lim, f"{what} {n}: rel-L2 {e:.3e} > {lim}"
        # every sequence of a full chunk or more on its own (short ones are few heavy-tailed numbers)
        for s, ln in enumerate(lens):
            if ln >= 64:
                a, b = int(cu[s]), int(cu[s + 1])
                e = rel_l2(got[i][a:b], ref[i][a:b])
                assert e <= 2 * lim, f"{what} {n} sequence {s} (len {ln}): rel-L2 {e:.3e}"
    if not c2:
        e = rel_l2(got[4], ref[4])
        assert e <= tol, f"{what} du: rel-L2 {e:.3e}"
    e = rel_l2(got[5], ref[5])
    assert e <= tol, f"{what} dstate_in: rel-L2 {e:.3e}"


LENS = [
    (64,), (1,), (63,), (65,), (200,),
    (64, 64), (1, 1, 1), (100, 0, 37, 64, 129), (0, 5), (7, 0), (0, 0, 3, 0),
    (300, 17, 128, 1, 255, 64),
]


@pytest.mark.parametrize("c2", [False, True])
@pytest.mark.parametrize("lens", LENS)
def test_packed_sequences_against_the_oracle(lens, c2):
    case = make(lens, 2, 7000 + sum(lens) + len(lens))
    got, ref = run_gpu(case, c2), run_oracle(case, c2)
    check(got, ref, case[-1].numpy(), c2, what=str(lens))


@pytest.mark.parametrize("c2", [False, True])
def test_empty_sequences_hand_the_state_gradient_through(c2):
    case = make((0, 70, 0), 2, 7100)
    got = run_gpu(case, c2)
    dsT = case[7].numpy()
    assert np.array_equal(got[5][0], dsT[0]) and np.array_equal(got[5][2], dsT[2])
    got0 = run_gpu(case, c2, dstate=False)
    assert np.count_nonzero(got0[5][0]) == 0 and np.count_nonzero(got0[5][2]) == 0


@pytest.mark.parametrize("c2", [False, True])
def test_equals_the_dense_call_sequence_by_sequence(c2):
    """Same kernel, same arithmetic per unit: bit-identical to dense calls on each sequence's rows."""
    import paper_2407_12077_b200 as gf
    lens = (130, 64, 7, 257)
    case = make(lens, 3, 7200)
    r, k, v, x, u, dy, s0, dsT, cu = case
    got = run_gpu(case, c2)
    du = np.zeros_like(got[4]) if not c2 else None
    for s, ln in enumerate(lens):
        a, b = int(cu[s]), int(cu[s + 1])
        sl = lambda t: t[a:b][None].contiguous().cuda()
        if c2:
            one = gf.backward_c2(sl(r), sl(k), sl(v), sl(x), sl(dy), s0[s][None].cuda(), dsT[s][None].cuda())
            one = list(one[:4]) + [None, one[4]]
        else:
            one = gf.backward(sl(r), sl(k), sl(v), sl(x), u.cuda(), sl(dy), s0[s][None].cuda(), dsT[s][None].cuda())
        torch.cuda.synchronize()
        for i in range(4):
            assert np.array_equal(got[i][a:b], one[i][0].float().cpu().numpy()), (s, i)
        assert np.array_equal(got[5][s], one[5][0].cpu().numpy())
        if not c2:
            du += one[4].cpu().numpy()
    if not c2:
        assert np.allclose(got[4], du, rtol=1e-5, atol=1e-5)


@pytest.mark.parametrize("c2", [False, True])
def test_serving_mix_of_lengths_more_units_than_sms(c2):
    """A mix like the batched-serving configuration's (many sequences of 128 .. 4096 tokens), scaled so that the
    oracle finishes in seconds: 40 sequences x 8 heads = 320 units, ragged tails everywhere."""
    rng = np.random.default_rng(7300)
    lens = tuple(int(n) for n in rng.integers(16, 700, size=40))
    case = make(lens, 8, 7300)
    got, ref = run_gpu(case, c2), run_oracle(case, c2)
    check(got, ref, case[-1].numpy(), c2, what="mix")


def test_serving_mix_at_full_size_every_unit():
    """The packed batch the benchmark's gradient row times (64 sequences of 128 .. 4096 tokens, 32 heads: 2048 units of
    different lengths on 148 SMs, longest first), every sequence against the oracle."""
    c = synth.CONFIGS["cfg4"]
    cu = synth.make_lengths(c["S"], c["len_min"], c["len_max"], seed=4000)
    lens = tuple(int(n) for n in np.diff(cu.numpy()))
    inp = synth.make_varlen(cu, c["H"], 64, "bf16", seed=4001, state_std=c["state_std"])
    g = torch.Generator().manual_seed(4002)
    dy = torch.randn(inp.r.shape, generator=g).to(torch.bfloat16)
    dsT = torch.randn(len(lens), c["H"], 64, 64, generator=g) * 0.1
    case = (inp.r, inp.k, inp.v, inp.x, inp.u, dy, inp.state_in, dsT, cu)
    got, ref = run_gpu(case), run_oracle(case)
    check(got, ref, cu.numpy(), what="cfg4")


@pytest.mark.parametrize("c2", [False, True])
@pytest.mark.parametrize("lens,H", [((4096, 100, 1000, 0), 2), ((2048,), 1), ((700, 3000), 4), ((1030, 1029, 1, 520), 8)])
def test_few_units_split_their_sequences(lens, H, c2):
    """Fewer (sequence, head) units than half the SMs: every sequence is cut into segments by the longest one (segments
    past a shorter sequence's end are empty) and the adjoint's segment summaries are folded, as in the dense call.
    Slow decays, so that what is handed across the cuts matters over the whole sequence."""
    import paper_2407_12077_b200 as gf
    case = make(lens, H, 7800 + len(lens), x_range=(-8.0, -4.0))
    n0 = gf.launch_count()
    got = run_gpu(case, c2)
    # order, forward summaries, checkpoints, adjoint summaries, gradient (and the bonus sum): the split was taken
    assert gf.launch_count() - n0 == (5 if c2 else 6)
    ref = run_oracle(case, c2)
    check(got, ref, case[-1].numpy(), c2, what=f"split {lens}")
    a, b = run_gpu(case, c2), got
    for p, q in zip(a, b):
        assert (p is None and q is None) or np.array_equal(p, q)


def test_fast_decays_take_the_token_path_in_some_sequences():
    lens = (150, 90, 64)
    case = make(lens, 2, 7400, x_range=(-2.0, 1.5))
    got, ref = run_gpu(case), run_oracle(case)
    check(got, ref, case[-1].numpy(), tol=4e-2, tol_dx=4e-2, what="fast")


def test_repeatable_bit_for_bit():
    case = make((100, 300, 50), 4, 7500)
    a, b = run_gpu(case), run_gpu(case)
    for p, q in zip(a, b):
        assert np.array_equal(p, q)


def test_argument_checks():
    import paper_2407_12077_b200 as gf
    lib = gf.load_library()
    case = make((70, 30), 2, 7600)
    r, k, v, x, u, dy, s0, dsT, cu = (None if t is None else t.cuda() for t in case)
    need = int(lib.gf_wkv6_backward_varlen_workspace_bytes(2, 100, 2, 64))
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    nmax = min(8, sms // 4) if 8 <= sms else 1            # the widest split 4 units may take
    assert need == (2 * (100 // 64 + 4) * 2048 + 4 * nmax * 64 + 4 * (nmax - 1) * (64 + 4096) + (16 + 2 + 3) // 4 * 4
                    + 2 * sms * 64 * 4096) * 4
    small = torch.empty(need - 16, dtype=torch.uint8, device="cuda")
    dr, dk, dv, dx = (torch.empty_like(r) for _ in range(4))
    du = torch.empty(2, 64, device="cuda")
    ds0 = torch.empty_like(dsT)
    p = lambda t: None if t is None else t.data_ptr()
    st = lib.gf_wkv6_backward_varlen(p(r), p(k), p(v), p(x), p(u), p(s0), p(dy), p(dsT), p(dr), p(dk), p(dv), p(dx), p(du),
                                     p(ds0), p(cu), 2, 100, 70, 2, 64, p(small), small.numel(), None)
    assert st == GF_ERR_WORKSPACE
    big = torch.empty(need, dtype=torch.uint8, device="cuda")
    st = lib.gf_wkv6_backward_varlen(p(r), p(k), p(v), p(x), p(u), p(s0), p(dy), p(dsT), p(dr), p(dk), p(dv), p(dx), p(du),
                                     p(dsT), p(cu), 2, 100, 70, 2, 64, p(big), big.numel(), None)
    assert st == GF_ERR_INVALID_ARG                   # dstate_in may not be dstate_out
    st = lib.gf_wkv6_backward_varlen(p(r), p(k), p(v), p(x), p(u), p(s0), p(dy), p(dsT), p(dr), p(dk), p(dv), p(dx), p(du),
                                     p(ds0), None, 2, 100, 70, 2, 64, p(big), big.numel(), None)
    assert st == GF_ERR_INVALID_ARG                   # no cu_seqlens
    st = lib.gf_wkv6_backward_varlen(p(r), p(k), p(v), p(x), p(u), p(s0), p(dy), p(dsT), p(dr), p(dk), p(dv), p(dx), p(du),
                                     p(ds0), p(cu), 2, 100, 70, 2, 32, p(big), big.numel(), None)
    assert st == GF_ERR_UNSUPPORTED
    torch.cuda.synchronize()


def test_more_sequences_than_the_order_kernel_ranks():
    """Past 8192 sequences the call keeps index order (no ranking): thousands of tiny sequences, many of them empty."""
    rng = np.random.default_rng(7700)
    lens = tuple(int(n) for n in rng.integers(0, 4, size=8300))
    case = make(lens, 1, 7700)
    got, ref = run_gpu(case), run_oracle(case)
    check(got, ref, case[-1].numpy(), what="8300 sequences")
    dsT = case[7].numpy()
    empty = np.flatnonzero(np.asarray(lens) == 0)
    assert len(empty) > 1000 and all(np.array_equal(got[5][s], dsT[s]) for s in empty[:50])


@pytest.mark.parametrize("c2", [False, True])
def test_split_sequences_with_fast_decays(c2):
    """The split with chunks that take the token-by-token path inside the segments (the adjoint's summaries never do:
    their operand cannot overflow)."""
    case = make((2048, 300), 2, 7900, x_range=(-2.0, 1.5))
    got, ref = run_gpu(case, c2), run_oracle(case, c2)
    check(got, ref, case[-1].numpy(), c2, tol=4e-2, tol_dx=4e-2, what="split, fast decays")
