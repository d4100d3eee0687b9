"""Pins of the oracle's gradients over a packed (cu_seqlens) batch, classic and Finch-C2 form.  What fixes them: the
recurrence never crosses a sequence boundary, so (a) every sequence's rows carry the dense gradient of that sequence
alone (the dense gradients are pinned by finite differences and reverse-mode differentiation in test_oracle_pins_bwd*.py),
(b) central differences of the pinned packed forward oracle, whose loss couples nothing across sequences, (c) two
neighbouring sequences chained through their states equal one sequence of both, (d) a token of one sequence has no
influence on another sequence's loss."""
import numpy as np
import pytest

from oracle import wkv6_oracle as orc


def _case(lens, H, N, seed):
    g = np.random.default_rng(seed)
    T, S = int(sum(lens)), len(lens)
    f = lambda *s: g.normal(size=s).astype(np.float32)
    r, k, v = f(T, H, N), (f(T, H, N) * 0.5).astype(np.float32), f(T, H, N)
    x = g.uniform(-3, 0.5, (T, H, N)).astype(np.float32)
    u = (f(H, N) * 0.5).astype(np.float32)
    s0 = (f(S, H, N, N) * 0.3).astype(np.float32)
    dy = g.normal(size=(T, H, N))
    dsT = g.normal(size=(S, H, N, N))
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    return r, k, v, x, u, s0, dy, dsT, cu


LENS = [(3, 0, 5, 1), (1,), (0, 4), (2, 2, 2), (7, 0)]


@pytest.mark.parametrize("lens", LENS)
def test_each_sequence_carries_its_own_dense_gradient(lens):
    H, N = 2, 4
    r, k, v, x, u, s0, dy, dsT, cu = _case(lens, H, N, 31)
    dr, dk, dv, dx, du, ds0 = orc.backward_varlen(r, k, v, x, u, dy, cu, s0, dsT)
    cr, ckk, cv, cx, cs0 = orc.backward_c2_varlen(r, k, v, x, dy, cu, s0, dsT)
    du_sum = np.zeros((H, N))
    for s, n in enumerate(lens):
        a, b = int(cu[s]), int(cu[s + 1])
        sl = lambda t: t[a:b][None]
        if n == 0:
            # no token: the state's gradient passes through, nothing else exists
            assert np.array_equal(ds0[s], dsT[s]) and np.array_equal(cs0[s], dsT[s])
            continue
        one = orc.backward(sl(r), sl(k), sl(v), sl(x), u, sl(dy), s0[s][None], dsT[s][None])
        for got, ref in zip((dr, dk, dv, dx), one[:4]):
            assert np.array_equal(got[a:b], ref[0])
        du_sum += one[4]
        assert np.array_equal(ds0[s], one[5][0])
        two = orc.backward_c2(sl(r), sl(k), sl(v), sl(x), sl(dy), s0[s][None], dsT[s][None])
        for got, ref in zip((cr, ckk, cv, cx), two[:4]):
            assert np.array_equal(got[a:b], ref[0])
        assert np.array_equal(cs0[s], two[4][0])
    assert np.allclose(du, du_sum, rtol=1e-14, atol=1e-14)


def _loss(form, r, k, v, x, u, s0, dy, dsT, cu):
    if form == "classic":
        y, sT = orc.prefill_varlen(r, k, v, x, u, cu, s0)
        return float((y * dy).sum() + (sT * dsT).sum())
    # the packed Finch-C2 forward, sequence by sequence through the dense oracle of that form (pinned on its own)
    tot = 0.0
    for s in range(len(cu) - 1):
        a, b = int(cu[s]), int(cu[s + 1])
        if a == b:
            tot += float((s0[s].astype(np.float64) * dsT[s]).sum())
            continue
        y, sT = orc.prefill_c2(r[a:b][None], k[a:b][None], v[a:b][None], x[a:b][None], None, s0[s][None])
        tot += float((y[0] * dy[a:b]).sum() + (sT[0] * dsT[s]).sum())
    return tot


@pytest.mark.parametrize("form", ["classic", "c2"])
def test_central_differences_of_the_packed_forward(form):
    """L = <y, dy> + <S_T, dS_T> over a packed batch; perturbations are powers of two that keep the float32 carriers exact."""
    lens, H, N = (3, 0, 4, 1), 2, 3
    r, k, v, x, u, s0, dy, dsT, cu = _case(lens, H, N, 41)
    args = dict(r=r, k=k, v=v, x=x, s0=s0)
    if form == "classic":
        args["u"] = u
    rng = np.random.default_rng(42)
    eps = 2.0 ** -10
    for name, arr in args.items():
        flat = arr.reshape(-1)
        for idx in rng.choice(flat.size, size=min(flat.size, 10), replace=False):
            base = np.float32(np.round(flat[idx] / eps) * eps)
            pts = {}
            for tag, val in (("plus", base + np.float32(eps)), ("minus", base - np.float32(eps)), ("mid", base)):
                a = arr.copy().reshape(-1)
                a[idx] = val
                pts[tag] = dict(args, u=args.get("u", u))
                pts[tag][name] = a.reshape(arr.shape)
            num = (_loss(form, dy=dy, dsT=dsT, cu=cu, **pts["plus"]) - _loss(form, dy=dy, dsT=dsT, cu=cu, **pts["minus"])) / (2 * eps)
            m = pts["mid"]
            if form == "classic":
                g = dict(zip(("r", "k", "v", "x", "u", "s0"),
                             orc.backward_varlen(m["r"], m["k"], m["v"], m["x"], m["u"], dy, cu, m["s0"], dsT)))
            else:
                g = dict(zip(("r", "k", "v", "x", "s0"),
                             orc.backward_c2_varlen(m["r"], m["k"], m["v"], m["x"], dy, cu, m["s0"], dsT)))
            ana = g[name].reshape(-1)[idx]
            tol = 1e-9 if name != "x" else 2e-5          # exact for the multilinear inputs, O(eps^2) for x
            assert abs(num - ana) <= tol * max(1.0, abs(ana)), (form, name, idx, num, ana)


@pytest.mark.parametrize("form", ["classic", "c2"])
def test_two_chained_sequences_are_one(form):
    """Sequence 1 started from sequence 0's final state (rounded to the float32 carrier) and its state gradient fed
    back: the packed gradients of both equal the gradient of the one sequence of all the rows."""
    H, N, n0, n1 = 2, 4, 3, 4
    r, k, v, x, u, s0, dy, dsT, cu = _case((n0, n1), H, N, 51)
    D = lambda t: t[None]
    if form == "classic":
        full = orc.backward(D(r), D(k), D(v), D(x), u, D(dy), s0[:1], dsT[1:])
        _, mid = orc.prefill(D(r[:n0]), D(k[:n0]), D(v[:n0]), D(x[:n0]), u, s0[:1])
    else:
        full = orc.backward_c2(D(r), D(k), D(v), D(x), D(dy), s0[:1], dsT[1:])
        _, mid = orc.prefill_c2(D(r[:n0]), D(k[:n0]), D(v[:n0]), D(x[:n0]), None, s0[:1])
    st = np.concatenate([s0[:1], mid.astype(np.float32)])
    # first the tail alone (its start-state gradient is what the head receives), then both in one packed call
    cu_tail = np.array([0, n1], dtype=np.int32)
    if form == "classic":
        tail = orc.backward_varlen(r[n0:], k[n0:], v[n0:], x[n0:], u, dy[n0:], cu_tail, st[1:], dsT[1:])
        both = orc.backward_varlen(r, k, v, x, u, dy, cu, st, np.concatenate([tail[5], dsT[1:]]))
    else:
        tail = orc.backward_c2_varlen(r[n0:], k[n0:], v[n0:], x[n0:], dy[n0:], cu_tail, st[1:], dsT[1:])
        both = orc.backward_c2_varlen(r, k, v, x, dy, cu, st, np.concatenate([tail[4], dsT[1:]]))
    tol = 1e-5                                            # the carrier rounds the state at the cut
    for i in range(4):
        assert np.allclose(both[i], full[i][0], rtol=tol, atol=tol)
    if form == "classic":
        assert np.allclose(both[4], full[4], rtol=tol, atol=tol)
        assert np.allclose(both[5][0], full[5][0], rtol=tol, atol=tol)
    else:
        assert np.allclose(both[4][0], full[4][0], rtol=tol, atol=tol)


def test_no_gradient_crosses_a_sequence_boundary():
    """Only sequence 1 has a loss: every gradient of the other sequences' rows and states is zero, exactly."""
    lens, H, N = (3, 4, 2), 2, 4
    r, k, v, x, u, s0, dy, dsT, cu = _case(lens, H, N, 61)
    a, b = int(cu[1]), int(cu[2])
    dy0 = np.zeros_like(dy)
    dy0[a:b] = dy[a:b]
    ds = np.zeros_like(dsT)
    ds[1] = dsT[1]
    for out in (orc.backward_varlen(r, k, v, x, u, dy0, cu, s0, ds), orc.backward_c2_varlen(r, k, v, x, dy0, cu, s0, ds)):
        for t in out[:4]:
            assert np.count_nonzero(t[:a]) == 0 and np.count_nonzero(t[b:]) == 0 and np.count_nonzero(t[a:b]) > 0
        ds0 = out[-1]
        assert np.count_nonzero(ds0[0]) == 0 and np.count_nonzero(ds0[2]) == 0 and np.count_nonzero(ds0[1]) > 0


def test_a_planted_mistake_fails():
    """An off-by-one in the row range of a sequence (rows taken from cu[s] + 1) changes every gradient of that
    sequence: the per-sequence comparison above would see it.  Planted here by shifting the packed inputs by hand."""
    lens, H, N = (3, 4), 1, 3
    r, k, v, x, u, s0, dy, dsT, cu = _case(lens, H, N, 71)
    good = orc.backward_varlen(r, k, v, x, u, dy, cu, s0, dsT)
    cu_bad = np.array([0, 4, 7], dtype=np.int32)          # boundary moved by one row
    bad = orc.backward_varlen(r, k, v, x, u, dy, cu_bad, s0, dsT)
    assert not np.allclose(good[0], bad[0], rtol=1e-3, atol=1e-6)
