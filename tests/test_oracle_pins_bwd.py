"""Pins of the oracle's gradient of the WKV recurrence (the adjoint of the wkv_t sum and the output r_t . wkv_t of
the Finch-C2 section, with the bonus term of the library's contract).  The forward oracle is pinned on its own
(test_oracle_pins.py); here its central finite differences in fp64 fix every gradient, and the structure of an
adjoint (linearity in the incoming gradients, split-and-carry through time, the one-token closed form) fixes the rest."""
import numpy as np
import pytest

from oracle import wkv6_oracle as orc


def _case(B, T, H, N, seed):
    g = np.random.default_rng(seed)
    f = lambda *s: g.normal(size=s).astype(np.float32)
    r, k, v = f(B, T, H, N), (f(B, T, H, N) * 0.5).astype(np.float32), f(B, T, H, N)
    x = g.uniform(-3, 0.5, (B, T, H, N)).astype(np.float32)
    u = (f(H, N) * 0.5).astype(np.float32)
    s0 = (f(B, H, N, N) * 0.3).astype(np.float32)
    dy = g.normal(size=(B, T, H, N))
    dsT = g.normal(size=(B, H, N, N))
    return r, k, v, x, u, s0, dy, dsT


def _loss(r, k, v, x, u, s0, dy, dsT):
    y, sT = orc.prefill(r, k, v, x, u, s0)
    return float((y * dy).sum() + (sT * dsT).sum())


@pytest.mark.parametrize("B,T,H,N,seed", [(1, 1, 1, 3, 0), (1, 4, 1, 4, 1), (2, 7, 2, 3, 2), (1, 8, 1, 5, 3)])
def test_central_differences_of_the_forward_oracle(B, T, H, N, seed):
    """L = <y, dy> + <S_T, dS_T> is linear in the outputs, so its gradient is the backward pass with those
    cotangents.  The inputs are float32 carriers: perturbations are powers of two that keep them exact."""
    r, k, v, x, u, s0, dy, dsT = _case(B, T, H, N, seed)
    dr, dk, dv, dx, du, ds0 = orc.backward(r, k, v, x, u, dy, s0, dsT)
    args = dict(r=r, k=k, v=v, x=x, u=u, s0=s0)
    grads = dict(r=dr, k=dk, v=dv, x=dx, u=du, s0=ds0)
    rng = np.random.default_rng(100 + seed)
    eps = 2.0 ** -10
    for name, arr in args.items():
        flat = arr.reshape(-1)
        for idx in rng.choice(flat.size, size=min(flat.size, 12), replace=False):
            # round the base value so that +-eps is exact in float32
            base = np.float32(np.round(flat[idx] / eps) * eps)
            plus, minus = dict(args), dict(args)
            for tgt, val in ((plus, base + np.float32(eps)), (minus, base - np.float32(eps))):
                a = arr.copy().reshape(-1)
                a[idx] = val
                tgt[name] = a.reshape(arr.shape)
            num = (_loss(dy=dy, dsT=dsT, **plus) - _loss(dy=dy, dsT=dsT, **minus)) / (2 * eps)
            # analytic gradient at the rounded base point
            mid = dict(args)
            a = arr.copy().reshape(-1)
            a[idx] = base
            mid[name] = a.reshape(arr.shape)
            g = dict(zip(("r", "k", "v", "x", "u", "s0"), orc.backward(mid["r"], mid["k"], mid["v"], mid["x"], mid["u"], dy, mid["s0"], dsT)))
            ana = g[name].reshape(-1)[idx]
            # central differences are exact for the (multi)linear inputs and O(eps^2) for x
            tol = 1e-9 if name != "x" else 2e-5
            assert abs(num - ana) <= tol * max(1.0, abs(ana)), (name, idx, num, ana)


def test_one_token_closed_form():
    """T = 1: y = r.(S_0 + diag(u) k^T v), S_1 = diag(w) S_0 + k^T v, so every gradient is a one-line expression."""
    N = 4
    r, k, v, x, u, s0, dy, dsT = _case(1, 1, 1, N, 5)
    dr, dk, dv, dx, du, ds0 = orc.backward(r, k, v, x, u, dy, s0, dsT)
    R, K, V, X, U = (a.reshape(N).astype(np.float64) for a in (r, k, v, x, u))
    S0, DY, G = s0.reshape(N, N).astype(np.float64), dy.reshape(N), dsT.reshape(N, N)
    w = np.exp(-np.exp(X))
    assert np.allclose(dr.reshape(N), S0 @ DY + U * K * (V @ DY), rtol=1e-13)
    assert np.allclose(dk.reshape(N), R * U * (V @ DY) + G @ V, rtol=1e-13)
    assert np.allclose(dv.reshape(N), (R * U * K).sum() * DY + K @ G, rtol=1e-13)
    assert np.allclose(dx.reshape(N), (G * S0).sum(axis=1) * (-w * np.exp(X)), rtol=1e-13)
    assert np.allclose(du.reshape(N), R * K * (V @ DY), rtol=1e-13)
    assert np.allclose(ds0.reshape(N, N), w[:, None] * G + np.outer(R, DY), rtol=1e-13)


def test_linear_in_the_incoming_gradients():
    r, k, v, x, u, s0, dy, dsT = _case(2, 6, 2, 4, 6)
    g = np.random.default_rng(7)
    dy2, dsT2 = g.normal(size=dy.shape), g.normal(size=dsT.shape)
    a, b = 0.75, -2.5
    g1 = orc.backward(r, k, v, x, u, dy, s0, dsT)
    g2 = orc.backward(r, k, v, x, u, dy2, s0, dsT2)
    g3 = orc.backward(r, k, v, x, u, a * dy + b * dy2, s0, a * dsT + b * dsT2)
    for p, q, s in zip(g1, g2, g3):
        assert np.allclose(s, a * p + b * q, rtol=1e-12, atol=1e-12)
    # no incoming gradient, no gradient; dS_T = None means zero
    z = orc.backward(r, k, v, x, u, np.zeros_like(dy), s0, None)
    assert all(np.count_nonzero(t) == 0 for t in z)
    assert all(np.array_equal(p, q) for p, q in zip(orc.backward(r, k, v, x, u, dy, s0, None),
                                                    orc.backward(r, k, v, x, u, dy, s0, np.zeros_like(dsT))))


@pytest.mark.parametrize("cut", [1, 3, 6])
def test_split_and_carry_of_the_adjoint(cut):
    """Backward over [0, T) = backward over [cut, T) from the forward state at the cut, then over [0, cut) with
    the state adjoint handed back; du adds up."""
    r, k, v, x, u, s0, dy, dsT = _case(1, 7, 2, 4, 8)
    full = orc.backward(r, k, v, x, u, dy, s0, dsT)
    _, s_cut = orc.prefill(r[:, :cut], k[:, :cut], v[:, :cut], x[:, :cut], u, s0)
    # the state at the cut as a float32 carrier would round it: keep the test exact by choosing it representable
    s_cut32 = s_cut.astype(np.float32)
    if not np.array_equal(s_cut32.astype(np.float64), s_cut):
        # compare against a full run that restarts from the rounded state instead
        tail = orc.backward(r[:, cut:], k[:, cut:], v[:, cut:], x[:, cut:], u, dy[:, cut:], s_cut32, dsT)
        head = orc.backward(r[:, :cut], k[:, :cut], v[:, :cut], x[:, :cut], u, dy[:, :cut], s0, tail[5])
        # tail gradients that read S_{t-1} see the rounded state: agreement to float32 rounding of the state
        tol = 1e-5
    else:
        tail = orc.backward(r[:, cut:], k[:, cut:], v[:, cut:], x[:, cut:], u, dy[:, cut:], s_cut32, dsT)
        head = orc.backward(r[:, :cut], k[:, :cut], v[:, :cut], x[:, :cut], u, dy[:, :cut], s0, tail[5])
        tol = 1e-12
    for i in range(4):
        assert np.allclose(np.concatenate([head[i], tail[i]], axis=1), full[i], rtol=tol, atol=tol)
    assert np.allclose(head[4] + tail[4], full[4], rtol=tol, atol=tol)
    assert np.allclose(head[5], full[5], rtol=tol, atol=tol)


def test_heads_and_batch_entries_are_independent_and_du_sums_over_the_batch():
    r, k, v, x, u, s0, dy, dsT = _case(2, 5, 2, 3, 9)
    full = orc.backward(r, k, v, x, u, dy, s0, dsT)
    du_sum = np.zeros_like(full[4])
    for b in range(2):
        one = orc.backward(r[b:b + 1], k[b:b + 1], v[b:b + 1], x[b:b + 1], u, dy[b:b + 1], s0[b:b + 1], dsT[b:b + 1])
        for i in (0, 1, 2, 3, 5):
            assert np.array_equal(one[i][0], full[i][b])
        du_sum += one[4]
    assert np.allclose(du_sum, full[4], rtol=1e-14)
    # bonus-free recurrence: u = 0 removes the bonus terms (the paper's own r_t . wkv_t form) and du's drivers stay
    z = orc.backward(r, k, v, x, np.zeros_like(u), dy, s0, dsT)
    assert np.allclose(z[4], full[4], rtol=1e-13)      # du does not depend on u


def test_against_reverse_mode_differentiation_of_the_definition_in_float64():
    """The recurrence written out token by token in torch (float64) and differentiated by the library's reverse mode:
    an independent route to every gradient at once (the oracle's adjoint recursion shares nothing with it)."""
    import torch
    B, T, H, N = 2, 9, 2, 5
    r, k, v, x, u, s0, dy, dsT = _case(B, T, H, N, 21)
    tr, tk, tv, tx, tu, ts0 = (torch.tensor(a.astype(np.float64), requires_grad=True) for a in (r, k, v, x, u, s0))
    S = ts0
    ys = []
    for t in range(T):
        w = torch.exp(-torch.exp(tx[:, t]))                                   # [B,H,N]
        kv = tk[:, t].unsqueeze(-1) * tv[:, t].unsqueeze(-2)                   # [B,H,N,N]
        ys.append(torch.einsum("bhi,bhij->bhj", tr[:, t], S + tu.unsqueeze(0).unsqueeze(-1) * kv))
        S = w.unsqueeze(-1) * S + kv
    y = torch.stack(ys, dim=1)
    loss = (y * torch.tensor(dy)).sum() + (S * torch.tensor(dsT)).sum()
    loss.backward()
    got = orc.backward(r, k, v, x, u, dy, s0, dsT)
    for name, a, b in zip(("dr", "dk", "dv", "dx", "du", "ds0"), got, (tr.grad, tk.grad, tv.grad, tx.grad, tu.grad, ts0.grad)):
        assert np.allclose(a, b.numpy(), rtol=1e-11, atol=1e-12), name
