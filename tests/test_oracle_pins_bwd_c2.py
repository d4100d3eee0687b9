"""Pins of the oracle's gradient of the Finch-C2 form of the recurrence (the layer the paper trains: keys times one
minus their decay, no bonus, second-value vector added to the output).  The forward oracle of this form is pinned on its
own (test_oracle_pins_c2.py); its central finite differences in fp64 fix every gradient here.  A second, independent
route: the gradient of the bonus-free classic recurrence on premultiplied keys (pinned in test_oracle_pins_bwd.py)
with the chain rule through k (1 - w) written out in numpy."""
import numpy as np
import pytest

from oracle import wkv6_oracle as orc


def _case(B, T, H, N, seed):
    g = np.random.default_rng(seed)
    f = lambda *s: g.normal(size=s).astype(np.float32)
    r, k, v = f(B, T, H, N), (f(B, T, H, N) * 0.5).astype(np.float32), f(B, T, H, N)
    x = g.uniform(-3, 0.5, (B, T, H, N)).astype(np.float32)
    s0 = (f(B, H, N, N) * 0.3).astype(np.float32)
    dy = g.normal(size=(B, T, H, N))
    dsT = g.normal(size=(B, H, N, N))
    return r, k, v, x, s0, dy, dsT


def _loss(r, k, v, x, s0, dy, dsT, u2=None):
    y, sT = orc.prefill_c2(r, k, v, x, u2, s0)
    return float((y * dy).sum() + (sT * dsT).sum())


@pytest.mark.parametrize("B,T,H,N,seed", [(1, 1, 1, 3, 0), (1, 4, 1, 4, 1), (2, 7, 2, 3, 2), (1, 8, 1, 5, 3)])
def test_central_differences_of_the_forward_oracle(B, T, H, N, seed):
    """L = <y, dy> + <S_T, dS_T>; perturbations are powers of two that keep the float32 carriers exact."""
    r, k, v, x, s0, dy, dsT = _case(B, T, H, N, seed)
    args = dict(r=r, k=k, v=v, x=x, s0=s0)
    rng = np.random.default_rng(100 + seed)
    eps = 2.0 ** -10
    for name, arr in args.items():
        flat = arr.reshape(-1)
        for idx in rng.choice(flat.size, size=min(flat.size, 12), replace=False):
            base = np.float32(np.round(flat[idx] / eps) * eps)
            pts = {}
            for tag, val in (("plus", base + np.float32(eps)), ("minus", base - np.float32(eps)), ("mid", base)):
                a = arr.copy().reshape(-1)
                a[idx] = val
                pts[tag] = dict(args)
                pts[tag][name] = a.reshape(arr.shape)
            num = (_loss(dy=dy, dsT=dsT, **pts["plus"]) - _loss(dy=dy, dsT=dsT, **pts["minus"])) / (2 * eps)
            m = pts["mid"]
            g = dict(zip(("r", "k", "v", "x", "s0"), orc.backward_c2(m["r"], m["k"], m["v"], m["x"], dy, m["s0"], dsT)))
            ana = g[name].reshape(-1)[idx]
            tol = 1e-9 if name != "x" else 2e-5          # exact for the multilinear inputs, O(eps^2) for x
            assert abs(num - ana) <= tol * max(1.0, abs(ana)), (name, idx, num, ana)


def test_reduces_to_the_classic_gradient_on_premultiplied_keys():
    """With w fixed, the C2 recurrence is the bonus-free classic one on k' = k (1 - w); x reaches the loss through w
    in the state decay (the classic dx) and through the key factor: dk = dk' (1 - w), dx = dx_classic + dk' k w e^x.
    The premultiplied key is not a float32 value, so it is fed through the decay-free entry (``w`` given) of the
    classic oracle only for the forward identity; the gradient identity is checked with keys chosen representable."""
    B, T, H, N = 2, 6, 2, 4
    r, k, v, x, s0, dy, dsT = _case(B, T, H, N, 11)
    # decays that are exact binary fractions, so that k (1 - w) is a float32 value: w in {1/2, 1/4, 3/4}
    g = np.random.default_rng(12)
    w = g.choice([0.5, 0.25, 0.75], size=x.shape)
    x = np.log(-np.log(w)).astype(np.float32)
    w32 = np.exp(-np.exp(x.astype(np.float64)))          # what the oracle sees (x rounded to float32)
    k = (np.round(k * 64) / 64).astype(np.float32)
    kp = (k.astype(np.float64) * (1.0 - w)).astype(np.float32)
    u0 = np.zeros((H, N), dtype=np.float32)
    dr, dk, dv, dx, ds0 = orc.backward_c2(r, k, v, x, dy, s0, dsT)
    cr, ckp, cv, cx, _, cs0 = orc.backward(r, kp, v, x, u0, dy, s0, dsT)
    # kp was formed with the exact w, the oracle uses w32: they differ by the rounding of x (1e-7 relative)
    tol = 5e-6
    assert np.allclose(dr, cr, rtol=tol, atol=tol) and np.allclose(dv, cv, rtol=tol, atol=tol)
    assert np.allclose(ds0, cs0, rtol=tol, atol=tol)
    assert np.allclose(dk, ckp * (1.0 - w32), rtol=tol, atol=tol)
    assert np.allclose(dx, cx + ckp * k * w32 * np.exp(x.astype(np.float64)), rtol=tol, atol=tol)


def test_one_token_closed_form():
    """T = 1: y = r . S_0 + u2, S_1 = diag(w) S_0 + (k (1 - w))^T v."""
    N = 4
    r, k, v, x, s0, dy, dsT = _case(1, 1, 1, N, 5)
    dr, dk, dv, dx, ds0 = orc.backward_c2(r, k, v, x, dy, s0, dsT)
    R, K, V, X = (a.reshape(N).astype(np.float64) for a in (r, k, v, x))
    S0, DY, G = s0.reshape(N, N).astype(np.float64), dy.reshape(N), dsT.reshape(N, N)
    w = np.exp(-np.exp(X))
    assert np.allclose(dr.reshape(N), S0 @ DY, rtol=1e-13)
    assert np.allclose(dk.reshape(N), (G @ V) * (1 - w), rtol=1e-13)
    assert np.allclose(dv.reshape(N), (K * (1 - w)) @ G, rtol=1e-13)
    assert np.allclose(dx.reshape(N), ((G * S0).sum(axis=1) - (G @ V) * K) * (-w * np.exp(X)), rtol=1e-13)
    assert np.allclose(ds0.reshape(N, N), w[:, None] * G + np.outer(R, DY), rtol=1e-13)


def test_linear_in_the_incoming_gradients_and_blind_to_the_second_value():
    r, k, v, x, s0, dy, dsT = _case(2, 6, 2, 4, 6)
    g = np.random.default_rng(7)
    dy2, dsT2 = g.normal(size=dy.shape), g.normal(size=dsT.shape)
    a, b = 0.75, -2.5
    g1 = orc.backward_c2(r, k, v, x, dy, s0, dsT)
    g2 = orc.backward_c2(r, k, v, x, dy2, s0, dsT2)
    g3 = orc.backward_c2(r, k, v, x, a * dy + b * dy2, s0, a * dsT + b * dsT2)
    for p, q, s in zip(g1, g2, g3):
        assert np.allclose(s, a * p + b * q, rtol=1e-12, atol=1e-12)
    z = orc.backward_c2(r, k, v, x, np.zeros_like(dy), s0, None)
    assert all(np.count_nonzero(t) == 0 for t in z)
    # u2 only adds to y: the loss is linear in it with gradient dy, and no other gradient depends on it
    u2 = g.normal(size=dy.shape).astype(np.float32)
    assert np.isclose(_loss(r, k, v, x, s0, dy, dsT, u2) - _loss(r, k, v, x, s0, dy, dsT), float((u2 * dy).sum()), rtol=1e-10)


@pytest.mark.parametrize("cut", [1, 3, 6])
def test_split_and_carry_of_the_adjoint(cut):
    r, k, v, x, s0, dy, dsT = _case(1, 7, 2, 4, 8)
    full = orc.backward_c2(r, k, v, x, dy, s0, dsT)
    _, s_cut = orc.prefill_c2(r[:, :cut], k[:, :cut], v[:, :cut], x[:, :cut], None, s0)
    s_cut32 = s_cut.astype(np.float32)                   # the carrier rounds the state at the cut: float32 agreement
    tail = orc.backward_c2(r[:, cut:], k[:, cut:], v[:, cut:], x[:, cut:], dy[:, cut:], s_cut32, dsT)
    head = orc.backward_c2(r[:, :cut], k[:, :cut], v[:, :cut], x[:, :cut], dy[:, :cut], s0, tail[4])
    tol = 1e-5
    for i in range(4):
        assert np.allclose(np.concatenate([head[i], tail[i]], axis=1), full[i], rtol=tol, atol=tol)
    assert np.allclose(head[4], full[4], rtol=tol, atol=tol)


def test_a_planted_mistake_fails():
    """The key factor's own dependence on x is the term a hasty derivation drops: without it the central differences
    of x disagree (checked on the formula in numpy, the oracle itself is not altered)."""
    N = 4
    r, k, v, x, s0, dy, dsT = _case(1, 1, 1, N, 5)
    _, _, _, dx, _ = orc.backward_c2(r, k, v, x, dy, s0, dsT)
    K, V, X = (a.reshape(N).astype(np.float64) for a in (k, v, x))
    S0, G = s0.reshape(N, N).astype(np.float64), dsT.reshape(N, N)
    w = np.exp(-np.exp(X))
    wrong = (G * S0).sum(axis=1) * (-w * np.exp(X))      # the classic dx: forgets that k (1 - w) depends on x
    assert not np.allclose(dx.reshape(N), wrong, rtol=1e-3)


def test_against_reverse_mode_differentiation_of_the_definition_in_float64():
    """The Finch-C2 recurrence written out token by token in torch (float64) and differentiated by the library's
    reverse mode; the second-value vector's gradient comes out as dy."""
    import torch
    B, T, H, N = 2, 9, 2, 5
    r, k, v, x, s0, dy, dsT = _case(B, T, H, N, 22)
    u2 = np.random.default_rng(23).normal(size=dy.shape).astype(np.float32)
    tr, tk, tv, tx, ts0, tu2 = (torch.tensor(a.astype(np.float64), requires_grad=True) for a in (r, k, v, x, s0, u2))
    S = ts0
    ys = []
    for t in range(T):
        w = torch.exp(-torch.exp(tx[:, t]))
        ys.append(torch.einsum("bhi,bhij->bhj", tr[:, t], S) + tu2[:, t])
        S = w.unsqueeze(-1) * S + (tk[:, t] * (1 - w)).unsqueeze(-1) * tv[:, t].unsqueeze(-2)
    y = torch.stack(ys, dim=1)
    loss = (y * torch.tensor(dy)).sum() + (S * torch.tensor(dsT)).sum()
    loss.backward()
    got = orc.backward_c2(r, k, v, x, dy, s0, dsT)
    for name, a, b in zip(("dr", "dk", "dv", "dx", "ds0"), got, (tr.grad, tk.grad, tv.grad, tx.grad, ts0.grad)):
        assert np.allclose(a, b.numpy(), rtol=1e-11, atol=1e-12), name
    assert np.allclose(tu2.grad.numpy(), dy, rtol=0, atol=0)
