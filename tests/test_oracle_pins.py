"""Pins for the fp64 CPU oracle: every check compares it with something fixed by the
paper's definition or by mathematics, never with the oracle's own formula retyped.

The wkv_t sum (Finch-C2 time-mixing section) is
    wkv_t = sum_{i=1}^{t-1} diag( prod_{j=i+1}^{t-1} w_j ) k_i^T v_i,
the output is r_t . wkv_t (plus classic Finch's diag(u) bonus on the current token),
and w_t = exp(-exp(x_t)).
"""
import json
import math
import os

import numpy as np
import pytest

from oracle import wkv6_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def rnd(shape, seed, scale=1.0):
    # float32-representable values so the float transport into the oracle is exact
    return (np.random.default_rng(seed).standard_normal(shape) * scale).astype(np.float32)


def make(B, T, H, N, seed, with_state=True):
    r = rnd((B, T, H, N), seed)
    k = rnd((B, T, H, N), seed + 1, 0.5)
    v = rnd((B, T, H, N), seed + 2)
    x = (np.random.default_rng(seed + 3).uniform(-3.0, 0.5, (B, T, H, N))).astype(np.float32)
    u = rnd((H, N), seed + 4, 0.5)
    s0 = rnd((B, H, N, N), seed + 5, 0.3) if with_state else None
    return r, k, v, x, u, s0


def brute_force(r, k, v, w, u, s0):
    """Literal expansion of the wkv_t sum for one head (double), products written out term by term.
    r,k,v,w: [T,N]; s0: [N,N].  The carried-in state is one more 'past' term decayed by every w so far."""
    T, N = r.shape
    y = np.zeros((T, N))
    for t in range(1, T + 1):                    # 1-based like the paper
        wkv = np.zeros((N, N))
        # initial state, decayed by w_1 .. w_{t-1}
        dec = np.ones(N)
        for j in range(1, t):
            dec = dec * w[j - 1]
        wkv += np.diag(dec) @ s0
        for i in range(1, t):                    # i = 1 .. t-1
            dec = np.ones(N)
            for j in range(i + 1, t):            # j = i+1 .. t-1 (empty for i = t-1)
                dec = dec * w[j - 1]
            wkv += np.diag(dec) @ np.outer(k[i - 1], v[i - 1])
        bonus = np.diag(u) @ np.outer(k[t - 1], v[t - 1])
        y[t - 1] = r[t - 1] @ (wkv + bonus)
    # final state = wkv_{T+1}
    S = np.zeros((N, N))
    dec = np.ones(N)
    for j in range(1, T + 1):
        dec = dec * w[j - 1]
    S += np.diag(dec) @ s0
    for i in range(1, T + 1):
        dec = np.ones(N)
        for j in range(i + 1, T + 1):
            dec = dec * w[j - 1]
        S += np.diag(dec) @ np.outer(k[i - 1], v[i - 1])
    return y, S


def test_hand_worked_example():
    g = json.load(open(os.path.join(GOLD, "wkv6_hand_example.json")))
    f = lambda a: np.asarray(a, dtype=np.float32)[None, :, None, :]       # [B=1,T,H=1,N]
    y, s = orc.prefill(f(g["r"]), f(g["k"]), f(g["v"]), None, np.asarray([g["u"]], np.float32),
                       np.asarray(g["state_in"], np.float32)[None, None],
                       w=np.asarray(g["w"], np.float64)[None, :, None, :])
    assert np.array_equal(y[0, :, 0, :], np.asarray(g["y"], np.float64))
    assert np.array_equal(s[0, 0], np.asarray(g["state_out"], np.float64))


@pytest.mark.parametrize("T", [1, 2, 3, 5, 8])
def test_brute_force_expansion_of_the_sum(T):
    B, H, N = 2, 3, 4
    r, k, v, x, u, s0 = make(B, T, H, N, seed=10 + T)
    y, s = orc.prefill(r, k, v, x, u, s0)
    w = np.exp(-np.exp(x.astype(np.float64)))
    for b in range(B):
        for h in range(H):
            yb, sb = brute_force(*(a[b, :, h].astype(np.float64) for a in (r, k, v)), w[b, :, h],
                                 u[h].astype(np.float64), s0[b, h].astype(np.float64))
            np.testing.assert_allclose(y[b, :, h], yb, rtol=1e-12, atol=1e-13)
            np.testing.assert_allclose(s[b, h], sb, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("via", ["w_direct", "x_minus_inf"])
def test_w_one_is_cumulative_sum_linear_attention(via):
    B, T, H, N = 1, 17, 2, 8
    r, k, v, x, u, s0 = make(B, T, H, N, seed=3)
    if via == "w_direct":
        y, s = orc.prefill(r, k, v, None, u, s0, w=np.ones(r.shape))
    else:
        y, s = orc.prefill(r, k, v, np.full(r.shape, -np.inf, np.float32), u, s0)
    r64, k64, v64 = (a.astype(np.float64) for a in (r, k, v))
    kv = np.einsum("bthi,bthj->bthij", k64, v64)
    csum = np.cumsum(kv, axis=1)                                   # inclusive sum of k_i^T v_i
    excl = csum - kv + s0.astype(np.float64)[:, None]              # S_0 + sum_{i<t}
    bonus = u.astype(np.float64)[None, None, :, :, None] * kv
    y_ref = np.einsum("bthi,bthij->bthj", r64, excl + bonus)
    np.testing.assert_allclose(y, y_ref, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(s, s0 + csum[:, -1], rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("via", ["w_direct", "x_plus_inf"])
def test_w_zero_keeps_only_bonus_and_previous_outer_product(via):
    B, T, H, N = 2, 9, 2, 8
    r, k, v, x, u, s0 = make(B, T, H, N, seed=5)
    if via == "w_direct":
        y, s = orc.prefill(r, k, v, None, u, s0, w=np.zeros(r.shape))
    else:
        y, s = orc.prefill(r, k, v, np.full(r.shape, np.inf, np.float32), u, s0)
    r64, k64, v64, u64 = (a.astype(np.float64) for a in (r, k, v, u))
    for t in range(T):
        prev = s0.astype(np.float64) if t == 0 else np.einsum("bhi,bhj->bhij", k64[:, t - 1], v64[:, t - 1])
        cur = u64[None, :, :, None] * np.einsum("bhi,bhj->bhij", k64[:, t], v64[:, t])
        np.testing.assert_allclose(y[:, t], np.einsum("bhi,bhij->bhj", r64[:, t], prev + cur),
                                   rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(s, np.einsum("bhi,bhj->bhij", k64[:, -1], v64[:, -1]), rtol=1e-13)


def test_constant_half_decay_geometric_closed_form():
    # x = ln(ln 2)  =>  exp(x) = ln 2  =>  w = 1/2 (up to the rounding of x to float32)
    B, T, H, N = 1, 12, 1, 6
    r, k, v, _, u, _ = make(B, T, H, N, seed=7, with_state=False)
    xval = np.float32(math.log(math.log(2.0)))
    w_exact = math.exp(-math.exp(float(xval)))
    assert abs(w_exact - 0.5) < 1e-7
    y, s = orc.prefill(r, k, v, np.full(r.shape, xval, np.float32), u, None)
    k64, v64 = k.astype(np.float64)[0, :, 0], v.astype(np.float64)[0, :, 0]
    S = sum(w_exact ** (T - i) * np.outer(k64[i - 1], v64[i - 1]) for i in range(1, T + 1))
    np.testing.assert_allclose(s[0, 0], S, rtol=1e-12, atol=1e-14)
    # and the weight w_t is not applied to the newest term when the output is formed
    t = 3
    wkv = sum(w_exact ** (t - 1 - i) * np.outer(k64[i - 1], v64[i - 1]) for i in range(1, t))
    y_ref = r.astype(np.float64)[0, t - 1, 0] @ (wkv + np.diag(u[0].astype(np.float64)) @ np.outer(k64[t - 1], v64[t - 1]))
    np.testing.assert_allclose(y[0, t - 1, 0], y_ref, rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("split", [1, 7, 19, 31])
def test_split_and_carry_equals_unsplit(split):
    B, T, H, N = 2, 32, 2, 8
    r, k, v, x, u, s0 = make(B, T, H, N, seed=11)
    y, s = orc.prefill(r, k, v, x, u, s0)
    y1, s1 = orc.prefill(r[:, :split], k[:, :split], v[:, :split], x[:, :split], u, s0)
    # the carried state must survive the float32 transport exactly for this identity: pass it as float64->float32 only if exact
    s1f = s1.astype(np.float32)
    y2, s2 = orc.prefill(r[:, split:], k[:, split:], v[:, split:], x[:, split:], u, s1f)
    # carried state was rounded to float32: the identity holds to float32 rounding of the state
    np.testing.assert_allclose(np.concatenate([y1, y2], 1), y, rtol=2e-6, atol=2e-6)
    np.testing.assert_allclose(s2, s, rtol=2e-6, atol=2e-6)
    assert np.array_equal(y1, y[:, :split])


def test_linearity_and_kv_rescaling():
    B, T, H, N = 1, 10, 2, 8
    r, k, v, x, u, s0 = make(B, T, H, N, seed=13)
    y, s = orc.prefill(r, k, v, x, u, s0)
    # y linear in r
    y2, s2 = orc.prefill(2 * r, k, v, x, u, s0)
    np.testing.assert_allclose(y2, 2 * y, rtol=1e-13)
    np.testing.assert_allclose(s2, s, rtol=0, atol=0)
    # (S_0, v) -> (a S_0, a v) scales y and S_T by a
    y3, s3 = orc.prefill(r, k, 4 * v, x, u, 4 * s0)
    np.testing.assert_allclose(y3, 4 * y, rtol=1e-13)
    np.testing.assert_allclose(s3, 4 * s, rtol=1e-13)
    # k -> 2k, v -> v/2 leaves everything unchanged when S_0 = 0 (powers of two: exact)
    ya, sa = orc.prefill(r, k, v, x, u, None)
    yb, sb = orc.prefill(r, 2 * k, v / 2, x, u, None)
    assert np.array_equal(ya, yb) and np.array_equal(sa, sb)


def test_heads_and_batches_are_independent():
    B, T, H, N = 3, 6, 4, 4
    r, k, v, x, u, s0 = make(B, T, H, N, seed=17)
    y, s = orc.prefill(r, k, v, x, u, s0)
    pb, ph = np.array([2, 0, 1]), np.array([3, 1, 0, 2])
    sel = lambda a: np.ascontiguousarray(a[pb][:, :, ph])
    y2, s2 = orc.prefill(sel(r), sel(k), sel(v), sel(x), np.ascontiguousarray(u[ph]),
                         np.ascontiguousarray(s0[pb][:, ph]))
    assert np.array_equal(y2, y[pb][:, :, ph])
    assert np.array_equal(s2, s[pb][:, ph])


def test_state_orientation_key_row_value_column():
    # S[i][j]: i is contracted with r and decayed by w[i]; j indexes the output
    N = 4
    s0 = np.zeros((1, 1, N, N), np.float32)
    s0[0, 0, 1, 2] = 3.0
    z = np.zeros((1, 2, 1, N), np.float32)
    r = z.copy()
    r[0, :, 0, 1] = 1.0                                           # r = e_1 on both steps
    w = np.ones((1, 2, 1, N))
    w[0, 0, 0, 1] = 0.5                                           # decays row 1
    w[0, 0, 0, 2] = 0.125                                         # must NOT touch entry (1,2)
    y, s = orc.prefill(r, z, z, None, np.zeros((1, N), np.float32), s0, w=w)
    assert np.array_equal(y[0, 0, 0], np.array([0, 0, 3.0, 0]))   # before any decay
    assert np.array_equal(y[0, 1, 0], np.array([0, 0, 1.5, 0]))   # row 1 decayed by w_1[1]
    assert s[0, 0, 1, 2] == 1.5 and np.count_nonzero(s) == 1


def test_zero_bonus_reduces_to_r_dot_wkv():
    B, T, H, N = 1, 7, 1, 4
    r, k, v, x, u, _ = make(B, T, H, N, seed=19, with_state=False)
    y, _ = orc.prefill(r, k, v, x, np.zeros_like(u), None)
    w = np.exp(-np.exp(x.astype(np.float64)))[0, :, 0]
    k64, v64, r64 = (a.astype(np.float64)[0, :, 0] for a in (k, v, r))
    for t in range(1, T + 1):
        wkv = np.zeros((N, N))
        for i in range(1, t):
            wkv += np.diag(np.prod(w[i:t - 1], axis=0)) @ np.outer(k64[i - 1], v64[i - 1])
        np.testing.assert_allclose(y[0, t - 1, 0], r64[t - 1] @ wkv, rtol=1e-12, atol=1e-14)


def test_bonus_scales_key_channel_of_current_token_only():
    # y_t(u) - y_t(0) = (sum_i r_t[i] u[i] k_t[i]) * v_t
    B, T, H, N = 1, 5, 2, 4
    r, k, v, x, u, s0 = make(B, T, H, N, seed=23)
    y1, s1 = orc.prefill(r, k, v, x, u, s0)
    y0, s00 = orc.prefill(r, k, v, x, np.zeros_like(u), s0)
    coef = np.einsum("bthi,hi,bthi->bth", r.astype(np.float64), u.astype(np.float64), k.astype(np.float64))
    np.testing.assert_allclose(y1 - y0, coef[..., None] * v.astype(np.float64), rtol=1e-10, atol=1e-12)
    assert np.array_equal(s1, s00)                                 # the bonus never enters the state


def test_varlen_equals_per_sequence_dense_and_handles_empty():
    H, N = 2, 4
    lens = [5, 0, 1, 9]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    total = int(cu[-1])
    r, k, v, x, u, _ = make(1, total, H, N, seed=29, with_state=False)
    r, k, v, x = (a[0] for a in (r, k, v, x))
    s0 = rnd((len(lens), H, N, N), 31, 0.3)
    y, s = orc.prefill_varlen(r, k, v, x, u, cu, s0)
    for i, L in enumerate(lens):
        a, b = cu[i], cu[i + 1]
        yd, sd = orc.prefill(r[None, a:b], k[None, a:b], v[None, a:b], x[None, a:b], u, s0[i:i + 1])
        assert np.array_equal(y[a:b], yd[0]) and np.array_equal(s[i], sd[0])
    assert np.array_equal(s[1], s0[1].astype(np.float64))          # empty sequence: state passes through


def test_step_is_prefill_of_length_one_and_chains():
    B, T, H, N = 2, 6, 2, 4
    r, k, v, x, u, s0 = make(B, T, H, N, seed=37)
    y, s = orc.prefill(r, k, v, x, u, s0)
    st = s0
    for t in range(T):
        yt, st64 = orc.step(r[:, t], k[:, t], v[:, t], x[:, t], u, st)
        np.testing.assert_allclose(yt, y[:, t], rtol=2e-6, atol=2e-6)
        st = st64.astype(np.float32)
    np.testing.assert_allclose(st, s, rtol=2e-6, atol=2e-6)


def test_bf16_inputs_are_widened_exactly():
    torch = pytest.importorskip("torch")
    g = torch.Generator().manual_seed(0)
    shp = (1, 4, 1, 4)
    r, k, v = (torch.randn(shp, generator=g).bfloat16() for _ in range(3))
    x = (torch.rand(shp, generator=g) * 5 - 6).bfloat16()
    u = torch.randn((1, 4), generator=g)
    y1, s1 = orc.prefill(r, k, v, x, u, None)
    y2, s2 = orc.prefill(r.float().numpy(), k.float().numpy(), v.float().numpy(), x.float().numpy(), u.numpy(), None)
    assert np.array_equal(y1, y2) and np.array_equal(s1, s2)
