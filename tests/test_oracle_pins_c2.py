"""Pins for the Finch-C2 form of the oracle (``prefill_c2``): the paper's Finch-C2 block multiplies the
key by one minus the decay of its own token, drops the bonus and adds the second-value vector u'_t to
r_t . wkv_t.  Each check compares with something the paper's equations or plain mathematics fix."""
import numpy as np
import pytest

from oracle import wkv6_oracle as orc


def rnd(shape, seed, scale=1.0):
    return (np.random.default_rng(seed).standard_normal(shape) * scale).astype(np.float32)


def make(B, T, H, N, seed):
    r, k, v = rnd((B, T, H, N), seed), rnd((B, T, H, N), seed + 1, 0.5), rnd((B, T, H, N), seed + 2)
    x = np.random.default_rng(seed + 3).uniform(-3.0, 0.5, (B, T, H, N)).astype(np.float32)
    u2 = rnd((B, T, H, N), seed + 4)
    s0 = rnd((B, H, N, N), seed + 5, 0.3)
    return r, k, v, x, u2, s0


def brute_force_c2(r, k, v, w, u2, s0):
    """The wkv_t sum of the Finch-C2 section written out term by term for one head, with the Finch-C2
    key k_i (1 - w_i), and o_t's per-head part r_t . wkv_t + u'_t.  r,k,v,w,u2: [T,N]; s0: [N,N]."""
    T, N = r.shape
    y = np.zeros((T, N))

    def wkv_at(t):                                # wkv_t, 1-based t; valid for t = 1 .. T+1
        acc = np.zeros((N, N))
        dec = np.ones(N)
        for j in range(1, t):
            dec = dec * w[j - 1]
        acc += dec[:, None] * s0                  # carried-in state: one more past term
        for i in range(1, t):
            dec = np.ones(N)
            for j in range(i + 1, t):
                dec = dec * w[j - 1]
            acc += dec[:, None] * np.outer(k[i - 1] * (1.0 - w[i - 1]), v[i - 1])
        return acc

    for t in range(1, T + 1):
        y[t - 1] = r[t - 1] @ wkv_at(t) + u2[t - 1]
    return y, wkv_at(T + 1)


@pytest.mark.parametrize("T", [1, 2, 5, 8])
def test_c2_brute_force_expansion(T):
    B, H, N = 1, 2, 4
    r, k, v, x, u2, s0 = make(B, T, H, N, 50 + T)
    y, s = orc.prefill_c2(r, k, v, x, u2, s0)
    w = np.exp(-np.exp(x.astype(np.float64)))
    for h in range(H):
        yb, sb = brute_force_c2(*(a[0, :, h].astype(np.float64) for a in (r, k, v)), w[0, :, h],
                                u2[0, :, h].astype(np.float64), s0[0, h].astype(np.float64))
        np.testing.assert_allclose(y[0, :, h], yb, rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(s[0, h], sb, rtol=1e-12, atol=1e-13)


def test_c2_reduces_to_the_bonus_free_recurrence_on_premultiplied_keys():
    """With keys k (1 - w) formed outside (exactly representable w) and u = 0 the classic recurrence, whose
    oracle is pinned separately, must give the same state and y - u2."""
    B, T, H, N = 2, 9, 2, 8
    r, k, v, _, u2, s0 = make(B, T, H, N, 70)
    w = np.random.default_rng(71).choice([0.0, 0.25, 0.5, 0.75, 1.0], size=(B, T, H, N))   # exact in binary
    k = np.round(k * 8) / 8                                                                   # k (1-w) exact in fp32
    kp = (k.astype(np.float64) * (1.0 - w)).astype(np.float32)
    y2, s2 = orc.prefill_c2(r, k, v, None, u2, s0, w=w)
    y1, s1 = orc.prefill(r, kp, v, None, np.zeros((H, N), np.float32), s0, w=w)
    np.testing.assert_allclose(y2 - u2, y1, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(s2, s1, rtol=1e-12, atol=1e-12)


def test_c2_w_one_freezes_the_state():
    """w == 1: keys are multiplied by 0 and nothing decays, so S_t = S_0 and y_t = r_t S_0 + u2_t."""
    B, T, H, N = 1, 6, 2, 4
    r, k, v, _, u2, s0 = make(B, T, H, N, 80)
    y, s = orc.prefill_c2(r, k, v, None, u2, s0, w=np.ones((B, T, H, N)))
    np.testing.assert_allclose(s, s0.astype(np.float64), rtol=0, atol=0)
    expect = np.einsum("bthi,bhij->bthj", r.astype(np.float64), s0.astype(np.float64)) + u2
    np.testing.assert_allclose(y, expect, rtol=1e-13, atol=1e-13)


def test_c2_w_zero_keeps_only_the_previous_token():
    """w == 0: the key passes unchanged and the state is forgotten every step: S_t = k_t^T v_t,
    y_t = r_t k_{t-1}^T v_{t-1} + u2_t (y_1 = u2_1 from a zero start)."""
    B, T, H, N = 1, 5, 1, 4
    r, k, v, _, u2, _ = make(B, T, H, N, 90)
    y, s = orc.prefill_c2(r, k, v, None, u2, None, w=np.zeros((B, T, H, N)))
    rd, kd, vd = (a[0, :, 0].astype(np.float64) for a in (r, k, v))
    np.testing.assert_allclose(y[0, 0, 0], u2[0, 0, 0], rtol=0, atol=0)
    for t in range(1, T):
        np.testing.assert_allclose(y[0, t, 0], (rd[t] @ kd[t - 1]) * vd[t - 1] + u2[0, t, 0], rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(s[0, 0], np.outer(kd[-1], vd[-1]), rtol=1e-13, atol=1e-13)


def test_c2_constant_half_decay_closed_form_and_split_carry():
    """x = ln ln 2 gives w = 1/2: S_T = 2^-T S_0 + sum_i 2^-(T-i) (k_i / 2)^T v_i; and splitting the
    sequence with the state handed over reproduces the unsplit run."""
    B, T, H, N = 1, 7, 1, 4
    r, k, v, _, u2, s0 = make(B, T, H, N, 95)
    x = np.full((B, T, H, N), np.log(np.log(2.0)), dtype=np.float64).astype(np.float32)
    y, s = orc.prefill_c2(r, k, v, x, u2, s0)
    w = float(np.exp(-np.exp(np.float64(x[0, 0, 0, 0]))))
    expect = w ** T * s0[0, 0].astype(np.float64)
    for i in range(1, T + 1):
        expect += w ** (T - i) * np.outer(k[0, i - 1, 0].astype(np.float64) * (1 - w), v[0, i - 1, 0].astype(np.float64))
    np.testing.assert_allclose(s[0, 0], expect, rtol=1e-12, atol=1e-13)
    for cut in (1, 3, 6):
        ya, sa = orc.prefill_c2(r[:, :cut], k[:, :cut], v[:, :cut], x[:, :cut], u2[:, :cut], s0)
        yb, sb = orc.prefill_c2(r[:, cut:], k[:, cut:], v[:, cut:], x[:, cut:], u2[:, cut:], sa.astype(np.float32))
        # the hand-over goes through float32, so allow its rounding
        np.testing.assert_allclose(np.concatenate([ya, yb], 1), y, rtol=1e-6, atol=1e-6)
        np.testing.assert_allclose(sb, s, rtol=1e-6, atol=1e-6)


def test_c2_without_second_value_is_y_minus_u2():
    B, T, H, N = 1, 4, 2, 4
    r, k, v, x, u2, s0 = make(B, T, H, N, 99)
    y0, s0_ = orc.prefill_c2(r, k, v, x, None, s0)
    y1, s1 = orc.prefill_c2(r, k, v, x, u2, s0)
    np.testing.assert_allclose(y1 - u2, y0, rtol=1e-13, atol=1e-13)
    np.testing.assert_array_equal(s0_, s1)
