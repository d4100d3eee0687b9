"""Pins of the oracle's decay logit d_t = lora_omega(ddlerp_d(x_t, x_{t-1})) (Finch-C2 section: the lerp, lora and
ddlerp operator definitions and the d_t equation).  Each test fixes the function against something other than
itself: end points and special cases of the operators that have closed forms, an exactly invertible outer lora that
exposes the inner ddlerp, a scalar loop written from the formulas with the standard library's tanh, the vectorised
library routines in fp64, a value worked out by hand, and the token-shift laws."""
import math

import numpy as np
import pytest

from oracle import wkv6_oracle as orc


def _weights(D, Rd, Rw, seed, scale=0.3):
    g = np.random.default_rng(seed)
    return dict(mu_x=g.uniform(0, 1, D), A_d=g.normal(0, scale, (D, Rd)), B_d=g.normal(0, scale, (Rd, D)),
                lambda_d=g.uniform(0, 1, D), A_w=g.normal(0, scale, (D, Rw)), B_w=g.normal(0, scale, (Rw, D)),
                lambda_w=g.normal(-3, 1, D))


def _call(x, w, x_prev=None):
    return orc.decay_logit(x, w["mu_x"], w["A_d"], w["B_d"], w["lambda_d"], w["A_w"], w["B_w"], w["lambda_w"], x_prev)


def _expose_inner(D, w):
    """An outer lora that can be undone exactly: A = B = identity, so d = lambda_w + tanh(m) and m = atanh(d - lambda_w)."""
    w = dict(w)
    w["A_w"], w["B_w"] = np.eye(D), np.eye(D)
    return w


def test_outer_lora_with_zero_A_is_lambda():
    D = 6
    w = _weights(D, 3, 4, 1)
    w["A_w"] = np.zeros_like(w["A_w"])
    x = np.random.default_rng(2).normal(size=(2, 5, D))
    assert np.allclose(_call(x, w), np.broadcast_to(w["lambda_w"], x.shape), rtol=0, atol=1e-15)


def test_ddlerp_end_points_and_plain_lerp():
    """With A_d = 0 the inner lora is the constant lambda_d, so ddlerp(a, b) = lerp(a, b, lambda_d): lambda_d = 0
    gives a = x_t, lambda_d = 1 gives b = x_{t-1}, and a general lambda_d the plain interpolation."""
    D = 5
    g = np.random.default_rng(3)
    x = g.uniform(-0.9, 0.9, (1, 4, D)) * 0.5          # |m| < 1 so that tanh can be undone accurately
    xp = g.uniform(-0.4, 0.4, (1, D))
    w = _expose_inner(D, _weights(D, 2, D, 4))
    w["A_d"] = np.zeros_like(w["A_d"])
    shifted = np.concatenate([xp[:, None], x[:, :-1]], axis=1)
    for lam, expect in ((np.zeros(D), x), (np.ones(D), shifted)):
        w["lambda_d"] = lam
        m = np.arctanh(_call(x, w, xp) - w["lambda_w"])
        assert np.allclose(m, expect, rtol=0, atol=1e-13)
    w["lambda_d"] = g.uniform(0, 1, D)
    m = np.arctanh(_call(x, w, xp) - w["lambda_w"])
    assert np.allclose(m, x + (shifted - x) * w["lambda_d"], rtol=0, atol=1e-13)


def test_inner_lora_sees_the_mu_x_interpolation():
    """B_d = 0 removes the data dependence again; with B_d != 0 the inner lora must be evaluated at
    a + (b - a) mu_x: mu_x = 0 and mu_x = 1 move its argument from x_t to x_{t-1}."""
    D, Rd = 4, 2
    g = np.random.default_rng(5)
    x = g.uniform(-0.3, 0.3, (1, 3, D))
    xp = g.uniform(-0.3, 0.3, (1, D))
    shifted = np.concatenate([xp[:, None], x[:, :-1]], axis=1)
    w = _expose_inner(D, _weights(D, Rd, D, 6, scale=0.5))
    for mu, arg in ((np.zeros(D), x), (np.ones(D), shifted)):
        w["mu_x"] = mu
        mix = w["lambda_d"] + np.tanh(arg @ w["A_d"]) @ w["B_d"]
        m = np.arctanh(_call(x, w, xp) - w["lambda_w"])
        assert np.allclose(m, x + (shifted - x) * mix, rtol=0, atol=1e-12)


def test_scalar_loops_from_the_formulas():
    """Every operator as nested Python loops with math.tanh, non-square ranks so that a transposed A or B cannot pass."""
    B, T, D, Rd, Rw = 2, 3, 5, 2, 3
    w = _weights(D, Rd, Rw, 7, scale=0.6)
    g = np.random.default_rng(8)
    x, xp = g.normal(size=(B, T, D)), g.normal(size=(B, D))
    d = _call(x, w, xp)

    def lora(vec, A, Bm, lam, R):
        h = [math.tanh(sum(vec[c] * A[c][q] for c in range(D))) for q in range(R)]
        return [lam[c] + sum(h[q] * Bm[q][c] for q in range(R)) for c in range(D)]

    for b in range(B):
        for t in range(T):
            a = x[b, t]
            prev = x[b, t - 1] if t > 0 else xp[b]
            inner = [a[c] + (prev[c] - a[c]) * w["mu_x"][c] for c in range(D)]
            mix = lora(inner, w["A_d"], w["B_d"], w["lambda_d"], Rd)
            m = [a[c] + (prev[c] - a[c]) * mix[c] for c in range(D)]
            ref = lora(m, w["A_w"], w["B_w"], w["lambda_w"], Rw)
            assert np.allclose(d[b, t], ref, rtol=1e-13, atol=1e-14)


def test_library_routines_in_fp64():
    B, T, D, Rd, Rw = 3, 17, 48, 8, 16
    w = _weights(D, Rd, Rw, 9, scale=0.2)
    g = np.random.default_rng(10)
    x, xp = g.normal(size=(B, T, D)), g.normal(size=(B, D))
    shifted = np.concatenate([xp[:, None], x[:, :-1]], axis=1)
    delta = shifted - x
    mix = w["lambda_d"] + np.tanh((x + delta * w["mu_x"]) @ w["A_d"]) @ w["B_d"]
    ref = w["lambda_w"] + np.tanh((x + delta * mix) @ w["A_w"]) @ w["B_w"]
    assert np.allclose(_call(x, w, xp), ref, rtol=1e-12, atol=1e-13)


def test_value_worked_out_by_hand():
    """D = 1, ranks 1: x_t = 1, x_{t-1} = 3, mu_x = 1/2 -> inner = 2; lora_d = 0 + tanh(2 * 1) * 1;
    mixed = 1 + 2 tanh 2; d = -3 + 2 tanh(mixed / 2).  tanh 2 = (e^4 - 1)/(e^4 + 1)."""
    th2 = (math.exp(4) - 1) / (math.exp(4) + 1)
    mixed = 1 + 2 * th2
    e = math.exp(mixed)                                  # tanh(mixed / 2) = (e^mixed - 1)/(e^mixed + 1)
    expect = -3 + 2 * (e - 1) / (e + 1)
    d = orc.decay_logit(np.array([[[1.0]]]), [0.5], [[1.0]], [[1.0]], [0.0], [[0.5]], [[2.0]], [-3.0], np.array([[3.0]]))
    assert d.shape == (1, 1, 1) and abs(d[0, 0, 0] - expect) < 1e-14


def test_token_shift_first_token_default_and_split():
    B, T, D = 2, 9, 6
    w = _weights(D, 2, 3, 11)
    g = np.random.default_rng(12)
    x = g.normal(size=(B, T, D))
    d0 = _call(x, w)                                                   # the token before the first one is zero
    assert np.array_equal(d0, _call(x, w, np.zeros((B, D))))
    # cutting the sequence and handing the last token over as x_prev changes nothing
    d_tail = _call(x[:, 4:], w, x[:, 3])
    assert np.array_equal(d0[:, 4:], d_tail)
    # a token's logit depends on itself and its predecessor only
    x2 = x.copy()
    x2[:, 6] += 1.0
    d2 = _call(x2, w)
    changed = np.any(d2 != d0, axis=(0, 2))
    assert list(np.nonzero(changed)[0]) == [6, 7]
    # batch entries are independent
    assert np.array_equal(_call(x[::-1].copy(), w), d0[::-1])


def test_the_logit_gives_a_decay_inside_the_unit_interval():
    D = 8
    w = _weights(D, 2, 3, 13)
    x = np.random.default_rng(14).normal(size=(1, 5, D))
    dec = np.exp(-np.exp(_call(x, w)))                                 # w_t = exp(-exp(d_t)) of the same block
    assert np.all((dec > 0) & (dec < 1))
