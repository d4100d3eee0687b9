"""Pins of the oracle's LayerNorm across all heads (the normalisation of the o_t equation of the
Finch-C2 block) to facts that do not come from the oracle: closed forms, special rows, the library
LayerNorm in float64, laws the operator obeys, and the difference to the per-head norm it replaces."""
import numpy as np
import pytest
import torch

from oracle import wkv6_oracle as orc


def test_arithmetic_progression_closed_form():
    # y = 0, 1, ..., D-1: mean (D-1)/2, biased variance (D^2 - 1)/12
    for D in (2, 7, 64, 2048):
        y = np.arange(D, dtype=np.float64)[None]
        eps = 1e-5
        want = (y - (D - 1) / 2) / np.sqrt((D * D - 1) / 12 + eps)
        np.testing.assert_allclose(orc.layernorm_heads(y, eps=eps), want, rtol=1e-13, atol=1e-13)


def test_two_element_row_is_minus_one_plus_one_without_eps():
    out = orc.layernorm_heads(np.array([[3.0, 11.0], [5.0, -2.5]]), eps=0.0)
    np.testing.assert_allclose(out, [[-1.0, 1.0], [1.0, -1.0]], rtol=0, atol=1e-15)


def test_eps_sits_inside_the_square_root():
    # row (-1, +1): mean 0, variance 1 -> out = +-1/sqrt(1 + eps); eps = 3 gives exactly +-1/2
    out = orc.layernorm_heads(np.array([[-1.0, 1.0]]), eps=3.0)
    np.testing.assert_allclose(out, [[-0.5, 0.5]], rtol=0, atol=1e-15)


def test_constant_row_gives_beta():
    D = 96
    beta = np.linspace(-1, 1, D)
    out = orc.layernorm_heads(np.full((3, D), 7.25), gamma=np.full(D, 5.0), beta=beta, eps=1e-5)
    np.testing.assert_array_equal(out, np.broadcast_to(beta, (3, D)))


def test_matches_library_layernorm_in_float64():
    g = torch.Generator().manual_seed(11)
    for rows, H, N in ((5, 4, 64), (3, 32, 64), (17, 1, 8)):
        D = H * N
        y = torch.randn(rows, H, N, generator=g, dtype=torch.float64) * 3 + 0.7
        gamma = torch.randn(D, generator=g, dtype=torch.float64)
        beta = torch.randn(D, generator=g, dtype=torch.float64)
        want = torch.nn.functional.layer_norm(y.reshape(rows, D), (D,), gamma, beta, eps=1e-5).reshape(rows, H, N)
        got = orc.layernorm_heads(y, gamma, beta, eps=1e-5)
        np.testing.assert_allclose(got, want.numpy(), rtol=1e-12, atol=1e-12)


def test_output_moments_without_affine():
    rng = np.random.default_rng(5)
    y = rng.normal(2.0, 4.0, size=(9, 512))
    eps = 0.25
    out = orc.layernorm_heads(y, eps=eps)
    var = y.var(axis=1)                                     # biased, like the operator's
    np.testing.assert_allclose(out.mean(axis=1), 0.0, atol=1e-13)
    np.testing.assert_allclose(out.var(axis=1), var / (var + eps), rtol=1e-12)


def test_shift_and_scale_laws():
    rng = np.random.default_rng(6)
    y = rng.normal(size=(4, 256))
    base = orc.layernorm_heads(y, eps=1e-3)
    np.testing.assert_allclose(orc.layernorm_heads(y + 123.5, eps=1e-3), base, rtol=0, atol=1e-10)
    a = 7.0                                                 # LN(a y; a^2 eps) = LN(y; eps),  LN(-y) = -LN(y)
    np.testing.assert_allclose(orc.layernorm_heads(a * y, eps=a * a * 1e-3), base, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(orc.layernorm_heads(-y, eps=1e-3), -base, rtol=0, atol=1e-15)


def test_normalises_over_all_heads_not_per_head():
    # heads with different offsets: one group over D channels (the paper's choice) keeps the offsets
    # between heads, a per-head norm (Finch's GroupNorm, which the paper replaces) would erase them
    g = torch.Generator().manual_seed(12)
    rows, H, N = 6, 4, 16
    y = torch.randn(rows, H, N, generator=g, dtype=torch.float64) + torch.arange(H, dtype=torch.float64)[None, :, None] * 5
    got = orc.layernorm_heads(y, eps=1e-5)
    one_group = torch.nn.functional.group_norm(y.reshape(rows, H * N), 1, eps=1e-5).reshape(rows, H, N).numpy()
    per_head = torch.nn.functional.group_norm(y.reshape(rows, H * N), H, eps=1e-5).reshape(rows, H, N).numpy()
    np.testing.assert_allclose(got, one_group, rtol=1e-12, atol=1e-12)
    assert np.abs(got - per_head).max() > 0.5
    assert np.abs(got.mean(axis=2)).min() > 0.1            # head means survive
    np.testing.assert_allclose(got.reshape(rows, -1).mean(axis=1), 0.0, atol=1e-13)


def test_gamma_and_beta_are_indexed_by_channel_and_rows_are_independent():
    rng = np.random.default_rng(7)
    rows, D = 5, 40
    y = rng.normal(size=(rows, D))
    plain = orc.layernorm_heads(y, eps=1e-5)
    for c in (0, 13, D - 1):
        gamma = np.zeros(D)
        gamma[c] = 2.0
        beta = np.zeros(D)
        beta[(c + 1) % D] = -3.0
        out = orc.layernorm_heads(y, gamma, beta, eps=1e-5)
        want = np.zeros_like(y)
        want[:, c] = 2.0 * plain[:, c]
        want[:, (c + 1) % D] += -3.0
        np.testing.assert_allclose(out, want, rtol=0, atol=1e-15)
    perm = np.array([3, 0, 4, 1, 2])
    np.testing.assert_array_equal(orc.layernorm_heads(y[perm], eps=1e-5), plain[perm])
    # a row's result does not depend on the other rows
    np.testing.assert_array_equal(orc.layernorm_heads(y[2:3], eps=1e-5), plain[2:3])


def test_brute_force_python_loop_on_a_tiny_case():
    y = [[0.5, -1.25, 2.0], [4.0, 4.5, 3.0]]
    gamma, beta, eps = [1.5, -2.0, 0.25], [0.1, 0.2, -0.3], 0.01
    want = []
    for row in y:
        mu = sum(row) / 3
        var = sum((a - mu) ** 2 for a in row) / 3
        want.append([(a - mu) / (var + eps) ** 0.5 * g + b for a, g, b in zip(row, gamma, beta)])
    np.testing.assert_allclose(orc.layernorm_heads(np.array(y), np.array(gamma), np.array(beta), eps), want, rtol=1e-14)


def test_accepts_bf16_and_widens_exactly():
    g = torch.Generator().manual_seed(13)
    y = torch.randn(3, 2, 64, generator=g).bfloat16()
    np.testing.assert_array_equal(orc.layernorm_heads(y), orc.layernorm_heads(y.double().numpy()))
