"""Pins of the oracle's GOLD key compression c_t = x_t W^{KD} to facts that do not come from the oracle."""
import numpy as np
import torch

from oracle import wkv6_oracle as orc


def test_brute_force_loops_on_a_tiny_case():
    x = [[1.0, -2.0, 0.5], [0.25, 4.0, -1.0]]
    w = [[2.0, -1.0], [0.5, 3.0], [-4.0, 0.125]]
    want = [[sum(x[t][k] * w[k][n] for k in range(3)) for n in range(2)] for t in range(2)]
    np.testing.assert_allclose(orc.key_compress(np.array(x), np.array(w)), want, rtol=0, atol=1e-15)


def test_selection_matrix_picks_every_sixteenth_channel():
    rng = np.random.default_rng(1)
    D, Dc = 256, 16
    x = rng.normal(size=(7, D))
    w = np.zeros((D, Dc))
    w[16 * np.arange(Dc), np.arange(Dc)] = 1.0
    np.testing.assert_array_equal(orc.key_compress(x, w), x[:, ::16])


def test_all_ones_matrix_gives_row_sums():
    x = np.arange(5 * 64, dtype=np.float64).reshape(5, 64)       # integers: sums are exact
    out = orc.key_compress(x, np.ones((64, 4)))
    np.testing.assert_array_equal(out, np.repeat(x.sum(axis=1, keepdims=True), 4, axis=1))


def test_single_weight_fixes_the_orientation():
    rng = np.random.default_rng(2)
    D, Dc, k0, n0 = 48, 8, 37, 5
    x = rng.normal(size=(4, D))
    w = np.zeros((D, Dc))
    w[k0, n0] = 3.0
    want = np.zeros((4, Dc))
    want[:, n0] = 3.0 * x[:, k0]
    np.testing.assert_array_equal(orc.key_compress(x, w), want)


def test_linearity_and_leading_dimensions():
    rng = np.random.default_rng(3)
    x, y, w = rng.normal(size=(2, 3, 32)), rng.normal(size=(2, 3, 32)), rng.normal(size=(32, 2))
    lhs = orc.key_compress(2.0 * x - 0.5 * y, w)
    np.testing.assert_allclose(lhs, 2.0 * orc.key_compress(x, w) - 0.5 * orc.key_compress(y, w), rtol=1e-13, atol=1e-13)
    assert lhs.shape == (2, 3, 2)


def test_matches_the_library_matrix_product_in_float64():
    g = torch.Generator().manual_seed(4)
    x = torch.randn(33, 2048, generator=g, dtype=torch.float64)
    w = torch.randn(2048, 128, generator=g, dtype=torch.float64) / 45
    np.testing.assert_allclose(orc.key_compress(x, w), (x @ w).numpy(), rtol=1e-12, atol=1e-12)


def test_accepts_bf16_and_widens_exactly():
    g = torch.Generator().manual_seed(5)
    x = torch.randn(3, 64, generator=g).bfloat16()
    w = torch.randn(64, 4, generator=g).bfloat16()
    np.testing.assert_array_equal(orc.key_compress(x, w), orc.key_compress(x.double().numpy(), w.double().numpy()))
