"""GPU parity of the GOLD key compression c_t = x_t W^{KD} (gf_gold_key_compress) against the fp64 oracle:
bf16 operands, fp32 accumulation, one bf16 rounding of the result.  Relative L2 <= 5e-3 as for the other bf16
kernels, and every element within one bf16 rounding of the oracle's value plus the fp32 accumulation error."""
import numpy as np
import pytest
import torch

import paper_2407_12077_b200 as gf
from oracle import wkv6_oracle as orc

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def draw(rows, D, Dc, seed):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(rows, D, generator=g).bfloat16()
    w = (torch.randn(D, Dc, generator=g) / D ** 0.5).bfloat16()
    return x, w


def compare(c, ref, what):
    out = c.float().cpu().numpy().astype(np.float64)
    scale = np.sqrt((ref ** 2).mean()) if ref.size else 1.0
    bound = 2.0 ** -8 * np.abs(ref) + 2e-5 * scale
    bad = int((np.abs(out - ref) > bound).sum())
    assert bad == 0, f"{what}: {bad} elements off, worst {np.abs(out - ref).max():.3e}"
    e = orc.rel_l2(out, ref)
    assert np.isfinite(e) and e <= 5e-3, f"{what}: rel-L2 {e:.3e}"


@pytest.mark.parametrize("rows", [1, 63, 64, 65, 255, 256, 257, 1000])
@pytest.mark.parametrize("D,Dc", [(64, 64), (128, 128), (768, 48), (1024, 64), (2048, 128), (3072, 192), (4096, 256), (200, 8), (1000, 136)])
def test_key_compress_matches_oracle(rows, D, Dc):
    x, w = draw(rows, D, Dc, seed=rows + D)
    canary = torch.full((rows + 2, Dc), 777.0, dtype=torch.bfloat16, device=DEV)
    before = gf.launch_count()
    gf.key_compress(x.to(DEV), w.to(DEV), out=canary[1:rows + 1])
    gf.last_device_status()
    assert gf.launch_count() - before == 1
    assert torch.all(canary[0] == 777.0) and torch.all(canary[rows + 1] == 777.0)      # nothing outside the rows
    compare(canary[1:rows + 1], orc.key_compress(x, w), f"rows {rows} D {D} Dc {Dc}")


def test_orientation_with_a_selection_matrix_is_exact():
    rows, D, Dc = 300, 2048, 128
    x, _ = draw(rows, D, Dc, seed=3)
    w = torch.zeros(D, Dc)
    w[16 * torch.arange(Dc), torch.arange(Dc)] = 1.0
    c = gf.key_compress(x.to(DEV), w.bfloat16().to(DEV))
    gf.last_device_status()
    assert torch.equal(c.cpu(), x[:, ::16])


@pytest.mark.parametrize("D,Dc", [(2048, 128), (3072, 192), (4096, 256), (768, 48)])
def test_more_row_tiles_than_sms_and_leading_dimensions(D, Dc):
    """[B, T, D] input with enough rows for several tiles per persistent CTA (40000 rows, 157 tiles of 256)."""
    B, T = 4, 10000
    g = torch.Generator().manual_seed(9)
    x = torch.randn(B, T, D, generator=g).bfloat16()
    w = (torch.randn(D, Dc, generator=g) / D ** 0.5).bfloat16()
    c = gf.key_compress(x.to(DEV), w.to(DEV))
    gf.last_device_status()
    assert c.shape == (B, T, Dc)
    idx = torch.randint(0, B * T, (600,), generator=g)
    idx = torch.cat([idx, torch.tensor([0, 255, 256, B * T - 1])])
    ref = orc.key_compress(x.reshape(B * T, D)[idx], w)
    compare(c.reshape(B * T, Dc)[idx.to(DEV)], ref, "40000 rows, sampled")


def test_benchmark_size_on_sampled_rows():
    """The launch the benchmark's key-compression row times (65536 tokens x 2048 -> 128: 256 row tiles over the persistent
    CTAs), rows sampled over the whole tensor plus the tile edges, every element of a row within one bf16 rounding."""
    rows, D, Dc = 65536, 2048, 128
    g = torch.Generator().manual_seed(19)
    x = torch.randn(rows, D, generator=g).bfloat16()
    w = (torch.randn(D, Dc, generator=g) / D ** 0.5).bfloat16()
    c = gf.key_compress(x.to(DEV), w.to(DEV))
    gf.last_device_status()
    idx = torch.randint(0, rows, (1500,), generator=g)
    idx = torch.cat([idx, torch.tensor([0, 255, 256, 257, 256 * 147, 256 * 148 - 1, 256 * 148, 256 * 255, rows - 1])])
    ref = orc.key_compress(x[idx], w)
    got = c[idx.to(DEV)].float().cpu().numpy()
    assert np.isfinite(c.float().cpu().numpy()).all()
    compare(c[idx.to(DEV)], ref, "65536 rows, sampled")
    assert (np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-3).all()
