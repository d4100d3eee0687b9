"""GPU parity of the LayerNorm across all heads (gf_c2_layernorm, the normalisation of the o_t equation
of the Finch-C2 block) against the fp64 oracle, element by element: bf16 results within one bf16 rounding
of the oracle's value (plus the fp32 arithmetic error), fp32 results to 1e-5; relative L2 as for the other
kernels (5e-3 bf16, 1e-4 fp32)."""
import numpy as np
import pytest
import torch

import paper_2407_12077_b200 as gf
from oracle import wkv6_oracle as orc
from paper_2407_12077_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def draw(rows, H, N, dtype, seed, mean=0.3, std=2.0, affine=True):
    g = torch.Generator().manual_seed(seed)
    y = (torch.randn(rows, H, N, generator=g) * std + mean).to(dtype)
    gamma = (1 + 0.5 * torch.randn(H * N, generator=g)) if affine else None
    beta = (0.5 * torch.randn(H * N, generator=g)) if affine else None
    return y, gamma, beta


def compare(out, ref, dtype, what):
    out = out.float().cpu().numpy().astype(np.float64)
    err = np.abs(out - ref)
    if dtype == torch.bfloat16:
        bound = 2.0 ** -8 * np.abs(ref) + 1e-5           # half an ulp of bf16 is 2^-9 |ref|; the rest covers fp32 arithmetic
        tol = 5e-3
    else:
        bound = 1e-5 * np.abs(ref) + 1e-5
        tol = 1e-4
    bad = int((err > bound).sum())
    assert bad == 0, f"{what}: {bad} elements off, worst {err.max():.3e}"
    e = orc.rel_l2(out, ref)
    assert np.isfinite(e) and e <= tol, f"{what}: rel-L2 {e:.3e}"
    return e


def run(y, gamma, beta, eps=1e-5, in_place=False):
    d = y.to(DEV)
    out = gf.layernorm_heads(d, None if gamma is None else gamma.to(DEV), None if beta is None else beta.to(DEV), eps,
                             out=d if in_place else None)
    gf.last_device_status()
    return out


# widths that reach every (slices per lane, warps per row) variant of the kernel, full and ragged
WIDTHS = [(1, 8), (1, 64), (4, 64), (8, 64), (12, 64), (16, 64), (20, 64), (24, 64), (28, 64), (32, 64), (33, 64),
          (40, 64), (48, 64), (56, 64), (64, 64), (65, 64), (80, 64), (96, 64), (112, 64), (128, 64), (7, 24), (45, 8)]


@pytest.mark.parametrize("rows", [1, 3, 8, 1001])
@pytest.mark.parametrize("H,N", WIDTHS)
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_layernorm_matches_oracle_over_widths_and_ragged_row_counts(rows, H, N, dtype):
    y, gamma, beta = draw(rows, H, N, dtype, seed=rows * 1000 + H * N)
    ref = orc.layernorm_heads(y, gamma, beta, 1e-5)
    compare(run(y, gamma, beta), ref, dtype, f"rows {rows} H {H} N {N}")


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_no_affine_in_place_and_other_eps(dtype):
    y, _, _ = draw(37, 32, 64, dtype, seed=5, affine=False)
    ref = orc.layernorm_heads(y, None, None, 0.5)
    compare(run(y, None, None, eps=0.5, in_place=True), ref, dtype, "in place, eps 0.5")
    ref0 = orc.layernorm_heads(y, None, None, 0.0)
    compare(run(y, None, None, eps=0.0), ref0, dtype, "eps 0")


def test_rows_with_a_large_common_offset_and_constant_rows():
    # mean 200, spread 1: the variance must come from the deviations, not from E[y^2] - mean^2
    y, gamma, beta = draw(64, 32, 64, torch.float32, seed=6, mean=200.0, std=1.0)
    ref = orc.layernorm_heads(y, gamma, beta, 1e-5)
    out = run(y, gamma, beta).cpu().numpy().astype(np.float64)
    assert np.abs(out - ref).max() < 2e-4                     # fp32 carries y - mean to about 200 * 2^-24 / 1
    yc = torch.full((5, 32, 64), 3.75, dtype=torch.bfloat16)
    out = run(yc, gamma, beta, eps=1e-5)
    assert torch.equal(out.cpu(), beta.reshape(32, 64).bfloat16().expand(5, 32, 64))


def test_outputs_outside_the_rows_stay_untouched():
    y, gamma, beta = draw(10, 12, 64, torch.bfloat16, seed=7)
    d = y.to(DEV)
    buf = torch.full((12, 12, 64), 777.0, dtype=torch.bfloat16, device=DEV)
    gf.layernorm_heads(d, gamma.to(DEV), beta.to(DEV), 1e-5, out=buf[1:11])
    gf.last_device_status()
    assert torch.all(buf[0] == 777.0) and torch.all(buf[11] == 777.0)
    compare(buf[1:11], orc.layernorm_heads(y, gamma, beta, 1e-5), torch.bfloat16, "into a slice")


def test_finch_c2_prefill_followed_by_layernorm_matches_the_oracle_chain():
    """The o_t equation up to W^O: LayerNorm(concat_h(r_t . wkv_t + u'_t)), both steps on the GPU against both
    steps of the oracle in fp64."""
    B, T, H = 2, 333, 6
    inp = synth.make_dense(B, T, H, 64, "bf16", seed=77, state_std=0.1)
    g = torch.Generator().manual_seed(78)
    u2 = torch.randn(inp.r.shape, generator=g).bfloat16()
    gamma, beta = 1 + 0.3 * torch.randn(H * 64, generator=g), 0.2 * torch.randn(H * 64, generator=g)
    d = inp.to(DEV)
    y, _ = gf.prefill_c2(d.r, d.k, d.v, d.x, u2.to(DEV), d.state_in)
    o = gf.layernorm_heads(y, gamma.to(DEV), beta.to(DEV), 1e-5)
    gf.last_device_status()
    y_ref, _ = orc.prefill_c2(inp.r, inp.k, inp.v, inp.x, u2, inp.state_in)
    o_ref = orc.layernorm_heads(y_ref, gamma, beta, 1e-5)
    e = orc.rel_l2(o.float().cpu().numpy(), o_ref)
    assert e <= 5e-3, e


def test_full_size_token_count_of_the_prefill_benchmark():
    """65536 tokens x 2048 channels (the prefill benchmark's B*T and H*N), in the launch configuration
    the timing case uses; every row against the oracle."""
    c = synth.CONFIGS["cfg2"]
    rows, H = c["B"] * c["T"], c["H"]
    y, gamma, beta = draw(rows, H, 64, torch.bfloat16, seed=8)
    before = gf.launch_count()
    out = run(y, gamma, beta)
    assert gf.launch_count() - before == 1
    compare(out, orc.layernorm_heads(y, gamma, beta, 1e-5), torch.bfloat16, "65536 x 2048")
