"""Seeded random shapes for the gradient calls (dense and packed, classic and Finch-C2 form, every decay range, with
and without states), two properties each:
  * the bf16 chunked gradient agrees with the fp64 oracle within the tolerances of test_gpu_parity_bwd_bf16.py
    (a little wider for the decay-logit gradient and for fast decays, where chunks take the token-by-token path);
  * the training pair (forward pass that keeps its chunk-start states + gradient from them) agrees bit for bit with
    the separate calls whenever the gradient call does not split its sequences.
The second property is what exposes a race: both sides run the same arithmetic, only their timing differs."""
import numpy as np
import pytest
import torch

import paper_2407_12077_b200 as gf
from oracle import wkv6_oracle as orc
from paper_2407_12077_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
RANGES = [(-6.0, -1.0), (-8.0, -4.0), (-3.0, 0.5), (-12.0, -8.0), (-2.0, 1.5)]


def _rel(a, b):
    a, b = a.double(), b.double()
    d = b.norm().item()
    return (a - b).norm().item() / d if d > 0 else a.norm().item()


def _packed_case(rng, H, lo, hi, std):
    S = int(rng.integers(1, 7))
    lens = [int(rng.integers(0, 500)) for _ in range(S)]
    if sum(lens) == 0:
        lens[0] = 5
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32)
    inp = synth.make_varlen(cu, H, 64, "bf16", seed=int(rng.integers(0, 1 << 30)), device=DEV, state_std=std, x_lo=lo, x_hi=hi)
    return lens, cu, inp


@pytest.mark.parametrize("seed", [101, 102, 103])
def test_chunked_gradient_against_the_oracle(seed):
    rng = np.random.default_rng(seed)
    g = torch.Generator().manual_seed(seed)
    for case in range(30):
        packed, c2 = rng.random() < 0.5, rng.random() < 0.4
        H = int(rng.integers(1, 6))
        lo, hi = RANGES[int(rng.integers(0, len(RANGES)))]
        std = 0.0 if rng.random() < 0.3 else 0.2
        with_d = rng.random() < 0.7
        fast = hi > 0
        dev = lambda t: None if t is None else t.to(DEV)
        if packed:
            S = int(rng.integers(1, 7))
            lens = [int(rng.integers(0, 500)) for _ in range(S)]
            if sum(lens) == 0:
                lens[0] = 5
            cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32)
            inp = synth.make_varlen(cu, H, 64, "bf16", seed=int(rng.integers(0, 1 << 30)), state_std=std, x_lo=lo, x_hi=hi)
            tot = sum(lens)
            dy = torch.randn((tot, H, 64), generator=g).bfloat16()
            dsT = torch.randn((S, H, 64, 64), generator=g) * 0.1 if with_d else None
            out = gf.backward_varlen(dev(inp.r), dev(inp.k), dev(inp.v), dev(inp.x), dev(inp.u), dev(dy), dev(cu), max(lens),
                                     dev(inp.state_in), dev(dsT), c2=c2)
            dyn, dsn = dy.double().numpy(), None if dsT is None else dsT.double().numpy()
            if c2:
                r = orc.backward_c2_varlen(inp.r, inp.k, inp.v, inp.x, dyn, cu, inp.state_in, dsn)
                ref = [r[0], r[1], r[2], r[3], None, r[4]]
            else:
                ref = list(orc.backward_varlen(inp.r, inp.k, inp.v, inp.x, inp.u, dyn, cu, inp.state_in, dsn))
            few = tot < 64
            what = ("packed", lens, H, c2, (lo, hi))
        else:
            B, T = int(rng.integers(1, 5)), int(rng.integers(1, 700))
            inp = synth.make_dense(B, T, H, 64, "bf16", seed=int(rng.integers(0, 1 << 30)), state_std=std, x_lo=lo, x_hi=hi)
            dy = torch.randn(inp.r.shape, generator=g).bfloat16()
            dsT = torch.randn((B, H, 64, 64), generator=g) * 0.1 if with_d else None
            dyn, dsn = dy.double().numpy(), None if dsT is None else dsT.double().numpy()
            if c2:
                o = gf.backward_c2(dev(inp.r), dev(inp.k), dev(inp.v), dev(inp.x), dev(dy), dev(inp.state_in), dev(dsT))
                out = [o[0], o[1], o[2], o[3], None, o[4]]
                r = orc.backward_c2(inp.r, inp.k, inp.v, inp.x, dyn, inp.state_in, dsn)
                ref = [r[0], r[1], r[2], r[3], None, r[4]]
            else:
                out = gf.backward(dev(inp.r), dev(inp.k), dev(inp.v), dev(inp.x), dev(inp.u), dev(dy), dev(inp.state_in), dev(dsT))
                ref = list(orc.backward(inp.r, inp.k, inp.v, inp.x, inp.u, dyn, inp.state_in, dsn))
            few = T < 64
            what = ("dense", B, T, H, c2, (lo, hi))
        gf.last_device_status()
        for i, (a, b) in enumerate(zip(out, ref)):
            if a is None:
                continue
            a = a.float().cpu().numpy().astype(np.float64)
            assert np.isfinite(a).all(), (what, i)
            lim = 4e-2 if fast else (1e-2 if i == 3 else 6e-3)
            if few:                     # a handful of rounded numbers: heavy-tailed ratio
                lim = max(lim, 3e-2)
            assert orc.rel_l2(a, b) <= lim, (what, i, orc.rel_l2(a, b))


@pytest.mark.parametrize("seed", [201, 202, 203])
def test_training_pair_against_the_separate_calls(seed):
    rng = np.random.default_rng(seed)
    g = torch.Generator(device=DEV).manual_seed(seed)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    for case in range(40):
        packed, c2 = rng.random() < 0.5, rng.random() < 0.5
        H = int(rng.integers(1, 9))
        lo, hi = RANGES[int(rng.integers(0, len(RANGES)))]
        if packed:
            lens, cu, inp = _packed_case(rng, H, lo, hi, 0.2)
            tot, S, mx = sum(lens), len(lens), max(lens)
            dy = torch.randn((tot, H, 64), device=DEV, generator=g).bfloat16()
            u2 = torch.randn((tot, H, 64), device=DEV, generator=g).bfloat16() if c2 else None
            dsT = torch.randn((S, H, 64, 64), device=DEV, generator=g) * 0.1
            ws = torch.empty(gf.backward_varlen_workspace_bytes(S, tot, H, 64), dtype=torch.uint8, device=DEV).fill_(case & 255)
            y, s = gf.prefill_varlen_train(inp.r, inp.k, inp.v, inp.x, inp.u, inp.cu_seqlens, mx, ws, inp.state_in, c2=c2, u2=u2)
            ga = gf.backward_varlen(inp.r, inp.k, inp.v, inp.x, inp.u, dy, inp.cu_seqlens, mx, inp.state_in, dsT, workspace=ws, c2=c2, saved=True)
            gb = gf.backward_varlen(inp.r, inp.k, inp.v, inp.x, inp.u, dy, inp.cu_seqlens, mx, inp.state_in, dsT, c2=c2)
            if c2:
                y0, s0 = gf.prefill_varlen_c2(inp.r, inp.k, inp.v, inp.x, u2, inp.cu_seqlens, mx, inp.state_in, split=False)
            else:
                y0, s0 = gf.prefill_varlen(inp.r, inp.k, inp.v, inp.x, inp.u, inp.cu_seqlens, mx, inp.state_in, split=False)
            split = 2 * S * H <= sms and (mx + 63) // 64 >= 16
            what = ("packed", lens, H, c2, (lo, hi))
        else:
            B, T = int(rng.integers(1, 5)), int(rng.integers(1, 900))
            inp = synth.make_dense(B, T, H, 64, "bf16", seed=int(rng.integers(0, 1 << 30)), device=DEV, state_std=0.2, x_lo=lo, x_hi=hi)
            dy = torch.randn(inp.r.shape, device=DEV, generator=g).bfloat16()
            u2 = torch.randn(inp.r.shape, device=DEV, generator=g).bfloat16() if c2 else None
            dsT = torch.randn((B, H, 64, 64), device=DEV, generator=g) * 0.1
            ws = torch.empty(gf.backward_workspace_bytes(B, T, H, 64), dtype=torch.uint8, device=DEV).fill_(case & 255)
            y, s = gf.prefill_train(inp.r, inp.k, inp.v, inp.x, inp.u, ws, inp.state_in, c2=c2, u2=u2)
            if c2:
                ga = gf.backward_c2(inp.r, inp.k, inp.v, inp.x, dy, inp.state_in, dsT, workspace=ws, saved=True)
                gb = gf.backward_c2(inp.r, inp.k, inp.v, inp.x, dy, inp.state_in, dsT)
                y0, s0 = gf.prefill_c2(inp.r, inp.k, inp.v, inp.x, u2, inp.state_in)
            else:
                ga = gf.backward(inp.r, inp.k, inp.v, inp.x, inp.u, dy, inp.state_in, dsT, workspace=ws, saved=True)
                gb = gf.backward(inp.r, inp.k, inp.v, inp.x, inp.u, dy, inp.state_in, dsT)
                y0, s0 = gf.prefill(inp.r, inp.k, inp.v, inp.x, inp.u, inp.state_in)
            split = gf.split_plan(B, T, H, sms)[0] != 1
            what = ("dense", B, T, H, c2, (lo, hi))
        gf.last_device_status()
        assert torch.equal(y, y0) and torch.equal(s, s0), what
        for i, (p, q) in enumerate(zip(ga, gb)):
            if p is None:
                continue
            if split:       # the gradient call's own checkpoint pass runs in segments: equal to rounding
                assert _rel(p.float(), q.float()) <= 3e-3, (what, i)
            else:
                assert torch.equal(p, q), (what, i)
