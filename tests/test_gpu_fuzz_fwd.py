"""Seeded random packed batches for the prefill calls (few long sequences, dozens of middling ones, hundreds of short
ones: below and above the SM count, so that the plain, the split and the persistent launch all come up).  Properties:
the call repeats bit for bit; with the workspace (persistent launch for many units) it equals the plain launch bit for
bit, or to rounding where it splits its sequences; a third of the cases are held to the fp64 oracle as well."""
import numpy as np
import pytest
import torch

import paper_2407_12077_b200 as gf
from oracle import wkv6_oracle as orc
from paper_2407_12077_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
RANGES = [(-6.0, -1.0), (-8.0, -4.0), (-3.0, 0.5), (-2.0, 1.5)]


@pytest.mark.parametrize("seed", [301, 302, 303])
def test_packed_prefill_launch_forms_agree(seed):
    rng = np.random.default_rng(seed)
    g = torch.Generator(device=DEV).manual_seed(seed)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    for case in range(40):
        c2 = rng.random() < 0.4
        H = int(rng.integers(1, 9))
        lo, hi = RANGES[int(rng.integers(0, len(RANGES)))]
        mode = int(rng.integers(0, 3))
        S, mxl = [(int(rng.integers(1, 8)), 600), (int(rng.integers(20, 120)), 200), (int(rng.integers(150, 500)), 80)][mode]
        lens = [int(rng.integers(0, mxl)) for _ in range(S)]
        if sum(lens) == 0:
            lens[0] = 3
        cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32)
        inp = synth.make_varlen(cu, H, 64, "bf16", seed=int(rng.integers(0, 1 << 30)), device=DEV, state_std=0.2, x_lo=lo, x_hi=hi)
        tot, mx = sum(lens), max(lens)
        u2 = torch.randn((tot, H, 64), device=DEV, generator=g).bfloat16() if c2 else None

        def call(split):
            if c2:
                return gf.prefill_varlen_c2(inp.r, inp.k, inp.v, inp.x, u2, inp.cu_seqlens, mx, inp.state_in, split=split)
            return gf.prefill_varlen(inp.r, inp.k, inp.v, inp.x, inp.u, inp.cu_seqlens, mx, inp.state_in, split=split)

        y, s = call(True)
        y2, s2 = call(True)
        y3, s3 = call(False)
        gf.last_device_status()
        what = (S, H, c2, (lo, hi), tot, mx)
        assert torch.equal(y, y2) and torch.equal(s, s2), what
        if 2 * S * H <= sms and (mx + 63) // 64 >= 16:          # the call with the workspace splits its sequences
            assert orc.rel_l2(y.float().cpu().numpy(), y3.float().cpu().numpy()) <= 3e-3, what
        else:
            assert torch.equal(y, y3) and torch.equal(s, s3), what
        if case % 3 == 0 and tot * H <= 40000:
            c = inp.to("cpu")
            if c2:
                # the packed Finch-C2 forward, sequence by sequence through the dense oracle of that form
                for q, ln in enumerate(lens):
                    a, b = int(cu[q]), int(cu[q + 1])
                    if ln < 64:
                        continue
                    yr, sr = orc.prefill_c2(c.r[a:b][None], c.k[a:b][None], c.v[a:b][None], c.x[a:b][None], u2[a:b][None].cpu(),
                                            c.state_in[q][None])
                    lim = 4e-2 if hi > 0 else 5e-3
                    assert orc.rel_l2(y[a:b].float().cpu().numpy(), yr[0]) <= lim, (what, q)
                    assert orc.rel_l2(s[q].cpu().numpy(), sr[0]) <= lim, (what, q)
            else:
                yr, sr = orc.prefill_varlen(c.r, c.k, c.v, c.x, c.u, cu, c.state_in)
                lim = 4e-2 if hi > 0 else 5e-3
                if tot >= 64:
                    assert orc.rel_l2(y.float().cpu().numpy(), yr) <= lim, what
                    assert orc.rel_l2(s.cpu().numpy(), sr) <= lim, what
