"""GPU parity of the Finch-C2 form (gf_wkv6_prefill_c2) against the fp64 oracle's Finch-C2 recurrence:
keys times one minus their decay, no bonus, second-value vector added to the output.  Same tolerance as
the other bf16 parity tests (relative L2 <= 5e-3 on y and on the final state)."""
import numpy as np
import pytest
import torch

import paper_2407_12077_b200 as gf
from oracle import wkv6_oracle as orc
from paper_2407_12077_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = 5e-3


def make(B, T, H, seed, state_std=0.1, with_u2=True, **kw):
    inp = synth.make_dense(B, T, H, 64, "bf16", seed=seed, state_std=state_std, **kw)
    g = torch.Generator().manual_seed(seed + 7)
    u2 = torch.randn(inp.r.shape, generator=g).bfloat16() if with_u2 else None
    return inp, u2


def run(inp, u2, **kw):
    d = inp.to(DEV)
    y, s = gf.prefill_c2(d.r, d.k, d.v, d.x, None if u2 is None else u2.to(DEV), d.state_in, **kw)
    gf.last_device_status()
    return y, s


def check(y, s, inp, u2, what):
    y_ref, s_ref = orc.prefill_c2(inp.r, inp.k, inp.v, inp.x, u2, inp.state_in)
    ey, es = orc.rel_l2(y.float().cpu().numpy(), y_ref), orc.rel_l2(s.cpu().numpy(), s_ref)
    assert np.isfinite(ey) and ey <= TOL, f"{what}: y rel-L2 {ey:.3e}"
    assert np.isfinite(es) and es <= TOL, f"{what}: state rel-L2 {es:.3e}"
    return ey, es


@pytest.mark.parametrize("T", [1, 2, 17, 63, 64, 65, 128, 200, 321, 1000])
@pytest.mark.parametrize("with_u2", [True, False])
def test_c2_ragged_lengths(T, with_u2):
    inp, u2 = make(2, T, 3, 300 + T, with_u2=with_u2)
    y, s = run(inp, u2)
    check(y, s, inp, u2, f"T={T} u2={with_u2}")


def test_c2_small_model_shape_full():
    c = synth.CONFIGS["cfg1"]
    inp, u2 = make(c["B"], c["T"], c["H"], 1100)
    y, s = run(inp, u2)
    check(y, s, inp, u2, "cfg1 shape")


@pytest.mark.parametrize("case", ["w_one", "fast_decay", "mixed_extreme", "slow_decay"])
def test_c2_extreme_decay_logits(case):
    inp, u2 = make(1, 200, 2, 810)
    g = torch.Generator().manual_seed(811)
    if case == "w_one":
        inp.x = torch.full_like(inp.x, float("-inf"))                              # keys vanish, state frozen
    elif case == "fast_decay":
        inp.x = (torch.rand(inp.x.shape, generator=g) * 4 - 1).bfloat16()          # token-by-token chunks
    elif case == "slow_decay":
        inp.x = (torch.rand(inp.x.shape, generator=g) * 3 - 9).bfloat16()          # 1 - w down to ~1e-4
    else:
        inp.x = (torch.rand(inp.x.shape, generator=g) * 16 - 8).bfloat16()
        inp.x[:, ::7, :, ::5] = float("-inf")
    y, s = run(inp, u2)
    assert torch.isfinite(y.float()).all() and torch.isfinite(s).all()
    check(y, s, inp, u2, case)


def test_c2_sequence_split_and_determinism():
    inp, u2 = make(1, 5000, 4, 820)
    assert gf.workspace_bytes(1, 5000, 4, 64) > 0
    y, s = run(inp, u2)
    y1, s1 = run(inp, u2, split=False)
    y2, s2 = run(inp, u2)
    assert torch.equal(y, y2) and torch.equal(s, s2)
    check(y, s, inp, u2, "split")
    check(y1, s1, inp, u2, "unsplit")


def test_c2_full_size_every_unit():
    """1.5B-class shape in the launch configuration the benchmark's Finch-C2 row times, with a start state: all 128
    units against the oracle, per tensor, per unit and per token (the bounds of the classic prefill's full-size test)."""
    c = synth.CONFIGS["cfg2"]
    B, T, H = c["B"], c["T"], c["H"]
    inp = synth.make_dense(B, T, H, 64, "bf16", seed=2100, state_std=0.1)
    u2 = torch.randn(inp.r.shape, generator=torch.Generator().manual_seed(5)).bfloat16()
    d = inp.to(DEV)
    y, s = gf.prefill_c2(d.r, d.k, d.v, d.x, u2.to(DEV), d.state_in)
    gf.last_device_status()
    yn, sn = y.float().cpu().numpy().astype(np.float64), s.cpu().numpy().astype(np.float64)
    assert np.isfinite(yn).all() and np.isfinite(sn).all()
    y_ref, s_ref = orc.prefill_c2(inp.r, inp.k, inp.v, inp.x, u2, inp.state_in)
    assert orc.rel_l2(yn, y_ref) <= TOL and orc.rel_l2(sn, s_ref) <= TOL
    row = ((yn - y_ref) ** 2).sum(axis=3)                        # [B, T, H]
    den = (y_ref ** 2).sum(axis=(1, 3))                          # [B, H]
    unit = np.sqrt(row.sum(axis=1) / den)
    assert unit.max() <= TOL, ("unit", float(unit.max()))
    tok = np.sqrt(row.max(axis=1) / (den / T))
    assert tok.max() <= 4e-2, ("token", float(tok.max()))
    su = np.sqrt(((sn - s_ref) ** 2).sum(axis=(2, 3)) / (s_ref ** 2).sum(axis=(2, 3)))
    assert su.max() <= TOL, ("state unit", float(su.max()))
    print("worst unit y / token / state", float(unit.max()), float(tok.max()), float(su.max()))


def test_c2_varlen_matches_per_sequence_oracle_including_empty_sequence():
    lens = [5, 0, 64, 1, 130, 77, 63, 200]
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32)
    H = 3
    inp = synth.make_varlen(cu, H, 64, "bf16", seed=830, state_std=0.1)
    u2 = torch.randn(inp.r.shape, generator=torch.Generator().manual_seed(831)).bfloat16()
    d = inp.to(DEV)
    y = torch.full_like(d.r, 12345.0)
    y, s = gf.prefill_varlen_c2(d.r, d.k, d.v, d.x, u2.to(DEV), d.cu_seqlens, max(lens), d.state_in, y=y)
    gf.last_device_status()
    for i, n in enumerate(lens):
        a, b = int(cu[i]), int(cu[i + 1])
        if n == 0:
            assert torch.equal(s[i].cpu(), inp.state_in[i])
            continue
        sl = lambda t: t[a:b][None].contiguous()
        y_ref, s_ref = orc.prefill_c2(sl(inp.r), sl(inp.k), sl(inp.v), sl(inp.x), sl(u2), inp.state_in[i][None].contiguous())
        ey = orc.rel_l2(y[a:b].float().cpu().numpy(), y_ref[0])
        es = orc.rel_l2(s[i].cpu().numpy(), s_ref[0])
        assert ey <= TOL and es <= TOL, (i, n, ey, es)


def test_c2_varlen_sequence_split_matches_per_sequence_oracle():
    """Packed Finch-C2 call with few units: cut by max_seqlen into segments, two launches."""
    lens = [2100, 0, 700, 3011]
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32)
    H = 2
    assert gf.workspace_bytes(len(lens), max(lens), H, 64) > 0
    inp = synth.make_varlen(cu, H, 64, "bf16", seed=832, state_std=0.1)
    u2 = torch.randn(inp.r.shape, generator=torch.Generator().manual_seed(833)).bfloat16()
    d = inp.to(DEV)
    before = gf.launch_count()
    y, s = gf.prefill_varlen_c2(d.r, d.k, d.v, d.x, u2.to(DEV), d.cu_seqlens, max(lens), d.state_in)
    assert gf.launch_count() - before == 2
    gf.last_device_status()
    for i, n in enumerate(lens):
        a, b = int(cu[i]), int(cu[i + 1])
        if n == 0:
            assert torch.equal(s[i].cpu(), inp.state_in[i])
            continue
        sl = lambda t: t[a:b][None].contiguous()
        y_ref, s_ref = orc.prefill_c2(sl(inp.r), sl(inp.k), sl(inp.v), sl(inp.x), sl(u2), inp.state_in[i][None].contiguous())
        ey = orc.rel_l2(y[a:b].float().cpu().numpy(), y_ref[0])
        es = orc.rel_l2(s[i].cpu().numpy(), s_ref[0])
        assert ey <= TOL and es <= TOL, (i, n, ey, es)


@pytest.mark.parametrize("with_u2", [True, False])
def test_c2_step_matches_oracle_and_chains_to_a_prefill(with_u2):
    B, H, T = 3, 5, 6
    inp, u2 = make(B, T, H, 840, with_u2=with_u2)
    d = inp.to(DEV)
    u2d = None if u2 is None else u2.to(DEV)
    st = d.state_in.clone()
    ys = []
    for t in range(T):
        yt, st = gf.step_c2(d.r[:, t].contiguous(), d.k[:, t].contiguous(), d.v[:, t].contiguous(), d.x[:, t].contiguous(),
                            None if u2d is None else u2d[:, t].contiguous(), st)
        ys.append(yt)
    gf.last_device_status()
    check(torch.stack(ys, 1), st, inp, u2, f"chain of step_c2 u2={with_u2}")


@pytest.mark.parametrize("with_u2", [True, False])
def test_c2_more_units_than_sms(with_u2):
    """Persistent launch of the Finch-C2 form: the second-value slab of a unit's first chunk is fetched when the
    stream reaches the unit."""
    inp, u2 = make(25, 210, 8, 880, with_u2=with_u2)
    y, s = run(inp, u2)
    check(y, s, inp, u2, f"persistent C2 u2={with_u2}")


def test_c2_packed_more_units_than_sms():
    import random
    rng = random.Random(9)
    lens = [rng.choice([0, 1, 64, rng.randint(2, 260)]) for _ in range(50)]
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32)
    H = 4
    inp = synth.make_varlen(cu, H, 64, "bf16", seed=890, state_std=0.1)
    u2 = torch.randn(inp.r.shape, generator=torch.Generator().manual_seed(891)).bfloat16()
    d = inp.to(DEV)
    y, s = gf.prefill_varlen_c2(d.r, d.k, d.v, d.x, u2.to(DEV), d.cu_seqlens, max(lens), d.state_in)
    gf.last_device_status()
    for i, n in enumerate(lens):
        a, b = int(cu[i]), int(cu[i + 1])
        if n == 0:
            assert torch.equal(s[i].cpu(), inp.state_in[i])
            continue
        sl = lambda t: t[a:b][None].contiguous()
        y_ref, s_ref = orc.prefill_c2(sl(inp.r), sl(inp.k), sl(inp.v), sl(inp.x), sl(u2), inp.state_in[i][None].contiguous())
        ey = orc.rel_l2(y[a:b].float().cpu().numpy(), y_ref[0])
        es = orc.rel_l2(s[i].cpu().numpy(), s_ref[0])
        assert ey <= TOL and es <= TOL, (i, n, ey, es)
