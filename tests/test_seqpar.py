"""Sequence-parallel prefill (one sequence cut along time over ranks): the exchange logic on two gloo ranks
with the fp64 oracle standing in for the three device steps, and the device steps themselves on one GPU
with the ranks played one after the other."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from oracle import wkv6_oracle as orc                      # noqa: E402
from paper_2407_12077_b200 import synth                     # noqa: E402

F = 64 + 64 * 64


class OracleOps:
    """CPU stand-ins for the device steps, written from the definition (test only)."""

    def summary(self, k, v, x):
        B, T, H, N = k.shape
        zeros = torch.zeros_like(k)
        _, dS = orc.prefill(zeros, k, v, x, np.zeros((H, N), np.float32), None)      # state reached from zero
        w = np.exp(-np.exp(x.float().numpy().astype(np.float64)))
        D = np.prod(w, axis=1)                                                       # [B, H, N]
        out = np.concatenate([D, dS.reshape(B, H, N * N)], axis=2)
        return torch.from_numpy(out.astype(np.float32))

    def fold(self, state_in, gathered, n_fold):
        P, B, H, _ = gathered.shape
        S = torch.zeros((B, H, 64, 64), dtype=torch.float64) if state_in is None else state_in.double()
        for p in range(n_fold):
            D, dS = gathered[p, :, :, :64].double(), gathered[p, :, :, 64:].double().reshape(B, H, 64, 64)
            S = D[..., None] * S + dS
        return S.float()

    def prefill(self, r, k, v, x, u, state_in):
        y, s = orc.prefill(r, k, v, x, u, state_in)
        return torch.from_numpy(y), torch.from_numpy(s.astype(np.float32))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2407_12077_b200 import seqpar
    inp = synth.make_dense(2, 48, 2, 64, "bf16", seed=77, state_std=0.1)
    cut = [0, 29, 48]                                               # unequal slices
    sl = slice(cut[rank], cut[rank + 1])
    y, s = seqpar.prefill_sequence_parallel(inp.r[:, sl].contiguous(), inp.k[:, sl].contiguous(), inp.v[:, sl].contiguous(),
                                            inp.x[:, sl].contiguous(), inp.u, inp.state_in, ops=OracleOps())
    torch.save({"y": y, "s": s}, os.path.join(out_dir, f"r{rank}.pt"))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_reproduce_the_unsplit_sequence(tmp_path):
    mp.spawn(_worker, args=(2, _free_port(), str(tmp_path)), nprocs=2, join=True)
    inp = synth.make_dense(2, 48, 2, 64, "bf16", seed=77, state_std=0.1)
    y_ref, s_ref = orc.prefill(inp.r, inp.k, inp.v, inp.x, inp.u, inp.state_in)
    out = [torch.load(tmp_path / f"r{r}.pt") for r in range(2)]
    y = torch.cat([o["y"] for o in out], 1).numpy()
    # summaries travel as float32, so agreement is to float32 rounding of the handed-over state
    assert orc.rel_l2(y, y_ref) < 1e-6
    assert orc.rel_l2(out[1]["s"].numpy(), s_ref) < 1e-6


@pytest.mark.gpu
@pytest.mark.parametrize("c2", [False, True])
def test_device_steps_with_ranks_played_in_turn(c2):
    """One GPU plays four ranks one after the other: summaries of the four pieces, the fold each rank would do
    after the all-gather, then each piece's prefill from its folded start state, against the oracle."""
    import paper_2407_12077_b200 as gf
    dev = "cuda:0"
    B, T, H, P = 2, 2000, 3, 4
    inp = synth.make_dense(B, T, H, 64, "bf16", seed=88, state_std=0.1)
    u2 = torch.randn(inp.r.shape, generator=torch.Generator().manual_seed(89)).bfloat16()
    d = inp.to(dev)
    cuts = [0, 500, 1037, 1500, T]
    pieces = [slice(cuts[p], cuts[p + 1]) for p in range(P)]
    cut = lambda t, p: t[:, pieces[p]].contiguous()
    gathered = torch.stack([gf.sequence_summary(cut(d.k, p), cut(d.v, p), cut(d.x, p), c2=c2) for p in range(P)])
    ys, state = [], None
    for p in range(P):
        start = d.state_in if p == 0 else gf.fold_summaries(d.state_in, gathered, p)
        if c2:
            y, state = gf.prefill_c2(cut(d.r, p), cut(d.k, p), cut(d.v, p), cut(d.x, p), cut(u2.to(dev), p), start)
        else:
            y, state = gf.prefill(cut(d.r, p), cut(d.k, p), cut(d.v, p), cut(d.x, p), d.u, start)
        ys.append(y)
    gf.last_device_status()
    y = torch.cat(ys, 1)
    if c2:
        y_ref, s_ref = orc.prefill_c2(inp.r, inp.k, inp.v, inp.x, u2, inp.state_in)
    else:
        y_ref, s_ref = orc.prefill(inp.r, inp.k, inp.v, inp.x, inp.u, inp.state_in)
    ey, es = orc.rel_l2(y.float().cpu().numpy(), y_ref), orc.rel_l2(state.cpu().numpy(), s_ref)
    assert ey <= 5e-3 and es <= 5e-3, (ey, es)
    # the fold of all four summaries over the initial state is the final state as well
    s_all = gf.fold_summaries(d.state_in, gathered, P)
    assert orc.rel_l2(s_all.cpu().numpy(), s_ref) <= 5e-3


def _device_worker(rank, world, port, out_dir, c2):
    """One rank of the real thing: the library's kernels around a collective of a process group.  Both ranks use
    cuda:0 (they meet on the host, in the gather, never inside a kernel); gloo carries the summaries."""
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import paper_2407_12077_b200 as gf
    from paper_2407_12077_b200 import seqpar
    dev = "cuda:0"
    inp, u2, cut = _device_case()
    sl = slice(cut[rank], cut[rank + 1])
    mv = lambda t: t[:, sl].contiguous().to(dev)
    u_arg = mv(u2) if c2 else inp.u.to(dev)
    y, s = seqpar.prefill_sequence_parallel(mv(inp.r), mv(inp.k), mv(inp.v), mv(inp.x), u_arg, inp.state_in.to(dev),
                                            ops=seqpar.DeviceOps(c2=c2))
    gf.last_device_status()
    torch.save({"y": y.cpu(), "s": s.cpu(), "launches": gf.launch_count()}, os.path.join(out_dir, f"d{rank}.pt"))
    dist.barrier()
    dist.destroy_process_group()


def _device_case():
    # slow decays (w about 0.998 .. 0.99995): the state a rank inherits still weighs on its last token
    inp = synth.make_dense(2, 2300, 3, 64, "bf16", seed=90, state_std=0.5, x_lo=-10.0, x_hi=-6.0)
    u2 = torch.randn(inp.r.shape, generator=torch.Generator().manual_seed(91)).bfloat16()
    return inp, u2, [0, 1237, 2300]


@pytest.mark.gpu
@pytest.mark.parametrize("c2", [False, True])
def test_two_ranks_with_the_device_steps_under_a_process_group(tmp_path, c2):
    """prefill_sequence_parallel with DeviceOps end to end: summary kernel -> all_gather -> fold kernel -> prefill,
    two processes, against the unsplit oracle."""
    mp.spawn(_device_worker, args=(2, _free_port(), str(tmp_path), c2), nprocs=2, join=True)
    inp, u2, cut = _device_case()
    if c2:
        y_ref, s_ref = orc.prefill_c2(inp.r, inp.k, inp.v, inp.x, u2, inp.state_in)
    else:
        y_ref, s_ref = orc.prefill(inp.r, inp.k, inp.v, inp.x, inp.u, inp.state_in)
    out = [torch.load(tmp_path / f"d{r}.pt") for r in range(2)]
    assert out[0]["launches"] >= 2 and out[1]["launches"] >= 3      # rank 1: summary, fold, prefill
    y = torch.cat([o["y"] for o in out], 1).float().numpy()
    assert orc.rel_l2(y, y_ref) <= 5e-3
    assert orc.rel_l2(y[:, cut[1]:], y_ref[:, cut[1]:]) <= 5e-3      # the second rank's piece on its own
    assert orc.rel_l2(out[1]["s"].numpy(), s_ref) <= 5e-3
    # the hand-over matters here: without the first piece the second rank's answer is far off
    wrong, _ = (orc.prefill_c2 if c2 else orc.prefill)(inp.r[:, cut[1]:], inp.k[:, cut[1]:], inp.v[:, cut[1]:], inp.x[:, cut[1]:],
                                                        (u2[:, cut[1]:] if c2 else inp.u), None)
    assert orc.rel_l2(wrong, y_ref[:, cut[1]:]) > 0.05
