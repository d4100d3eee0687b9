"""Sequence-parallel prefill: ONE long sequence per batch entry, cut along time over the ranks of a
``torch.distributed`` group (rank order = sequence order).

Over a run of tokens the WKV recurrence acts on the state as the affine map S -> diag(D) S + dS (D: product
of the run's decays, dS: state reached from zero; the wkv_t sum of the Finch-C2 section restricted to the
run).  These maps compose in order, so the only exchange is one all-gather of every rank's (D, dS) summary
(B*H*(64 + 4096) fp32 per rank): each rank folds the summaries of the ranks before it over the sequence's
initial state and then runs the ordinary prefill on its own piece.  Ranks after the first read k, v, x twice.

The three device steps are the library's entry points (gf_wkv6_sequence_summary, gf_wkv6_fold_summaries,
gf_wkv6_prefill / gf_wkv6_prefill_c2); this module only orders them around the collective.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


class DeviceOps:
    """The device steps, bound to the CUDA library."""

    def __init__(self, c2: bool = False):
        import paper_2407_12077_b200 as gf
        self.gf, self.c2 = gf, c2

    def summary(self, k, v, x):
        return self.gf.sequence_summary(k, v, x, c2=self.c2)

    def fold(self, state_in, gathered, n_fold):
        return self.gf.fold_summaries(state_in, gathered, n_fold)

    def prefill(self, r, k, v, x, u, state_in):
        if self.c2:
            return self.gf.prefill_c2(r, k, v, x, u, state_in)
        return self.gf.prefill(r, k, v, x, u, state_in)


def prefill_sequence_parallel(r, k, v, x, u, state_in=None, group=None, ops=None):
    """Each rank passes its own time slice r,k,v,x [B, T_local, H, N] (slices may differ in length) and the
    same u ([H,N] bonus, or the local slice of the second-value tensor / None with ``DeviceOps(c2=True)``)
    and state_in (the sequence's initial state [B,H,N,N] or None).  Returns (y_local, state): state is the
    state after this rank's last token, so the last rank holds the sequence's final state."""
    ops = ops or DeviceOps()
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    if world == 1:
        return ops.prefill(r, k, v, x, u, state_in)
    mine = ops.summary(k, v, x).contiguous()                         # [B, H, 64 + 4096]
    if mine.is_cuda and dist.get_backend(group) != "nccl":
        # a backend that gathers host memory only (gloo): stage the summaries through the host
        host = torch.empty((world,) + tuple(mine.shape), dtype=mine.dtype)
        dist.all_gather(list(host.unbind(0)), mine.cpu(), group=group)
        gathered = host.to(mine.device)
    else:
        gathered = torch.empty((world,) + tuple(mine.shape), dtype=mine.dtype, device=mine.device)
        dist.all_gather(list(gathered.unbind(0)), mine, group=group)  # the one exchange step
    start = state_in if rank == 0 else ops.fold(state_in, gathered, rank)
    return ops.prefill(r, k, v, x, u, start)
