"""Seeded synthetic inputs for the WKV-6 prefill / decode workloads.

This module holds no arithmetic of the method: it only draws the random tensors
(shapes, dtypes and value distributions of the benchmark configurations) that both
the CUDA library and the CPU oracle are fed.  Generation uses a seeded
``torch.Generator`` on the requested device, so a (seed, device) pair always yields
the same bits; to give the oracle the same bits as the GPU, generate once and copy.

Distributions (Finch-C2 activations stand-in): r, k, v ~ N(0,1) with k scaled by 1/8;
decay logit x ~ U(-6,-1) so that w = exp(-exp(x)) lies in about [0.69, 0.998];
bonus u ~ N(0, 0.5) (0.5 read as the standard deviation); state_in ~ N(0, 0.1) (std)
or zero.  Values are drawn in fp32 and rounded (nearest-even) to the storage dtype.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

CONFIGS = {
    # name: B, T, H, N, dtype, state_std (0 = zero state)
    "cfg0": dict(B=1, T=256, H=4, N=64, dtype="f32", state_std=0.0),
    "cfg1": dict(B=8, T=4096, H=12, N=64, dtype="bf16", state_std=0.1),
    "cfg2": dict(B=4, T=16384, H=32, N=64, dtype="bf16", state_std=0.0, calls=16),
    "cfg3": dict(B=1, T=131072, H=32, N=64, dtype="bf16", state_std=0.0, segments=8),
    "cfg4": dict(S=64, len_min=128, len_max=4096, H=32, N=64, dtype="bf16", state_std=0.1,
                 decode_steps=256),
}


def torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


@dataclass
class Wkv6Inputs:
    r: torch.Tensor
    k: torch.Tensor
    v: torch.Tensor
    x: torch.Tensor
    u: torch.Tensor
    state_in: torch.Tensor | None
    cu_seqlens: torch.Tensor | None = None

    def to(self, device):
        mv = lambda t: None if t is None else t.to(device)
        return Wkv6Inputs(mv(self.r), mv(self.k), mv(self.v), mv(self.x), mv(self.u),
                          mv(self.state_in), mv(self.cu_seqlens))


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _draw(shape, n_states, H, N, dtype, seed, device, state_std, x_lo, x_hi):
    g = _gen(seed, device)
    dt = torch_dtype(dtype) if isinstance(dtype, str) else dtype
    f = dict(device=device, dtype=torch.float32, generator=g)
    r = torch.randn(shape, **f).to(dt)
    k = (torch.randn(shape, **f) * 0.125).to(dt)
    v = torch.randn(shape, **f).to(dt)
    x = (torch.rand(shape, **f) * (x_hi - x_lo) + x_lo).to(dt)
    u = torch.randn((H, N), **f) * 0.5
    s = torch.randn((n_states, H, N, N), **f) * state_std if state_std > 0 else None
    return r, k, v, x, u, s


def make_dense(B, T, H, N=64, dtype="bf16", seed=0, device="cpu", state_std=0.0,
               x_lo=-6.0, x_hi=-1.0) -> Wkv6Inputs:
    """Inputs of one dense prefill call: r,k,v,x [B,T,H,N], u [H,N], state_in [B,H,N,N] or None."""
    r, k, v, x, u, s = _draw((B, T, H, N), B, H, N, dtype, seed, device, state_std, x_lo, x_hi)
    return Wkv6Inputs(r, k, v, x, u, s)


def make_lengths(S, len_min, len_max, seed=0) -> torch.Tensor:
    """Sequence lengths uniform on {len_min..len_max} and their exclusive prefix sum
    (int32 cu_seqlens of S+1 entries), drawn on the CPU."""
    g = _gen(seed, "cpu")
    lens = torch.randint(len_min, len_max + 1, (S,), generator=g, dtype=torch.int64)
    cu = torch.zeros(S + 1, dtype=torch.int32)
    cu[1:] = torch.cumsum(lens, 0).to(torch.int32)
    return cu


def make_varlen(cu_seqlens, H, N=64, dtype="bf16", seed=0, device="cpu", state_std=0.1,
                x_lo=-6.0, x_hi=-1.0) -> Wkv6Inputs:
    """Packed variable-length inputs: r,k,v,x [total_T,H,N], state_in [S,H,N,N]."""
    cu = torch.as_tensor(cu_seqlens, dtype=torch.int32)
    total, S = int(cu[-1]), cu.numel() - 1
    r, k, v, x, u, s = _draw((total, H, N), S, H, N, dtype, seed, device, state_std, x_lo, x_hi)
    return Wkv6Inputs(r, k, v, x, u, s, cu.to(device))


def make_step(B, H, N=64, dtype="bf16", seed=0, device="cpu", state_std=0.1) -> Wkv6Inputs:
    """Inputs of one decode step: r,k,v,x [B,H,N], state_in [B,H,N,N]."""
    r, k, v, x, u, s = _draw((B, H, N), B, H, N, dtype, seed, device, state_std, -6.0, -1.0)
    return Wkv6Inputs(r, k, v, x, u, s)


def make_decay_lora(D, Rd=32, Rw=64, seed=0, device="cpu"):
    """Weights of the decay-logit producer of a Finch-C2 block (stand-ins for trained ones): mu_x, lambda_d ~ U(0,1)
    (token-shift mixes), A ~ N(0, 1/D) so that the low-rank pre-activations are O(1), B ~ N(0, 1/R) so that each
    lora adds a vector of about unit scale, lambda_w ~ U(-6,-1) (the decay-logit range of the prefill workloads).
    Matrices are rounded to bf16, vectors stay fp32.  Returns a dict of tensors."""
    g = _gen(seed, device)
    f = dict(device=device, dtype=torch.float32, generator=g)
    bf = torch.bfloat16
    return dict(mu_x=torch.rand(D, **f), lambda_d=torch.rand(D, **f), lambda_w=torch.rand(D, **f) * 5 - 6,
                A_d=(torch.randn((D, Rd), **f) / D ** 0.5).to(bf), B_d=(torch.randn((Rd, D), **f) / Rd ** 0.5).to(bf),
                A_w=(torch.randn((D, Rw), **f) / D ** 0.5).to(bf), B_w=(torch.randn((Rw, D), **f) / Rw ** 0.5).to(bf))


def make_block_input(B, T, D, seed=0, device="cpu", with_prev=True):
    """Input of a Finch-C2 block (a normalised residual stream stand-in): x ~ N(0,1) [B,T,D] bf16 and the token
    before each sequence's first one [B,D] (or None)."""
    g = _gen(seed, device)
    f = dict(device=device, dtype=torch.float32, generator=g)
    x = torch.randn((B, T, D), **f).to(torch.bfloat16)
    xp = torch.randn((B, D), **f).to(torch.bfloat16) if with_prev else None
    return x, xp
