"""Python binding of the gf_wkv6 C-ABI CUDA library (argument marshalling only).

Every function mirrors the entry point of the same name in ``include/gf_wkv6.h``:
torch tensors supply device memory and the current CUDA stream, all arithmetic runs
in the library's kernels.  There is no CPU or PyTorch fallback: if the shared library
is missing or a tensor is not on a CUDA device the call raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import _build

__all__ = [
    "GfError", "load_library", "library_path", "prefill", "prefill_varlen", "step", "bind_step",
    "sequence_summary", "fold_summaries", "SUMMARY_FLOATS", "backward", "backward_c2", "prefill_train", "backward_workspace_bytes", "backward_varlen", "backward_varlen_workspace_bytes", "prefill_varlen_train", "decay_logit", "prefill_c2", "prefill_varlen_c2", "step_c2", "prefill_static", "STATIC_SCRATCH_BYTES", "prefill_host", "host_workspace_bytes", "workspace_bytes", "split_plan", "set_workspace", "set_kernel", "last_device_status",
    "launch_count", "status_string", "version", "set_wait_limit", "selftest_wait_timeout",
    "KERNEL_AUTO", "KERNEL_EXACT", "KERNEL_CHUNKED",
]

KERNEL_AUTO, KERNEL_EXACT, KERNEL_CHUNKED = 0, 1, 2
GF_OK = 0

_lib = None
_vp, _i, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t

# name -> (restype, argtypes); the single place the ABI is mirrored in Python
_SIGNATURES = {
    "gf_wkv6_prefill": (_i, [_vp] * 8 + [_i] * 4 + [_vp]),
    "gf_wkv6_prefill_f32": (_i, [_vp] * 8 + [_i] * 4 + [_vp]),
    "gf_wkv6_prefill_static": (_i, [_vp] * 8 + [_i] * 4 + [_vp]),
    "gf_wkv6_backward_f32": (_i, [_vp] * 14 + [_i] * 4 + [_vp, _sz, _vp]),
    "gf_wkv6_backward_workspace_bytes": (_sz, [_i] * 4),
    "gf_wkv6_backward": (_i, [_vp] * 14 + [_i] * 4 + [_vp, _sz, _vp]),
    "gf_wkv6_backward_bf16_workspace_bytes": (_sz, [_i] * 4),
    "gf_wkv6_backward_c2": (_i, [_vp] * 12 + [_i] * 4 + [_vp, _sz, _vp]),
    "gf_wkv6_backward_varlen": (_i, [_vp] * 15 + [_i] * 5 + [_vp, _sz, _vp]),
    "gf_wkv6_backward_varlen_c2": (_i, [_vp] * 13 + [_i] * 5 + [_vp, _sz, _vp]),
    "gf_wkv6_backward_varlen_workspace_bytes": (_sz, [_i] * 4),
    "gf_wkv6_backward_varlen_saved": (_i, [_vp] * 15 + [_i] * 5 + [_vp, _sz, _vp]),
    "gf_wkv6_backward_varlen_c2_saved": (_i, [_vp] * 13 + [_i] * 5 + [_vp, _sz, _vp]),
    "gf_wkv6_prefill_varlen_train": (_i, [_vp] * 9 + [_i] * 5 + [_vp, _sz, _vp]),
    "gf_wkv6_prefill_varlen_c2_train": (_i, [_vp] * 9 + [_i] * 5 + [_vp, _sz, _vp]),
    "gf_wkv6_backward_saved": (_i, [_vp] * 14 + [_i] * 4 + [_vp, _sz, _vp]),
    "gf_wkv6_backward_c2_saved": (_i, [_vp] * 12 + [_i] * 4 + [_vp, _sz, _vp]),
    "gf_wkv6_prefill_train": (_i, [_vp] * 8 + [_i] * 4 + [_vp, _sz, _vp]),
    "gf_wkv6_prefill_c2_train": (_i, [_vp] * 8 + [_i] * 4 + [_vp, _sz, _vp]),
    "gf_wkv6_prefill_c2": (_i, [_vp] * 8 + [_i] * 4 + [_vp]),
    "gf_wkv6_prefill_varlen_c2": (_i, [_vp] * 9 + [_i] * 5 + [_vp]),
    "gf_wkv6_step_c2": (_i, [_vp] * 8 + [_i] * 3 + [_vp]),
    "gf_wkv6_prefill_varlen": (_i, [_vp] * 9 + [_i] * 5 + [_vp]),
    "gf_wkv6_prefill_varlen_f32": (_i, [_vp] * 9 + [_i] * 5 + [_vp]),
    "gf_wkv6_step": (_i, [_vp] * 8 + [_i] * 3 + [_vp]),
    "gf_wkv6_step_f32": (_i, [_vp] * 8 + [_i] * 3 + [_vp]),
    "gf_wkv6_prefill_host": (_i, [_vp] * 8 + [_i] * 4 + [_vp, _sz, _vp]),
    "gf_wkv6_host_workspace_bytes": (_sz, [_i] * 4),
    "gf_wkv6_workspace_bytes": (_sz, [_i] * 4),
    "gf_wkv6_set_workspace": (_i, [_vp, _sz]),
    "gf_wkv6_split_plan": (_i, [_i] * 5 + [_sz, _vp, _vp, _vp]),
    "gf_wkv6_sequence_summary": (_i, [_vp] * 4 + [_i] * 5 + [_vp]),
    "gf_wkv6_fold_summaries": (_i, [_vp, _vp] + [_i] * 4 + [_vp, _vp]),
    "gf_c2_layernorm": (_i, [_vp, _vp, _vp, ctypes.c_float, _vp, ctypes.c_longlong, _i, _i, _vp]),
    "gf_c2_layernorm_f32": (_i, [_vp, _vp, _vp, ctypes.c_float, _vp, ctypes.c_longlong, _i, _i, _vp]),
    "gf_gold_key_compress": (_i, [_vp, _vp, _vp, ctypes.c_longlong, _i, _i, _vp]),
    "gf_c2_decay_logit": (_i, [_vp] * 10 + [_i] * 5 + [_vp]),
    "gf_wkv6_set_kernel": (_i, [_i]),
    "gf_wkv6_last_device_status": (_i, [_vp]),
    "gf_wkv6_set_wait_limit": (_i, [ctypes.c_uint]),
    "gf_wkv6_selftest_wait_timeout": (_i, [ctypes.c_uint, _vp]),
    "gf_wkv6_launch_count": (ctypes.c_uint64, []),
    "gf_status_string": (ctypes.c_char_p, [_i]),
    "gf_wkv6_version": (_i, []),
}


class GfError(RuntimeError):
    """A gf_wkv6 call returned a status other than GF_OK."""

    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: {status_string(status)} (gf_status_t {int(status)})")


def library_path() -> str:
    return _build.LIB_PATH


def load_library(build_if_missing: bool = True):
    """dlopen libgfwkv6.so (building it with nvcc first if it is absent or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB_PATH
    if build_if_missing and _build.is_stale():
        _build.build()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_2407_12077_b200._build`; "
                           "there is no fallback path")
    lib = ctypes.CDLL(path)
    for name, (res, args) in _SIGNATURES.items():
        fn = getattr(lib, name)            # AttributeError here = header / library mismatch
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().gf_status_string(int(status)).decode()


def version() -> int:
    return int(load_library().gf_wkv6_version())


def launch_count() -> int:
    return int(load_library().gf_wkv6_launch_count())


def set_kernel(kernel: int) -> None:
    _check(load_library().gf_wkv6_set_kernel(int(kernel)), "gf_wkv6_set_kernel")


def _check(status: int, where: str) -> None:
    if status != GF_OK:
        raise GfError(status, where)


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream) if hasattr(stream, "cuda_stream") else int(stream)


def _dev(t: torch.Tensor | None, name: str, dtype=None, shape=None):
    """Device pointer of a contiguous CUDA tensor (None -> NULL)."""
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (no CPU fallback exists)")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} must have shape {tuple(shape)}, got {tuple(t.shape)}")
    return t.data_ptr()


def _suffix(dtype) -> str:
    if dtype == torch.bfloat16:
        return ""
    if dtype == torch.float32:
        return "_f32"
    raise TypeError(f"r,k,v,x must be bfloat16 or float32, got {dtype}")


_workspace = None            # the registered scratch tensor is kept alive here


def workspace_bytes(B, T, H, N=64) -> int:
    """Scratch gf_wkv6_prefill(B,T,H,N) would use on the current device (0: the call does not split)."""
    return int(load_library().gf_wkv6_workspace_bytes(int(B), int(T), int(H), int(N)))


def split_plan(B, T, H, n_sm, scratch_cap=0, N=64):
    """gf_wkv6_split_plan: (segments per sequence, chunks per segment, scratch bytes) of a bf16 prefill call on a GPU
    of n_sm SMs with at most scratch_cap bytes of scratch (0: unlimited).  Host arithmetic, needs no device."""
    nseg, sc, nb = ctypes.c_int(), ctypes.c_int(), ctypes.c_size_t()
    _check(load_library().gf_wkv6_split_plan(int(B), int(T), int(H), int(N), int(n_sm), int(scratch_cap),
                                             ctypes.byref(nseg), ctypes.byref(sc), ctypes.byref(nb)), "gf_wkv6_split_plan")
    return nseg.value, sc.value, nb.value


def set_workspace(buf: torch.Tensor | None) -> None:
    """gf_wkv6_set_workspace: register a CUDA byte tensor as the library's scratch (None unregisters)."""
    global _workspace
    lib = load_library()
    if buf is None:
        _check(lib.gf_wkv6_set_workspace(None, 0), "gf_wkv6_set_workspace")
    else:
        _check(lib.gf_wkv6_set_workspace(_dev(buf, "workspace"), buf.numel() * buf.element_size()), "gf_wkv6_set_workspace")
    _workspace = buf


def _ensure_workspace(B, T, H, N, device) -> None:
    """Device memory is torch's job: grow the registered scratch when a call could use more."""
    need = workspace_bytes(B, T, H, N)
    have = 0 if _workspace is None or _workspace.device != device else _workspace.numel()
    if need > have:
        set_workspace(torch.empty(need, dtype=torch.uint8, device=device))


def last_device_status(stream=None) -> None:
    """Synchronise the stream and raise if a kernel gave up on a bounded wait."""
    _check(load_library().gf_wkv6_last_device_status(_stream(stream)), "gf_wkv6_last_device_status")


def set_wait_limit(microseconds: int) -> None:
    """gf_wkv6_set_wait_limit: bound of every device-side wait of later launches (0: the default of 2 s)."""
    _check(load_library().gf_wkv6_set_wait_limit(int(microseconds)), "gf_wkv6_set_wait_limit")


def selftest_wait_timeout(microseconds: int, stream=None) -> None:
    """gf_wkv6_selftest_wait_timeout: enqueue the one-warp kernel whose bounded wait runs out after `microseconds`."""
    _check(load_library().gf_wkv6_selftest_wait_timeout(int(microseconds), _stream(stream)), "gf_wkv6_selftest_wait_timeout")


def prefill(r, k, v, x, u, state_in=None, state_out=None, y=None, stream=None, want_state=True, split=True):
    """gf_wkv6_prefill / gf_wkv6_prefill_f32.  r,k,v,x: [B,T,H,N] CUDA tensors (bf16 or fp32);
    u: [H,N] fp32; state_in: [B,H,N,N] fp32 or None (zero).  Returns (y, state_out);
    both are allocated here unless passed in (state_out may be state_in).  split=False unregisters
    the scratch workspace first, so that a call with few (b,h) units runs as a single launch."""
    lib = load_library()
    B, T, H, N = r.shape
    sfx = _suffix(r.dtype)
    if y is None:
        y = torch.empty_like(r)
    if state_out is None and want_state:
        state_out = torch.empty((B, H, N, N), device=r.device, dtype=torch.float32)
    args = [_dev(r, "r", shape=(B, T, H, N)), _dev(k, "k", r.dtype, r.shape), _dev(v, "v", r.dtype, r.shape),
            _dev(x, "x", r.dtype, r.shape), _dev(u, "u", torch.float32, (H, N)),
            _dev(state_in, "state_in", torch.float32, (B, H, N, N)),
            _dev(state_out, "state_out", torch.float32, (B, H, N, N)), _dev(y, "y", r.dtype, r.shape)]
    with torch.cuda.device(r.device):
        if sfx == "" and split:
            _ensure_workspace(B, T, H, N, r.device)
        elif not split and _workspace is not None:
            set_workspace(None)
        _check(getattr(lib, "gf_wkv6_prefill" + sfx)(*args, B, T, H, N, _stream(stream)), "gf_wkv6_prefill" + sfx)
    return y, state_out


def backward(r, k, v, x, u, dy, state_in=None, dstate_out=None, want_dstate=True, stream=None, workspace=None, saved=False):
    """gf_wkv6_backward (bf16 tensors: chunked on the tensor cores) or gf_wkv6_backward_f32 (fp32 tensors: token by
    token): gradient of the prefill.  r,k,v,x,dy: [B,T,H,N] CUDA tensors of one dtype, u: [H,N] fp32,
    state_in / dstate_out: [B,H,N,N] fp32 or None.  Returns (dr, dk, dv, dx, du, dstate_in); outputs (and the
    workspace, unless a uint8 tensor of enough bytes is passed) are allocated here."""
    lib = load_library()
    B, T, H, N = r.shape
    f32 = torch.float32
    dt = r.dtype
    if dt not in (torch.bfloat16, f32):
        raise TypeError("backward: r must be bfloat16 or float32")
    sfx, wsfn = ("_f32", "gf_wkv6_backward_workspace_bytes") if dt == f32 else ("", "gf_wkv6_backward_bf16_workspace_bytes")
    if saved:       # the workspace holds the checkpoints of prefill_train() of the same inputs
        if dt == f32 or workspace is None:
            raise ValueError("backward(saved=True) needs bf16 tensors and the workspace prefill_train() filled")
        sfx = "_saved"
    dr, dk, dv, dx = (torch.empty_like(r) for _ in range(4))
    du = torch.empty((H, N), device=r.device, dtype=f32)
    ds0 = torch.empty((B, H, N, N), device=r.device, dtype=f32) if want_dstate else None
    with torch.cuda.device(r.device):
        nbytes = int(getattr(lib, wsfn)(B, T, H, N))
        ws = workspace if workspace is not None and workspace.numel() >= nbytes else torch.empty(max(nbytes, 16), dtype=torch.uint8, device=r.device)
        args = [_dev(r, "r", dt), _dev(k, "k", dt, r.shape), _dev(v, "v", dt, r.shape), _dev(x, "x", dt, r.shape),
                _dev(u, "u", f32, (H, N)), _dev(state_in, "state_in", f32, (B, H, N, N)), _dev(dy, "dy", dt, r.shape),
                _dev(dstate_out, "dstate_out", f32, (B, H, N, N)), _dev(dr, "dr"), _dev(dk, "dk"), _dev(dv, "dv"),
                _dev(dx, "dx"), _dev(du, "du"), _dev(ds0, "dstate_in")]
        _check(getattr(lib, "gf_wkv6_backward" + sfx)(*args, B, T, H, N, _dev(ws, "workspace"), ws.numel(), _stream(stream)),
               "gf_wkv6_backward" + sfx)
    return dr, dk, dv, dx, du, ds0


def backward_c2(r, k, v, x, dy, state_in=None, dstate_out=None, want_dstate=True, stream=None, workspace=None, saved=False):
    """gf_wkv6_backward_c2: gradient of prefill_c2 (bf16 tensors; k is the key before the (1 - w) factor; the
    second-value vector's gradient is dy itself).  Returns (dr, dk, dv, dx, dstate_in)."""
    lib = load_library()
    B, T, H, N = r.shape
    bf, f32 = torch.bfloat16, torch.float32
    dr, dk, dv, dx = (torch.empty_like(r) for _ in range(4))
    ds0 = torch.empty((B, H, N, N), device=r.device, dtype=f32) if want_dstate else None
    with torch.cuda.device(r.device):
        nbytes = int(lib.gf_wkv6_backward_bf16_workspace_bytes(B, T, H, N))
        ws = workspace if workspace is not None and workspace.numel() >= nbytes else torch.empty(max(nbytes, 16), dtype=torch.uint8, device=r.device)
        args = [_dev(r, "r", bf), _dev(k, "k", bf, r.shape), _dev(v, "v", bf, r.shape), _dev(x, "x", bf, r.shape),
                _dev(state_in, "state_in", f32, (B, H, N, N)), _dev(dy, "dy", bf, r.shape),
                _dev(dstate_out, "dstate_out", f32, (B, H, N, N)), _dev(dr, "dr"), _dev(dk, "dk"), _dev(dv, "dv"),
                _dev(dx, "dx"), _dev(ds0, "dstate_in")]
        if saved and workspace is None:
            raise ValueError("backward_c2(saved=True) needs the workspace prefill_c2_train() filled")
        fn = "gf_wkv6_backward_c2_saved" if saved else "gf_wkv6_backward_c2"
        _check(getattr(lib, fn)(*args, B, T, H, N, _dev(ws, "workspace"), ws.numel(), _stream(stream)), fn)
    return dr, dk, dv, dx, ds0


def backward_varlen(r, k, v, x, u, dy, cu_seqlens, max_seqlen, state_in=None, dstate_out=None, want_dstate=True,
                    stream=None, workspace=None, c2=False, saved=False):
    """gf_wkv6_backward_varlen / gf_wkv6_backward_varlen_c2 (saved=True: their _saved forms, from the states that
    prefill_varlen_train() left in `workspace`): gradient of the packed prefill (bf16 tensors).  r,k,v,x,dy:
    [total_T,H,N]; cu_seqlens: int32 CUDA [S+1]; u: [H,N] fp32 (ignored with c2=True); state_in / dstate_out:
    [S,H,N,N] fp32 or None.  Returns (dr, dk, dv, dx, du, dstate_in), du None with c2=True."""
    lib = load_library()
    total_T, H, N = r.shape
    S = cu_seqlens.numel() - 1
    bf, f32 = torch.bfloat16, torch.float32
    dr, dk, dv, dx = (torch.empty_like(r) for _ in range(4))
    du = None if c2 else torch.empty((H, N), device=r.device, dtype=f32)
    ds0 = torch.empty((S, H, N, N), device=r.device, dtype=f32) if want_dstate else None
    with torch.cuda.device(r.device):
        nbytes = int(lib.gf_wkv6_backward_varlen_workspace_bytes(S, total_T, H, N))
        ws = workspace if workspace is not None and workspace.numel() >= nbytes else torch.empty(max(nbytes, 16), dtype=torch.uint8, device=r.device)
        args = [_dev(r, "r", bf), _dev(k, "k", bf, r.shape), _dev(v, "v", bf, r.shape), _dev(x, "x", bf, r.shape)]
        if not c2:
            args.append(_dev(u, "u", f32, (H, N)))
        args += [_dev(state_in, "state_in", f32, (S, H, N, N)), _dev(dy, "dy", bf, r.shape),
                 _dev(dstate_out, "dstate_out", f32, (S, H, N, N)), _dev(dr, "dr"), _dev(dk, "dk"), _dev(dv, "dv"), _dev(dx, "dx")]
        if not c2:
            args.append(_dev(du, "du"))
        args += [_dev(ds0, "dstate_in"), _dev(cu_seqlens, "cu_seqlens", torch.int32)]
        fn = "gf_wkv6_backward_varlen_c2" if c2 else "gf_wkv6_backward_varlen"
        if saved:
            if workspace is None or workspace.numel() < nbytes:
                raise ValueError("backward_varlen(saved=True) needs the workspace prefill_varlen_train() filled")
            fn += "_saved"
        _check(getattr(lib, fn)(*args, S, total_T, int(max_seqlen), H, N, _dev(ws, "workspace"), ws.numel(), _stream(stream)), fn)
    return dr, dk, dv, dx, du, ds0


def prefill_train(r, k, v, x, u, workspace, state_in=None, c2=False, u2=None, stream=None):
    """gf_wkv6_prefill_train / gf_wkv6_prefill_c2_train: the forward pass of a training step.  As prefill() /
    prefill_c2() (u is ignored with c2=True, u2 without), and `workspace` (uint8 CUDA tensor of
    backward_workspace_bytes(B,T,H,N) bytes) receives the chunk-start states for backward(..., saved=True).
    Returns (y, state_out)."""
    lib = load_library()
    B, T, H, N = r.shape
    bf, f32 = torch.bfloat16, torch.float32
    y = torch.empty_like(r)
    s_out = torch.empty((B, H, N, N), device=r.device, dtype=f32)
    with torch.cuda.device(r.device):
        base = [_dev(r, "r", bf), _dev(k, "k", bf, r.shape), _dev(v, "v", bf, r.shape), _dev(x, "x", bf, r.shape)]
        mid = _dev(u2, "u2", bf, r.shape) if c2 else _dev(u, "u", f32, (H, N))
        fn = "gf_wkv6_prefill_c2_train" if c2 else "gf_wkv6_prefill_train"
        _check(getattr(lib, fn)(*base, mid, _dev(state_in, "state_in", f32, (B, H, N, N)), _dev(s_out, "state_out"),
                                _dev(y, "y"), B, T, H, N, _dev(workspace, "workspace"), workspace.numel(), _stream(stream)), fn)
    return y, s_out


def backward_workspace_bytes(B, T, H, N, dtype=torch.bfloat16):
    """Bytes of workspace backward() needs for tensors of this dtype on the current device."""
    lib = load_library()
    fn = "gf_wkv6_backward_workspace_bytes" if dtype == torch.float32 else "gf_wkv6_backward_bf16_workspace_bytes"
    return int(getattr(lib, fn)(B, T, H, N))


def prefill_varlen_train(r, k, v, x, u, cu_seqlens, max_seqlen, workspace, state_in=None, c2=False, u2=None, stream=None):
    """gf_wkv6_prefill_varlen_train / gf_wkv6_prefill_varlen_c2_train: the packed forward pass of a training step.  As
    prefill_varlen() / prefill_varlen_c2() (u is ignored with c2=True, u2 without); `workspace` (uint8 CUDA tensor of
    backward_varlen_workspace_bytes(S,total_T,H,N) bytes) receives the chunk-start states for
    backward_varlen(..., saved=True).  Returns (y, state_out)."""
    lib = load_library()
    total_T, H, N = r.shape
    S = cu_seqlens.numel() - 1
    bf, f32 = torch.bfloat16, torch.float32
    y = torch.empty_like(r)
    s_out = torch.empty((S, H, N, N), device=r.device, dtype=f32)
    with torch.cuda.device(r.device):
        base = [_dev(r, "r", bf), _dev(k, "k", bf, r.shape), _dev(v, "v", bf, r.shape), _dev(x, "x", bf, r.shape)]
        mid = _dev(u2, "u2", bf, r.shape) if c2 else _dev(u, "u", f32, (H, N))
        fn = "gf_wkv6_prefill_varlen_c2_train" if c2 else "gf_wkv6_prefill_varlen_train"
        _check(getattr(lib, fn)(*base, mid, _dev(state_in, "state_in", f32, (S, H, N, N)), _dev(s_out, "state_out"),
                                _dev(y, "y"), _dev(cu_seqlens, "cu_seqlens", torch.int32), S, total_T, int(max_seqlen), H, N,
                                _dev(workspace, "workspace"), workspace.numel(), _stream(stream)), fn)
    return y, s_out


def backward_varlen_workspace_bytes(S, total_T, H, N):
    """Bytes of workspace backward_varlen() needs on the current device."""
    return int(load_library().gf_wkv6_backward_varlen_workspace_bytes(S, total_T, H, N))


def prefill_c2(r, k, v, x, u2=None, state_in=None, state_out=None, y=None, stream=None, want_state=True, split=True):
    """gf_wkv6_prefill_c2: the Finch-C2 form.  r,k,v,x (and u2, the per-token second-value vector, or
    None): [B,T,H,N] bf16 CUDA tensors; k is the key before the (1 - w) factor.  Returns (y, state_out)."""
    lib = load_library()
    B, T, H, N = r.shape
    bf = torch.bfloat16
    if y is None:
        y = torch.empty_like(r)
    if state_out is None and want_state:
        state_out = torch.empty((B, H, N, N), device=r.device, dtype=torch.float32)
    args = [_dev(r, "r", bf), _dev(k, "k", bf, r.shape), _dev(v, "v", bf, r.shape), _dev(x, "x", bf, r.shape),
            _dev(u2, "u2", bf, r.shape), _dev(state_in, "state_in", torch.float32, (B, H, N, N)),
            _dev(state_out, "state_out", torch.float32, (B, H, N, N)), _dev(y, "y", bf, r.shape)]
    with torch.cuda.device(r.device):
        if split:
            _ensure_workspace(B, T, H, N, r.device)
        elif _workspace is not None:
            set_workspace(None)
        _check(lib.gf_wkv6_prefill_c2(*args, B, T, H, N, _stream(stream)), "gf_wkv6_prefill_c2")
    return y, state_out


def prefill_varlen_c2(r, k, v, x, u2, cu_seqlens, max_seqlen, state_in=None, state_out=None, y=None,
                      stream=None, want_state=True, split=True):
    """gf_wkv6_prefill_varlen_c2: packed Finch-C2 prefill.  r,k,v,x,u2 (u2 may be None): [total_T,H,N] bf16."""
    lib = load_library()
    total_T, H, N = r.shape
    S = cu_seqlens.numel() - 1
    bf = torch.bfloat16
    if y is None:
        y = torch.empty_like(r)
    if state_out is None and want_state:
        state_out = torch.empty((S, H, N, N), device=r.device, dtype=torch.float32)
    args = [_dev(r, "r", bf), _dev(k, "k", bf, r.shape), _dev(v, "v", bf, r.shape), _dev(x, "x", bf, r.shape),
            _dev(u2, "u2", bf, r.shape), _dev(state_in, "state_in", torch.float32, (S, H, N, N)),
            _dev(state_out, "state_out", torch.float32, (S, H, N, N)), _dev(y, "y", bf, r.shape),
            _dev(cu_seqlens, "cu_seqlens", torch.int32)]
    with torch.cuda.device(r.device):
        if split:
            _ensure_workspace(S, int(max_seqlen), H, N, r.device)
        elif _workspace is not None:
            set_workspace(None)
        _check(lib.gf_wkv6_prefill_varlen_c2(*args, S, total_T, int(max_seqlen), H, N, _stream(stream)),
               "gf_wkv6_prefill_varlen_c2")
    return y, state_out


def step_c2(r, k, v, x, u2, state_in, state_out=None, y=None, stream=None):
    """gf_wkv6_step_c2: one Finch-C2 decode token per sequence.  r,k,v,x,u2 (u2 may be None): [B,H,N] bf16;
    state_out defaults to state_in (in-place update)."""
    lib = load_library()
    B, H, N = r.shape
    bf = torch.bfloat16
    if y is None:
        y = torch.empty_like(r)
    if state_out is None:
        state_out = state_in if state_in is not None else torch.empty((B, H, N, N), device=r.device, dtype=torch.float32)
    args = [_dev(r, "r", bf), _dev(k, "k", bf, r.shape), _dev(v, "v", bf, r.shape), _dev(x, "x", bf, r.shape),
            _dev(u2, "u2", bf, r.shape), _dev(state_in, "state_in", torch.float32, (B, H, N, N)),
            _dev(state_out, "state_out", torch.float32, (B, H, N, N)), _dev(y, "y", bf, r.shape)]
    with torch.cuda.device(r.device):
        _check(lib.gf_wkv6_step_c2(*args, B, H, N, _stream(stream)), "gf_wkv6_step_c2")
    return y, state_out


SUMMARY_FLOATS = 64 + 64 * 64         # per (b,h): decay product D[64], then dS[64][64]


def sequence_summary(k, v, x, c2=False, out=None, stream=None):
    """gf_wkv6_sequence_summary: (D, dS) of every (b,h) of a bf16 [B,T,H,N] run -> fp32 [B,H,64+4096]."""
    lib = load_library()
    B, T, H, N = k.shape
    bf = torch.bfloat16
    if out is None:
        out = torch.empty((B, H, SUMMARY_FLOATS), device=k.device, dtype=torch.float32)
    with torch.cuda.device(k.device):
        _check(lib.gf_wkv6_sequence_summary(_dev(k, "k", bf), _dev(v, "v", bf, k.shape), _dev(x, "x", bf, k.shape),
                                            _dev(out, "summary", torch.float32, (B, H, SUMMARY_FLOATS)), B, T, H, N,
                                            1 if c2 else 0, _stream(stream)), "gf_wkv6_sequence_summary")
    return out


def fold_summaries(state_in, summaries, n_fold, state_out=None, stream=None):
    """gf_wkv6_fold_summaries: apply the first n_fold of summaries [P,B,H,64+4096] to state_in ([B,H,N,N] or None)."""
    lib = load_library()
    P, B, H, F = summaries.shape
    assert F == SUMMARY_FLOATS and 0 <= n_fold <= P
    if state_out is None:
        state_out = torch.empty((B, H, 64, 64), device=summaries.device, dtype=torch.float32)
    with torch.cuda.device(summaries.device):
        _check(lib.gf_wkv6_fold_summaries(_dev(state_in, "state_in", torch.float32, (B, H, 64, 64)),
                                          _dev(summaries, "summaries", torch.float32), int(n_fold), B, H, 64,
                                          _dev(state_out, "state_out", torch.float32, (B, H, 64, 64)), _stream(stream)),
               "gf_wkv6_fold_summaries")
    return state_out


def layernorm_heads(y, gamma=None, beta=None, eps=1e-5, out=None, stream=None):
    """gf_c2_layernorm(_f32): LayerNorm over all H*N channels of every token.  y: [..., H, N] CUDA tensor
    (bf16 or fp32, contiguous); gamma, beta: fp32 [H*N] (or [H, N]) or None.  out defaults to a new tensor
    (pass out=y for in place).  Returns out."""
    lib = load_library()
    H, N = y.shape[-2], y.shape[-1]
    rows = y.numel() // (H * N) if H * N else 0
    sfx = _suffix(y.dtype)
    if out is None:
        out = torch.empty_like(y)
    with torch.cuda.device(y.device):
        _check(getattr(lib, "gf_c2_layernorm" + sfx)(
            _dev(y, "y"), _dev(None if gamma is None else gamma.reshape(H * N), "gamma", torch.float32),
            _dev(None if beta is None else beta.reshape(H * N), "beta", torch.float32), float(eps),
            _dev(out, "out", y.dtype, y.shape), rows, H, N, _stream(stream)), "gf_c2_layernorm" + sfx)
    return out


def key_compress(x, w_kd, out=None, stream=None):
    """gf_gold_key_compress: c = x @ w_kd.  x: [..., D] bf16 CUDA tensor (contiguous), w_kd: [D, Dc] bf16.
    Returns c [..., Dc] bf16 (allocated here unless passed as out)."""
    lib = load_library()
    D, Dc = w_kd.shape
    assert x.shape[-1] == D
    rows = x.numel() // D if D else 0
    bf = torch.bfloat16
    if out is None:
        out = torch.empty(x.shape[:-1] + (Dc,), device=x.device, dtype=bf)
    with torch.cuda.device(x.device):
        _check(lib.gf_gold_key_compress(_dev(x, "x", bf), _dev(w_kd, "w_kd", bf, (D, Dc)), _dev(out, "c", bf, x.shape[:-1] + (Dc,)),
                                        rows, D, Dc, _stream(stream)), "gf_gold_key_compress")
    return out


def decay_logit(x, mu_x, A_d, B_d, lambda_d, A_w, B_w, lambda_w, x_prev=None, out=None, stream=None):
    """gf_c2_decay_logit: d = lora_omega(ddlerp_d(x_t, x_{t-1})).  x: [B,T,D] bf16 CUDA tensor (contiguous); mu_x,
    lambda_d, lambda_w: fp32 [D]; A_d [D,Rd], B_d [Rd,D], A_w [D,Rw], B_w [Rw,D]: bf16; x_prev: [B,D] bf16 or None.
    Returns d [B,T,D] bf16 (allocated here unless passed as out)."""
    lib = load_library()
    B, T, D = x.shape
    Rd, Rw = A_d.shape[1], A_w.shape[1]
    bf, f32 = torch.bfloat16, torch.float32
    if out is None:
        out = torch.empty_like(x)
    with torch.cuda.device(x.device):
        _check(lib.gf_c2_decay_logit(
            _dev(x, "x", bf), _dev(x_prev, "x_prev", bf, (B, D)), _dev(mu_x, "mu_x", f32, (D,)),
            _dev(A_d, "A_d", bf, (D, Rd)), _dev(B_d, "B_d", bf, (Rd, D)), _dev(lambda_d, "lambda_d", f32, (D,)),
            _dev(A_w, "A_w", bf, (D, Rw)), _dev(B_w, "B_w", bf, (Rw, D)), _dev(lambda_w, "lambda_w", f32, (D,)),
            _dev(out, "d", bf, x.shape), B, T, D, Rd, Rw, _stream(stream)), "gf_c2_decay_logit")
    return out


STATIC_SCRATCH_BYTES = 2121728       # GF_WKV6_STATIC_SCRATCH_BYTES


def prefill_static(r, k, v, x, u, state_in, state_out, y, stream=None) -> None:
    """gf_wkv6_prefill_static: the dense bf16 prefill for callers that cannot allocate.  Nothing is
    allocated here either: y [B,T,H,N] bf16 and state_out [B,H,N,N] fp32 (or None) are the caller's,
    and the sequence split uses the scratch built into the library (as many segments as fit into its
    STATIC_SCRATCH_BYTES).  Raises GfError(GF_ERR_WORKSPACE) when not even two segments fit."""
    lib = load_library()
    B, T, H, N = r.shape
    bf = torch.bfloat16
    args = [_dev(r, "r", bf), _dev(k, "k", bf, r.shape), _dev(v, "v", bf, r.shape), _dev(x, "x", bf, r.shape),
            _dev(u, "u", torch.float32, (H, N)), _dev(state_in, "state_in", torch.float32, (B, H, N, N)),
            _dev(state_out, "state_out", torch.float32, (B, H, N, N)), _dev(y, "y", bf, r.shape)]
    with torch.cuda.device(r.device):
        _check(lib.gf_wkv6_prefill_static(*args, B, T, H, N, _stream(stream)), "gf_wkv6_prefill_static")


def prefill_varlen(r, k, v, x, u, cu_seqlens, max_seqlen, state_in=None, state_out=None, y=None,
                   stream=None, want_state=True, split=True):
    """gf_wkv6_prefill_varlen(_f32).  r,k,v,x: [total_T,H,N]; cu_seqlens: int32 CUDA [S+1];
    states [S,H,N,N].  Returns (y, state_out).  split as for prefill (cut by max_seqlen)."""
    lib = load_library()
    total_T, H, N = r.shape
    S = cu_seqlens.numel() - 1
    sfx = _suffix(r.dtype)
    if y is None:
        y = torch.empty_like(r)
    if state_out is None and want_state:
        state_out = torch.empty((S, H, N, N), device=r.device, dtype=torch.float32)
    args = [_dev(r, "r"), _dev(k, "k", r.dtype, r.shape), _dev(v, "v", r.dtype, r.shape),
            _dev(x, "x", r.dtype, r.shape), _dev(u, "u", torch.float32, (H, N)),
            _dev(state_in, "state_in", torch.float32, (S, H, N, N)),
            _dev(state_out, "state_out", torch.float32, (S, H, N, N)), _dev(y, "y", r.dtype, r.shape),
            _dev(cu_seqlens, "cu_seqlens", torch.int32)]
    with torch.cuda.device(r.device):
        if sfx == "" and split:
            _ensure_workspace(S, int(max_seqlen), H, N, r.device)
        elif not split and _workspace is not None:
            set_workspace(None)
        _check(getattr(lib, "gf_wkv6_prefill_varlen" + sfx)(*args, S, total_T, int(max_seqlen), H, N, _stream(stream)),
               "gf_wkv6_prefill_varlen" + sfx)
    return y, state_out


def step(r, k, v, x, u, state_in, state_out=None, y=None, stream=None):
    """gf_wkv6_step(_f32): one decode token per sequence.  r,k,v,x: [B,H,N]; state [B,H,N,N].
    state_out defaults to state_in (in-place update).  Returns (y, state_out)."""
    lib = load_library()
    B, H, N = r.shape
    sfx = _suffix(r.dtype)
    if y is None:
        y = torch.empty_like(r)
    if state_out is None:
        state_out = state_in if state_in is not None else torch.empty((B, H, N, N), device=r.device, dtype=torch.float32)
    args = [_dev(r, "r"), _dev(k, "k", r.dtype, r.shape), _dev(v, "v", r.dtype, r.shape),
            _dev(x, "x", r.dtype, r.shape), _dev(u, "u", torch.float32, (H, N)),
            _dev(state_in, "state_in", torch.float32, (B, H, N, N)),
            _dev(state_out, "state_out", torch.float32, (B, H, N, N)), _dev(y, "y", r.dtype, r.shape)]
    with torch.cuda.device(r.device):
        _check(getattr(lib, "gf_wkv6_step" + sfx)(*args, B, H, N, _stream(stream)), "gf_wkv6_step" + sfx)
    return y, state_out


def bind_step(r, k, v, x, u, state, y=None, stream=None):
    """Pre-marshalled decode step for loops that reuse the same buffers (the caller refreshes r,k,v,x in
    place every token, the state is updated in place): checks and pointer extraction happen once here, the
    returned zero-argument callable is one C call.  Returns (callable, y)."""
    lib = load_library()
    B, H, N = r.shape
    sfx = _suffix(r.dtype)
    if y is None:
        y = torch.empty_like(r)
    args = [_dev(r, "r"), _dev(k, "k", r.dtype, r.shape), _dev(v, "v", r.dtype, r.shape),
            _dev(x, "x", r.dtype, r.shape), _dev(u, "u", torch.float32, (H, N)),
            _dev(state, "state", torch.float32, (B, H, N, N)), _dev(state, "state", torch.float32, (B, H, N, N)),
            _dev(y, "y", r.dtype, r.shape), B, H, N, _stream(stream)]
    fn = getattr(lib, "gf_wkv6_step" + sfx)
    keep = (r, k, v, x, u, state, y)                 # the bound buffers must outlive the callable
    index = r.device.index

    def call():
        if torch.cuda.current_device() != index:
            raise RuntimeError("bind_step: the bound tensors' device is not the current device")
        status = fn(*args)
        if status != GF_OK:
            raise GfError(status, "gf_wkv6_step" + sfx)

    call.buffers = keep
    return call, y


def host_workspace_bytes(B, T, H, N) -> int:
    return int(load_library().gf_wkv6_host_workspace_bytes(B, T, H, N))


def _host(t: torch.Tensor | None, name: str):
    if t is None:
        return None
    if t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous host tensor")
    return t.data_ptr()


def prefill_host(r, k, v, x, u, state_in, state_out, y, dev_ws, stream=None):
    """gf_wkv6_prefill_host: bf16 host tensors in (pinned for speed), y / state_out host tensors
    out, staged through the caller's CUDA byte buffer ``dev_ws``.  Asynchronous on the stream."""
    lib = load_library()
    B, T, H, N = r.shape
    args = [_host(r, "r"), _host(k, "k"), _host(v, "v"), _host(x, "x"), _host(u, "u"),
            _host(state_in, "state_in"), _host(state_out, "state_out"), _host(y, "y")]
    with torch.cuda.device(dev_ws.device):
        _check(lib.gf_wkv6_prefill_host(*args, B, T, H, N, _dev(dev_ws, "dev_ws"), dev_ws.numel() * dev_ws.element_size(),
                                        _stream(stream)), "gf_wkv6_prefill_host")
