"""ctypes front end of the fp64 CPU oracle (``wkv6_oracle.c``).

TEST INFRASTRUCTURE ONLY: the test-suite, the smoke check and the CPU-baseline leg
of the benchmark may import this module; the CUDA library and its Python binding
never do, and this module imports nothing from them.

All functions take numpy arrays or torch CPU tensors.  r, k, v, x may be float32 or
bfloat16 (torch); they are widened exactly to float32 for transport and to float64
inside the C code, so the oracle sees precisely the values the GPU sees.
"""
from __future__ import annotations

import ctypes
import hashlib
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "wkv6_oracle.c")
_lib = None


def _host_tag() -> str:
    """The library is compiled for the host it runs on (-march=native), so its file name carries a tag of the
    host's instruction-set flags: a copy built on another kind of machine is not picked up."""
    flags = ""
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags") or line.startswith("Features"):
                    flags = line
                    break
    except OSError:
        pass
    return hashlib.md5(flags.encode()).hexdigest()[:8]


_LIB = os.path.join(_HERE, f"libwkv6_oracle_{_host_tag()}.so")


def build(force: bool = False) -> str:
    """Compile the C oracle next to its source (gcc, OpenMP) and return the path.  -ffp-contract=off keeps every
    product and sum a rounding of its own, as the loops are written."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O3", "-march=native", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", "-std=c99",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.wkv6_oracle_threads.restype = ctypes.c_int
        _lib.wkv6_oracle_prefill.restype = None
        _lib.wkv6_oracle_prefill_varlen.restype = None
        _lib.wkv6_oracle_prefill_c2.restype = None
        _lib.c2_oracle_layernorm.restype = None
        _lib.gold_oracle_key_compress.restype = None
        _lib.c2_oracle_decay_logit.restype = None
        _lib.wkv6_oracle_backward.restype = None
    return _lib


def threads() -> int:
    """Number of host threads the oracle's OpenMP loops use."""
    return int(_load().wkv6_oracle_threads())


def _f32(a):
    """Exact float32 numpy copy of a numpy array / torch tensor (bf16 widens exactly)."""
    if a is None:
        return None
    if hasattr(a, "detach"):  # torch tensor
        a = a.detach().cpu().float().numpy()
    a = np.ascontiguousarray(a)
    if a.dtype == np.float64:
        b = a.astype(np.float32)
        if not np.array_equal(b.astype(np.float64), a, equal_nan=True):
            raise ValueError("float64 input is not exactly representable in float32")
        a = b
    if a.dtype != np.float32:
        raise TypeError(f"unsupported dtype {a.dtype}")
    return a


def _p(a, ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def prefill(r, k, v, x, u, state_in=None, w=None):
    """Dense WKV-6 prefill.  r,k,v,x: [B,T,H,N]; u: [H,N]; state_in: [B,H,N,N] or None.

    ``w`` (float64 [B,T,H,N]), if given, is used as the decay directly and ``x`` is
    ignored (x may then be None): this states the w == 1 / w == 0 invariants exactly.
    Returns (y float64 [B,T,H,N], state_out float64 [B,H,N,N]).
    """
    lib = _load()
    r, k, v, u = _f32(r), _f32(k), _f32(v), _f32(u)
    x = _f32(x)
    state_in = _f32(state_in)
    B, T, H, N = r.shape
    assert k.shape == r.shape and v.shape == r.shape and u.shape == (H, N)
    if w is not None:
        w = np.ascontiguousarray(np.asarray(w, dtype=np.float64))
        assert w.shape == r.shape
    else:
        assert x is not None and x.shape == r.shape
    if state_in is not None:
        assert state_in.shape == (B, H, N, N)
    y = np.zeros((B, T, H, N), dtype=np.float64)
    s_out = np.zeros((B, H, N, N), dtype=np.float64)
    f, d = ctypes.c_float, ctypes.c_double
    lib.wkv6_oracle_prefill(_p(r, f), _p(k, f), _p(v, f), _p(x, f), _p(w, d), _p(u, f),
                            _p(state_in, f), _p(s_out, d), _p(y, d),
                            ctypes.c_long(B), ctypes.c_long(T), ctypes.c_long(H), ctypes.c_long(N))
    return y, s_out


def prefill_c2(r, k, v, x, u2=None, state_in=None, w=None):
    """Finch-C2 form (the paper's Finch-C2 block): the key entering the state is k (1 - w), no bonus,
    y_t = r_t . wkv_t + u2_t.  r,k,v,x,u2: [B,T,H,N] (u2 may be None); ``w`` as in prefill().
    Returns (y float64 [B,T,H,N], state_out float64 [B,H,N,N])."""
    lib = _load()
    r, k, v, x, u2, state_in = _f32(r), _f32(k), _f32(v), _f32(x), _f32(u2), _f32(state_in)
    B, T, H, N = r.shape
    assert k.shape == r.shape and v.shape == r.shape and (u2 is None or u2.shape == r.shape)
    if w is not None:
        w = np.ascontiguousarray(np.asarray(w, dtype=np.float64))
        assert w.shape == r.shape
    else:
        assert x is not None and x.shape == r.shape
    y = np.zeros((B, T, H, N), dtype=np.float64)
    s_out = np.zeros((B, H, N, N), dtype=np.float64)
    f, d = ctypes.c_float, ctypes.c_double
    lib.wkv6_oracle_prefill_c2(_p(r, f), _p(k, f), _p(v, f), _p(x, f), _p(w, d), _p(u2, f),
                               _p(state_in, f), _p(s_out, d), _p(y, d),
                               ctypes.c_long(B), ctypes.c_long(T), ctypes.c_long(H), ctypes.c_long(N))
    return y, s_out


def prefill_varlen(r, k, v, x, u, cu_seqlens, state_in=None):
    """Packed variable-length prefill.  r,k,v,x: [total_T,H,N]; cu_seqlens: int32 [S+1];
    state_in: [S,H,N,N] or None.  Returns (y [total_T,H,N], state_out [S,H,N,N]) in float64."""
    lib = _load()
    r, k, v, x, u = _f32(r), _f32(k), _f32(v), _f32(x), _f32(u)
    state_in = _f32(state_in)
    if hasattr(cu_seqlens, "detach"):
        cu_seqlens = cu_seqlens.detach().cpu().numpy()
    cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int32))
    total_T, H, N = r.shape
    S = cu.shape[0] - 1
    assert cu[0] == 0 and cu[-1] == total_T and np.all(np.diff(cu) >= 0)
    if state_in is not None:
        assert state_in.shape == (S, H, N, N)
    y = np.zeros((total_T, H, N), dtype=np.float64)
    s_out = np.zeros((S, H, N, N), dtype=np.float64)
    f, d = ctypes.c_float, ctypes.c_double
    lib.wkv6_oracle_prefill_varlen(_p(r, f), _p(k, f), _p(v, f), _p(x, f), _p(u, f),
                                   _p(state_in, f), _p(s_out, d), _p(y, d),
                                   cu.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                   ctypes.c_long(S), ctypes.c_long(H), ctypes.c_long(N))
    return y, s_out


def step(r, k, v, x, u, state_in):
    """Single-token decode step: r,k,v,x [B,H,N]; state_in [B,H,N,N].  Defined as a
    prefill of length one (new-token generation runs the same recurrence)."""
    r, k, v, x = (_f32(a)[:, None] for a in (r, k, v, x))
    y, s = prefill(r, k, v, x, u, state_in)
    return y[:, 0], s


def layernorm_heads(y, gamma=None, beta=None, eps=1e-5):
    """LayerNorm over all D = H*N channels of each token (the o_t equation of the Finch-C2 block, before
    W^O).  y: [..., H, N] or [rows, D] (numpy / torch, any float type; widened exactly to float64 and
    flattened to rows of D); gamma, beta: [D] or None.  Returns float64 of y's shape."""
    lib = _load()
    if hasattr(y, "detach"):
        y = y.detach().cpu().double().numpy()
    y = np.ascontiguousarray(np.asarray(y, dtype=np.float64))
    D = y.shape[-1] * (y.shape[-2] if y.ndim >= 3 else 1)
    rows = y.size // D if D else 0
    cv = lambda a: None if a is None else np.ascontiguousarray(
        (a.detach().cpu().double().numpy() if hasattr(a, "detach") else np.asarray(a, dtype=np.float64)).reshape(D))
    gamma, beta = cv(gamma), cv(beta)
    out = np.zeros_like(y)
    d = ctypes.c_double
    lib.c2_oracle_layernorm(_p(y, d), _p(gamma, d), _p(beta, d), d(float(eps)), _p(out, d),
                            ctypes.c_long(rows), ctypes.c_long(D))
    return out


def key_compress(x, w_kd):
    """GOLD key compression c_t = x_t W^{KD} (the compressed key cache entry of every token).  x: [..., D]
    (numpy / torch, any float type, widened exactly to float64); w_kd: [D, Dc].  Returns float64 [..., Dc]."""
    lib = _load()
    cv = lambda a: np.ascontiguousarray(a.detach().cpu().double().numpy() if hasattr(a, "detach") else np.asarray(a, dtype=np.float64))
    x, w = cv(x), cv(w_kd)
    D, Dc = w.shape
    assert x.shape[-1] == D
    rows = x.size // D if D else 0
    c = np.zeros(x.shape[:-1] + (Dc,), dtype=np.float64)
    d = ctypes.c_double
    lib.gold_oracle_key_compress(_p(x, d), _p(w, d), _p(c, d), ctypes.c_long(rows), ctypes.c_long(D), ctypes.c_long(Dc))
    return c


def _f64(a, shape=None):
    """Exact float64 numpy copy of a numpy array / torch tensor of any float type."""
    if a is None:
        return None
    if hasattr(a, "detach"):
        a = a.detach().cpu().double().numpy()
    a = np.ascontiguousarray(np.asarray(a, dtype=np.float64))
    if shape is not None:
        assert a.shape == tuple(shape), (a.shape, shape)
    return a


def decay_logit(x, mu_x, A_d, B_d, lambda_d, A_w, B_w, lambda_w, x_prev=None):
    """The decay logit of the Finch-C2 block, d_t = lora_omega(ddlerp_d(x_t, x_{t-1})) (lerp / lora / ddlerp as the
    Finch-C2 section defines them).  x: [B,T,D]; mu_x, lambda_d, lambda_w: [D]; A_d: [D,Rd], B_d: [Rd,D] (the lora
    inside ddlerp_d); A_w: [D,Rw], B_w: [Rw,D] (lora_omega); x_prev: [B,D], the token before each sequence's first
    (None: zeros).  Any float type, widened exactly to float64.  Returns d float64 [B,T,D]."""
    lib = _load()
    x = _f64(x)
    B, T, D = x.shape
    A_d, A_w = _f64(A_d), _f64(A_w)
    Rd, Rw = A_d.shape[1], A_w.shape[1]
    assert A_d.shape == (D, Rd) and A_w.shape == (D, Rw)
    B_d, B_w = _f64(B_d, (Rd, D)), _f64(B_w, (Rw, D))
    mu_x, lambda_d, lambda_w = _f64(mu_x, (D,)), _f64(lambda_d, (D,)), _f64(lambda_w, (D,))
    x_prev = _f64(x_prev, (B, D)) if x_prev is not None else None
    d = np.zeros((B, T, D), dtype=np.float64)
    c = ctypes.c_double
    lib.c2_oracle_decay_logit(_p(x, c), _p(x_prev, c), _p(mu_x, c), _p(A_d, c), _p(B_d, c), _p(lambda_d, c),
                              ctypes.c_long(Rd), _p(A_w, c), _p(B_w, c), _p(lambda_w, c), ctypes.c_long(Rw),
                              _p(d, c), ctypes.c_long(B), ctypes.c_long(T), ctypes.c_long(D))
    return d


def backward(r, k, v, x, u, dy, state_in=None, dstate_out=None):
    """Gradient of prefill(): given dy = dL/dy [B,T,H,N] and dstate_out = dL/dS_T [B,H,N,N] (None: zero), returns
    (dr, dk, dv, dx [B,T,H,N], du [H,N] summed over the batch, dstate_in [B,H,N,N]) in float64.  r,k,v,x,u,state_in
    as for prefill() (float32 / bfloat16 carriers)."""
    lib = _load()
    r, k, v, x, u, state_in = _f32(r), _f32(k), _f32(v), _f32(x), _f32(u), _f32(state_in)
    B, T, H, N = r.shape
    dy = _f64(dy, (B, T, H, N))
    dsT = _f64(dstate_out, (B, H, N, N)) if dstate_out is not None else None
    outs = [np.zeros((B, T, H, N), dtype=np.float64) for _ in range(4)]
    du_b = np.zeros((B, H, N), dtype=np.float64)
    ds0 = np.zeros((B, H, N, N), dtype=np.float64)
    f, c = ctypes.c_float, ctypes.c_double
    lib.wkv6_oracle_backward(_p(r, f), _p(k, f), _p(v, f), _p(x, f), _p(u, f), _p(state_in, f), _p(dy, c), _p(dsT, c),
                             _p(outs[0], c), _p(outs[1], c), _p(outs[2], c), _p(outs[3], c), _p(du_b, c), _p(ds0, c),
                             ctypes.c_long(B), ctypes.c_long(T), ctypes.c_long(H), ctypes.c_long(N))
    return outs[0], outs[1], outs[2], outs[3], du_b.sum(axis=0), ds0


def backward_c2(r, k, v, x, dy, state_in=None, dstate_out=None):
    """Gradient of prefill_c2() (the Finch-C2 form: keys k (1 - w), no bonus; u2 only adds, so its gradient is dy
    itself and is not returned).  Returns (dr, dk, dv, dx [B,T,H,N], dstate_in [B,H,N,N]) in float64."""
    lib = _load()
    r, k, v, x, state_in = _f32(r), _f32(k), _f32(v), _f32(x), _f32(state_in)
    B, T, H, N = r.shape
    dy = _f64(dy, (B, T, H, N))
    dsT = _f64(dstate_out, (B, H, N, N)) if dstate_out is not None else None
    outs = [np.zeros((B, T, H, N), dtype=np.float64) for _ in range(4)]
    ds0 = np.zeros((B, H, N, N), dtype=np.float64)
    f, c = ctypes.c_float, ctypes.c_double
    lib.wkv6_oracle_backward_c2.restype = None
    lib.wkv6_oracle_backward_c2(_p(r, f), _p(k, f), _p(v, f), _p(x, f), _p(state_in, f), _p(dy, c), _p(dsT, c),
                                _p(outs[0], c), _p(outs[1], c), _p(outs[2], c), _p(outs[3], c), _p(ds0, c),
                                ctypes.c_long(B), ctypes.c_long(T), ctypes.c_long(H), ctypes.c_long(N))
    return outs[0], outs[1], outs[2], outs[3], ds0


def _cu(cu_seqlens, total_T):
    if hasattr(cu_seqlens, "detach"):
        cu_seqlens = cu_seqlens.detach().cpu().numpy()
    cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int32))
    assert cu[0] == 0 and cu[-1] == total_T and np.all(np.diff(cu) >= 0)
    return cu


def backward_varlen(r, k, v, x, u, dy, cu_seqlens, state_in=None, dstate_out=None):
    """Gradient of prefill_varlen(): r,k,v,x,dy [total_T,H,N], cu_seqlens int32 [S+1], state_in / dstate_out [S,H,N,N]
    or None (zero).  Returns (dr, dk, dv, dx [total_T,H,N], du [H,N] summed over the sequences, dstate_in [S,H,N,N])
    in float64."""
    lib = _load()
    r, k, v, x, u, state_in = _f32(r), _f32(k), _f32(v), _f32(x), _f32(u), _f32(state_in)
    total_T, H, N = r.shape
    cu = _cu(cu_seqlens, total_T)
    S = cu.shape[0] - 1
    dy = _f64(dy, (total_T, H, N))
    dsT = _f64(dstate_out, (S, H, N, N)) if dstate_out is not None else None
    outs = [np.zeros((total_T, H, N), dtype=np.float64) for _ in range(4)]
    du_s = np.zeros((S, H, N), dtype=np.float64)
    ds0 = np.zeros((S, H, N, N), dtype=np.float64)
    f, c = ctypes.c_float, ctypes.c_double
    lib.wkv6_oracle_backward_varlen.restype = None
    lib.wkv6_oracle_backward_varlen(_p(r, f), _p(k, f), _p(v, f), _p(x, f), _p(u, f), _p(state_in, f), _p(dy, c),
                                    _p(dsT, c), _p(outs[0], c), _p(outs[1], c), _p(outs[2], c), _p(outs[3], c),
                                    _p(du_s, c), _p(ds0, c), cu.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                    ctypes.c_long(S), ctypes.c_long(H), ctypes.c_long(N))
    return outs[0], outs[1], outs[2], outs[3], du_s.sum(axis=0), ds0


def backward_c2_varlen(r, k, v, x, dy, cu_seqlens, state_in=None, dstate_out=None):
    """Gradient of the Finch-C2 form over a packed batch (layouts as backward_varlen; no bonus, so no du).  Returns
    (dr, dk, dv, dx [total_T,H,N], dstate_in [S,H,N,N]) in float64."""
    lib = _load()
    r, k, v, x, state_in = _f32(r), _f32(k), _f32(v), _f32(x), _f32(state_in)
    total_T, H, N = r.shape
    cu = _cu(cu_seqlens, total_T)
    S = cu.shape[0] - 1
    dy = _f64(dy, (total_T, H, N))
    dsT = _f64(dstate_out, (S, H, N, N)) if dstate_out is not None else None
    outs = [np.zeros((total_T, H, N), dtype=np.float64) for _ in range(4)]
    ds0 = np.zeros((S, H, N, N), dtype=np.float64)
    f, c = ctypes.c_float, ctypes.c_double
    lib.wkv6_oracle_backward_c2_varlen.restype = None
    lib.wkv6_oracle_backward_c2_varlen(_p(r, f), _p(k, f), _p(v, f), _p(x, f), _p(state_in, f), _p(dy, c), _p(dsT, c),
                                       _p(outs[0], c), _p(outs[1], c), _p(outs[2], c), _p(outs[3], c), _p(ds0, c),
                                       cu.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                       ctypes.c_long(S), ctypes.c_long(H), ctypes.c_long(N))
    return outs[0], outs[1], outs[2], outs[3], ds0


def rel_l2(a, b) -> float:
    """||a - b||_2 / ||b||_2 in float64 (b is the reference)."""
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    den = float(np.linalg.norm(b))
    num = float(np.linalg.norm(a - b))
    return num / den if den > 0 else num
