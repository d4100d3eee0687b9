"""Runs one of the benchmark configurations of the WKV-6 library a few times on the current CUDA device and
prints one JSON line per case with CUDA-event timings (inputs resident in HBM, seeded synthetic data).

    python -m paper_2407_12077_b200.cases [--reps N] [--scale F] case [case ...]      (or: all)

cases: cfg0 cfg1 cfg2 cfg2-c2 cfg3 cfg3-segments cfg3-packed cfg4-prefill cfg4-decode cfg4-decode-layers ln-cfg1 ln-cfg2 ln-wide kc-cfg2 kc-wide
       dl-cfg1 dl-cfg2 bwd-cfg1 bwd-cfg2 bwd-cfg3 bwd-cfg3-packed bwd-cfg4 train-fwd-cfg2 train-bwd-cfg2
--scale shrinks the time axis (T, sequence lengths) for quick runs or profiler captures.

`bytes` is the algorithmic HBM traffic of one run of the case (r,k,v,x in, y out, states in/out), `frac` that
traffic over the time, relative to ``--peak-gbs`` (default: the measured copy bandwidth recorded in
MEASURED_PEAKS.json at the repository root when present, else 6650 GB/s).
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import torch

import paper_2407_12077_b200 as gf
from paper_2407_12077_b200 import synth

DEV = "cuda:0"


def _peak(default=6650.0):
    p = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(p))["hbm_gbs"])
    except Exception:
        return default


def _time(fn, reps):
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    gf.last_device_status()
    return e0.elapsed_time(e1) / reps


def _dense(name, B, T, H, dtype, state_std, reps, c2=False):
    inp = synth.make_dense(B, T, H, 64, dtype, seed=7, device=DEV, state_std=state_std)
    y = torch.empty_like(inp.r)
    s = torch.empty((B, H, 64, 64), device=DEV)
    esz = 2 if dtype == "bf16" else 4
    nbytes = B * T * H * 64 * esz * 5 + B * H * 16384 * (2 if state_std > 0 else 1)
    if c2:
        u2 = torch.randn(inp.r.shape, device=DEV).bfloat16()
        nbytes += B * T * H * 128
        fn = lambda: gf.prefill_c2(inp.r, inp.k, inp.v, inp.x, u2, inp.state_in, state_out=s, y=y)
    else:
        fn = lambda: gf.prefill(inp.r, inp.k, inp.v, inp.x, inp.u, inp.state_in, state_out=s, y=y)
    return dict(case=name, shape=f"B={B} T={T} H={H} {dtype}", units=B * T * H, bytes=nbytes, ms=_time(fn, reps))


def run(case, reps, scale):
    c = synth.CONFIGS
    sc = lambda t: max(64, int(t * scale) // 64 * 64)
    if case == "cfg0":
        k = c["cfg0"]
        return _dense(case, k["B"], k["T"], k["H"], "f32", 0.0, reps)
    if case == "cfg1":
        k = c["cfg1"]
        return _dense(case, k["B"], sc(k["T"]), k["H"], "bf16", 0.1, reps)
    if case in ("cfg2", "cfg2-c2"):
        k = c["cfg2"]
        return _dense(case, k["B"], sc(k["T"]), k["H"], "bf16", 0.0, reps, c2=case.endswith("c2"))
    if case == "cfg3":                      # one call over the whole context (splits into segments internally)
        k = c["cfg3"]
        return _dense(case, 1, sc(k["T"]), k["H"], "bf16", 0.0, reps)
    if case == "cfg3-segments":             # 8 calls with the state carried from one to the next
        k = c["cfg3"]
        T, H, nseg = sc(k["T"]), k["H"], k["segments"]
        inp = synth.make_dense(1, T, H, 64, "bf16", seed=7, device=DEV)
        seg = T // nseg
        parts = [tuple(t[:, i * seg:(i + 1) * seg].contiguous() for t in (inp.r, inp.k, inp.v, inp.x)) for i in range(nseg)]
        ys = [torch.empty_like(p[0]) for p in parts]
        st = torch.zeros((1, H, 64, 64), device=DEV)

        def fn():
            state = None
            for (r, kk, v, x), y in zip(parts, ys):
                _, state = gf.prefill(r, kk, v, x, inp.u, state, state_out=st, y=y)

        return dict(case=case, shape=f"B=1 T={nseg}x{seg} H={H} bf16", units=T * H, bytes=T * H * 640 + nseg * 2 * H * 16384,
                    ms=_time(fn, reps))
    if case == "cfg3-packed":               # two long contexts of different lengths in one packed call (split by max_seqlen)
        k = c["cfg3"]
        H, lens = k["H"], [sc(k["T"]), sc(k["T"] * 3 // 8) + 37]
        cu = torch.tensor([0, lens[0], lens[0] + lens[1]], dtype=torch.int32)
        inp = synth.make_varlen(cu, H, 64, "bf16", seed=3001, device=DEV, state_std=0.0)
        y = torch.empty_like(inp.r)
        s = torch.empty((2, H, 64, 64), device=DEV)
        fn = lambda: gf.prefill_varlen(inp.r, inp.k, inp.v, inp.x, inp.u, inp.cu_seqlens, max(lens), None, state_out=s, y=y)
        return dict(case=case, shape=f"S=2 lens={lens} H={H} bf16", units=sum(lens) * H,
                    bytes=sum(lens) * H * 640 + 2 * H * 16384, ms=_time(fn, reps))
    if case == "bwd-cfg3-packed":           # gradient of that packed call (64 units: the sequences split by the longer one)
        k = c["cfg3"]
        H, lens = k["H"], [sc(k["T"]), sc(k["T"] * 3 // 8) + 37]
        cu = torch.tensor([0, lens[0], lens[0] + lens[1]], dtype=torch.int32)
        inp = synth.make_varlen(cu, H, 64, "bf16", seed=3001, device=DEV, state_std=0.0)
        dy = torch.randn(inp.r.shape, device=DEV).bfloat16()
        ws = torch.empty(gf.backward_varlen_workspace_bytes(2, sum(lens), H, 64), dtype=torch.uint8, device=DEV)
        fn = lambda: gf.backward_varlen(inp.r, inp.k, inp.v, inp.x, inp.u, dy, inp.cu_seqlens, max(lens), None, None, workspace=ws)
        return dict(case=case, shape=f"S=2 lens={lens} H={H} bf16", units=sum(lens) * H,
                    bytes=sum(lens) * H * 64 * 2 * 9 + 2 * H * 16384, ms=_time(fn, reps))
    if case in ("ln-cfg1", "ln-cfg2", "ln-wide"):  # LayerNorm across all heads over the tokens of a prefill's output
        k = c["cfg1" if case == "ln-cfg1" else "cfg2"]
        rows, H = k["B"] * sc(k["T"]), (128 if case == "ln-wide" else k["H"])
        g = torch.Generator(device=DEV).manual_seed(9)
        y = torch.randn((rows, H, 64), device=DEV, generator=g).bfloat16()
        gamma, beta = torch.rand(H * 64, device=DEV, generator=g) + 0.5, torch.randn(H * 64, device=DEV, generator=g)
        out = torch.empty_like(y)
        fn = lambda: gf.layernorm_heads(y, gamma, beta, 1e-5, out=out)
        return dict(case=case, shape=f"rows={rows} D={H * 64} bf16", units=rows * H, bytes=rows * H * 64 * 4 + 8 * H * 64,
                    ms=_time(fn, reps))
    if case in ("kc-cfg2", "kc-wide"):      # GOLD key compression over the tokens of cfg2 (D = 2048 -> 128; wide: 4096 -> 256)
        k = c["cfg2"]
        rows, D = k["B"] * sc(k["T"]), (4096 if case == "kc-wide" else k["H"] * 64)
        g = torch.Generator(device=DEV).manual_seed(11)
        x = torch.randn((rows, D), device=DEV, generator=g).bfloat16()
        w = (torch.randn((D, D // 16), device=DEV, generator=g) / D ** 0.5).bfloat16()
        out = torch.empty((rows, D // 16), device=DEV, dtype=torch.bfloat16)
        fn = lambda: gf.key_compress(x, w, out=out)
        r = dict(case=case, shape=f"rows={rows} D={D} Dc={D // 16} bf16", units=rows, bytes=rows * D * 2 + rows * (D // 16) * 2 + D * (D // 16) * 2,
                 ms=_time(fn, reps))
        r["tflops"] = 2.0 * rows * D * (D // 16) / (r["ms"] * 1e-3) / 1e12
        return r
    if case in ("dl-cfg1", "dl-cfg2"):      # decay logit d = lora_omega(ddlerp_d(x_t, x_{t-1})) over the tokens of a prefill call
        k = c["cfg1" if case == "dl-cfg1" else "cfg2"]
        B, T, D, Rd, Rw = k["B"], sc(k["T"]), k["H"] * 64, 32, 64
        x, xp = synth.make_block_input(B, T, D, seed=13, device=DEV)
        w = synth.make_decay_lora(D, Rd, Rw, seed=14, device=DEV)
        out = torch.empty_like(x)
        fn = lambda: gf.decay_logit(x, w["mu_x"], w["A_d"], w["B_d"], w["lambda_d"], w["A_w"], w["B_w"], w["lambda_w"], x_prev=xp, out=out)
        r = dict(case=case, shape=f"B={B} T={T} D={D} Rd={Rd} Rw={Rw} bf16", units=B * T * k["H"],
                 bytes=2 * B * T * D * 2 + 4 * D * (Rd + Rw) + 12 * D, ms=_time(fn, reps))
        r["tflops"] = 2.0 * B * T * D * 2 * (Rd + Rw) / (r["ms"] * 1e-3) / 1e12
        return r
    if case in ("bwd-cfg1", "bwd-cfg2", "bwd-cfg3"):    # gradient of one prefill call (bf16, chunked on the tensor cores)
        k = c[{"bwd-cfg1": "cfg1", "bwd-cfg2": "cfg2", "bwd-cfg3": "cfg3"}[case]]     # (cfg3: 32 units, the sequences split)
        B, T, H = k["B"], sc(k["T"]), k["H"]
        inp = synth.make_dense(B, T, H, 64, "bf16", seed=7, device=DEV, state_std=k["state_std"])
        dy = torch.randn(inp.r.shape, device=DEV).bfloat16()
        ws = torch.empty(gf.backward_workspace_bytes(B, T, H, 64), dtype=torch.uint8, device=DEV)
        fn = lambda: gf.backward(inp.r, inp.k, inp.v, inp.x, inp.u, dy, inp.state_in, None, workspace=ws)
        # algorithmic traffic: r,k,v,x,dy read and dr,dk,dv,dx written once (bf16), the start state read, its adjoint
        # written; the checkpoints (one bf16 state per chunk, written by the first pass and read by the second, and
        # the first pass's second read of k,v,x) are this design's own and are not counted
        return dict(case=case, shape=f"B={B} T={T} H={H} bf16", units=B * T * H,
                    bytes=B * T * H * 64 * 2 * 9 + B * H * 16384 * (2 if k["state_std"] > 0 else 1),
                    design_bytes=B * T * H * 1792 + B * H * 16384 * 2, ms=_time(fn, reps))
    if case in ("train-fwd-cfg2", "train-bwd-cfg2"):    # a training step's pair: forward that keeps its chunk-start states, gradient from them
        k = c["cfg2"]
        B, T, H = k["B"], sc(k["T"]), k["H"]
        inp = synth.make_dense(B, T, H, 64, "bf16", seed=7, device=DEV, state_std=k["state_std"])
        dy = torch.randn(inp.r.shape, device=DEV).bfloat16()
        ws = torch.empty(gf.backward_workspace_bytes(B, T, H, 64), dtype=torch.uint8, device=DEV)
        gf.prefill_train(inp.r, inp.k, inp.v, inp.x, inp.u, ws, inp.state_in)
        if case == "train-fwd-cfg2":
            fn = lambda: gf.prefill_train(inp.r, inp.k, inp.v, inp.x, inp.u, ws, inp.state_in)
            nbytes = B * T * H * 640 + B * H * 16384
        else:
            fn = lambda: gf.backward(inp.r, inp.k, inp.v, inp.x, inp.u, dy, inp.state_in, None, workspace=ws, saved=True)
            nbytes = B * T * H * 64 * 2 * 9 + B * H * 16384
        # (the checkpoints, 128 B per token*head written by the one and read by the other, are the design's own)
        return dict(case=case, shape=f"B={B} T={T} H={H} bf16", units=B * T * H, bytes=nbytes, ms=_time(fn, reps))
    if case == "bwd-cfg4":       # gradient of the packed serving-mix prefill (64 sequences of 128..4096 tokens)
        k = c["cfg4"]
        S, H = k["S"], k["H"]
        cu = synth.make_lengths(S, max(1, int(k["len_min"] * scale)), max(2, int(k["len_max"] * scale)), seed=4000)
        inp = synth.make_varlen(cu, H, 64, "bf16", seed=4001, device=DEV, state_std=k["state_std"])
        total, mx = int(cu[-1]), int((cu[1:] - cu[:-1]).max())
        dy = torch.randn(inp.r.shape, device=DEV).bfloat16()
        ws = torch.empty(gf.backward_varlen_workspace_bytes(S, total, H, 64), dtype=torch.uint8, device=DEV)
        fn = lambda: gf.backward_varlen(inp.r, inp.k, inp.v, inp.x, inp.u, dy, inp.cu_seqlens, mx, inp.state_in, None, workspace=ws)
        return dict(case=case, shape=f"S={S} total_T={total} H={H} bf16", units=total * H,
                    bytes=total * H * 64 * 2 * 9 + 2 * S * H * 16384, ms=_time(fn, reps))
    if case in ("cfg4-prefill", "cfg4-decode", "cfg4-decode-layers"):
        k = c["cfg4"]
        S, H = k["S"], k["H"]
        cu = synth.make_lengths(S, max(1, int(k["len_min"] * scale)), max(2, int(k["len_max"] * scale)), seed=4000)
        if case == "cfg4-prefill":
            inp = synth.make_varlen(cu, H, 64, "bf16", seed=4001, device=DEV, state_std=k["state_std"])
            total, mx = int(cu[-1]), int((cu[1:] - cu[:-1]).max())
            y = torch.empty_like(inp.r)
            s = torch.empty((S, H, 64, 64), device=DEV)
            fn = lambda: gf.prefill_varlen(inp.r, inp.k, inp.v, inp.x, inp.u, inp.cu_seqlens, mx, inp.state_in, state_out=s, y=y)
            return dict(case=case, shape=f"S={S} total_T={total} H={H} bf16", units=total * H,
                        bytes=total * H * 640 + 2 * S * H * 16384, ms=_time(fn, reps))
        if case == "cfg4-decode-layers":
            # a decode loop over a stack of layers: every layer has its own state, so the states of one token step
            # (12 layers x 33.5 MB) do not fit L2 and every step streams its state from and to HBM
            layers = 12
            ds = [synth.make_step(S, H, 64, "bf16", seed=4100 + i, device=DEV) for i in range(layers)]
            ys = [torch.empty_like(d.r) for d in ds]
            g = torch.cuda.CUDAGraph()
            st = torch.cuda.Stream()
            with torch.cuda.stream(st):
                for d, y in zip(ds, ys):
                    gf.step(d.r, d.k, d.v, d.x, d.u, d.state_in, y=y, stream=st)
                torch.cuda.synchronize()
                with torch.cuda.graph(g, stream=st):
                    for d, y in zip(ds, ys):
                        gf.step(d.r, d.k, d.v, d.x, d.u, d.state_in, y=y, stream=st)
            ms = _time(g.replay, reps) / layers
            return dict(case=case, shape=f"S={S} H={H} bf16, {layers} layers with their own states per graph replay, in place",
                        units=S * H, bytes=S * H * (2 * 16384 + 5 * 128), ms=ms)
        d = synth.make_step(S, H, 64, "bf16", seed=4002, device=DEV)
        y = torch.empty_like(d.r)
        steps = 64
        g = torch.cuda.CUDAGraph()                       # a decode loop replays a captured step sequence
        st = torch.cuda.Stream()
        with torch.cuda.stream(st):
            gf.step(d.r, d.k, d.v, d.x, d.u, d.state_in, y=y, stream=st)
            torch.cuda.synchronize()
            with torch.cuda.graph(g, stream=st):
                for _ in range(steps):
                    gf.step(d.r, d.k, d.v, d.x, d.u, d.state_in, y=y, stream=st)
        ms = _time(g.replay, reps) / steps
        call, _ = gf.bind_step(d.r, d.k, d.v, d.x, d.u, d.state_in, y=y)
        loop_ms = _time(lambda: [call() for _ in range(steps)], reps) / steps
        return dict(case=case, shape=f"S={S} H={H} bf16, {steps} steps per graph replay, state updated in place",
                    units=S * H, bytes=S * H * (2 * 16384 + 5 * 128), ms=ms, ms_pre_marshalled_calls_no_graph=loop_ms)
    raise SystemExit(f"unknown case {case}")


ALL = ["cfg0", "cfg1", "cfg2", "cfg2-c2", "cfg3", "cfg3-segments", "cfg3-packed", "cfg4-prefill", "cfg4-decode", "cfg4-decode-layers", "ln-cfg1", "ln-cfg2", "ln-wide", "kc-cfg2", "kc-wide", "dl-cfg1", "dl-cfg2", "bwd-cfg1", "bwd-cfg2", "bwd-cfg3", "bwd-cfg3-packed", "bwd-cfg4", "train-fwd-cfg2", "train-bwd-cfg2"]


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("cases", nargs="+")
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--scale", type=float, default=1.0)
    ap.add_argument("--peak-gbs", type=float, default=None)
    a = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device: the library has no CPU path")
    gf.load_library()
    peak = a.peak_gbs or _peak()
    for case in (ALL if a.cases == ["all"] else a.cases):
        r = run(case, a.reps, a.scale)
        r["units_per_s"] = r["units"] / (r["ms"] * 1e-3)
        r["gbs"] = r["bytes"] / (r["ms"] * 1e-3) / 1e9
        r["frac"] = r["gbs"] / peak
        r["peak_gbs"] = peak
        print(json.dumps(r), flush=True)
        torch.cuda.empty_cache()


if __name__ == "__main__":
    sys.exit(main())
