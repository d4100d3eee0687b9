#!/usr/bin/env python
"""Benchmark of the WKV-6 prefill hot path on the 1.5B-class shape.

One step = one pass of the hot path over one batch: 16 sequential gf_wkv6_prefill calls
(B=4, T=16384, H=32, N=64, bf16 r/k/v/x/y, fp32 u/state, independent seeds), modelling the
Finch-C2 two thirds of a 24-layer stack.  Metric: tokens*heads per second (B*T*H*16 / step time).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 is launched by torch.distributed.run, one rank per GPU; the (batch, head) units are
independent, so every rank runs its own 16 calls (weak scaling) and there is no data-path
collective: only the timing barrier and a max-reduce of the elapsed time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "WKV-6 prefill tokens*heads/s at 1.5B-class shape"
UNIT = "token*heads/s"
WORKLOAD = dict(B=4, T=16384, H=32, N=64, calls=16)
BYTES_PER_TOKEN_HEAD = 640            # bf16 r,k,v,x in (4*64*2) + bf16 y out (64*2)
STATE_BYTES_PER_UNIT = 64 * 64 * 4    # fp32 final state written once per (b,h) (state_in is NULL)
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
# DRAM traffic per launch of the dominant kernel, from the ncu capture summarised under profiles/ (taken on a
# B=4 T=4096 H=32 launch; None once the kernel has changed since the counters were taken).  The reads grow in
# proportion to the tokens and are scaled to the timed launch; the writes of the capture miss the part of y
# that is still in L2 when the kernel ends (a fixed amount), so for the timed launch they are only bounded:
# at least the scaled figure, at most the algorithmic y + state bytes.
NCU_CAPTURE = {"profile": "profiles/ncu_wkv6_chunked_kernel_B4_T4096_H32.txt", "token_heads": 4 * 4096 * 32,
               "read_bytes": 268504832, "write_bytes": 50730496}


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--calls", type=int, default=WORKLOAD["calls"], help=argparse.SUPPRESS)
    ap.add_argument("--seq-len", type=int, default=WORKLOAD["T"], help=argparse.SUPPRESS)
    ap.add_argument("--no-e2e", action="store_true", help=argparse.SUPPRESS)
    ap.add_argument("--no-cpu-baseline", action="store_true", help=argparse.SUPPRESS)
    ap.add_argument("--no-extras", action="store_true", help=argparse.SUPPRESS)
    return ap.parse_args()


def measured_peaks():
    """(HBM GB/s, bf16 TFLOP/s burst, which) from MEASURED_PEAKS.json, else the fallback figures."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            j = json.load(open(p))
            return float(j["hbm_gbs"]), float(j.get("bf16_tflops", FALLBACK_BF16_TFLOPS)), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS, "fallback"


def traffic_of_launch(tokens_heads: int, alg_write_bytes: int):
    """DRAM traffic of one timed launch from the ncu capture (see NCU_CAPTURE), or None."""
    if not NCU_CAPTURE:
        return None
    scale = tokens_heads / NCU_CAPTURE["token_heads"]
    return {"read": int(NCU_CAPTURE["read_bytes"] * scale),
            "write_at_least": int(NCU_CAPTURE["write_bytes"] * scale), "write_at_most": int(alg_write_bytes),
            "note": "reads scaled by tokens from the capture in " + NCU_CAPTURE["profile"] +
                    "; writes: the capture misses the y rows still in L2 at kernel end"}


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU while the timed region runs: an NVML polling
    thread (read-only queries, every few ms) or, if NVML cannot be loaded, an nvidia-smi query loop."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int, period_s: float = 0.004):
        import threading
        self.proc, self.thread, self.samples, self.reasons, self.max_mhz = None, None, [], set(), None
        self._stop = threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = int(vis.split(",")[index]) if vis and vis.split(",")[index].isdigit() else index
            h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            bits = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}

            def poll():
                while not self._stop.is_set():
                    try:
                        self.samples.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                        r = int(pynvml.nvmlDeviceGetCurrentClocksEventReasons(h))
                        for n, b in bits.items():
                            if r & b:
                                self.reasons.add(n)
                    except Exception:
                        pass
                    self._stop.wait(period_s)

            self.thread = threading.Thread(target=poll, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.thread = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.thread is not None:
            self._stop.set()
            self.thread.join(timeout=2)
            sm = self.samples
            return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": self.max_mhz,
                    "reasons": sorted(self.reasons), "samples": len(sm), "source": "nvml"}
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "source": "none"}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        for line in out.splitlines():
            f = [s.strip() for s in line.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, val in zip(self.NAMES, f[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "source": "nvidia-smi"}


def rank_seed(rank: int, call: int) -> int:
    """Seed of one call's inputs on one rank: every rank draws its own (b,h) units (weak scaling)."""
    return 2000 + 100 * rank + call


def max_over_ranks(ms: float, world: int, device) -> float:
    """The job's time for a timed region is the slowest rank's device time."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank_step: int, world: int, ms_per_step: float) -> float:
    """Whole-job throughput: the units all ranks processed in a step over the (max-over-ranks) step time."""
    return units_per_rank_step * world / (ms_per_step * 1e-3)


def cpu_oracle_rate(calls_equiv: float, B, T, H, N, seed, passes: int = 1):
    """Times the fp64 oracle, as it stands, on `calls_equiv` calls' worth of the workload
    (whole (b,h) units of full length T), `passes` times over.  Returns (token*heads/s, threads, description, s)."""
    from oracle import wkv6_oracle as orc
    from paper_2407_12077_b200 import synth
    n_units = max(1, int(round(calls_equiv * B * H)))
    Hs = min(H, n_units)
    Bs = max(1, n_units // Hs)
    inp = synth.make_dense(Bs, T, Hs, N, "bf16", seed=seed)
    r, k, v, x = (t.float().numpy() for t in (inp.r, inp.k, inp.v, inp.x))
    u = inp.u.numpy()
    t0 = time.perf_counter()
    for _ in range(passes):
        orc.prefill(r, k, v, x, u, None)
    dt = time.perf_counter() - t0
    desc = f"{passes} x {Bs * Hs} whole (b,h) units of T={T} ({passes * Bs * Hs / (B * H):.3g} calls' worth)"
    return passes * Bs * T * Hs / dt, orc.threads(), desc, dt


def run_reference(args):
    """--impl reference: the CPU oracle on host cores, a bounded sample of the workload per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    B, T, H, N = WORKLOAD["B"], args.seq_len, WORKLOAD["H"], WORKLOAD["N"]
    rates, th, desc = [], 1, ""
    for i in range(args.warmup + args.steps):
        rate, th, desc, dt = cpu_oracle_rate(0.5, B, T, H, N, seed=2000 + i)
        if i >= args.warmup:
            rates.append((rate, dt))
    value = sum(r for r, _ in rates) / len(rates)
    units_per_step = B * T * H * args.calls
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": units_per_step / value * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"cfg2: {args.calls} x gf_wkv6_prefill B={B} T={T} H={H} N={N} bf16 inputs",
                   "note": "CPU oracle on a bounded sample per step; ms_per_step extrapolated to the full step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": th, "kind": "oracle", "sample": desc + " per step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    args = parse()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    import paper_2407_12077_b200 as gf
    from paper_2407_12077_b200 import synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)
    gf.load_library()

    B, T, H, N, calls = WORKLOAD["B"], args.seq_len, WORKLOAD["H"], WORKLOAD["N"], args.calls
    # ---- seeded synthetic inputs, resident in HBM, distinct buffers per call (1.34 GB each >> L2)
    batches = []
    for c in range(calls):
        inp = synth.make_dense(B, T, H, N, "bf16", seed=rank_seed(rank, c), device=dev)
        y = torch.empty_like(inp.r)
        s_out = torch.empty((B, H, N, N), device=dev, dtype=torch.float32)
        batches.append((inp, y, s_out))
    stream = torch.cuda.current_stream()

    def step(events=None):
        for c, (inp, y, s_out) in enumerate(batches):
            if events is not None:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
            gf.prefill(inp.r, inp.k, inp.v, inp.x, inp.u, None, state_out=s_out, y=y, stream=stream)
            if events is not None:
                e1.record(stream)
                events.append((e0, e1))

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    gf.last_device_status()

    # ---- timed region: exactly K steps between barriers, device time, max over ranks
    barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    launches0 = gf.launch_count()
    kernel_events = []
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_begin.record(stream)
    for _ in range(args.steps):
        step(kernel_events)
    t_end.record(stream)
    barrier()
    elapsed_ms = t_begin.elapsed_time(t_end)
    launches = gf.launch_count() - launches0
    clocks = sampler.stop() if sampler else None
    gf.last_device_status()
    elapsed_ms = max_over_ranks(elapsed_ms, world, dev)
    ms_per_step = elapsed_ms / args.steps
    units_per_step = B * T * H * calls * world
    value = whole_job_value(B * T * H * calls, world, ms_per_step)

    # ---- roofline of the dominant kernel (one prefill launch) from the live per-launch events
    per_launch = [a.elapsed_time(b) for a, b in kernel_events]
    launch_ms, launch_med = statistics.mean(per_launch), statistics.median(per_launch)
    alg_bytes = B * T * H * BYTES_PER_TOKEN_HEAD + B * H * STATE_BYTES_PER_UNIT
    peak, peak_tf, peak_kind = measured_peaks()
    gbs = lambda ms: alg_bytes / (ms * 1e-3) / 1e9
    achieved = gbs(launch_ms)
    # frac: from the mean of the per-launch events; frac_median: from their median; frac_step: from the step
    # time the headline value is made of (launch gaps included): the three differ when the clock drifts
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "frac_median": gbs(launch_med) / peak, "frac_step": gbs(ms_per_step / calls) / peak,
                "frac_best": gbs(min(per_launch)) / peak,
                "traffic": traffic_of_launch(B * T * H, B * T * H * N * 2 + B * H * STATE_BYTES_PER_UNIT),
                "peak_kind": f"of {peak_kind}", "kernel": "gf_wkv6_prefill (one launch)", "launch_ms": launch_ms,
                "launch_ms_median": launch_med, "launch_ms_min": min(per_launch), "launch_ms_max": max(per_launch),
                "algorithmic_bytes": alg_bytes, "launches_timed": len(per_launch)}

    # ---- the step that follows the WKV output in the o_t equation (LayerNorm across all heads), timed on its own
    # over the y of every call, outside the step and its numbers: reported beside them, not in them
    g_ln = torch.Generator(device=dev).manual_seed(77)
    gamma = torch.rand(H * N, device=dev, generator=g_ln) + 0.5
    beta = torch.randn(H * N, device=dev, generator=g_ln)
    o_ln = torch.empty_like(batches[0][1])
    for _, y, _ in batches[:3]:
        gf.layernorm_heads(y, gamma, beta, 1e-5, out=o_ln, stream=stream)
    ln_a, ln_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ln_a.record(stream)
    for _, y, _ in batches:
        gf.layernorm_heads(y, gamma, beta, 1e-5, out=o_ln, stream=stream)
    ln_b.record(stream)
    torch.cuda.synchronize()
    ln_ms = ln_a.elapsed_time(ln_b) / len(batches)
    ln_bytes = 2 * B * T * H * N * 2
    layernorm = {"kernel": "gf_c2_layernorm (one launch over the y of one call)", "launch_ms": ln_ms, "bound": "hbm",
                 "achieved": ln_bytes / (ln_ms * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                 "frac": ln_bytes / (ln_ms * 1e-3) / 1e9 / peak, "algorithmic_bytes": ln_bytes}

    # ---- batched serving prefill (packed variable-length call, 64 sequences of 128..4096 tokens: more units than SMs,
    # one persistent CTA per SM), timed on its own after the step like the LayerNorm above
    packed = None
    if world == 1:
        c4 = synth.CONFIGS["cfg4"]
        cu = synth.make_lengths(c4["S"], c4["len_min"], c4["len_max"], seed=4000)
        vin = synth.make_varlen(cu, c4["H"], N, "bf16", seed=4001, device=dev, state_std=c4["state_std"])
        v_total, v_max = int(cu[-1]), int((cu[1:] - cu[:-1]).max())
        v_y = torch.empty_like(vin.r)
        v_s = torch.empty((c4["S"], c4["H"], N, N), device=dev)
        v_call = lambda: gf.prefill_varlen(vin.r, vin.k, vin.v, vin.x, vin.u, vin.cu_seqlens, v_max, vin.state_in,
                                           state_out=v_s, y=v_y, stream=stream)
        for _ in range(3):
            v_call()
        v_a, v_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        v_a.record(stream)
        for _ in range(10):
            v_call()
        v_b.record(stream)
        torch.cuda.synchronize()
        gf.last_device_status()
        v_ms = v_a.elapsed_time(v_b) / 10
        v_bytes = v_total * c4["H"] * BYTES_PER_TOKEN_HEAD + 2 * c4["S"] * c4["H"] * STATE_BYTES_PER_UNIT
        packed = {"kernel": "gf_wkv6_prefill_varlen (one call: rank kernel + persistent prefill kernel)",
                  "workload": f"cfg4: {c4['S']} sequences of {c4['len_min']}..{c4['len_max']} tokens, {v_total} tokens, H={c4['H']}",
                  "call_ms": v_ms, "value": v_total * c4["H"] / (v_ms * 1e-3), "unit": UNIT, "bound": "hbm",
                  "achieved": v_bytes / (v_ms * 1e-3) / 1e9, "peak": peak, "frac": v_bytes / (v_ms * 1e-3) / 1e9 / peak,
                  "algorithmic_bytes": v_bytes}
        del vin, v_y, v_s

    # ---- the other rows of the path, each timed on its own after the step (a few launches each, seeded inputs
    # of its configuration resident in HBM): not part of the headline value, reported beside it
    others = None
    if world == 1 and not args.no_extras:
        from paper_2407_12077_b200 import cases
        others = {}
        for key, case, what in (
                ("cfg1", "cfg1", "gf_wkv6_prefill, small-model shape B=8 T=4096 H=12 (96 units: one CTA each)"),
                ("cfg3_one_call", "cfg3", "gf_wkv6_prefill, B=1 T=131072 H=32 in one call (sequence split: 2 launches)"),
                ("cfg3_eight_segments", "cfg3-segments", "8 x gf_wkv6_prefill of 16384 tokens, state carried in place"),
                ("prefill_c2", "cfg2-c2", "gf_wkv6_prefill_c2 with the second-value tensor, cfg2 shape (768 B per token*head)"),
                ("key_compress", "kc-cfg2", "gf_gold_key_compress 65536 x 2048 -> 128"),
                ("decay_logit", "dl-cfg2", "gf_c2_decay_logit, 65536 tokens x 2048 channels, ranks 32 and 64 (x read, d written)"),
                ("backward", "bwd-cfg2", "gf_wkv6_backward, cfg2 shape: checkpoint pass + chunked gradient kernel, two chunks in flight per SM (1152 B per token*head counted; the design moves 1792)"),
                ("backward_long_context", "bwd-cfg3", "gf_wkv6_backward, B=1 T=131072 H=32: 32 units, sequences split 4-way with the adjoint's segment summaries (5 launches)"),
                ("backward_packed", "bwd-cfg4", "gf_wkv6_backward_varlen, the serving mix's shape (64 packed sequences of 128..4096 tokens, 32 heads: 2048 units, longest first)"),
                ("train_forward", "train-fwd-cfg2", "gf_wkv6_prefill_train, cfg2 shape: the prefill that also keeps its chunk-start states (128 B per token*head more, not counted)"),
                ("train_backward", "train-bwd-cfg2", "gf_wkv6_backward_saved, cfg2 shape: the gradient kernel alone, from the states the forward pass kept"),
                ("decode_step", "cfg4-decode", "gf_wkv6_step, 64 sequences x 32 heads, 64 steps per graph replay (states stay in L2)"),
                ("decode_step_layer_stack", "cfg4-decode-layers", "gf_wkv6_step over 12 layers with their own states (streams from HBM)")):
            r = cases.run(case, 5, 1.0)
            ms = r["ms"]
            o = {"kernel": what, "call_ms": ms, "algorithmic_bytes": r["bytes"], "bound": "hbm",
                 "achieved": r["bytes"] / (ms * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                 "value": r["units"] / (ms * 1e-3), "value_unit": "tokens/s" if key == "key_compress" else ("step*heads/s" if key.startswith("decode_step") else "token*heads/s")}
            o["frac"] = o["achieved"] / peak
            if key in ("key_compress", "decay_logit"):
                # near the crossing of the two rooflines: the bound is the slower of bytes at HBM rate and flops at tensor rate
                flops = r["tflops"] * 1e12 * ms * 1e-3
                t_hbm, t_tc = r["bytes"] / (peak * 1e9), flops / (peak_tf * 1e12)
                o.update(tflops=r["tflops"], peak_tflops=peak_tf, bound="hbm" if t_hbm >= t_tc else "tensor",
                         frac=max(t_hbm, t_tc) / (ms * 1e-3))
            if "design_bytes" in r:
                o["design_bytes"] = r["design_bytes"]
            if "ms_pre_marshalled_calls_no_graph" in r:
                o["call_ms_pre_marshalled_no_graph"] = r["ms_pre_marshalled_calls_no_graph"]
            others[key] = o
            torch.cuda.empty_cache()

    # ---- end to end through the host-buffer entry point: pinned host inputs -> y on the host
    e2e = None
    if not args.no_e2e:
        inp0 = batches[0][0]
        host = [t.cpu().pin_memory() for t in (inp0.r, inp0.k, inp0.v, inp0.x, inp0.u)]
        # Two streams, each with its own device workspace and host result buffers, take the calls in turn:
        # the host->device copy of one call overlaps the device->host copy of the previous one (PCIe is
        # full duplex), which is how a user of the host-buffer entry point would pipeline a layer stack.
        lanes = []
        for _ in range(2):
            lanes.append((torch.cuda.Stream(device=dev),
                          torch.empty(gf.host_workspace_bytes(B, T, H, N), dtype=torch.uint8, device=dev),
                          torch.empty(inp0.r.shape, dtype=torch.bfloat16).pin_memory(),
                          torch.empty((B, H, N, N), dtype=torch.float32).pin_memory()))

        def e2e_step():
            for c in range(calls):
                st_c, ws_c, y_c, s_c = lanes[c & 1]
                gf.prefill_host(host[0], host[1], host[2], host[3], host[4], None, s_c, y_c, ws_c, stream=st_c)

        def timed(fn):
            """Device time of fn's work on both lanes: start after everything before, end after both lanes."""
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for st_c, *_ in lanes:
                st_c.wait_event(a)
            fn()
            for st_c, *_ in lanes:
                done = torch.cuda.Event()
                done.record(st_c)
                stream.wait_event(done)
            b.record(stream)
            return a, b

        e2e_steps = max(1, min(args.steps, 2))
        e2e_step()
        barrier()
        a, b = timed(lambda: [e2e_step() for _ in range(e2e_steps)])
        barrier()
        e_ms = a.elapsed_time(b)
        e_ms = max_over_ranks(e_ms, world, dev)
        tok = B * T * H * N * 2
        e2e = {"value": units_per_step / (e_ms / e2e_steps * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": calls * (4 * tok + H * N * 4),
               "d2h_bytes_per_step": calls * (tok + B * H * N * N * 4), "steps": e2e_steps,
               "streams": len(lanes)}
        del lanes

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        rate, th, desc, dt = cpu_oracle_rate(2.0, B, T, H, N, seed=2000, passes=6)
        cpu_baseline = {"value": rate, "unit": UNIT, "cores": th, "kind": "oracle",
                        "sample": f"{desc}, {dt:.1f} s wall on {th} threads"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": f"cfg2: {calls} x gf_wkv6_prefill B={B} T={T} H={H} N={N}, bf16 r/k/v/x/y, "
                                   f"fp32 u/state, independent seeds per call",
                       "precision": "bf16 r/k/v/x/y and tensor-core operands, fp32 accumulation, decay sums and state",
                       "l2": "inputs larger than L2 (1.34 GB per call, distinct buffers per call)",
                       "parallelism": f"(b,h) units replicated per GPU x{world}, no collective"},
            "roofline": roofline, "layernorm_heads": layernorm, "packed_prefill": packed, "other_rows": others,
            "cpu_baseline": cpu_baseline,
            "e2e": e2e,
            "gpu_launches": launches,
            "clocks": clocks,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
