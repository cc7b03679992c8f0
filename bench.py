#!/usr/bin/env python
"""Benchmark of the LongGen efficient-layer attention path on B200.

A step is one pass of the hot path over one batch of synthetic input: the block-index
build, the sparse forward (with LSE) and the backward of the 128K length-extension
workload (Llama-2-7B-shaped, sink + sliding window).  The other configurations (32K
prefill sparse vs full-causal, 70B-shaped strided GQA fwd+bwd, 70B-shaped decode over the
sink+window ring cache vs a dense cache) are measured once each and reported under
"other".  One JSON line is printed by rank 0.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--quick]

With N > 1 (launched under torch.distributed.run) every rank runs the same workload on its
own GPU -- the path has no exchange step, ranks are replicas -- and the value is the sum
over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
from dataclasses import replace
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2410_01485_b200 import synth

METRIC = "128K sparse attn fwd+bwd TFLOP/s (useful)"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_burst": p["bf16_tflops"], "bf16_sustained": p["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


def pairs_per_head(cfg) -> int:
    """Exact number of visible (query, key) pairs of one head: full blocks count Bs^2,
    diagonal blocks Bs(Bs+1)/2 (closed form of the pattern; the oracle's mask count agrees)."""
    Bs, nB = cfg.block, cfg.L // cfg.block
    if cfg.mode == synth.MODE_FULL_CAUSAL:
        off = nB * (nB - 1) // 2
    elif cfg.mode == synth.MODE_SINK_WINDOW:
        ns, nw = cfg.sink_tokens // Bs, cfg.window_tokens // Bs
        off = sum(min(qb + 1, nw) - 1 + min(ns, max(qb + 1 - nw, 0)) for qb in range(nB))
    else:
        nl, s = cfg.local_blocks, cfg.stride_blocks
        off = sum(min(qb + 1, nl) - 1 + -(-max(qb - nl + 1, 0) // s) for qb in range(nB))
    return off * Bs * Bs + nB * Bs * (Bs + 1) // 2


def flops(cfg, fwd=True, bwd=True) -> float:
    per_pair = (4 if fwd else 0) + (10 if bwd else 0)
    return float(pairs_per_head(cfg)) * cfg.B * cfg.Hq * cfg.D * per_pair


# ------------------------------------------------------------------------------ clocks

class ClockSampler:
    """Samples nvidia-smi while the timed region runs (reads settings only)."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.QUERY,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def __exit__(self, *exc):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self):
        sm, mx, reasons = [], 0.0, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx = max(mx, float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx or None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------ oracle timing

def oracle_sample(cfg, fraction=8):
    """Time the CPU oracle, as it stands, on a bounded sample of the workload: two kv heads with
    their query heads, the first L/fraction tokens, forward + backward.  The value is the sample's
    own rate (its own useful FLOPs / its own time): it is not extrapolated to the whole workload.
    Returns (useful TFLOP/s, description, cores, seconds)."""
    from oracle import lg_oracle as O
    small = replace(cfg, B=1, Hq=2 * (cfg.Hq // cfg.Hkv), Hkv=2, L=cfg.L // fraction)
    inp = synth.make_attn_inputs(small, "cpu", seed=0, with_do=True)
    q, k, v, do = (synth.to_f64(inp[x][0]) for x in ("q", "k", "v", "do"))
    t0 = time.perf_counter()
    O.attn_backward(q, k, v, do, O.Pattern.of(small), 1.0 / math.sqrt(cfg.D), rows_per_slab=cfg.block)
    dt = time.perf_counter() - t0
    tf = flops(small) / dt / 1e12
    desc = ("sample, not extrapolated: %s pattern, %d query heads / 2 kv heads, first %d of %d tokens, fwd+bwd, "
            "fp64 numpy, %.1f s" % (cfg.name, small.Hq, small.L, cfg.L, dt))
    return tf, desc, os.cpu_count(), dt


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = synth.CFG3
    vals = []
    for i in range(args.warmup + args.steps):
        tf, desc, cores, dt = oracle_sample(cfg)
        if i >= args.warmup:
            vals.append((tf, dt))
    tf = float(np.mean([v[0] for v in vals]))
    ms = float(np.mean([v[1] for v in vals])) * 1e3
    line = {"impl": "reference", "metric": METRIC, "value": tf, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "sample": desc},
            "cpu_baseline": {"value": tf, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": tf, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------- GPU timing

def time_cuda(fn, warmup, steps):
    """Median-free plain timing: total of `steps` calls between two events on the current stream."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def max_over_ranks(ms: float, dist, device) -> float:
    """Step time of the job = the slowest rank's device time (ranks are independent replicas)."""
    if dist is None:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(flops_per_rank: float, world: int, ms_step: float) -> float:
    """Whole-job useful TFLOP/s: every rank does the same work in the time of the slowest one."""
    return flops_per_rank * world / ms_step / 1e9


def bwd_kernel_ms(lg, p, inp, o, lse, dq, dk, dv, ws, reps):
    """Mean durations (ms) of the backward's three kernels: the caller's events are recorded between them
    by lg_sparse_attn_bwd_marked; nothing synchronises inside the library."""
    ev = lg.timing_events(4)
    acc = np.zeros(3)
    for _ in range(reps):
        lg.lg_sparse_attn_bwd_marked(p, inp["q"], inp["k"], inp["v"], o, lse, inp["do"], dq, dk, dv, ws, ev)
        torch.cuda.synchronize()
        acc += [ev[i].elapsed_time(ev[i + 1]) for i in range(3)]
    return acc / reps


def dram_traffic_record(kernel: str):
    """DRAM bytes per launch of `kernel` from the committed ncu summary, or None when the kernel sources
    have changed since that capture (the record carries a hash of them)."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "dram_traffic_cfg3.json")
    if not os.path.exists(path):
        return None, "no record"
    with open(path) as f:
        rec = json.load(f)
    h = hashlib.sha256()
    for name in rec["sources"]:
        with open(os.path.join(ROOT, name), "rb") as f:
            h.update(f.read())
    if h.hexdigest() != rec["sources_sha256"]:
        return None, "kernel sources changed since the capture %s" % rec["capture"]
    return rec, rec["capture"]


def bench_attn(lg, cfg, warmup, steps, want_bwd, profile_kernels=False):
    p = lg.params_of(cfg)
    inp = synth.make_attn_inputs(cfg, "cuda", seed=0, with_do=want_bwd)
    ws = lg.attn_workspace(p, want_bwd)
    lg.lg_sparse_attn_prepare(p, ws, want_bwd)       # lists and schedules once; the timed calls launch attention kernels only
    o = torch.empty_like(inp["q"])
    lse = torch.empty(inp["q"].shape[:3], dtype=torch.float32, device="cuda")
    out = {"config": cfg.name}
    f_fwd = lambda: lg.lg_sparse_attn_fwd(p, inp["q"], inp["k"], inp["v"], o=o, lse=lse, workspace=ws)
    out["fwd_ms"] = time_cuda(f_fwd, warmup, steps)
    out["fwd_tflops"] = flops(cfg, True, False) / out["fwd_ms"] / 1e9
    if want_bwd:
        dq, dk, dv = torch.empty_like(inp["q"]), torch.empty_like(inp["k"]), torch.empty_like(inp["v"])
        f_bwd = lambda: lg.lg_sparse_attn_bwd(p, inp["q"], inp["k"], inp["v"], o, lse, inp["do"], dq=dq, dk=dk,
                                              dv=dv, workspace=ws)
        out["bwd_ms"] = time_cuda(f_bwd, warmup, steps)
        out["bwd_tflops"] = flops(cfg, False, True) / out["bwd_ms"] / 1e9
        out["bwd_variant"] = lg.bwd_variant_name(p)
        out["fwd_bwd_ms"] = out["fwd_ms"] + out["bwd_ms"]
        out["fwd_bwd_tflops"] = flops(cfg) / out["fwd_bwd_ms"] / 1e9
        if profile_kernels:
            ks = bwd_kernel_ms(lg, p, inp, o, lse, dq, dk, dv, ws, max(steps, 3))
            out["bwd_kernel_ms"] = dict(zip(("delta", "dkdv", "dq"), [float(x) for x in ks]))
    assert lg.lg_last_status(ws) == 0, "device-side wait expired"
    return out, (p, inp, ws, o, lse)


def bench_decode(lg, c, warmup, steps, dense=False, copies=4, graph=True):
    cap = c.n_tokens if dense else c.sink_tokens + c.window_tokens
    p = lg.decode_params(c.B, c.Hq, c.Hkv, c.D, 0 if dense else c.sink_tokens, cap if dense else c.window_tokens)
    if dense:
        copies = 1                      # 8.6 GB per copy: far larger than L2 already
    sets = [synth.make_decode_inputs(c, "cuda", seed=s, capacity=cap) for s in range(copies)]
    n_t = torch.full((c.B,), c.n_tokens, dtype=torch.int64, device="cuda")
    ws = lg.decode_workspace(p)
    o = torch.empty_like(sets[0]["q"])
    state = {"i": 0}

    # a serving loop's call: fixed buffers, arguments (the stream too) marshalled once per cache copy
    calls = [lg.decode_call(p, s["q"], s["k_cache"], s["v_cache"], n_t, o, None, ws) for s in sets]

    def fn_bound():
        state["i"] += 1
        calls[state["i"] % copies]()

    def fn():   # the plain call, on whatever stream is current (graph capture below)
        s = sets[state["i"] % copies]
        state["i"] += 1
        lg.lg_sparse_decode(p, s["q"], s["k_cache"], s["v_cache"], n_t, o=o, workspace=ws, want_lse=False)

    ms_enqueue = time_cuda(fn if dense else fn_bound, warmup, steps)
    nbytes = 2.0 * c.B * c.Hkv * cap * c.D * 2
    assert lg.lg_last_status(ws) == 0
    out = {"config": c.name + ("_dense" if dense else ""), "bytes": nbytes,
           "l2": "rotating over %d cache copies (%.0f MB each)" % (copies, nbytes / 1e6)}
    if dense or not graph:
        out.update(ms=ms_enqueue, gbs=nbytes / ms_enqueue / 1e6, launch="one host call per step")
        return out
    # A decode step of ~60 us is launch-sensitive, and a serving loop replays it from a CUDA graph:
    # capture a few steps (one per cache copy, several rounds) and time whole-graph replays.
    per_graph = copies * 5
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for _ in range(per_graph):
                fn()
    torch.cuda.current_stream().wait_stream(side)
    replays = max(1, steps // per_graph)
    ms = time_cuda(g.replay, 2, replays) / per_graph
    assert lg.lg_last_status(ws) == 0
    out.update(ms=ms, gbs=nbytes / ms / 1e6, launch="CUDA graph replay, %d steps per graph" % per_graph,
               ms_host_call_per_step=ms_enqueue, gbs_host_call_per_step=nbytes / ms_enqueue / 1e6)
    return out


def bench_chunk_prefill(lg, c, T, warmup, steps):
    """A chunk of T tokens served against the full sink + window ring of the decode configuration."""
    p = lg.decode_params(1, c.Hq, c.Hkv, c.D, c.sink_tokens, c.window_tokens)
    cap = c.sink_tokens + c.window_tokens
    gen = torch.Generator(device="cuda").manual_seed(0)
    mk = lambda *shape: torch.randn(*shape, generator=gen, device="cuda").to(torch.bfloat16)
    q, kc, vc = mk(1, c.Hq, T, c.D), mk(1, c.Hkv, T, c.D), mk(1, c.Hkv, T, c.D)
    k_cache, v_cache = mk(1, c.Hkv, cap, c.D), mk(1, c.Hkv, cap, c.D)
    n0 = c.n_tokens - T
    ws = lg.chunk_prefill_workspace(p, T, n0)
    o = torch.empty_like(q)
    lse = torch.empty(1, c.Hq, T, dtype=torch.float32, device="cuda")
    ms = time_cuda(lambda: lg.lg_chunk_prefill(p, q, kc, vc, k_cache, v_cache, n0, o=o, lse=lse, workspace=ws),
                   warmup, steps)
    assert lg.lg_last_status(ws) == 0
    pairs = float(T) * cap          # every chunk token sees the sink and a full window
    flop = 4.0 * c.D * pairs * c.Hq
    return {"config": "%s_chunk_prefill_T%d" % (c.name, T), "ms": ms, "tflops": flop / ms / 1e9,
            "note": "ring linearisation + block-index build + forward, one sequence"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--quick", action="store_true", help="headline workload only (no other configs, no e2e)")
    ap.add_argument("--no-oracle", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--case", default="full", choices=["full", "small", "decode"],
                    help="small: the headline pattern at 8 heads x 32K tokens, for profiler captures "
                         "(implies --quick --no-oracle; its numbers are not benchmark values); "
                         "decode: only the 70B-shaped decode over the sink+window ring, for profiler captures")
    args = ap.parse_args()
    if args.case == "small":
        args.quick = args.no_oracle = True
    else:
        args.warmup = max(args.warmup, 3)

    if args.impl == "reference":
        run_reference(args)
        return

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    from paper_2410_01485_b200 import binding as lg, build
    if rank == 0:
        build.build()
    if dist is not None:
        dist.barrier()
    lg.load_library()
    peaks = load_peaks()
    if args.case == "decode":
        d5 = bench_decode(lg, synth.CFG5, args.warmup, max(args.steps, 1))
        print(json.dumps({"case": "decode", **d5}), flush=True)
        return
    cfg = synth.CFG3
    if args.case == "small":
            cfg = replace(cfg, name=cfg.name + "_small", Hq=8, Hkv=8, L=32768)

    # ---- headline: K timed steps of fwd + bwd, device-resident inputs ----------------------
    p = lg.params_of(cfg)
    inp = synth.make_attn_inputs(cfg, "cuda", seed=0, with_do=True)
    ws = lg.attn_workspace(p, True)
    o = torch.empty_like(inp["q"])
    lse = torch.empty(inp["q"].shape[:3], dtype=torch.float32, device="cuda")
    dq, dk, dv = torch.empty_like(inp["q"]), torch.empty_like(inp["k"]), torch.empty_like(inp["v"])

    # The block lists and tile schedules are static (same pattern, same L every step): built once here,
    # timed by itself, and every step below launches the four attention kernels only.
    index_ms = time_cuda(lambda: lg.lg_sparse_attn_prepare(p, ws, True), 1, 3)

    def step():
        lg.lg_sparse_attn_fwd(p, inp["q"], inp["k"], inp["v"], o=o, lse=lse, workspace=ws)
        lg.lg_sparse_attn_bwd(p, inp["q"], inp["k"], inp["v"], o, lse, inp["do"], dq=dq, dk=dk, dv=dv, workspace=ws)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    with ClockSampler(local) as clocks:
        torch.cuda.synchronize()
        launches0 = lg.kernel_launches()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
        torch.cuda.synchronize()
        launches = lg.kernel_launches() - launches0
        # per-kernel durations inside the same clock-sampled region
        fwd_ms = time_cuda(lambda: lg.lg_sparse_attn_fwd(p, inp["q"], inp["k"], inp["v"], o=o, lse=lse, workspace=ws),
                           0, args.steps)
        kms = bwd_kernel_ms(lg, p, inp, o, lse, dq, dk, dv, ws, args.steps)
    assert lg.lg_last_status(ws) == 0, "device-side wait expired"
    ms_step = max_over_ranks(e0.elapsed_time(e1) / args.steps, dist, "cuda")
    value = aggregate_value(flops(cfg), world, ms_step)
    clk = clocks.summary()

    pairs = float(pairs_per_head(cfg)) * cfg.B * cfg.Hq
    kern = {"fwd": (fwd_ms, pairs * cfg.D * 4), "bwd_dkdv": (float(kms[1]), pairs * cfg.D * 8),
            "bwd_dq": (float(kms[2]), pairs * cfg.D * 2), "bwd_delta": (float(kms[0]), 0.0)}
    dom = max(("fwd", "bwd_dkdv", "bwd_dq"), key=lambda n: kern[n][0])
    achieved = kern[dom][1] / kern[dom][0] / 1e9
    # dram__bytes_read + dram__bytes_write of one launch come from the committed ncu summary of the same kernels
    # on this very workload (a single-pass capture; no scaling: the L2 behaves differently at other sizes);
    # null for a workload that was not captured and once the kernel sources differ from the captured ones
    rec, rec_note = dram_traffic_record(dom)
    traffic = None
    if rec is not None:
        traffic = rec["workloads"].get(cfg.name, {}).get(dom)
        if traffic is None:
            rec_note = "workload %s is not in the capture %s" % (cfg.name, rec["capture"])
    kernel_ms = {k: v[0] for k, v in kern.items()}
    kernel_ms["index_build_once"] = index_ms
    roofline = {"bound": "tensor", "kernel": dom, "achieved": achieved, "peak": peaks["bf16_sustained"],
                "unit": "TFLOP/s", "frac": achieved / peaks["bf16_sustained"], "traffic": traffic,
                "traffic_note": "bytes per launch; " + rec_note,
                "peak_source": "%s sustained bf16 matmul" % peaks["source"],
                "frac_of_nominal_2250": achieved / NOMINAL_BF16_TFLOPS,
                "kernel_ms": kernel_ms,
                "note": "algorithmic FLOPs per launch: fwd 4D, dK/dV pass 8D, dQ pass 2D per visible pair (the dQ pass of "
                        "the keep_ds variant is one product that reads dS back from HBM: it is bandwidth-bound)"}

    mhz = clk.get("sm_mhz")
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": cfg.name, "B": cfg.B, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "L": cfg.L, "D": cfg.D,
                       "block": cfg.block, "sink_tokens": cfg.sink_tokens, "window_tokens": cfg.window_tokens,
                       "useful_flop_per_step": flops(cfg), "parallelism": "replicas x%d" % world,
                       "bwd_variant": lg.bwd_variant_name(p),
                       "l2": "inputs (8.6 GB) far larger than L2; no flush",
                       "lists": "block lists and tile schedules built once before the timed region "
                                "(lg_sparse_attn_prepare, %.3f ms); a step = forward + backward kernels" % index_ms},
            "pct_of_nominal_bf16_peak": 100.0 * value / world / NOMINAL_BF16_TFLOPS,
            "pct_of_measured_bf16_sustained": 100.0 * value / world / peaks["bf16_sustained"],
            "roofline": roofline, "clocks": clk,
            "kernel_ms": kernel_ms,
            "kernel_ms_x_sm_mhz": {k: v * mhz for k, v in kernel_ms.items()} if mhz else None,
            "gpu_launches": launches,
            "gpu_launches_note": "counted by the library (lg_debug_kernel_launches) around the timed region: "
                                 "%.1f per step" % (launches / float(args.steps))}

    del dq, dk, dv
    others = []
    if rank == 0 and not args.quick:
        # ---- e2e: host buffers, copies inside the timed region -----------------------------
        host = {k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True).copy_(v) for k, v in inp.items()}
        h_out = {"o": torch.empty(o.shape, dtype=o.dtype, pin_memory=True),
                 "lse": torch.empty(lse.shape, dtype=lse.dtype, pin_memory=True),
                 "dq": torch.empty(o.shape, dtype=o.dtype, pin_memory=True),
                 "dk": torch.empty(inp["k"].shape, dtype=o.dtype, pin_memory=True),
                 "dv": torch.empty(inp["v"].shape, dtype=o.dtype, pin_memory=True)}
        dq, dk, dv = torch.empty_like(inp["q"]), torch.empty_like(inp["k"]), torch.empty_like(inp["v"])

        n_grp = next((g for g in (16, 8, 4, 2) if cfg.Hkv % g == 0), 1)
        p_host = lg.params_of(cfg)
        ws_g = lg.host_step_workspace(p_host, n_grp)

        def e2e_step():
            # the library's host-buffer entry point (C ABI): head groups pipelined over copy-in / compute /
            # copy-out streams inside the call
            lg.sparse_attn_fwd_bwd_host(p_host, host, h_out, dev=(inp, o, lse, dq, dk, dv, ws_g), head_groups=n_grp)

        e2e_ms = time_cuda(e2e_step, 1, max(2, min(args.steps, 3)))
        h2d = sum(t.numel() * t.element_size() for t in host.values())
        d2h = sum(t.numel() * t.element_size() for t in h_out.values())
        line["e2e"] = {"value": flops(cfg) / e2e_ms / 1e9, "unit": UNIT, "ms_per_step": e2e_ms,
                       "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                       "entry_point": "lg_sparse_attn_fwd_bwd_host (C ABI, host pointers)",
                       "pipeline": "%d head groups over copy-in / compute / copy-out streams" % n_grp}
        del host, h_out, dq, dk, dv, ws_g
    del inp, o, lse, ws
    torch.cuda.empty_cache()

    if rank == 0 and not args.quick:
        r2, _ = bench_attn(lg, synth.CFG2, 3, 5, want_bwd=False)
        r2f, _ = bench_attn(lg, synth.CFG2.full_causal(), 3, 3, want_bwd=False)
        torch.cuda.empty_cache()
        r4, _ = bench_attn(lg, synth.CFG4, 3, 3, want_bwd=True, profile_kernels=True)
        torch.cuda.empty_cache()
        # the same with the backward that recomputes S and dP in its dQ pass (the default keeps dS where its
        # buffer, 73 GB here, is at most 40 % of the device's memory)
        prev_var = os.environ.get("LG_BWD_VARIANT")
        os.environ["LG_BWD_VARIANT"] = "two_pass"
        try:
            r4k, _ = bench_attn(lg, synth.CFG4, 3, 3, want_bwd=True, profile_kernels=True)
            r4["with_LG_BWD_VARIANT_two_pass"] = {k: r4k[k] for k in ("bwd_ms", "bwd_variant", "fwd_bwd_ms", "fwd_bwd_tflops",
                                                                      "bwd_kernel_ms")}
        finally:
            if prev_var is None:
                del os.environ["LG_BWD_VARIANT"]
            else:
                os.environ["LG_BWD_VARIANT"] = prev_var
        del r4k, _
        torch.cuda.empty_cache()
        d5 = bench_decode(lg, synth.CFG5, 5, 200)
        d5["pct_of_nominal_8tbs"] = 100 * d5["gbs"] / NOMINAL_HBM_GBS
        d5["pct_of_measured_copy"] = 100 * d5["gbs"] / peaks["hbm_gbs"]
        torch.cuda.empty_cache()
        d5d = bench_decode(lg, synth.CFG5, 2, 5, dense=True)
        d5d["pct_of_measured_copy"] = 100 * d5d["gbs"] / peaks["hbm_gbs"]
        # the paper's own pattern settings (Section 4.1) on the Llama-2-7B shape at 128K
        rp1, _ = bench_attn(lg, synth.PAPER_SINK, 3, 3, want_bwd=True)
        torch.cuda.empty_cache()
        rp2, _ = bench_attn(lg, synth.PAPER_STRIDED, 3, 3, want_bwd=True)
        torch.cuda.empty_cache()
        cp = bench_chunk_prefill(lg, synth.CFG5, 8192, 3, 10)
        # modelled 32-layer mix (Section 4.1: 12 full-attention layers in the middle, 20 sparse ones), attention
        # only, from the measured times of the paper's sink + window setting and of full causal attention
        rpf, _ = bench_attn(lg, synth.PAPER_SINK.full_causal(), 1, 2, want_bwd=True)
        torch.cuda.empty_cache()
        mix = {"config": "modelled_mix_12_full_20_sparse_of_32",
               "full_causal_fwd_ms": rpf["fwd_ms"], "full_causal_fwd_bwd_ms": rpf["fwd_bwd_ms"],
               "full_causal_fwd_bwd_tflops": rpf["fwd_bwd_tflops"],
               "attention_train_speedup": 32 * rpf["fwd_bwd_ms"] / (12 * rpf["fwd_bwd_ms"] + 20 * rp1["fwd_bwd_ms"]),
               "attention_prefill_speedup": 32 * rpf["fwd_ms"] / (12 * rpf["fwd_ms"] + 20 * rp1["fwd_ms"]),
               "note": "attention kernels only, Llama-2-7B shape at 128K; the paper's 1.55x (training) and 1.67x "
                       "(prefill) are end-to-end model numbers on other hardware"}
        # packed documents (exponential lengths, 8K tokens on average) on the headline pattern and on full
        # causal attention: one sequence, so the documents also prune the block lists
        ds = synth.make_doc_start(cfg.L, seed=0, mean_len=8192).view(1, -1).cuda()
        docs = {"config": "cfg3_packed_documents_mean8k", "documents": int(ds.unique().numel())}
        for name, c in (("sink_window", cfg), ("full_causal", cfg.full_causal())):
            pd_ = lg.params_of(c, doc_start=ds)
            inp_d = synth.make_attn_inputs(c, "cuda", seed=0, with_do=True)
            ws_d = lg.attn_workspace(pd_, True)
            o_d = torch.empty_like(inp_d["q"])
            lse_d = torch.empty(inp_d["q"].shape[:3], dtype=torch.float32, device="cuda")
            g_d = [torch.empty_like(inp_d[x]) for x in ("q", "k", "v")]

            def step_d():
                lg.lg_sparse_attn_fwd(pd_, inp_d["q"], inp_d["k"], inp_d["v"], o=o_d, lse=lse_d, workspace=ws_d)
                lg.lg_sparse_attn_bwd(pd_, inp_d["q"], inp_d["k"], inp_d["v"], o_d, lse_d, inp_d["do"], dq=g_d[0],
                                      dk=g_d[1], dv=g_d[2], workspace=ws_d)
            docs[name + "_fwd_bwd_ms"] = time_cuda(step_d, 2, 3)
            assert lg.lg_last_status(ws_d) == 0
            del inp_d, ws_d, o_d, lse_d, g_d
            torch.cuda.empty_cache()
        others = [r2, r2f, r4, d5, d5d, rp1, rp2, cp, mix, docs]
        line["other"] = others
        line["decode_hbm_gbs"] = d5["gbs"]
        line["decode_roofline"] = {"bound": "hbm", "kernel": "decode_stream_kernel", "achieved": d5["gbs"],
                                   "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": d5["gbs"] / peaks["hbm_gbs"],
                                   "frac_of_nominal_8000": d5["gbs"] / NOMINAL_HBM_GBS,
                                   "peak_source": "%s copy bandwidth" % peaks["source"]}
    if rank == 0 and not args.no_oracle and world == 1:
        tf, desc, cores, _ = oracle_sample(cfg, fraction=4)
        line["cpu_baseline"] = {"value": tf, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
