#!/usr/bin/env python
"""Benchmark of the batch LoRA linear layer (paper Section 3.4) on B200.

A step is one pass of the whole hot path over one synthetic batch: routing plan, shrink, base
product, expand/combine -- i.e. one ``edgelora_lora_linear`` call.  The default workload is the
Llama-3.1-8B q_proj decode batch (4096 -> 4096, 32 resident rank-16 adapters, 32 tokens each on
its own adapter), which is bound by HBM traffic.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank runs an independent replica on its
own GPU: the layer has no exchange step, so there is no data-path collective; only the timing
barrier and the max over ranks use torch.distributed.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2507_01438_b200 import workloads as wl  # noqa: E402

METRIC = "batched multi-adapter LoRA linear tokens/s"
L2_BYTES = 126 * 1024 * 1024
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

WORKLOADS = {
    # name: (builder, bound, description)
    "q_proj_decode": (lambda: wl.q_proj_decode(), "hbm",
                      "configs[1]: Llama-3.1-8B q_proj decode 4096->4096, 32 adapters r16, T=32 distinct ids"),
    "gate_up_prefill": (lambda: wl.gate_up_prefill(), "tensor",
                        "configs[2]: gate/up prefill 4096->14336, 8 adapters r16, 8 x 512-token segments"),
    "down_proj_many_tenant": (lambda: wl.down_proj_many_tenant(), "hbm",
                              "configs[3]: down_proj 14336->4096, 1000 adapters r64, T=256 Zipf(1.1), 10% base-only"),
    "tiny": (lambda: wl.tiny(), "hbm", "configs[0]: 256->256, 4 adapters r8, T=16"),
    # smaller resident pool, same layer and batch recipe: sized for multi-pass ncu captures
    "down_proj_200_tenants": (lambda: wl.down_proj_many_tenant(n_adapters=200), "hbm",
                              "profiling-size variant of configs[3]: down_proj 14336->4096, 200 adapters r64, T=256"),
}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured (MEASURED_PEAKS.json)"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback (earlier measurement on this pool)"
    return p


def ncu_traffic(workload):
    """DRAM bytes per launch of the dominant kernel from the committed ncu summary, if any."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.txt")
    if not os.path.exists(path):
        return None
    for line in open(path):
        parts = line.split("#")[0].split("=")
        if len(parts) == 2 and parts[0].strip() == workload:
            try:
                return float(parts[1])
            except ValueError:
                return None
    return None


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed loops run."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.samples = []
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50", "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.time(), line.strip()))

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self, windows):
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.samples:
            if not any(a <= ts <= b for a, b in windows):
                continue
            f = [s.strip() for s in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                smax.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(smax)) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def max_over_ranks(value, world, device):
    """The slowest rank's time: every rank runs its own replica, the job is as fast as the slowest."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tokens_per_s(tokens_per_rank_step, steps, world, seconds):
    """Whole-job throughput of `world` replicas that each did `steps` steps in `seconds` (max over ranks)."""
    return world * tokens_per_rank_step * steps / seconds


def time_oracle(w, tokens, reps):
    import oracle
    from oracle import AdapterSet
    s = AdapterSet(w.n_slots)
    for a, ad in w.adapters.items():
        s.put(a, ad.A, ad.B, ad.scale)
    x = np.ascontiguousarray(w.x[:tokens])
    ids = np.ascontiguousarray(w.ids[:tokens])
    t0 = time.perf_counter()
    for _ in range(reps):
        oracle.lora_linear(w.W, x, ids, s)
    return time.perf_counter() - t0


def cpu_baseline(w, budget_s=10.0):
    """The CPU oracle, as it stands, on a bounded sample of the same workload."""
    import oracle
    tokens = min(w.T, 64)
    t1 = time_oracle(w, tokens, 1)
    reps = int(max(1, min(200, budget_s / max(t1, 1e-6))))
    t = time_oracle(w, tokens, reps)
    return {"value": tokens * reps / t, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"first {tokens} of {w.T} tokens (all columns), {reps} passes, {t:.1f} s wall"}


def run_reference(args, w, desc):
    """--impl reference: the CPU oracle timed as the reference arm (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    total = args.steps + args.warmup
    t_full = time_oracle(w, min(w.T, 32), 1) / min(w.T, 32)          # seconds per token
    per_step_budget = 120.0 / max(total, 1)
    tokens = int(max(1, min(w.T, per_step_budget / max(t_full, 1e-9))))
    time_oracle(w, tokens, args.warmup)
    t = time_oracle(w, tokens, args.steps)
    value = tokens * args.steps / t
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": desc, "tokens_per_step": tokens},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": f"first {tokens} of {w.T} tokens per step (all columns)"},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default="q_proj_decode", choices=sorted(WORKLOADS) + ["full_projection_set"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-graph", action="store_true", help="time plain stream launches instead of CUDA-graph replay")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--pdl", type=int, default=None, help="EDGELORA_OPT_PDL value (0, 1, 2); default: library default")
    ap.add_argument("--decode-splits", type=int, default=0, help="tuning: EDGELORA_OPT_DECODE_SPLITS")
    ap.add_argument("--shrink-items", type=int, default=0, help="tuning: EDGELORA_OPT_SHRINK_ITEMS")
    args = ap.parse_args()

    if args.workload == "full_projection_set":   # configs[4]: 224 sites, its own driver
        if args.impl == "reference" or int(os.environ.get("WORLD_SIZE", "1")) > 1:
            raise SystemExit("full_projection_set: single GPU, --impl ours only")
        import torch
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
        torch.cuda.set_device(0)
        from paper_2507_01438_b200 import full_set_bench
        print(json.dumps(full_set_bench.run(args, peaks(), ClockSampler, max_over_ranks)), flush=True)
        return

    builder, bound, desc = WORKLOADS[args.workload]
    decode_like = bound == "hbm"
    if args.steps is None:
        args.steps = 100000 if decode_like else 2000
    if args.warmup is None:
        args.warmup = 200 if decode_like else 10
    args.warmup = max(args.warmup, 3)

    w = builder()
    if args.impl == "reference":
        run_reference(args, w, desc)
        return

    import torch
    import torch.distributed as dist
    from paper_2507_01438_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    # ---- resident state: n_rep replicas of (W, pool) so that every step reads cold data from HBM
    ws_bytes = w.algorithmic_bytes()
    n_rep = 1 if not decode_like else max(2, int(np.ceil(3 * L2_BYTES / ws_bytes)))
    if args.workload == "gate_up_prefill":
        n_rep = 2   # 273 MB per step already exceeds L2; two replicas keep W from being re-hit
    # The timed steps are independent batches (their W, x and ids are not produced by the step
    # before), so the library may let a step's first kernel start under the previous step's tail
    # (EDGELORA_OPT_PDL = 2).  The number for calls that depend on each other (mode 1, the
    # library's default) is measured as well and reported under "dependent_calls".
    pdl_mode = args.pdl if args.pdl is not None else (2 if decode_like else 1)
    to_bf16 = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)
    Ws, pools = [], []
    for r in range(n_rep):
        Ws.append(to_bf16(w.W) if r == 0 else Ws[0].clone())
        pool = B.Pool(w.h_in, w.h_out, w.n_slots, w.max_rank, max_tokens=w.T)
        pool.load_all(w.adapters)
        B.edgelora_pool_set_option(pool.handle, B.OPT_PDL, pdl_mode)
        if args.decode_splits:
            B.edgelora_pool_set_option(pool.handle, B.OPT_DECODE_SPLITS, args.decode_splits)
        if args.shrink_items:
            B.edgelora_pool_set_option(pool.handle, B.OPT_SHRINK_ITEMS, args.shrink_items)
        pools.append(pool)
    x = to_bf16(w.x)
    ids = torch.from_numpy(w.ids).cuda()
    ys = [torch.empty((w.T, w.h_out), dtype=torch.bfloat16, device="cuda") for _ in range(n_rep)]
    stream = torch.cuda.Stream()

    def step(i):
        r = i % n_rep
        B.edgelora_lora_linear(pools[r].handle, Ws[r], x, ids, ys[r], stream)

    graph = None
    # a graph holds several rotations of the replicas, so that the gap between two replays
    # (about 20 us) is spread over many steps
    per_graph = n_rep * (10 if decode_like else 1)
    with torch.cuda.stream(stream):
        for i in range(args.warmup):
            step(i)
        stream.synchronize()
        for pool in pools:
            rc, bits = pool.status()
            if rc != 0 or bits != 0:
                raise SystemExit(f"device status after warm-up: rc={rc} bits={bits:#x} ({B.strerror(rc)})")
        if not args.no_graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                for i in range(per_graph):
                    step(i)
            for _ in range(3):
                graph.replay()
            stream.synchronize()
    info = B.edgelora_pool_last_launch(pools[0].handle)

    def run_steps(k):
        with torch.cuda.stream(stream):
            if graph is not None:
                for _ in range(k // per_graph):
                    graph.replay()
                for i in range(k % per_graph):
                    step(i)
            else:
                for i in range(k):
                    step(i)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(torch.cuda.current_device() if "CUDA_VISIBLE_DEVICES" not in os.environ else
                           os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local])
    windows = []
    if rank == 0:
        sampler.start()
        time.sleep(0.2)

    # ---- timed region: exactly K steps, device time, max over ranks
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_start = time.time()
    e0.record(stream)
    run_steps(args.steps)
    e1.record(stream)
    barrier()
    windows.append((t_start, time.time()))
    ms = e0.elapsed_time(e1)
    ms = max_over_ranks(ms, world, "cuda")
    value = aggregate_tokens_per_s(w.T, args.steps, world, ms * 1e-3)

    # ---- spread over 20 windows of the same steps (one event at every window boundary)
    n_win = 20
    win_steps = per_graph if graph is not None else max(1, args.steps // (n_win * 5))
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_win + 1)]
    barrier()
    t_start = time.time()
    evs[0].record(stream)
    for i in range(n_win):
        run_steps(win_steps)
        evs[i + 1].record(stream)
    barrier()
    windows.append((t_start, time.time()))
    per_step = sorted(evs[i].elapsed_time(evs[i + 1]) / win_steps for i in range(n_win))
    iterations = {"windows": n_win, "steps_per_window": int(win_steps),
                  "ms_per_step_median": 0.5 * (per_step[n_win // 2 - 1] + per_step[n_win // 2]),
                  "ms_per_step_best": per_step[0], "ms_per_step_worst": per_step[-1]}

    # ---- the same step on ONE replica (W and, for small pools, the adapters stay in L2): labelled
    # warm, never the headline; and the latency of a single un-graphed call on cold data
    warm = None
    if graph is not None:
        wg = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            for _ in range(3):
                step(0)
            stream.synchronize()
            with torch.cuda.graph(wg, stream=stream):
                for _ in range(per_graph):
                    step(0)
            wg.replay()
        barrier()
        n_w = 10
        w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_start = time.time()
        w0.record(stream)
        with torch.cuda.stream(stream):
            for _ in range(n_w):
                wg.replay()
        w1.record(stream)
        barrier()
        windows.append((t_start, time.time()))
        warm = {"ms_per_step": w0.elapsed_time(w1) / (n_w * per_graph), "steps": n_w * per_graph,
                "note": "warm L2: one replica of W and the pool, not the cold rotation the headline uses"}
    lat = []
    for i in range(1, 41):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        with torch.cuda.stream(stream):
            step(i)
        stream.synchronize()
        lat.append((time.perf_counter() - t0) * 1e3)
    lat.sort()
    single_call = {"ms_median": 0.5 * (lat[19] + lat[20]), "ms_best": lat[0], "calls": 40,
                   "note": "one un-graphed call, launch to stream synchronise, wall clock, cold rotation"}

    dependent = None
    if pdl_mode == 2:   # same steps with the library's default launch mode, plain stream launches
        for p_ in pools:
            B.edgelora_pool_set_option(p_.handle, B.OPT_PDL, 1)
        k_dep = int(min(args.steps, 20000))
        with torch.cuda.stream(stream):
            for i in range(20):
                step(i)
        barrier()
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        d0.record(stream)
        with torch.cuda.stream(stream):
            for i in range(k_dep):
                step(i)
        d1.record(stream)
        barrier()
        ms_dep = d0.elapsed_time(d1)
        dependent = {"value": world * w.T * k_dep / (ms_dep * 1e-3), "unit": "tokens/s", "steps": k_dep,
                     "ms_per_step": ms_dep / k_dep, "launch": "plain stream launches, EDGELORA_OPT_PDL=1"}
        for p_ in pools:
            B.edgelora_pool_set_option(p_.handle, B.OPT_PDL, pdl_mode)

    # ---- end to end through the pipelined host-buffer entry point: every step copies x and the ids
    # from page-locked host memory and reads y back into page-locked host memory; the library
    # overlaps the copies of neighbouring steps with the layer (two sets of device mirrors per pool)
    k_e2e = int(min(args.steps, 3000 if decode_like else 200))
    hx = torch.from_numpy(np.ascontiguousarray(w.x).view(np.int16)).pin_memory()
    hids = torch.from_numpy(np.ascontiguousarray(w.ids)).pin_memory()
    hys = [torch.empty((w.T, w.h_out), dtype=torch.int16).pin_memory() for _ in range(2 * n_rep)]

    def e2e_step(i):
        r = i % n_rep
        B.edgelora_lora_linear_host_async(pools[r].handle, Ws[r], hx, hids, hys[2 * r + ((i // n_rep) & 1)], stream)

    for i in range(2 * n_rep + 1):
        e2e_step(i)
    for p_ in pools:
        B.edgelora_pool_host_sync(p_.handle)
    barrier()
    t_start = time.time()
    t0 = time.perf_counter()
    for i in range(k_e2e):
        e2e_step(i)
    for p_ in pools:
        B.edgelora_pool_host_sync(p_.handle)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    windows.append((t_start, time.time()))
    e2e_s = max_over_ranks(e2e_s, world, "cuda")
    e2e = {"value": world * w.T * k_e2e / e2e_s, "unit": "tokens/s", "steps": k_e2e,
           "h2d_bytes_per_step": int(w.x.nbytes + w.ids.nbytes), "d2h_bytes_per_step": int(w.T * w.h_out * 2),
           "api": "edgelora_lora_linear_host_async per step, edgelora_pool_host_sync at the end (wall clock)"}

    # ---- dominant kernel (base product): CUDA events around every launch, cold data
    k_prof = int(min(args.steps, 2000 if decode_like else 100))
    for p in pools:
        B.edgelora_pool_set_option(p.handle, B.OPT_PROFILE, 1)
        B.edgelora_pool_kernel_times(p.handle, reset=True)
    t_start = time.time()
    with torch.cuda.stream(stream):
        for i in range(k_prof):
            step(i)
    torch.cuda.synchronize()
    windows.append((t_start, time.time()))
    kt = {}
    for p in pools:
        for name, v in B.edgelora_pool_kernel_times(p.handle, reset=True).items():
            acc = kt.setdefault(name, {"ms": 0.0, "launches": 0})
            acc["ms"] += v["ms"]
            acc["launches"] += v["launches"]
        B.edgelora_pool_set_option(p.handle, B.OPT_PROFILE, 0)
    gemm_us = 1e3 * kt["base_gemm"]["ms"] / max(kt["base_gemm"]["launches"], 1)
    pk = peaks()
    if bound == "hbm":
        # the base-product kernel reads W once, x once and each distinct adapter's B once, and
        # writes y once; its fp32 split-K partials are not counted
        gemm_bytes = 2 * w.h_in * w.h_out + 2 * w.T * (w.h_in + w.h_out) + \
            sum(2 * w.adapters[a].rank * w.h_out for a in w.distinct_adapters())
        achieved = gemm_bytes / (gemm_us * 1e-6) / 1e9
        peak = pk["hbm_gbs"]
        roof = {"bound": "hbm", "kernel": "lora_gemm_kernel (decode mode)", "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak, "traffic": ncu_traffic(args.workload),
                "algorithmic_bytes": gemm_bytes, "kernel_us": gemm_us, "peak_source": pk["_source"] + ", burst copy",
                "frac_of_nominal": achieved / 7700.0, "nominal": "7.7 TB/s HBM3e (HGX B200)"}
        step_frac = (ws_bytes / (ms * 1e-3 / args.steps) / 1e9) / peak
    else:
        gemm_flops = 2.0 * w.T * w.h_in * w.h_out + 2.0 * sum(w.adapters[int(a)].rank for a in w.ids if a >= 0) * w.h_out
        achieved = gemm_flops / (gemm_us * 1e-6) / 1e12
        peak = pk["bf16_tflops"]
        roof = {"bound": "tensor", "kernel": "lora_gemm_kernel (prefill mode)", "achieved": achieved, "peak": peak,
                "unit": "TFLOP/s", "frac": achieved / peak, "traffic": ncu_traffic(args.workload),
                "algorithmic_flops": gemm_flops, "kernel_us": gemm_us, "peak_source": pk["_source"] + ", burst",
                "frac_of_nominal": achieved / 2250.0, "nominal": "2.25 PFLOP/s dense bf16"}
        step_frac = (w.algorithmic_flops() / (ms * 1e-3 / args.steps) / 1e12) / peak

    if rank == 0:
        time.sleep(0.1)
        sampler.stop()
    for p in pools:
        p.close()
    if world > 1:
        dist.destroy_process_group()
    if rank != 0:
        return

    line = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": desc, "T": w.T, "h_in": w.h_in, "h_out": w.h_out, "n_slots": w.n_slots,
                   "max_rank": w.max_rank, "distinct_adapters": len(w.distinct_adapters()),
                   "regime": info["regime"], "split_k": info["split_k"], "gemm_grid": info["gemm_grid"],
                   "stages": info["stages"], "pdl_mode": pdl_mode, "launch": "plain stream launches" if graph is None else
                   f"CUDA-graph replay of {per_graph} consecutive steps",
                   "l2": f"inputs larger than L2: {n_rep} replicas of W and the adapter pool used in rotation "
                         f"({n_rep * ws_bytes / 2**20:.0f} MiB)", "parallelism": f"replicas x{world}"},
        "clocks": sampler.summary(windows),
        "e2e": e2e,
        "gpu_launches": int(info["launches"] * args.steps),
        "kernels_per_step": info["launches"],
        "roofline": roof,
        "step_roofline_frac": step_frac,
        "iterations": iterations,
        "warm_l2": warm,
        "single_call_latency": single_call,
        "kernel_ms_profiled": {k: v for k, v in kt.items() if v["launches"]},
    }
    if dependent is not None:
        line["dependent_calls"] = dependent
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(w)
    print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
