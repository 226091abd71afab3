#!/usr/bin/env python
"""Benchmark of the batch LoRA linear layer (paper Section 3.4) on B200.

A step is one pass of the whole hot path over one synthetic batch: routing plan, shrink, base
product, expand/combine.  Four timed workloads (the Llama-3.1-8B-shaped configurations):

  q_proj_decode          4096 -> 4096, 32 adapters r16, 32 tokens each on its own adapter   (HBM)
  gate_up_prefill        4096 -> 14336, 8 adapters r16, 8 runs of 512 tokens                (tensor)
  down_proj_many_tenant  14336 -> 4096, 1000 adapters r64, 256 tokens Zipf(1.1), 10% base   (HBM)
  full_projection_set    7 projections x 32 layers = 224 sites, 128 adapters r{8,16,32},
                         64 decode tokens + 2 runs of 1024 tokens, one plan per batch      (tensor)

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME|all] [--impl reference]

With no --workload the headline (value, ms_per_step, roofline, e2e, cpu_baseline) is the largest
single-GPU workload, the full projection set, timed over exactly K steps after W warm-up steps; the
other three are measured in the same run and reported under "per_config".  One JSON line on rank 0.
With N > 1 every rank runs an independent replica on its own GPU: the layer has no exchange step,
so there is no data-path collective; only the timing barrier and the max over ranks use
torch.distributed.  `--gpus N` without a torchrun environment starts the N ranks itself.
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
NOMINAL_HBM_GBS, NOMINAL_BF16_TFLOPS = 7700.0, 2250.0

SITE_WORKLOADS = {
    # name: (builder, bound, description)
    "q_proj_decode": (lambda: wl.q_proj_decode(), "hbm",
                      "configs[1]: Llama-3.1-8B q_proj decode 4096->4096, 32 adapters r16, T=32 distinct ids"),
    "gate_up_prefill": (lambda: wl.gate_up_prefill(), "tensor",
                        "configs[2]: gate/up prefill 4096->14336, 8 adapters r16, 8 x 512-token segments"),
    "down_proj_many_tenant": (lambda: wl.down_proj_many_tenant(), "hbm",
                              "configs[3]: down_proj 14336->4096, 1000 adapters r64, T=256 Zipf(1.1), 10% base-only"),
    "tiny": (lambda: wl.tiny(), "hbm", "configs[0]: 256->256, 4 adapters r8, T=16"),
    # next row N2: the same batch over a pool that keeps A in Q8_0 (paper Section 5.1); only the
    # adapters the batch touches are drawn and loaded, the other slots of the 1000 stay empty
    "down_proj_many_tenant_q8": (lambda: wl.down_proj_many_tenant(only_used=True), "hbm",
                                 "configs[3] with Q8_0 adapters: down_proj 14336->4096, pool of 1000 slots keeping A "
                                 "in Q8_0, rank 64, T=256 Zipf(1.1), 10% base-only"),
    # smaller resident pool, same layer and batch recipe: sized for multi-pass profiler captures
    "down_proj_200_tenants": (lambda: wl.down_proj_many_tenant(n_adapters=200), "hbm",
                              "profiling-size variant of configs[3]: down_proj 14336->4096, 200 adapters r64, T=256"),
}
FULL_SET = "full_projection_set"
FULL_SET_DESC = ("configs[4]: full Llama-3.1-8B projection set x32 layers (224 sites), 128 adapters ranks "
                 "{8,16,32}, 64 decode tokens + 2 x 1024-token prefill runs, one plan for all sites")
DEFAULT_ORDER = ("q_proj_decode", "gate_up_prefill", "down_proj_many_tenant", FULL_SET)


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
    """DRAM bytes per launch of the dominant kernel from the committed profiler summary, if any."""
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
                 "-lms", "20", "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
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


# --------------------------------------------------------------------------- CPU oracle timing
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


def cpu_baseline_site(w, budget_s):
    """The CPU oracle, as it stands, on a bounded sample of one site's workload."""
    import oracle
    tokens = min(w.T, 64)
    t1 = time_oracle(w, tokens, 1)
    reps = int(max(1, min(200, budget_s / max(t1, 1e-6))))
    t = time_oracle(w, tokens, reps)
    return {"value": tokens * reps / t, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"first {tokens} of {w.T} tokens (all columns), {reps} passes, {t:.1f} s wall"}


class FullSetOracleSample:
    """The oracle on the seven sites of one decoder layer (numpy-generated values) over a token
    sample that holds decode tokens and tokens of both runs; a full step is 32 such layers."""

    def __init__(self):
        batch = wl.full_set_batch()
        self.rows = np.array(list(range(0, 64, 4)) + list(range(64, 2112, 128)))   # 16 decode + 16 prefill tokens
        self.sites = [wl.full_set_site(batch, 0, s) for s in range(len(wl.LLAMA8B_SITES))]
        for w in self.sites:
            w.x = np.ascontiguousarray(w.x[self.rows])
            w.ids = np.ascontiguousarray(batch.ids[self.rows])

    def one_pass(self):
        t0 = time.perf_counter()
        for w in self.sites:
            time_oracle(w, len(self.rows), 1)
        return time.perf_counter() - t0

    def tokens_per_s(self, seconds, passes):
        return 1.0 / (seconds / (passes * len(self.rows)) * wl.LLAMA8B_LAYERS)

    def sample(self, passes, seconds):
        return (f"{len(self.rows)} tokens (16 decode, 16 prefill) through the 7 sites of one layer, {passes} passes, "
                f"{seconds:.1f} s wall; tokens/s of a full step = 1 / (seconds per token and layer x 32 layers)")


def full_set_oracle_sample(budget_s):
    import oracle
    o = FullSetOracleSample()
    t, passes = 0.0, 0
    while passes == 0 or (t < budget_s and passes < 50):
        t += o.one_pass()
        passes += 1
    return {"value": o.tokens_per_s(t, passes), "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": o.sample(passes, t)}


def static_config(name):
    """The part of `config` that does not depend on the run (the reference arm prints the same)."""
    if name == FULL_SET:
        return {"workload": FULL_SET_DESC, "T": 2112, "sites": 224,
                "l2": "inputs larger than L2: 14 GB of weights and 2.7 GB of touched adapters per step",
                "launch": "plain stream launches through edgelora_siteset_run"}
    builder, bound, desc = SITE_WORKLOADS[name]
    return {"workload": desc}


def run_reference(args, name):
    """--impl reference: the CPU oracle timed as the reference arm (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    total = args.steps + args.warmup
    if name == FULL_SET:
        # a step = one pass of the bounded sample (see FullSetOracleSample)
        o = FullSetOracleSample()
        for _ in range(min(args.warmup, 2)):
            o.one_pass()
        t = sum(o.one_pass() for _ in range(args.steps))
        value = o.tokens_per_s(t, args.steps)
        sample = o.sample(args.steps, t)
        ms_step = 1e3 * t / args.steps
    else:
        w = SITE_WORKLOADS[name][0]()
        t_full = time_oracle(w, min(w.T, 32), 1) / min(w.T, 32)          # seconds per token
        per_step_budget = 120.0 / max(total, 1)
        tokens = int(max(1, min(w.T, per_step_budget / max(t_full, 1e-9))))
        time_oracle(w, tokens, args.warmup)
        t = time_oracle(w, tokens, args.steps)
        value = tokens * args.steps / t
        sample = f"first {tokens} of {w.T} tokens per step (all columns)"
        ms_step = 1e3 * t / args.steps
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": static_config(name),
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- one linear site
def bench_site(name, ctx, steps=None, warmup=None, pdl=None, graph=True, cpu_budget=4.0):
    """One linear site: the timed steps, the spread over 20 windows, launch-mode variants, the
    dominant kernel, the end-to-end number and the oracle beside it.  Returns a dict."""
    import torch
    from paper_2507_01438_b200 import binding as B
    world, barrier, sampler = ctx["world"], ctx["barrier"], ctx["sampler"]
    builder, bound, desc = SITE_WORKLOADS[name]
    decode_like = bound == "hbm"
    q8 = name.endswith("_q8")
    w = builder()
    warmup = max(3, warmup if warmup is not None else (50 if decode_like else 5))

    # ---- resident state: n_rep replicas of (W, pool) so that every step reads cold data from HBM
    ws_bytes = w.algorithmic_bytes()
    q8_blocks = {}
    if q8:   # A in Q8_0: 34 bytes per 32 values instead of 64
        ws_bytes -= sum(w.adapters[a].rank * w.h_in * 2 - w.adapters[a].rank * (w.h_in // 32) * 34
                        for a in w.distinct_adapters())
        cpu_budget = 0.0
        for a, ad in w.adapters.items():
            q8_blocks[a] = (wl.q8_0_encode(wl.bf16_bits_to_f32(ad.A)), wl.q8_0_encode(wl.bf16_bits_to_f32(ad.B)))
    n_rep = 2 if not decode_like else max(2, int(np.ceil(3 * L2_BYTES / ws_bytes)))
    pdl_mode = pdl if pdl is not None else 1            # the library's default: calls may depend on each other
    to_bf16 = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)
    Ws, pools = [], []
    for r in range(n_rep):
        Ws.append(to_bf16(w.W) if r == 0 else Ws[0].clone())
        pool = B.Pool(w.h_in, w.h_out, w.n_slots, w.max_rank, max_tokens=w.T, flags=B.FLAG_A_Q8 if q8 else 0)
        if q8:
            for a, ad in w.adapters.items():
                B.edgelora_pool_load_slot_q8(pool.handle, a, ad.rank, ad.scale, q8_blocks[a][0], q8_blocks[a][1])
            B.edgelora_pool_wait_loads(pool.handle)
        else:
            pool.load_all(w.adapters)
        B.edgelora_pool_set_option(pool.handle, B.OPT_PDL, pdl_mode)
        pools.append(pool)
    x = to_bf16(w.x)
    ids = torch.from_numpy(w.ids).cuda()
    ys = [torch.empty((w.T, w.h_out), dtype=torch.bfloat16, device="cuda") for _ in range(n_rep)]
    stream = torch.cuda.Stream()

    def step(i):
        r = i % n_rep
        B.edgelora_lora_linear(pools[r].handle, Ws[r], x, ids, ys[r], stream)

    def set_pdl(mode):
        for p_ in pools:
            B.edgelora_pool_set_option(p_.handle, B.OPT_PDL, mode)

    def capture(n_steps):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            with torch.cuda.graph(g, stream=stream):
                for i in range(n_steps):
                    step(i)
            g.replay()
            stream.synchronize()
        return g

    with torch.cuda.stream(stream):
        for i in range(warmup):
            step(i)
        stream.synchronize()
    for pool in pools:
        rc, bits = pool.status()
        if rc != 0 or bits != 0:
            raise SystemExit(f"{name}: device status after warm-up: rc={rc} bits={bits:#x} ({B.strerror(rc)})")
    info = B.edgelora_pool_last_launch(pools[0].handle)

    # a graph holds several rotations of the replicas, so that the gap between two replays (about
    # 20 us) is spread over many steps; with few steps asked for, a graph of that many steps (but
    # never less than one rotation)
    per_graph = n_rep * (10 if decode_like else 1)
    if steps is not None and steps < per_graph:
        per_graph = max(n_rep, steps - steps % n_rep) if steps >= n_rep else n_rep
    g_main = capture(per_graph) if graph else None

    def run_steps(k, g):
        """k steps: whole replays of g, the rest as plain launches.  Returns (replays, plain)."""
        with torch.cuda.stream(stream):
            if g is None:
                for i in range(k):
                    step(i)
                return 0, k
            for _ in range(k // per_graph):
                g.replay()
            for i in range(k % per_graph):
                step(i)
            return k // per_graph, k % per_graph

    def timed(k, g):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t_start = time.time()
        e0.record(stream)
        shape = run_steps(k, g)
        e1.record(stream)
        barrier()
        ctx["windows"].append((t_start, time.time()))
        return max_over_ranks(e0.elapsed_time(e1), world, "cuda"), shape

    # ---- timed region: exactly `steps` steps (default: about a second of them), device time
    if steps is None:
        probe_ms, _ = timed(per_graph, g_main)
        steps = int(max(per_graph, min(200000, (1000.0 / max(probe_ms, 1e-3)) * per_graph)))
        steps -= steps % per_graph
    ms, (n_replays, n_plain) = timed(steps, g_main)
    value = aggregate_tokens_per_s(w.T, steps, world, ms * 1e-3)
    if g_main is None:
        launch = f"{steps} plain stream launches"
    else:
        launch = f"{n_replays} replays of a CUDA graph of {per_graph} consecutive steps" + \
                 (f" + {n_plain} plain launches" if n_plain else "")

    # ---- spread over 20 windows (one event at every window boundary), each about 50 ms
    n_win = 20
    win_steps = max(per_graph, int(steps / 20) - int(steps / 20) % per_graph)
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_win + 1)]
    barrier()
    t_start = time.time()
    evs[0].record(stream)
    for i in range(n_win):
        run_steps(win_steps, g_main)
        evs[i + 1].record(stream)
    barrier()
    ctx["windows"].append((t_start, time.time()))
    per_step = sorted(evs[i].elapsed_time(evs[i + 1]) / win_steps for i in range(n_win))
    iterations = {"windows": n_win, "steps_per_window": int(win_steps),
                  "ms_per_step_median": 0.5 * (per_step[n_win // 2 - 1] + per_step[n_win // 2]),
                  "ms_per_step_best": per_step[0], "ms_per_step_worst": per_step[-1]}

    # ---- other launch modes of the same steps: plain launches in the default mode; and, for decode,
    # EDGELORA_OPT_PDL = 2 ("independent calls": a call's first kernel may start under the previous
    # call's tail, valid when the calls do not feed each other, e.g. q/k/v of one layer)
    variants = {}
    k_var = int(min(steps, 20000))
    ms_plain, _ = timed(k_var, None)
    variants["plain_launches"] = {"ms_per_step": ms_plain / k_var, "steps": k_var,
                                  "launch": f"plain stream launches, EDGELORA_OPT_PDL={pdl_mode}"}
    if decode_like and pdl is None and graph:
        set_pdl(2)
        with torch.cuda.stream(stream):
            for i in range(n_rep):
                step(i)
            stream.synchronize()
        g2 = capture(per_graph)
        k2 = max(per_graph, k_var - k_var % per_graph)
        ms2, _ = timed(k2, g2)
        variants["independent_calls"] = {"ms_per_step": ms2 / k2, "steps": k2,
                                         "tokens_per_s": world * w.T * k2 / (ms2 * 1e-3),
                                         "launch": f"CUDA-graph replay of {per_graph} steps, EDGELORA_OPT_PDL=2 "
                                                   "(calls that do not depend on each other)"}
        del g2
        set_pdl(pdl_mode)

    # ---- the same step on ONE replica (W and, for small pools, the adapters stay in L2): labelled
    # warm, never the headline; and the latency of a single un-graphed call on cold data
    warm = None
    if graph:
        with torch.cuda.stream(stream):
            for _ in range(3):
                step(0)
            stream.synchronize()
        wg = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            with torch.cuda.graph(wg, stream=stream):
                for _ in range(per_graph):
                    step(0)
            wg.replay()
        barrier()
        n_w = 10
        w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        w0.record(stream)
        with torch.cuda.stream(stream):
            for _ in range(n_w):
                wg.replay()
        w1.record(stream)
        barrier()
        warm = {"ms_per_step": w0.elapsed_time(w1) / (n_w * per_graph), "steps": n_w * per_graph,
                "note": "warm L2: one replica of W and the pool, not the cold rotation the headline uses"}
        del wg
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

    # ---- adapter swaps beside the layer (Section 3.3 / 4.2: a missing adapter is loaded into a free
    # block while serving goes on): plain launches with 0, 1 and 4 loads per step into blocks the
    # batch does not use, from page-locked host memory, copies on the pool's side stream
    swap = None
    if decode_like and w.n_slots <= 64 and not q8:
        spare_pools = []
        for r in range(n_rep):
            sp = B.Pool(w.h_in, w.h_out, w.n_slots + 4, w.max_rank, max_tokens=w.T)
            sp.load_all(w.adapters)
            spare_pools.append(sp)
        ad0 = w.adapters[sorted(w.adapters)[0]]
        Rp = 16 if w.max_rank <= 16 else (32 if w.max_rank <= 32 else 64)
        if ad0.rank == Rp:
            pa = torch.from_numpy(ad0.A.view(np.int16).copy()).pin_memory()
            pb = torch.from_numpy(ad0.B.view(np.int16).copy()).pin_memory()
            swap = {"adapter_bytes": int(ad0.A.nbytes + ad0.B.nbytes), "per_step": {}}
            for n_sw in (0, 1, 4):
                k_sw = 2000
                for timed_pass in (False, True):
                    torch.cuda.synchronize()
                    t0 = time.perf_counter()
                    for i in range(k_sw if timed_pass else 50):
                        r = i % n_rep
                        for j in range(n_sw):
                            B.edgelora_pool_load_slot_pinned(spare_pools[r].handle, w.n_slots + j, Rp, ad0.scale, pa, pb)
                        B.edgelora_lora_linear(spare_pools[r].handle, Ws[r], x, ids, ys[r], stream)
                    torch.cuda.synchronize()
                    dt = time.perf_counter() - t0
                swap["per_step"][str(n_sw)] = {"us_per_step_wall": 1e6 * dt / k_sw, "swaps_per_s": n_sw * k_sw / dt,
                                               "adapter_gb_per_s": n_sw * k_sw * swap["adapter_bytes"] / dt / 1e9}
        for sp in spare_pools:
            sp.close()

    # ---- end to end through the pipelined host-buffer entry point: every step copies x and the ids
    # from page-locked host memory and reads y back into page-locked host memory; the library
    # overlaps the copies of neighbouring steps with the layer (two sets of device mirrors per pool)
    k_e2e = int(min(steps, 3000 if decode_like else 100))
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
    ctx["windows"].append((t_start, time.time()))
    e2e_s = max_over_ranks(e2e_s, world, "cuda")
    e2e = {"value": world * w.T * k_e2e / e2e_s, "unit": "tokens/s", "steps": k_e2e,
           "h2d_bytes_per_step": int(w.x.nbytes + w.ids.nbytes), "d2h_bytes_per_step": int(w.T * w.h_out * 2),
           "api": "edgelora_lora_linear_host_async per step, edgelora_pool_host_sync at the end (wall clock)"}

    # ---- dominant kernel (base product): CUDA events around every launch, cold data.  A serialised
    # latency: launch gap included, nothing overlapped, so it is not a share of the step time above.
    k_prof = int(min(steps, 2000 if decode_like else 100))
    for p in pools:
        B.edgelora_pool_set_option(p.handle, B.OPT_PROFILE, 1)
        B.edgelora_pool_kernel_times(p.handle, reset=True)
    t_start = time.time()
    with torch.cuda.stream(stream):
        for i in range(k_prof):
            step(i)
    torch.cuda.synchronize()
    ctx["windows"].append((t_start, time.time()))
    kt = {}
    for p in pools:
        for kname, v in B.edgelora_pool_kernel_times(p.handle, reset=True).items():
            acc = kt.setdefault(kname, {"ms": 0.0, "launches": 0})
            acc["ms"] += v["ms"]
            acc["launches"] += v["launches"]
        B.edgelora_pool_set_option(p.handle, B.OPT_PROFILE, 0)
    gemm_us = 1e3 * kt["base_gemm"]["ms"] / max(kt["base_gemm"]["launches"], 1)
    pk = ctx["peaks"]
    us_step = 1e3 * ms / steps
    if bound == "hbm":
        # the base-product kernel reads W once, x once and each distinct adapter's B once, and
        # writes y once; its fp32 split-K partials are not counted
        gemm_bytes = 2 * w.h_in * w.h_out + 2 * w.T * (w.h_in + w.h_out) + \
            sum(2 * w.adapters[a].rank * w.h_out for a in w.distinct_adapters())
        kernel_name = "lora_gemm_kernel (decode mode)"
        if not any(kt.get(k, {}).get("launches", 0) for k in ("shrink_small_decode", "shrink_tiles", "plan")):
            # one launch per call: the same kernel also reads every distinct A_a (its shrink teams)
            gemm_bytes = ws_bytes
            kernel_name = "lora_gemm_kernel (decode mode with the shrink teams in its grid: the whole call)"
        achieved = gemm_bytes / (gemm_us * 1e-6) / 1e9
        peak = pk["hbm_gbs"]
        roof = {"bound": "hbm", "kernel": kernel_name, "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak, "traffic": ncu_traffic(name),
                "algorithmic_bytes": gemm_bytes, "kernel_us": gemm_us,
                "kernel_us_is": "serialised latency of one launch between two CUDA events (launch gap included)",
                "peak_source": pk["_source"] + ", burst copy",
                "frac_of_nominal": achieved / NOMINAL_HBM_GBS, "nominal": "7.7 TB/s HBM3e (HGX B200)"}
        step_work = {"algorithmic_bytes": ws_bytes, "achieved_gbs": ws_bytes / (us_step * 1e-6) / 1e9}
        step_frac = step_work["achieved_gbs"] / peak
        step_frac_nominal = step_work["achieved_gbs"] / NOMINAL_HBM_GBS
    else:
        gemm_flops = 2.0 * w.T * w.h_in * w.h_out + 2.0 * sum(w.adapters[int(a)].rank for a in w.ids if a >= 0) * w.h_out
        achieved = gemm_flops / (gemm_us * 1e-6) / 1e12
        peak = pk["bf16_tflops"]
        roof = {"bound": "tensor", "kernel": "lora_gemm_kernel (prefill mode)", "achieved": achieved, "peak": peak,
                "unit": "TFLOP/s", "frac": achieved / peak, "traffic": ncu_traffic(name),
                "algorithmic_flops": gemm_flops, "kernel_us": gemm_us,
                "kernel_us_is": "serialised latency of one launch between two CUDA events (launch gap included)",
                "peak_source": pk["_source"] + ", burst",
                "frac_of_nominal": achieved / NOMINAL_BF16_TFLOPS, "nominal": "2.25 PFLOP/s dense bf16"}
        step_work = {"algorithmic_flops": w.algorithmic_flops(),
                     "achieved_tflops": w.algorithmic_flops() / (us_step * 1e-6) / 1e12}
        step_frac = step_work["achieved_tflops"] / peak
        step_frac_nominal = step_work["achieved_tflops"] / NOMINAL_BF16_TFLOPS

    res = {
        "name": name, "value": value, "unit": "tokens/s", "steps": steps, "warmup": warmup,
        "ms_per_step": ms / steps,
        "config": {**static_config(name), "T": w.T, "h_in": w.h_in, "h_out": w.h_out, "n_slots": w.n_slots,
                   "max_rank": w.max_rank, "G": len(w.distinct_adapters()),
                   "launch": launch + f", EDGELORA_OPT_PDL={pdl_mode}",
                   "l2": f"inputs larger than L2: {n_rep} replicas of W and the adapter pool used in rotation "
                         f"({n_rep * ws_bytes / 2**20:.0f} MiB)", "parallelism": f"replicas x{world}"},
        "launch_info": {"regime": info["regime"], "split_k": info["split_k"], "gemm_grid": info["gemm_grid"],
                        "stages": info["stages"], "kernels_per_step": info["launches"]},
        "gpu_launches": int(info["launches"] * steps),
        "iterations": iterations, "step_work": step_work, "step_roofline_frac": step_frac,
        "step_roofline_frac_of_nominal": step_frac_nominal, "roofline": roof, "e2e": e2e,
        "variants": variants, "warm_l2": warm, "single_call_latency": single_call, "adapter_swaps": swap,
        "kernel_ms_profiled": {k: v for k, v in kt.items() if v["launches"]},
    }
    if ctx["rank"] == 0 and world == 1 and cpu_budget > 0:
        res["cpu_baseline"] = cpu_baseline_site(w, cpu_budget)
    for p in pools:
        p.close()
    del Ws, ys, x
    torch.cuda.empty_cache()
    return res


# --------------------------------------------------------------------------- the 224-site set
def bench_full_set(ctx, steps=None, warmup=None, cpu_budget=12.0, layers=wl.LLAMA8B_LAYERS):
    """Only the ids, the ranks and x come from the seeded numpy recipe (workloads.full_set_batch);
    the 14 GB of weights are drawn on the device and one host adapter per (rank, shape) serves every
    slot of that shape: values do not change the timing (parity of this configuration is checked on
    sampled sites by the GPU tests, with the numpy-generated values)."""
    import torch
    from paper_2507_01438_b200 import binding as B
    world, barrier = ctx["world"], ctx["barrier"]
    steps = steps if steps is not None else 20
    warmup = max(3, warmup if warmup is not None else 3)
    batch = wl.full_set_batch()
    T = len(batch.ids)
    used = sorted(set(int(a) for a in batch.ids if a >= 0))
    rng = np.random.Generator(np.random.PCG64(4))
    host = {}
    gen = torch.Generator(device="cuda")
    gen.manual_seed(4)
    sites = []
    for layer in range(layers):
        for sname, h_in, h_out in wl.LLAMA8B_SITES:
            W = (torch.randn((h_out, h_in), generator=gen, device="cuda", dtype=torch.float32) * wl.STD_W).to(torch.bfloat16)
            pool = B.Pool(h_in, h_out, batch.n_slots, batch.max_rank, max_tokens=T)
            for a in used:
                r = int(batch.ranks[a])
                key = (r, h_in, h_out)
                if key not in host:
                    host[key] = (wl.normal_bf16(rng, (r, h_in), wl.STD_W), wl.normal_bf16(rng, (h_out, r), wl.STD_W))
                pool.load(a, host[key][0], host[key][1], wl.SCALE)
            B.edgelora_pool_wait_loads(pool.handle)
            sites.append((sname, h_in, h_out, W, pool))
    to_bf16 = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)
    widths = (4096, 14336)
    xs = [to_bf16(batch.x4096), to_bf16(batch.x14336)]
    ids = torch.from_numpy(batch.ids).cuda()
    ybuf = {h: torch.empty((T, h), dtype=torch.bfloat16, device="cuda") for h in (1024, 4096, 14336)}
    ys = [ybuf[s[2]] for s in sites]
    sset = B.edgelora_siteset_create([s[4].handle for s in sites], [s[3] for s in sites],
                                     [widths.index(s[1]) for s in sites], 2, T)
    stream = torch.cuda.Stream()

    def step():
        B.edgelora_siteset_run(sset, xs, ids, ys, stream)

    with torch.cuda.stream(stream):
        for _ in range(warmup):
            step()
    stream.synchronize()
    for s in sites:
        rc, bits = s[4].status()
        if rc != 0 or bits != 0:
            raise SystemExit(f"full set: device status after warm-up: rc={rc} bits={bits:#x}")

    def timed(k):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t_start = time.time()
        e0.record(stream)
        with torch.cuda.stream(stream):
            for _ in range(k):
                step()
        e1.record(stream)
        barrier()
        ctx["windows"].append((t_start, time.time()))
        return max_over_ranks(e0.elapsed_time(e1), world, "cuda")

    ms = timed(steps)
    value = aggregate_tokens_per_s(T, steps, world, ms * 1e-3)
    # spread: 20 single steps, one event per boundary
    n_win = 20
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_win + 1)]
    barrier()
    t_start = time.time()
    evs[0].record(stream)
    with torch.cuda.stream(stream):
        for i in range(n_win):
            step()
            evs[i + 1].record(stream)
    barrier()
    ctx["windows"].append((t_start, time.time()))
    per_step = sorted(evs[i].elapsed_time(evs[i + 1]) for i in range(n_win))
    iterations = {"windows": n_win, "steps_per_window": 1,
                  "ms_per_step_median": 0.5 * (per_step[n_win // 2 - 1] + per_step[n_win // 2]),
                  "ms_per_step_best": per_step[0], "ms_per_step_worst": per_step[-1]}

    # end to end through the host-buffer call of the set: x (both widths) and the ids from pinned
    # host memory every step, the seven results of the last decoder layer read back
    hx = [torch.from_numpy(np.ascontiguousarray(b).view(np.int16)).pin_memory() for b in (batch.x4096, batch.x14336)]
    hids = torch.from_numpy(batch.ids).pin_memory()
    n_back = len(wl.LLAMA8B_SITES)
    hys = [None] * (len(sites) - n_back) + \
          [torch.empty((T, s[2]), dtype=torch.int16).pin_memory() for s in sites[-n_back:]]
    k_e2e = max(3, min(steps, 10))
    B.edgelora_siteset_run_host(sset, hx, hids, hys, stream)
    barrier()
    t_start = time.time()
    t0 = time.perf_counter()
    for _ in range(k_e2e):
        B.edgelora_siteset_run_host(sset, hx, hids, hys, stream)
    e2e_s = time.perf_counter() - t0
    ctx["windows"].append((t_start, time.time()))
    e2e_s = max_over_ranks(e2e_s, world, "cuda")
    e2e = {"value": world * T * k_e2e / e2e_s, "unit": "tokens/s", "steps": k_e2e,
           "h2d_bytes_per_step": int(batch.x4096.nbytes + batch.x14336.nbytes + batch.ids.nbytes),
           "d2h_bytes_per_step": int(sum(T * s[2] * 2 for s in sites[-n_back:])),
           "api": "edgelora_siteset_run_host: pinned H2D of both inputs and the ids, 224 sites, D2H of the last "
                  "decoder layer's seven results, stream synchronise (wall clock)"}

    # dominant kernel: the base product of every site, one CUDA-event pair per launch (serialised)
    for s in sites:
        B.edgelora_pool_set_option(s[4].handle, B.OPT_PROFILE, 1)
        B.edgelora_pool_kernel_times(s[4].handle, reset=True)
    with torch.cuda.stream(stream):
        step()
    torch.cuda.synchronize()
    kt = {}
    per_site = {}     # site name -> [device ms of its base-product launches, launches, flops of one launch]
    for s in sites:
        for kname, v in B.edgelora_pool_kernel_times(s[4].handle, reset=True).items():
            acc = kt.setdefault(kname, {"ms": 0.0, "launches": 0})
            acc["ms"] += v["ms"]
            acc["launches"] += v["launches"]
            if kname == "base_gemm":
                ps = per_site.setdefault(s[0], [0.0, 0, 2.0 * T * s[1] * s[2]])
                ps[0] += v["ms"]
                ps[1] += v["launches"]
        B.edgelora_pool_set_option(s[4].handle, B.OPT_PROFILE, 0)
    per_site_us = {k: {"kernel_us": 1e3 * v[0] / max(v[1], 1),
                       "base_tflops": v[2] / (1e-3 * v[0] / max(v[1], 1)) / 1e12 if v[0] > 0 else None}
                   for k, v in per_site.items()}
    # kernels of one step in the timed configuration
    before = sum(B.edgelora_pool_last_launch(s[4].handle)["total_launches"] for s in sites)
    with torch.cuda.stream(stream):
        step()
    torch.cuda.synchronize()
    launches_per_step = 1 + sum(B.edgelora_pool_last_launch(s[4].handle)["total_launches"] for s in sites) - before

    rank_sum = sum(int(batch.ranks[a]) for a in batch.ids if a >= 0)
    flops = sum(2 * T * h_in * h_out + 2 * rank_sum * (h_in + h_out) for _, h_in, h_out, _, _ in sites)
    pk = ctx["peaks"]
    gemm_ms = kt["base_gemm"]["ms"]
    peak = pk.get("bf16_tflops_sustained", pk["bf16_tflops"])
    achieved = flops / (gemm_ms * 1e-3) / 1e12
    step_tflops = flops / (ms * 1e-3 / steps) / 1e12
    res = {
        "name": FULL_SET, "value": value, "unit": "tokens/s", "steps": steps, "warmup": warmup,
        "ms_per_step": ms / steps,
        "config": {**static_config(FULL_SET), "G": len(used), "parallelism": f"replicas x{world}"},
        "launch_info": {"regime": "prefill", "kernels_per_step": launches_per_step,
                        "note": "the shrink of site i+1 is issued with the kernels of site i"},
        "gpu_launches": int(launches_per_step * steps),
        "iterations": iterations,
        "step_work": {"algorithmic_flops": flops, "achieved_tflops": step_tflops},
        "step_roofline_frac": step_tflops / peak,
        "step_roofline_frac_of_nominal": step_tflops / NOMINAL_BF16_TFLOPS,
        "roofline": {"bound": "tensor", "kernel": "lora_gemm_kernel (prefill mode), all 224 sites of a step",
                     "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak, "traffic": (ncu_traffic("full_projection_set_per_layer") or 0) * layers or None,
                     "algorithmic_flops": flops, "kernel_us": 1e3 * gemm_ms / max(kt["base_gemm"]["launches"], 1),
                     "kernel_us_is": "serialised latency of one launch between two CUDA events (launch gap included), "
                                     "mean over the 224 sites; with events between the kernels nothing overlaps",
                     "peak_source": pk["_source"] + ", sustained (the kernel runs inside a long step)",
                     "frac_of_nominal": achieved / NOMINAL_BF16_TFLOPS, "nominal": "2.25 PFLOP/s dense bf16"},
        "e2e": e2e,
        "kernel_ms_profiled": {k: v for k, v in kt.items() if v["launches"]},
        # per projection site, mean over the layers: serialised device time of its launch (its base product
        # and the next site's shrink tiles) and the base product's flops over that time
        "per_site": per_site_us,
    }
    if ctx["rank"] == 0 and world == 1 and cpu_budget > 0:
        res["cpu_baseline"] = full_set_oracle_sample(cpu_budget)
    B.edgelora_siteset_destroy(sset)
    for s in sites:
        s[4].close()
    del sites, xs, ys, ybuf
    torch.cuda.empty_cache()
    return res


# --------------------------------------------------------------------------- serving trace
SERVING = "serving_trace"


def bench_serving(ctx, layers=wl.LLAMA8B_LAYERS):
    """The request batcher (slot state machine) driving the layer over a synthetic trace (paper
    Section 5.1 workload: Gamma arrivals, power-law adapters, uniform lengths; gamma slots, top-k
    candidates).  The model is one decoder layer's seven projection sites (random values); a step
    costs the measured GPU time of the site set over the step's batch, times the number of layers:
    the clock is virtual, the arrival rate is scaled to a B200 instead of an edge device."""
    import torch
    from paper_2507_01438_b200 import binding as B
    n_adapters, n_blocks, gamma, top_k, rank = 200, 64, 20, 3, 16
    max_tokens = 2112
    trace = wl.serving_trace(seed=5, n_adapters=n_adapters, alpha=1.0, rate=25.0, cv=1.0, duration=20.0,
                             in_range=(8, 256), out_range=(8, 128), top_k=top_k)
    rng = np.random.Generator(np.random.PCG64(6))
    gen = torch.Generator(device="cuda")
    gen.manual_seed(6)
    sites, templates = [], {}
    for sname, h_in, h_out in wl.LLAMA8B_SITES:
        W = (torch.randn((h_out, h_in), generator=gen, device="cuda", dtype=torch.float32) * wl.STD_W).to(torch.bfloat16)
        pool = B.Pool(h_in, h_out, n_blocks, rank, max_tokens=max_tokens)
        templates[sname] = [(wl.normal_bf16(rng, (rank, h_in), wl.STD_W), wl.normal_bf16(rng, (h_out, rank), wl.STD_W))
                            for _ in range(4)]        # adapter key -> one of four value sets (timing only)
        sites.append((sname, h_in, h_out, W, pool))
    widths = (4096, 14336)
    xs = [(torch.randn((max_tokens, w_), generator=gen, device="cuda", dtype=torch.float32)).to(torch.bfloat16) for w_ in widths]
    ybuf = {h: torch.empty((max_tokens, h), dtype=torch.bfloat16, device="cuda") for h in (1024, 4096, 14336)}
    sset = B.edgelora_siteset_create([s[4].handle for s in sites], [s[3] for s in sites],
                                     [widths.index(s[1]) for s in sites], 2, max_tokens)
    cache = B.edgelora_cache_create(n_blocks)
    # Section 4.2: the cache starts full of randomly chosen adapters
    start_keys = rng.choice(n_adapters, size=n_blocks, replace=False)
    for key, block in zip(start_keys, B.edgelora_cache_prefill(cache, start_keys)):
        for sname, _, _, _, pool in sites:
            A_, B_ = templates[sname][int(key) % 4]
            pool.load(int(block), A_, B_, wl.SCALE)
    for s in sites:
        B.edgelora_pool_wait_loads(s[4].handle)
    nb = B.edgelora_batcher_create(gamma, max_tokens, top_k, cache)
    for i in range(len(trace.arrival)):
        B.edgelora_batcher_submit(nb, i, trace.arrival[i], trace.in_len[i], trace.out_len[i], trace.candidates[i])
    stream = torch.cuda.Stream()
    ids_host = torch.zeros(max_tokens, dtype=torch.int32).pin_memory()
    ids_dev = torch.zeros(max_tokens, dtype=torch.int32, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    steps = swaps = tokens = 0
    gpu_ms = 0.0
    t_wall = time.perf_counter()
    t_start = time.time()
    while True:
        b = B.edgelora_batcher_next_batch(nb, max_tokens, gamma)
        if b is None:
            break
        for key, block in b["loads"]:                 # the adapters this step admits (side-stream copies)
            for sname, _, _, _, pool in sites:
                A_, B_ = templates[sname][key % 4]
                pool.load(block, A_, B_, wl.SCALE)
            swaps += 1
        T = len(b["token_block"])
        ids_host[:T] = torch.from_numpy(b["token_block"])
        with torch.cuda.stream(stream):
            ids_dev[:T].copy_(ids_host[:T], non_blocking=True)
            e0.record(stream)
            B.edgelora_siteset_run(sset, [x[:T] for x in xs], ids_dev[:T], [ybuf[s[2]][:T] for s in sites], stream)
            e1.record(stream)
        stream.synchronize()
        ms = e0.elapsed_time(e1)
        gpu_ms += ms
        B.edgelora_batcher_complete_step(nb, ms * 1e-3 * layers)
        steps += 1
        tokens += T
    wall = time.perf_counter() - t_wall
    ctx["windows"].append((t_start, time.time()))
    for s in sites:
        rc, bits = s[4].status()
        if rc != 0 or bits != 0:
            raise SystemExit(f"serving trace: device status rc={rc} bits={bits:#x}")
    fin = B.edgelora_batcher_finished(nb)
    n = len(fin["id"])
    span = float(fin["finish"].max() - fin["arrival"].min())
    first = fin["first_token"] - fin["arrival"]
    st = B.edgelora_cache_stats(cache)
    res = {"name": SERVING, "requests": n, "value": n / span, "unit": "requests/s (virtual clock)",
           "avg_latency_s": float(np.mean(fin["finish"] - fin["arrival"])),
           "avg_first_token_s": float(np.mean(first)), "slo_attainment_6s": float(np.mean(first <= 6.0)),
           "hit_rate": float(np.mean(fin["hit"])), "cache": st,
           "steps": steps, "tokens_per_step": tokens / max(steps, 1), "adapter_swaps": swaps,
           "gpu_ms_per_step_one_layer": gpu_ms / max(steps, 1), "generated_tokens_per_s": float(trace.out_len.sum()) / span,
           "swaps_per_virtual_s": swaps / span, "wall_s": wall,
           "config": {"workload": "next row N3: Gamma arrivals R=25/s cv=1, 200 adapters power law alpha=1, "
                                  "lengths U[8,256] / U[8,128], gamma=20 slots, top-3 candidates, 64 cache blocks; "
                                  "one decoder layer's seven sites measured per step, step time x 32 layers",
                      "note": "the paper's rates (0.2-1 request/s) are for edge devices; the rate here keeps a B200 busy"}}
    B.edgelora_batcher_destroy(nb)
    B.edgelora_cache_destroy(cache)
    B.edgelora_siteset_destroy(sset)
    for s in sites:
        s[4].close()
    torch.cuda.empty_cache()
    return res


def spawn_ranks(args):
    """`--gpus N` outside a torchrun environment: start the N ranks (one per GPU) ourselves."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default="all", choices=["all", FULL_SET, SERVING] + sorted(SITE_WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-graph", action="store_true", help="time plain stream launches instead of CUDA-graph replay")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--pdl", type=int, default=None, help="EDGELORA_OPT_PDL value (0, 1, 2); default: library default")
    ap.add_argument("--layers", type=int, default=wl.LLAMA8B_LAYERS,
                    help="decoder layers of the projection set (fewer only for profiler captures)")
    args = ap.parse_args()

    headline = FULL_SET if args.workload == "all" else args.workload
    if args.impl == "reference":
        args.steps = args.steps if args.steps is not None else 5
        args.warmup = args.warmup if args.warmup is not None else 1
        run_reference(args, headline)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_ranks(args)

    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    sampler = ClockSampler(vis.split(",")[local] if vis else torch.cuda.current_device())
    ctx = {"world": world, "rank": rank, "barrier": barrier, "sampler": sampler, "windows": [], "peaks": peaks()}
    if rank == 0:
        sampler.start()
        time.sleep(0.2)
    cpu = 0.0 if args.no_cpu_baseline else None

    per_config = []
    if args.workload == "all" and world == 1:
        for name in DEFAULT_ORDER[:-1]:
            ctx["windows"] = []
            r = bench_site(name, ctx, graph=not args.no_graph, **({"cpu_budget": 0.0} if cpu == 0.0 else {}))
            r["clocks"] = sampler.summary(ctx["windows"])
            per_config.append(r)
    serving = None
    if (args.workload == "all" and world == 1) or args.workload == SERVING:
        ctx["windows"] = []
        serving = bench_serving(ctx)
        serving["clocks"] = sampler.summary(ctx["windows"])
        if args.workload == SERVING:
            if rank == 0:
                sampler.stop()
                print(json.dumps(serving), flush=True)
            return
    ctx["windows"] = []
    if headline == FULL_SET:
        head = bench_full_set(ctx, args.steps, args.warmup, layers=args.layers,
                              **({"cpu_budget": 0.0} if cpu == 0.0 else {}))
    else:
        head = bench_site(headline, ctx, args.steps, args.warmup, args.pdl, not args.no_graph,
                          **({"cpu_budget": 0.0} if cpu == 0.0 else {"cpu_budget": 10.0}))
    if rank == 0:
        time.sleep(0.1)
        sampler.stop()
    head["clocks"] = sampler.summary(ctx["windows"])
    if world > 1:
        dist.destroy_process_group()
    if rank != 0:
        return

    line = {"metric": METRIC, "value": head["value"], "unit": "tokens/s", "n_gpus": world, "steps": head["steps"],
            "warmup": head["warmup"], "ms_per_step": head["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic"}
    for k in ("config", "launch_info", "clocks", "e2e", "gpu_launches", "roofline", "step_work", "step_roofline_frac",
              "step_roofline_frac_of_nominal", "iterations", "variants", "warm_l2", "single_call_latency",
              "kernel_ms_profiled", "per_site", "adapter_swaps", "cpu_baseline"):
        if k in head:
            line[k] = head[k]
    if per_config:
        per_config.append({k: v for k, v in head.items()})
        line["per_config"] = per_config
    if serving is not None:
        line["serving_trace"] = serving
    print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
