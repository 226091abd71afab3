"""Timing of the full Llama-3.1-8B projection set: 7 sites x 32 layers = 224 independent LoRA
linear sites over one mixed batch (64 decode tokens + 2 prefill runs of 1024 tokens, 128 adapters
with ranks from {8, 16, 32}), one routing plan shared by all sites.

Called by ``bench.py --workload full_projection_set``.  Only the ids, the ranks and x come from the
seeded numpy recipe (``workloads.full_set_batch``); the 14 GB of weights and the adapter values are
drawn on the device / reused across slots, since their values do not change the timing (parity of
this configuration is checked on sampled sites by the GPU tests with the numpy-generated values).
"""
import time

import numpy as np

from . import binding as B
from . import workloads as wl


def build(torch, layers: int):
    batch = wl.full_set_batch()
    used = sorted(set(int(a) for a in batch.ids if a >= 0))
    rng = np.random.Generator(np.random.PCG64(4))
    host = {}      # one host adapter per (rank, h_in, h_out), reused for every slot of that shape
    gen = torch.Generator(device="cuda")
    gen.manual_seed(4)
    sites = []
    for layer in range(layers):
        for name, h_in, h_out in wl.LLAMA8B_SITES:
            W = (torch.randn((h_out, h_in), generator=gen, device="cuda", dtype=torch.float32) * wl.STD_W).to(torch.bfloat16)
            pool = B.Pool(h_in, h_out, batch.n_slots, batch.max_rank, max_tokens=len(batch.ids))
            for a in used:
                r = int(batch.ranks[a])
                key = (r, h_in, h_out)
                if key not in host:
                    host[key] = (wl.normal_bf16(rng, (r, h_in), wl.STD_W), wl.normal_bf16(rng, (h_out, r), wl.STD_W))
                pool.load(a, host[key][0], host[key][1], wl.SCALE)
            B.edgelora_pool_wait_loads(pool.handle)
            sites.append((name, h_in, h_out, W, pool))
    return batch, used, sites


def flops_per_step(batch, sites):
    T = len(batch.ids)
    rank_sum = sum(int(batch.ranks[a]) for a in batch.ids if a >= 0)
    f = 0
    for _, h_in, h_out, _, _ in sites:
        f += 2 * T * h_in * h_out + 2 * rank_sum * (h_in + h_out)
    return f


def run(args, peaks, sampler_cls, max_over_ranks):
    import torch
    layers = 32
    batch, used, sites = build(torch, layers)
    T = len(batch.ids)
    to_bf16 = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)
    xs = {4096: to_bf16(batch.x4096), 14336: to_bf16(batch.x14336)}
    ids = torch.from_numpy(batch.ids).cuda()
    ys = {h: torch.empty((T, h), dtype=torch.bfloat16, device="cuda") for h in (1024, 4096, 14336)}
    plan = B.edgelora_plan_create(T, batch.n_slots)
    stream = torch.cuda.Stream()

    def step():
        B.edgelora_plan_build(plan, ids, stream)
        for _, h_in, h_out, W, pool in sites:
            B.edgelora_lora_linear_planned(pool.handle, plan, W, xs[h_in], ys[h_out], stream)

    steps = args.steps if args.steps is not None else 20
    warmup = max(args.warmup if args.warmup is not None else 3, 3)
    with torch.cuda.stream(stream):
        for _ in range(warmup):
            step()
    stream.synchronize()
    for s in sites:
        rc, bits = s[4].status()
        if rc != 0 or bits != 0:
            raise SystemExit(f"device status after warm-up: rc={rc} bits={bits:#x}")

    sampler = sampler_cls(torch.cuda.current_device())
    sampler.start()
    time.sleep(0.2)
    windows = []
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t_start = time.time()
    e0.record(stream)
    with torch.cuda.stream(stream):
        for _ in range(steps):
            step()
    e1.record(stream)
    torch.cuda.synchronize()
    windows.append((t_start, time.time()))
    ms = max_over_ranks(e0.elapsed_time(e1), 1, "cuda")
    value = T * steps / (ms * 1e-3)

    # end to end: x and ids from pinned host memory every step, the last site's y read back
    hx = {h: torch.from_numpy(np.ascontiguousarray(b).view(np.int16)).pin_memory() for h, b in
          ((4096, batch.x4096), (14336, batch.x14336))}
    hids = torch.from_numpy(batch.ids).pin_memory()
    hy = torch.empty((T, 4096), dtype=torch.int16).pin_memory()
    k_e2e = min(steps, 10)
    torch.cuda.synchronize()
    t_start = time.time()
    t0 = time.perf_counter()
    for _ in range(k_e2e):
        with torch.cuda.stream(stream):
            for h in (4096, 14336):
                xs[h].view(torch.int16).copy_(hx[h], non_blocking=True)
            ids.copy_(hids, non_blocking=True)
            step()
            hy.copy_(ys[4096].view(torch.int16), non_blocking=True)
        stream.synchronize()
    e2e_s = time.perf_counter() - t0
    windows.append((t_start, time.time()))
    e2e = {"value": T * k_e2e / e2e_s, "unit": "tokens/s", "steps": k_e2e,
           "h2d_bytes_per_step": int(batch.x4096.nbytes + batch.x14336.nbytes + batch.ids.nbytes),
           "d2h_bytes_per_step": int(T * 4096 * 2),
           "api": "edgelora_plan_build + 224 x edgelora_lora_linear_planned; pinned H2D of x and ids, D2H of the last site's y"}

    # dominant kernel: the base product of every site, one CUDA-event pair per launch
    for s in sites:
        B.edgelora_pool_set_option(s[4].handle, B.OPT_PROFILE, 1)
        B.edgelora_pool_kernel_times(s[4].handle, reset=True)
    t_start = time.time()
    with torch.cuda.stream(stream):
        step()
    torch.cuda.synchronize()
    windows.append((t_start, time.time()))
    kt = {}
    for s in sites:
        for name, v in B.edgelora_pool_kernel_times(s[4].handle, reset=True).items():
            acc = kt.setdefault(name, {"ms": 0.0, "launches": 0})
            acc["ms"] += v["ms"]
            acc["launches"] += v["launches"]
        B.edgelora_pool_set_option(s[4].handle, B.OPT_PROFILE, 0)
    info = B.edgelora_pool_last_launch(sites[0][4].handle)
    time.sleep(0.1)
    sampler.stop()

    flops = flops_per_step(batch, sites)
    gemm_ms = kt["base_gemm"]["ms"]
    peak = peaks["bf16_tflops_sustained"] if "bf16_tflops_sustained" in peaks else peaks["bf16_tflops"]
    achieved = flops / (gemm_ms * 1e-3) / 1e12
    launches_per_step = 1 + len(sites) * info["launches"]
    line = {
        "metric": "batched multi-adapter LoRA linear tokens/s", "value": value, "unit": "tokens/s", "n_gpus": 1,
        "steps": steps, "warmup": warmup, "ms_per_step": ms / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "configs[4]: full Llama-3.1-8B projection set x32 layers (224 sites), 128 adapters "
                               "ranks {8,16,32}, 64 decode tokens + 2 x 1024-token prefill runs, one plan for all sites",
                   "T": T, "sites": len(sites), "distinct_adapters": len(used), "regime": info["regime"],
                   "launch": "plain stream launches",
                   "l2": "inputs larger than L2: 14 GB of weights and 2.7 GB of touched adapters per step",
                   "parallelism": "replicas x1"},
        "clocks": sampler.summary(windows), "e2e": e2e,
        "gpu_launches": int(launches_per_step * steps), "kernels_per_step": launches_per_step,
        "roofline": {"bound": "tensor", "kernel": "lora_gemm_kernel (prefill mode), all 224 sites of a step",
                     "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak, "traffic": None,
                     "algorithmic_flops": flops, "kernel_us": 1e3 * gemm_ms / max(kt["base_gemm"]["launches"], 1),
                     "peak_source": peaks["_source"] + ", sustained (the kernel runs inside a 40 ms step)",
                     "frac_of_nominal": achieved / 2250.0, "nominal": "2.25 PFLOP/s dense bf16"},
        "step_roofline_frac": (flops / (ms * 1e-3 / steps) / 1e12) / peak,
        "kernel_ms_profiled": {k: v for k, v in kt.items() if v["launches"]},
    }
    B.edgelora_plan_destroy(plan)
    for s in sites:
        s[4].close()
    return line
