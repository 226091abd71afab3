"""The task's full-size workloads (gate/up prefill, many-tenant down_proj, the 224-site projection set)
run in the launch configuration the benchmark uses.

gate/up prefill and the many-tenant down_proj are compared with the oracle on EVERY element (the
oracle needs seconds to a minute for them).  The projection set is 224 sites: there every row of
the first 128-token tile (the 64 decode tokens and the first tokens of the first long run) plus the
boundary rows of the long runs are compared element by element on the sampled sites.  The
projection p[t] = sum_j v[j] y[t][j] over all tokens stays as an extra check, not the carrier.
"""
import numpy as np
import pytest

import oracle
from paper_2507_01438_b200 import binding as B
from paper_2507_01438_b200 import workloads as wl
from helpers import adapter_set, assert_parity, oracle_of
from gpu_helpers import from_dev_bf16, make_pool, run_gpu, to_dev_bf16

pytestmark = pytest.mark.gpu


def boundary_rows(ids, extra, seed):
    """First and last token of every run (capped), plus `extra` random tokens."""
    start, _ = oracle.segments(ids)
    rows = set()
    runs = list(zip(start[:-1], start[1:]))
    if len(runs) > 24:                                  # many short runs: sample the runs too
        rng = np.random.Generator(np.random.PCG64(seed))
        runs = [runs[i] for i in rng.choice(len(runs), 24, replace=False)]
    for a, b in runs:
        rows.update((int(a), int(b - 1)))
    rng = np.random.Generator(np.random.PCG64(seed + 1))
    rows.update(int(t) for t in rng.choice(len(ids), size=min(extra, len(ids)), replace=False))
    return np.array(sorted(rows))


def projection_check(w, y, seed):
    """Every token: <v, y[t]> against the oracle, v a seeded +-1 vector.

    Allowed error: the sum of h_out independent bf16 roundings of size <= 2^-9 |y| grows like
    sqrt(h_out); 1e-2 * sqrt(h_out) * rms(y) is > 5x that and far below the change a dropped or
    misrouted adapter makes (its term is >= 10 % of rms(y) on every output)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    v = rng.choice(np.array([-1.0, 1.0]), size=w.h_out)
    p_ref = oracle.lora_projection(w.W, w.x, w.ids, adapter_set(w.n_slots, w.adapters), v)
    p_gpu = y.astype(np.float64) @ v
    rms_y = float(np.sqrt(np.mean(y.astype(np.float64) ** 2)))
    tol = 1e-2 * np.sqrt(w.h_out) * rms_y
    bad = np.abs(p_gpu - p_ref) > tol
    assert not bad.any(), f"{w.name}: projection off for tokens {np.where(bad)[0][:10]}, " \
                          f"worst {np.abs(p_gpu - p_ref).max() / tol:.2f}x tol"


def test_gate_up_prefill_full_size():
    w = wl.gate_up_prefill()
    assert (w.T, w.h_in, w.h_out) == (4096, 4096, 14336)
    y = run_gpu(w)
    assert_parity(y, oracle_of(w), "gate_up_prefill, all 4096 x 14336 elements")
    projection_check(w, y, 3)


def test_down_proj_many_tenant_full_size():
    w = wl.down_proj_many_tenant(only_used=False)       # all 1000 slots resident (2.36 GB)
    assert (w.T, w.h_in, w.h_out, len(w.adapters)) == (256, 14336, 4096, 1000)
    y = run_gpu(w)
    assert_parity(y, oracle_of(w), "down_proj many-tenant, all 256 x 4096 elements")
    projection_check(w, y, 4)


def full_set_single_sites():
    """One site (rotating through the seven projections) of every layer except 0, 15 and 31."""
    return [(l, l % 7) for l in range(32) if l not in (0, 15, 31)]


def full_set_rows(batch):
    # the whole first token tile (64 decode tokens + the head of the first run), run boundaries, a
    # few random rows
    rows = boundary_rows(batch.ids, 4, 5)
    return np.array(sorted(set(range(128)) | set(rows.tolist()[:10]) | {1087, 1088, 2111}))


@pytest.mark.parametrize("layer", [0, 15, 31])
def test_full_projection_set_whole_layers_through_the_site_set(layer):
    # the seven projections of a decoder layer as one set of sites: one plan, the sites back to
    # back with the next site's shrink riding on the current site's launches (what bench.py times)
    import torch
    batch = wl.full_set_batch()
    assert batch.ids.shape[0] == 2112
    rows = full_set_rows(batch)
    sites = [wl.full_set_site(batch, layer, s) for s in range(7)]
    pools = [make_pool(w, 2112) for w in sites]
    Ws = [to_dev_bf16(w.W) for w in sites]
    widths = (4096, 14336)
    sset = B.edgelora_siteset_create([p.handle for p in pools], Ws, [widths.index(w.h_in) for w in sites], 2, 2112)
    try:
        ys = [torch.full((2112, w.h_out), float("nan"), dtype=torch.bfloat16, device="cuda") for w in sites]
        B.edgelora_siteset_run(sset, [to_dev_bf16(batch.x4096), to_dev_bf16(batch.x14336)],
                               torch.from_numpy(batch.ids).cuda(), ys)
        torch.cuda.synchronize()
        for w, pool, y in zip(sites, pools, ys):
            assert pool.status() == (0, 0)
            yh = from_dev_bf16(y)
            assert_parity(yh[rows], oracle_of(w, rows), w.name)
            projection_check(w, yh, 5 + layer)
    finally:
        B.edgelora_siteset_destroy(sset)
        for p in pools:
            p.close()


def test_full_projection_set_sampled_sites():
    import torch
    batch = wl.full_set_batch()
    rows = full_set_rows(batch)
    ids_dev = torch.from_numpy(batch.ids).cuda()
    plan = B.edgelora_plan_create(2112, batch.n_slots)
    xs = {4096: to_dev_bf16(batch.x4096), 14336: to_dev_bf16(batch.x14336)}
    try:
        B.edgelora_plan_build(plan, ids_dev)             # one plan reused by every site
        for (layer, site) in full_set_single_sites():
            w = wl.full_set_site(batch, layer, site)
            pool = make_pool(w, 2112)
            try:
                y = torch.empty((w.T, w.h_out), dtype=torch.bfloat16, device="cuda")
                B.edgelora_lora_linear_planned(pool.handle, plan, to_dev_bf16(w.W), xs[w.h_in], y)
                assert pool.status() == (0, 0)
                yh = from_dev_bf16(y)
                assert_parity(yh[rows], oracle_of(w, rows), w.name)
            finally:
                pool.close()
    finally:
        B.edgelora_plan_destroy(plan)


def test_largest_batch_a_pool_takes():
    # T = 32768 (the limit of max_tokens), small widths so that the oracle covers every element:
    # 256 token tiles, long runs (segment tiles), short runs and scattered tokens (gather tiles), a
    # ragged last row tile, ragged ranks
    from test_gpu_parity import random_workload
    from gpu_helpers import run_gpu
    T = 32768
    base = random_workload(9900, 64, 136, 200, ranks=[16, 8, 3, 16, 12, 5, 16, 1], max_rank=16)
    rng = np.random.Generator(np.random.PCG64(9901))
    parts, left = [], T
    while left > 0:
        n = int(min(left, rng.choice([1, 2, 5, 17, 40, 130, 700, 3000])))
        parts.append(np.full(n, rng.integers(-1, 8)))
        left -= n
    ids = np.concatenate(parts).astype(np.int32)
    x = wl.normal_bf16(rng, (T, base.h_in), 1.0)
    w = wl.Workload("max_T", base.h_in, base.h_out, base.n_slots, base.max_rank, base.W, x, ids, base.adapters)
    y, plan = run_gpu(w, 0, return_plan=True)
    assert_parity(y, oracle_of(w), "T = 32768")
    from test_gpu_parity import check_plan
    check_plan(plan, ids, w.n_slots)


@pytest.mark.parametrize("T", [40, 300])
def test_largest_pool_and_smallest_widths(T):
    # 65534 slots (the limit), adapters in the first, a middle and the last slot; and the smallest widths
    # the library takes (8 -> 8), where every operand tile is mostly zero fill
    from gpu_helpers import run_gpu
    rng = np.random.Generator(np.random.PCG64(9950 + T))
    S, h_in, h_out = 65534, 64, 72
    slots = [0, 1, 32767, 65533]
    ad = {a: wl.Adapter(wl.normal_bf16(rng, (r, h_in), 0.05), wl.normal_bf16(rng, (h_out, r), 0.05), 1.0)
          for a, r in zip(slots, [16, 5, 12, 16])}
    ids = rng.choice(np.array([-1] + slots), size=T).astype(np.int32)
    w = wl.Workload("max_slots", h_in, h_out, S, 16, wl.normal_bf16(rng, (h_out, h_in), 0.05),
                    wl.normal_bf16(rng, (T, h_in), 1.0), ids, ad)
    assert_parity(run_gpu(w, 0), oracle_of(w), f"65534 slots, T = {T}")
    tiny = {0: wl.Adapter(wl.normal_bf16(rng, (8, 8), 0.3), wl.normal_bf16(rng, (8, 8), 0.3), 2.0),
            1: wl.Adapter(wl.normal_bf16(rng, (3, 8), 0.3), wl.normal_bf16(rng, (8, 3), 0.3), 0.5)}
    w8 = wl.Workload("min_widths", 8, 8, 2, 8, wl.normal_bf16(rng, (8, 8), 0.3), wl.normal_bf16(rng, (T, 8), 1.0),
                     rng.integers(-1, 2, size=T).astype(np.int32), tiny)
    assert_parity(run_gpu(w8, 0), oracle_of(w8), f"8 -> 8, T = {T}")
