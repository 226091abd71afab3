"""A set of linear sites over one batch (edgelora_siteset_*): one routing plan, the sites run back
to back with the next site's shrink issued alongside the current site's kernels.  Every site's
result is compared with the CPU oracle of that site, element by element; the plan bit for bit.
"""
import numpy as np
import pytest

import oracle
from paper_2507_01438_b200 import binding as B
from paper_2507_01438_b200 import workloads as wl
from helpers import assert_parity, oracle_of
from gpu_helpers import from_dev_bf16, make_pool, to_dev_bf16

pytestmark = pytest.mark.gpu


def make_sites(seed, T, shapes, ranks, max_rank, ids):
    """Sites with their own W and adapters (one rank per adapter, the same at all its sites)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    xs = {}
    sites = []
    for (h_in, h_out) in shapes:
        if h_in not in xs:
            xs[h_in] = wl.normal_bf16(rng, (T, h_in), 1.0)
        W = wl.normal_bf16(rng, (h_out, h_in), 0.05)
        ad = {a: wl.Adapter(wl.normal_bf16(rng, (r, h_in), 0.05), wl.normal_bf16(rng, (h_out, r), 0.05),
                            float(rng.choice([0.5, 1.0, 2.0]))) for a, r in enumerate(ranks) if r > 0}
        sites.append(wl.Workload(f"site{len(sites)}_{h_in}x{h_out}", h_in, h_out, len(ranks), max_rank, W,
                                 xs[h_in], ids, ad))
    return xs, sites


def mixed_ids(seed, n_decode, runs, n_slots):
    rng = np.random.Generator(np.random.PCG64(seed))
    parts = [rng.integers(-1, n_slots, size=n_decode)]
    for a, n in runs:
        parts.append(np.full(n, a))
    return np.concatenate(parts).astype(np.int32)


def run_set(sites, xs, ids, max_tokens, host=False):
    import torch
    widths = sorted(xs)
    pools = [make_pool(w, max_tokens) for w in sites]
    Ws = [to_dev_bf16(w.W) for w in sites]
    s = B.edgelora_siteset_create([p.handle for p in pools], Ws, [widths.index(w.h_in) for w in sites],
                                  len(widths), max_tokens)
    try:
        T = len(ids)
        if host:
            pin = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a).view(dt)).pin_memory()
            ys = [torch.zeros((T, w.h_out), dtype=torch.int16).pin_memory() if i % 2 == 0 else None
                  for i, w in enumerate(sites)]
            B.edgelora_siteset_run_host(s, [pin(xs[h], np.int16) for h in widths], pin(ids, np.int32), ys)
            out = [None if y is None else wl.bf16_bits_to_f32(y.numpy().view(np.uint16)) for y in ys]
        else:
            ys = [torch.full((T, w.h_out), float("nan"), dtype=torch.bfloat16, device="cuda") for w in sites]
            B.edgelora_siteset_run(s, [to_dev_bf16(xs[h]) for h in widths], torch.from_numpy(ids).cuda(), ys)
            torch.cuda.synchronize()
            out = [from_dev_bf16(y) for y in ys]
        for p in pools:
            assert p.status() == (0, 0)
        plan = B.edgelora_plan_export(B.edgelora_siteset_plan(s), T)
        return out, plan
    finally:
        B.edgelora_siteset_destroy(s)
        for p in pools:
            p.close()


def check_plan(plan, ids, n_slots):
    s0, s1 = oracle.segments(ids)
    g0, g1, g2 = oracle.groups(ids, n_slots)
    assert np.array_equal(plan["seg_start"], s0) and np.array_equal(plan["seg_adapter"], s1)
    assert np.array_equal(plan["perm"], g0)
    assert np.array_equal(plan["group_start"], g1) and np.array_equal(plan["group_adapter"], g2)


@pytest.mark.parametrize("host", [False, True])
def test_prefill_sized_set_with_ragged_ranks(host):
    # 40 scattered tokens, then runs of 300 / 70 / 20 tokens (long runs go through the segment shrink
    # that rides on the previous site's launch, the short ones through the gather shrink beside it)
    ranks = [8, 16, 32, 4, 0, 32, 12]
    ids = mixed_ids(3, 40, [(2, 300), (5, 70), (0, 20), (-1, 37)], len(ranks))
    ids[ids == 4] = -1                                   # slot 4 is empty
    shapes = [(256, 320), (256, 72), (512, 256), (256, 1032), (512, 136)]
    xs, sites = make_sites(17, len(ids), shapes, ranks, 32, ids)
    out, plan = run_set(sites, xs, ids, 512, host)
    for w, y in zip(sites, out):
        if y is not None:
            assert_parity(y, oracle_of(w), w.name)
    check_plan(plan, ids, len(ranks))


def test_repeated_runs_and_decode_sized_batches():
    import torch
    ranks = [16, 8, 16]
    shapes = [(256, 256), (256, 384), (384, 256)]
    for T, runs in ((300, [(1, 200)]), (64, []), (300, [(0, 130), (2, 100)])):
        ids = mixed_ids(5 + T, T - sum(n for _, n in runs), runs, len(ranks))
        xs, sites = make_sites(23 + len(runs), len(ids), shapes, ranks, 16, ids)
        out, plan = run_set(sites, xs, ids, 512)
        for w, y in zip(sites, out):
            assert_parity(y, oracle_of(w), f"{w.name} T={T}")
        check_plan(plan, ids, len(ranks))


def test_one_set_run_three_times_gives_the_same_bits():
    import torch
    ranks = [16, 32, 8, 32]
    ids = mixed_ids(9, 30, [(1, 260), (3, 129)], len(ranks))
    shapes = [(256, 264), (256, 512), (256, 128)]
    xs, sites = make_sites(31, len(ids), shapes, ranks, 32, ids)
    pools = [make_pool(w, 512) for w in sites]
    Ws = [to_dev_bf16(w.W) for w in sites]
    s = B.edgelora_siteset_create([p.handle for p in pools], Ws, [0, 0, 0], 1, 512)
    try:
        x = to_dev_bf16(xs[256])
        idt = torch.from_numpy(ids).cuda()
        ys = [torch.zeros((len(ids), w.h_out), dtype=torch.bfloat16, device="cuda") for w in sites]
        first = None
        for _ in range(3):
            B.edgelora_siteset_run(s, [x], idt, ys)
            torch.cuda.synchronize()
            got = [from_dev_bf16(y) for y in ys]
            if first is None:
                first = got
                for w, y in zip(sites, got):
                    assert_parity(y, oracle_of(w), w.name)
            else:
                for a, b in zip(first, got):
                    assert np.array_equal(a, b)
            for y in ys:
                y.zero_()
        for p in pools:
            assert p.status() == (0, 0)
    finally:
        B.edgelora_siteset_destroy(s)
        for p in pools:
            p.close()


def test_host_buffer_call_twice_on_one_set():
    # the set's second stream, its events and its device mirrors are reused by the second call, which
    # has other inputs and another batch size: both calls must match the oracle
    import torch
    ranks = [16, 8, 16]
    shapes = [(256, 264), (512, 128), (256, 520)]
    pin = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a).view(dt)).pin_memory()
    ids1 = mixed_ids(31, 30, [(1, 280)], len(ranks))
    ids2 = mixed_ids(32, 12, [(0, 150), (2, 200)], len(ranks))
    xs1, sites1 = make_sites(41, len(ids1), shapes, ranks, 16, ids1)
    rng = np.random.Generator(np.random.PCG64(43))
    xs2 = {h: wl.normal_bf16(rng, (len(ids2), h), 1.0) for h in xs1}       # the same W and adapters, other inputs
    sites2 = [wl.Workload(w.name, w.h_in, w.h_out, w.n_slots, w.max_rank, w.W, xs2[w.h_in], ids2, w.adapters)
              for w in sites1]
    widths = sorted(xs1)
    pools = [make_pool(w, 512) for w in sites1]
    Ws = [to_dev_bf16(w.W) for w in sites1]
    s = B.edgelora_siteset_create([p.handle for p in pools], Ws, [widths.index(w.h_in) for w in sites1],
                                  len(widths), 512)
    try:
        for xs, ids, sites in ((xs1, ids1, sites1), (xs2, ids2, sites2)):
            ys = [torch.zeros((len(ids), w.h_out), dtype=torch.int16).pin_memory() for w in sites]
            B.edgelora_siteset_run_host(s, [pin(xs[h], np.int16) for h in widths], pin(ids, np.int32), ys)
            for p in pools:
                assert p.status() == (0, 0)
            for w, y in zip(sites, ys):
                assert_parity(wl.bf16_bits_to_f32(y.numpy().view(np.uint16)), oracle_of(w), w.name)
    finally:
        B.edgelora_siteset_destroy(s)
        for p in pools:
            p.close()
