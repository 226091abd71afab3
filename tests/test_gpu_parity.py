"""Parity of the CUDA path (through the C ABI) against the CPU oracle, element by element.

Tolerance (fixed by the task): |y_gpu - y_ref| <= 1e-2 |y_ref| + 1e-2 rms(y_ref); bf16 inputs, fp32
accumulation, bf16 output.  Routing arrays must match bit for bit.
"""
import numpy as np
import pytest

import oracle
from paper_2507_01438_b200 import binding as B
from paper_2507_01438_b200 import workloads as wl
from helpers import adapter_set, assert_parity, oracle_of
from gpu_helpers import from_dev_bf16, make_pool, run_gpu, to_dev_bf16

pytestmark = pytest.mark.gpu


def check_plan(plan, ids, n_slots):
    s0, s1 = oracle.segments(ids)
    g0, g1, g2 = oracle.groups(ids, n_slots)
    assert np.array_equal(plan["ids_valid"], ids)
    assert np.array_equal(plan["seg_start"], s0) and np.array_equal(plan["seg_adapter"], s1)
    assert np.array_equal(plan["perm"], g0)
    assert np.array_equal(plan["group_start"], g1) and np.array_equal(plan["group_adapter"], g2)


def random_workload(seed, T, h_in, h_out, ranks, max_rank, id_mode="uniform", run_len=1):
    rng = np.random.Generator(np.random.PCG64(seed))
    S = len(ranks)
    W = wl.normal_bf16(rng, (h_out, h_in), 0.05)
    ad = {}
    for a, r in enumerate(ranks):
        if r > 0:
            ad[a] = wl.Adapter(wl.normal_bf16(rng, (r, h_in), 0.05), wl.normal_bf16(rng, (h_out, r), 0.05),
                               float(rng.choice([0.5, 1.0, 2.0])))
    x = wl.normal_bf16(rng, (T, h_in), 1.0)
    loaded = sorted(ad)
    if id_mode == "uniform":
        ids = rng.choice(np.array([-1] + loaded), size=T)
    elif id_mode == "runs":
        n_runs = (T + run_len - 1) // run_len
        ids = np.repeat(rng.choice(np.array([-1] + loaded), size=n_runs), run_len)[:T]
    elif id_mode == "base":
        ids = np.full(T, -1)
    else:
        ids = np.full(T, loaded[int(id_mode)])
    return wl.Workload(f"rand{seed}", h_in, h_out, S, max_rank, W, x, ids.astype(np.int32), ad)


# ------------------------------------------------------------------ configs 1 and 2, full oracle
@pytest.mark.parametrize("regime", [0, 1, 2])
def test_tiny(regime):
    w = wl.tiny()
    y, plan = run_gpu(w, regime, return_plan=True)
    assert_parity(y, oracle_of(w), "tiny")
    check_plan(plan, w.ids, w.n_slots)


def test_q_proj_decode_full_size():
    w = wl.q_proj_decode()
    y, plan = run_gpu(w, 0, return_plan=True)
    assert_parity(y, oracle_of(w), "q_proj_decode")
    check_plan(plan, w.ids, w.n_slots)
    # the low-rank term is visible: dropping it would break parity
    base = oracle.lora_linear(w.W, w.x, np.full_like(w.ids, -1), oracle.AdapterSet(w.n_slots))
    from helpers import parity_violations
    assert parity_violations(base, oracle_of(w))[0] > 1000


# ------------------------------------------------------------------ ragged shapes, both regimes
@pytest.mark.parametrize("T,h_in,h_out,regime", [
    (1, 64, 64, 0), (5, 200, 136, 1), (5, 200, 136, 2), (33, 328, 264, 1), (130, 328, 264, 1),
    (130, 328, 264, 2), (256, 512, 384, 0), (257, 512, 384, 0), (300, 200, 136, 0), (700, 456, 520, 0),
])
def test_ragged_shapes(T, h_in, h_out, regime):
    w = random_workload(T * 7 + h_in, T, h_in, h_out, ranks=[8, 16, 4, 12, 0, 16], max_rank=16)
    y, plan = run_gpu(w, regime, return_plan=True)
    assert_parity(y, oracle_of(w), f"T={T} {h_in}->{h_out} regime={regime}")
    check_plan(plan, w.ids, w.n_slots)


@pytest.mark.parametrize("max_rank,ranks", [(8, [8, 3, 1]), (32, [8, 16, 32, 24]), (64, [64, 40, 8, 33])])
@pytest.mark.parametrize("T", [48, 400])
def test_ragged_ranks(max_rank, ranks, T):
    w = random_workload(max_rank + T, T, 256, 384, ranks=ranks, max_rank=max_rank, id_mode="runs",
                        run_len=7 if T < 100 else 50)
    assert_parity(run_gpu(w), oracle_of(w), f"ranks {ranks}")


@pytest.mark.parametrize("T,h_in,h_out,max_rank,ranks", [
    (24, 2048, 1024, 64, [64, 40, 8, 33, 64]),      # 8 K splits, expand by the reduction owners, rank 64
    (64, 2048, 1024, 16, [16, 8, 3, 16, 12, 16]),   # same path at its largest token count
    (64, 1024, 2048, 64, [64, 64, 17]),             # too many B loads per owner: LoRA K blocks, 64 tokens
    (200, 1024, 1024, 32, [32, 8, 24, 16]),         # LoRA K blocks with both halves of the 256-token tile
    (255, 1536, 1000, 64, [64, 8, 32, 16, 50]),     # 8 K splits of a 256-token tile, ragged last row tile and token quad
    (97, 2048, 520, 32, [32, 5, 16]),               # 128-token tile through the wide cluster reduction
])
def test_small_and_medium_decode_paths(T, h_in, h_out, max_rank, ranks):
    w = random_workload(T + h_out + max_rank, T, h_in, h_out, ranks=ranks, max_rank=max_rank)
    y, plan = run_gpu(w, 1, return_plan=True)
    assert_parity(y, oracle_of(w), f"decode T={T} {h_in}->{h_out} ranks {ranks}")
    check_plan(plan, w.ids, w.n_slots)


@pytest.mark.parametrize("mode", ["base", "0", "2"])
@pytest.mark.parametrize("T", [40, 384])
def test_degenerate_batches(mode, T):
    # all base-only, or every token on one adapter (the merged-weight case)
    w = random_workload(5 + T, T, 256, 256, ranks=[16, 8, 16], max_rank=16, id_mode=mode)
    y, plan = run_gpu(w, return_plan=True)
    assert_parity(y, oracle_of(w), f"mode {mode}")
    check_plan(plan, w.ids, w.n_slots)


def test_mixed_long_and_short_runs_prefill():
    # long runs (segment shrink), short runs and scattered tokens (gather shrink) in one batch,
    # with runs that are not aligned to the 128-token tiles
    rng = np.random.Generator(np.random.PCG64(77))
    w = random_workload(77, 1000, 384, 520, ranks=[16, 8, 16, 12, 16], max_rank=16)
    pieces = [np.full(37, 0), rng.integers(-1, 5, size=20), np.full(301, 3), np.full(31, 1),
              np.full(200, -1), np.full(33, 2), rng.integers(-1, 5, size=50), np.full(328, 4)]
    w.ids = np.concatenate(pieces).astype(np.int32)
    assert w.ids.shape[0] == 1000
    y, plan = run_gpu(w, return_plan=True)
    assert_parity(y, oracle_of(w), "mixed runs")
    check_plan(plan, w.ids, w.n_slots)


def test_empty_batch_is_a_noop():
    import torch
    w = wl.tiny()
    pool = make_pool(w)
    try:
        W = to_dev_bf16(w.W)
        x = torch.empty((0, w.h_in), dtype=torch.bfloat16, device="cuda")
        ids = torch.empty((0,), dtype=torch.int32, device="cuda")
        y = torch.empty((0, w.h_out), dtype=torch.bfloat16, device="cuda")
        B.edgelora_lora_linear(pool.handle, W, x, ids, y)
        assert pool.status() == (0, 0)
    finally:
        pool.close()


def test_run_to_run_determinism():
    w = random_workload(3, 200, 512, 512, ranks=[16, 16, 8], max_rank=16)
    a = run_gpu(w)
    b = run_gpu(w)
    assert np.array_equal(a, b)
    w2 = random_workload(4, 900, 512, 512, ranks=[16, 16, 8], max_rank=16, id_mode="runs", run_len=150)
    assert np.array_equal(run_gpu(w2), run_gpu(w2))


# ------------------------------------------------------------------ pool behaviour (Section 3.3 / 4.2)
def test_slot_reload_and_evict():
    import torch
    w = random_workload(9, 64, 256, 256, ranks=[16, 8, 16], max_rank=16)
    pool = make_pool(w)
    try:
        W, x = to_dev_bf16(w.W), to_dev_bf16(w.x)
        ids = torch.from_numpy(w.ids).cuda()
        y1 = from_dev_bf16(pool.linear(W, x, ids))
        assert_parity(y1, oracle_of(w), "before reload")
        # a different adapter goes into slot 1; the other slots are untouched
        rng = np.random.Generator(np.random.PCG64(123))
        new = wl.Adapter(wl.normal_bf16(rng, (12, 256), 0.05), wl.normal_bf16(rng, (256, 12), 0.05), 1.5)
        pool.load(1, new.A, new.B, new.scale)          # async; the next call waits for it
        y2 = from_dev_bf16(pool.linear(W, x, ids))
        w.adapters[1] = new
        ref2 = oracle_of(w)
        assert_parity(y2, ref2, "after reload")
        other = w.ids != 1
        assert np.array_equal(y1[other], y2[other])
        assert not np.array_equal(y1[~other], y2[~other])
        # evicted slot: its tokens fall back to base-only and the status word says so
        B.edgelora_pool_evict_slot(pool.handle, 1)
        y3 = from_dev_bf16(pool.linear(W, x, ids))
        rc, bits = pool.status()
        assert rc == B.ERR_SLOT_EMPTY and bits == B.STATUS_SLOT_EMPTY
        ids_fallback = np.where(w.ids == 1, -1, w.ids).astype(np.int32)
        ref3 = oracle.lora_linear(w.W, w.x, ids_fallback, adapter_set(w.n_slots, w.adapters))
        assert_parity(y3, ref3, "after evict")
        assert pool.status() == (0, 0)                 # reading the status clears it
    finally:
        pool.close()


def test_out_of_range_ids_fall_back_to_base_and_raise_status():
    import torch
    w = random_workload(10, 40, 256, 256, ranks=[16, 16], max_rank=16)
    bad = w.ids.copy()
    bad[3], bad[17], bad[30] = 2, -5, 1000
    pool = make_pool(w)
    try:
        y = from_dev_bf16(pool.linear(to_dev_bf16(w.W), to_dev_bf16(w.x), torch.from_numpy(bad).cuda()))
        rc, bits = pool.status()
        assert rc == B.ERR_BAD_ADAPTER_ID and bits & B.STATUS_BAD_ADAPTER_ID
        fixed = bad.copy()
        fixed[[3, 17, 30]] = -1
        ref = oracle.lora_linear(w.W, w.x, fixed, adapter_set(w.n_slots, w.adapters))
        assert_parity(y, ref, "bad ids")
    finally:
        pool.close()


def test_argument_errors():
    w = wl.tiny()
    pool = make_pool(w, max_tokens=32)
    try:
        ad = w.adapters[0]
        with pytest.raises(B.EdgeLoraError) as e:
            B.edgelora_pool_load_slot(pool.handle, 4, 8, 1.0, ad.A, ad.B)
        assert e.value.code == B.ERR_BAD_SLOT
        big = np.zeros((9, 256), dtype=np.uint16)
        with pytest.raises(B.EdgeLoraError) as e:
            B.edgelora_pool_load_slot(pool.handle, 0, 9, 1.0, big, np.zeros((256, 9), dtype=np.uint16))
        assert e.value.code == B.ERR_RANK_TOO_LARGE
        w33 = random_workload(1, 33, 256, 256, ranks=[8] * 4, max_rank=8)
        with pytest.raises(B.EdgeLoraError) as e:
            run_gpu(w33, pool=pool)
        assert e.value.code == B.ERR_TOO_MANY_TOKENS
    finally:
        pool.close()


def test_caller_owned_arena():
    import torch
    w = wl.tiny()
    need = B.edgelora_pool_bytes_required(w.h_in, w.h_out, w.n_slots, w.max_rank)
    small = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.EdgeLoraError) as e:
        B.Pool(w.h_in, w.h_out, w.n_slots, w.max_rank, arena=small)
    assert e.value.code == B.ERR_ARENA_TOO_SMALL
    arena = torch.empty(need, dtype=torch.uint8, device="cuda")
    pool = B.Pool(w.h_in, w.h_out, w.n_slots, w.max_rank, max_tokens=64, arena=arena)
    try:
        pool.load_all(w.adapters)
        assert_parity(run_gpu(w, pool=pool), oracle_of(w), "arena")
        # the blocks really live in the caller's memory: A of slot 0 is at the start of the arena
        got = arena[: 8 * 256 * 2].cpu().numpy().view(np.uint16).reshape(8, 256)
        assert np.array_equal(got, w.adapters[0].A)
    finally:
        pool.close()


def test_one_plan_serves_two_sites():
    import torch
    wa = random_workload(21, 300, 256, 384, ranks=[16, 8, 16], max_rank=16, id_mode="runs", run_len=40)
    wb = random_workload(22, 300, 384, 256, ranks=[16, 8, 16], max_rank=16)
    wb.ids = wa.ids
    plan = B.edgelora_plan_create(512, 3)
    pa, pb = make_pool(wa, 512), make_pool(wb, 512)
    try:
        ids = torch.from_numpy(wa.ids).cuda()
        B.edgelora_plan_build(plan, ids)
        for w, pool in ((wa, pa), (wb, pb)):
            y = torch.empty((w.T, w.h_out), dtype=torch.bfloat16, device="cuda")
            B.edgelora_lora_linear_planned(pool.handle, plan, to_dev_bf16(w.W), to_dev_bf16(w.x), y)
            assert pool.status() == (0, 0)
            assert_parity(from_dev_bf16(y), oracle_of(w), w.name)
        check_plan(B.edgelora_plan_export(plan, wa.T), wa.ids, 3)
    finally:
        pa.close()
        pb.close()
        B.edgelora_plan_destroy(plan)


def test_host_buffer_entry_point():
    w = random_workload(31, 96, 256, 384, ranks=[16, 8, 16], max_rank=16)
    pool = make_pool(w, 128)
    try:
        y = np.zeros((w.T, w.h_out), dtype=np.uint16)
        B.edgelora_lora_linear_host(pool.handle, to_dev_bf16(w.W), w.x, w.ids, y)
        assert pool.status() == (0, 0)
        assert_parity(wl.bf16_bits_to_f32(y), oracle_of(w), "host entry")
        assert np.array_equal(wl.bf16_bits_to_f32(y), run_gpu(w, pool=pool))
    finally:
        pool.close()


def test_pipelined_host_buffer_entry_point():
    # five calls in flight over two sets of device mirrors: every y must match its own inputs
    import torch
    base = random_workload(900, 40, 256, 384, ranks=[8, 16, 4, 12], max_rank=16)
    pool = make_pool(base, 128)
    try:
        W = to_dev_bf16(base.W)
        rng = np.random.Generator(np.random.PCG64(901))
        batches = []
        for i in range(5):
            T = 40 + 17 * i
            x = wl.normal_bf16(rng, (T, base.h_in), 1.0)
            ids = rng.integers(-1, 4, size=T).astype(np.int32)
            batches.append(wl.Workload(f"pipelined{i}", base.h_in, base.h_out, base.n_slots, base.max_rank,
                                       base.W, x, ids, base.adapters))
        pin = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a).view(dt)).pin_memory()
        xs = [pin(b.x, np.int16) for b in batches]
        ids = [pin(b.ids, np.int32) for b in batches]
        ys = [torch.zeros((b.T, b.h_out), dtype=torch.int16).pin_memory() for b in batches]
        for x, i, y in zip(xs, ids, ys):
            B.edgelora_lora_linear_host_async(pool.handle, W, x, i, y)
        B.edgelora_pool_host_sync(pool.handle)
        assert pool.status() == (0, 0)
        for b, y in zip(batches, ys):
            got = wl.bf16_bits_to_f32(y.numpy().view(np.uint16))
            assert_parity(got, oracle_of(b), f"pipelined T={b.T}")
            assert np.array_equal(got, run_gpu(b, pool=pool))
    finally:
        pool.close()


@pytest.mark.parametrize("pdl", [1, 2])
@pytest.mark.parametrize("T,h_in,h_out,max_rank", [(32, 4096, 4096, 16), (200, 1024, 1024, 32), (256, 2048, 512, 64), (400, 512, 640, 16)])
def test_cuda_graph_replay_in_the_benchmarks_launch_configuration(pdl, T, h_in, h_out, max_rank):
    # bench.py replays a CUDA graph of consecutive calls, with programmatic dependent launch inside
    # a call (1) or also across calls (2: the next call's shrink starts under this call's base
    # product).  Three different batches through one pool, captured twice over, replayed three times.
    import torch
    base = random_workload(500 + T, T, h_in, h_out, ranks=[max_rank, 8, max_rank, 4, 16, 8], max_rank=max_rank)
    rng = np.random.Generator(np.random.PCG64(600 + T))
    batches = []
    for i in range(3):
        x = wl.normal_bf16(rng, (T, h_in), 1.0)
        ids = rng.integers(-1, 6, size=T).astype(np.int32)
        batches.append(wl.Workload(f"graph{i}", h_in, h_out, base.n_slots, max_rank, base.W, x, ids, base.adapters))
    pool = make_pool(base)
    try:
        B.edgelora_pool_set_option(pool.handle, B.OPT_PDL, pdl)
        W = to_dev_bf16(base.W)
        xs = [to_dev_bf16(b.x) for b in batches]
        ids = [torch.from_numpy(b.ids).cuda() for b in batches]
        ys = [torch.zeros((T, h_out), dtype=torch.bfloat16, device="cuda") for _ in batches]
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            for i in range(3):
                B.edgelora_lora_linear(pool.handle, W, xs[i], ids[i], ys[i], stream)
        stream.synchronize()
        eager = [from_dev_bf16(y) for y in ys]
        for y in ys:
            y.zero_()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for i in range(6):
                B.edgelora_lora_linear(pool.handle, W, xs[i % 3], ids[i % 3], ys[i % 3], stream)
        with torch.cuda.stream(stream):
            for _ in range(3):
                graph.replay()
        stream.synchronize()
        assert pool.status() == (0, 0)
        for b, y, e in zip(batches, ys, eager):
            got = from_dev_bf16(y)
            assert_parity(got, oracle_of(b), f"graph replay pdl={pdl} T={T}")
            assert np.array_equal(got, e)
    finally:
        pool.close()


def test_profiling_option_reports_every_kernel():
    w = random_workload(41, 300, 256, 256, ranks=[16, 16], max_rank=16, id_mode="runs", run_len=64)
    pool = make_pool(w, 512)
    try:
        B.edgelora_pool_set_option(pool.handle, B.OPT_PROFILE, 1)
        run_gpu(w, pool=pool)
        t = B.edgelora_pool_kernel_times(pool.handle)
        assert t["plan"]["launches"] == 1 and t["shrink_small_decode"]["launches"] == 0
        assert t["shrink_tiles"]["launches"] == 1 and t["base_gemm"]["launches"] == 1
        assert t["base_gemm"]["ms"] > 0
        info = B.edgelora_pool_last_launch(pool.handle)
        assert info["launches"] == 3 and info["regime"] == "prefill"
    finally:
        pool.close()
