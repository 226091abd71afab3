"""Host-side state of a pool under awkward use, checked against the CPU oracle through the C ABI:
many distinct (x, T) pairs through one pool (descriptor cache), the time-out status path, the
documented rule for CUDA graphs and slot loads, calls from several streams after a load, and the
status word of a plan that is built on its own.
"""
import numpy as np
import pytest

from paper_2507_01438_b200 import binding as B
from paper_2507_01438_b200 import workloads as wl
from helpers import assert_parity, oracle_of
from gpu_helpers import from_dev_bf16, make_pool, to_dev_bf16
from test_gpu_parity import random_workload

pytestmark = pytest.mark.gpu


def variant(base, seed, T, n_ids):
    rng = np.random.Generator(np.random.PCG64(seed))
    x = wl.normal_bf16(rng, (T, base.h_in), 1.0)
    ids = rng.integers(-1, n_ids, size=T).astype(np.int32)
    return wl.Workload(f"{base.name}_v{seed}", base.h_in, base.h_out, base.n_slots, base.max_rank,
                       base.W, x, ids, base.adapters)


def test_many_distinct_inputs_through_one_pool():
    # 48 calls, alternating decode-sized and prefill-sized batches, every call with a fresh x tensor
    # and its own T: far more distinct tensor-map keys than the pool's descriptor cache holds.  Every
    # result must still belong to its own inputs.
    import torch
    base = random_workload(77, 8, 320, 264, ranks=[8, 16, 4, 12, 16], max_rank=16)
    pool = make_pool(base, 512)
    try:
        W = to_dev_bf16(base.W)
        keep = []                                        # keeps every x alive: no address is reused
        for i in range(48):
            T = (3 + 5 * i) if i % 2 == 0 else (260 + 3 * i)
            w = variant(base, 1000 + i, T, 5)
            x = to_dev_bf16(w.x)
            keep.append(x)
            y = torch.full((T, w.h_out), float("nan"), dtype=torch.bfloat16, device="cuda")
            B.edgelora_lora_linear(pool.handle, W, x, torch.from_numpy(w.ids).cuda(), y)
            assert pool.status() == (0, 0)
            assert_parity(from_dev_bf16(y), oracle_of(w), f"call {i} T={T}")
    finally:
        pool.close()


def test_bounded_wait_runs_out_and_the_pool_stays_usable():
    import torch
    w = random_workload(78, 40, 256, 256, ranks=[16, 8], max_rank=16)
    pool = make_pool(w, 64)
    try:
        # refused at the default limit (the kernel would spin for seconds)
        assert B.edgelora_pool_selftest_wait(pool.handle) == B.ERR_INVALID_ARG
        B.edgelora_pool_set_option(pool.handle, B.OPT_WAIT_CYCLES, 100)      # about 1e5 cycles
        assert B.edgelora_pool_selftest_wait(pool.handle) == B.OK
        rc, bits = pool.status()
        assert rc == B.ERR_TIMEOUT and bits & B.STATUS_TIMEOUT
        assert pool.status() == (0, 0)                   # reading the status cleared it
        # the same pool, same lowered limit (still far above any real wait of this size): correct
        y = torch.empty((w.T, w.h_out), dtype=torch.bfloat16, device="cuda")
        B.edgelora_lora_linear(pool.handle, to_dev_bf16(w.W), to_dev_bf16(w.x), torch.from_numpy(w.ids).cuda(), y)
        assert pool.status() == (0, 0)
        assert_parity(from_dev_bf16(y), oracle_of(w), "after the time-out")
        B.edgelora_pool_set_option(pool.handle, B.OPT_WAIT_CYCLES, 0)
        assert B.edgelora_pool_selftest_wait(pool.handle) == B.ERR_INVALID_ARG
    finally:
        pool.close()


@pytest.mark.parametrize("T", [24, 300])
def test_graph_replay_after_a_slot_reload_follows_the_documented_rule(T):
    # A captured call does not wait for slot loads by itself.  The rule: edgelora_pool_wait_loads
    # before capture and before a replay that follows a load.  Then the replay sees the new adapter.
    import torch
    w = random_workload(79 + T, T, 256, 384, ranks=[16, 8, 16], max_rank=16)
    pool = make_pool(w, 512)
    try:
        W, x = to_dev_bf16(w.W), to_dev_bf16(w.x)
        ids = torch.from_numpy(w.ids).cuda()
        y = torch.zeros((T, w.h_out), dtype=torch.bfloat16, device="cuda")
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            B.edgelora_lora_linear(pool.handle, W, x, ids, y, stream)     # warm-up outside capture
        stream.synchronize()
        B.edgelora_pool_wait_loads(pool.handle)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            B.edgelora_lora_linear(pool.handle, W, x, ids, y, stream)
        with torch.cuda.stream(stream):
            graph.replay()
        stream.synchronize()
        assert_parity(from_dev_bf16(y), oracle_of(w), "replay before the reload")
        # new contents for slot 0 (other values, other rank), then the rule, then replay
        rng = np.random.Generator(np.random.PCG64(5))
        new = wl.Adapter(wl.normal_bf16(rng, (4, w.h_in), 0.05), wl.normal_bf16(rng, (w.h_out, 4), 0.05), 1.5)
        pool.load(0, new.A, new.B, new.scale)
        B.edgelora_pool_wait_loads(pool.handle)
        with torch.cuda.stream(stream):
            graph.replay()
        stream.synchronize()
        assert pool.status() == (0, 0)
        w2 = wl.Workload("reloaded", w.h_in, w.h_out, w.n_slots, w.max_rank, w.W, w.x, w.ids,
                         {**w.adapters, 0: new})
        assert_parity(from_dev_bf16(y), oracle_of(w2), "replay after the reload")
    finally:
        pool.close()


def test_every_stream_waits_for_a_load():
    # a load, then calls on two different streams (one after the other: calls of one pool share its
    # workspaces and must not overlap): both must see the loaded adapter
    import torch
    w = random_workload(81, 48, 512, 256, ranks=[16, 16], max_rank=16, id_mode=0)
    pool = B.Pool(w.h_in, w.h_out, w.n_slots, w.max_rank, max_tokens=64)
    try:
        W, x = to_dev_bf16(w.W), to_dev_bf16(w.x)
        ids = torch.from_numpy(w.ids).cuda()
        s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
        y1 = torch.zeros((w.T, w.h_out), dtype=torch.bfloat16, device="cuda")
        y2 = torch.zeros_like(y1)
        torch.cuda.synchronize()
        for a, ad in w.adapters.items():
            pool.load(a, ad.A, ad.B, ad.scale)           # no wait_loads: the calls must order themselves
        B.edgelora_lora_linear(pool.handle, W, x, ids, y1, s1)
        s1.synchronize()
        B.edgelora_lora_linear(pool.handle, W, x, ids, y2, s2)
        torch.cuda.synchronize()
        assert pool.status() == (0, 0)
        ref = oracle_of(w)
        assert_parity(from_dev_bf16(y1), ref, "first stream")
        assert_parity(from_dev_bf16(y2), ref, "second stream")
    finally:
        pool.close()


def test_status_of_a_plan_built_on_its_own():
    import torch
    ids = np.array([0, 1, 7, -1, 2, -5, 1], dtype=np.int32)      # 7 and -5 are outside [-1, 3)
    plan = B.edgelora_plan_create(16, 3)
    try:
        B.edgelora_plan_build(plan, torch.from_numpy(ids).cuda())
        rc, bits = B.edgelora_plan_sync_status(plan)
        assert rc == B.ERR_BAD_ADAPTER_ID and bits == B.STATUS_BAD_ADAPTER_ID
        assert B.edgelora_plan_sync_status(plan) == (0, 0)
        got = B.edgelora_plan_export(plan, len(ids))
        assert got["ids_valid"].tolist() == [0, 1, -1, -1, 2, -1, 1]
    finally:
        B.edgelora_plan_destroy(plan)


def test_load_from_page_locked_memory():
    import torch
    w = random_workload(83, 50, 256, 384, ranks=[16, 16, 16], max_rank=16)
    pool = B.Pool(w.h_in, w.h_out, w.n_slots, w.max_rank, max_tokens=64)
    try:
        keep = []
        for a, ad in w.adapters.items():
            A = torch.from_numpy(ad.A.view(np.int16).copy()).pin_memory()
            Bm = torch.from_numpy(ad.B.view(np.int16).copy()).pin_memory()
            keep += [A, Bm]
            assert B.edgelora_pool_load_slot_pinned(pool.handle, a, 16, ad.scale, A, Bm) == B.OK
        y = pool.linear(to_dev_bf16(w.W), to_dev_bf16(w.x), torch.from_numpy(w.ids).cuda())
        assert pool.status() == (0, 0)
        assert_parity(from_dev_bf16(y), oracle_of(w), "adapters loaded from page-locked memory")
        pageable = torch.from_numpy(w.adapters[0].A.view(np.int16).copy())
        assert B.edgelora_pool_load_slot_pinned(pool.handle, 0, 16, 1.0, pageable, keep[1]) == B.ERR_INVALID_ARG
        assert B.edgelora_pool_load_slot_pinned(pool.handle, 0, 8, 1.0, keep[0], keep[1]) == B.ERR_INVALID_ARG
    finally:
        pool.close()
