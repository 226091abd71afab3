"""The tensor-core gather shrink (stacked A blocks of several adapters against the gathered rows of
their tokens): the corners of its tiling, each against the CPU oracle element by element.
"""
import numpy as np
import pytest

from paper_2507_01438_b200 import binding as B
from paper_2507_01438_b200 import workloads as wl
from helpers import assert_parity, oracle_of
from gpu_helpers import run_gpu
from test_gpu_parity import check_plan, random_workload

pytestmark = pytest.mark.gpu

# decode batches take the tensor-core gather shrink only when asked to (a tuning option)
GATHER = {B.OPT_GATHER_MIN_T: 16}


@pytest.mark.parametrize("splits", [0, 3])
@pytest.mark.parametrize("T,n_adapters,max_rank,h_in", [
    (256, 1, 16, 512),     # one adapter, 256 tokens: one tile, four passes of 64 tokens
    (200, 3, 64, 1088),    # rank 64: two adapters per tile, ~67 tokens each, ragged K (17 K blocks)
    (100, 40, 16, 768),    # eight adapters per tile, five tiles
    (130, 9, 32, 2048),    # four per tile, K splits chosen on the device
    (65, 65, 8, 256),      # as many adapters as tokens (one token each), nine tiles
    (256, 100, 64, 896),   # 50 tiles of two adapters
])
def test_decode_sized_batches(T, n_adapters, max_rank, h_in, splits):
    rng = np.random.Generator(np.random.PCG64(T + n_adapters))
    ranks = [int(r) for r in rng.integers(1, max_rank + 1, size=n_adapters)]
    ranks[0] = max_rank
    w = random_workload(1000 + T + n_adapters, T, h_in, 264, ranks=ranks, max_rank=max_rank)
    if n_adapters == 1:
        w.ids[:] = 0
    elif n_adapters >= T:
        w.ids = rng.permutation(n_adapters)[:T].astype(np.int32)
    y, plan = run_gpu(w, 1, return_plan=True, options={**GATHER, B.OPT_GATHER_SPLITS: splits})
    assert_parity(y, oracle_of(w), f"T={T} adapters={n_adapters} rank<={max_rank}")
    check_plan(plan, w.ids, w.n_slots)


def test_empty_slot_inside_a_tile():
    # the second adapter of a tile has nothing loaded: its tokens are base-only, the status says so,
    # the tile's other adapters are unaffected
    import torch
    w = random_workload(4242, 120, 512, 256, ranks=[16, 0, 16, 8, 16], max_rank=16)
    rng = np.random.Generator(np.random.PCG64(7))
    ids = rng.integers(-1, 5, size=120).astype(np.int32)
    from gpu_helpers import from_dev_bf16, make_pool, to_dev_bf16
    pool = make_pool(w)
    try:
        B.edgelora_pool_set_option(pool.handle, B.OPT_GATHER_MIN_T, 16)
        y = from_dev_bf16(pool.linear(to_dev_bf16(w.W), to_dev_bf16(w.x), torch.from_numpy(ids).cuda()))
        rc, bits = pool.status()
        assert rc == B.ERR_SLOT_EMPTY and bits == B.STATUS_SLOT_EMPTY
        w.ids = np.where(ids == 1, -1, ids).astype(np.int32)
        assert_parity(y, oracle_of(w), "empty slot in a gather tile")
    finally:
        pool.close()


def test_prefill_with_many_short_tokens_on_one_adapter():
    # runs of 20 tokens alternating between two adapters: every token is "short", so each adapter
    # has hundreds of tokens in the gather tiles (several passes), beside two long runs
    pieces = []
    for i in range(30):
        pieces.append(np.full(20, i % 2))
    pieces += [np.full(150, 2), np.full(17, -1), np.full(200, 0)]
    ids = np.concatenate(pieces).astype(np.int32)
    w = random_workload(99, len(ids), 384, 520, ranks=[32, 8, 20], max_rank=32)
    w.ids = ids
    y, plan = run_gpu(w, return_plan=True)
    assert_parity(y, oracle_of(w), "many short tokens")
    check_plan(plan, w.ids, w.n_slots)


def test_repeated_calls_reuse_the_arrival_counters():
    # the per-tile arrival counters must be back at zero after every call
    w = random_workload(555, 180, 1024, 256, ranks=[64, 32, 64, 8, 64, 16, 64], max_rank=64)
    from gpu_helpers import make_pool
    pool = make_pool(w)
    try:
        first = run_gpu(w, pool=pool, options=GATHER)
        assert_parity(first, oracle_of(w), "first call")
        for _ in range(3):
            assert np.array_equal(run_gpu(w, pool=pool, options=GATHER), first)
    finally:
        pool.close()
