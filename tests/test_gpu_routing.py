"""The routing plan built on the GPU equals the CPU routing oracle bit for bit."""
import numpy as np
import pytest

import oracle
from paper_2507_01438_b200 import binding as B
from paper_2507_01438_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def gpu_plan(ids, n_slots, max_tokens=0):
    import torch
    plan = B.edgelora_plan_create(max_tokens or max(len(ids), 1), n_slots)
    try:
        B.edgelora_plan_build(plan, torch.from_numpy(np.ascontiguousarray(ids, dtype=np.int32)).cuda())
        return B.edgelora_plan_export(plan, len(ids))
    finally:
        B.edgelora_plan_destroy(plan)


def check(ids, n_slots):
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    p = gpu_plan(ids, n_slots)
    s0, s1 = oracle.segments(ids)
    g0, g1, g2 = oracle.groups(ids, n_slots)
    assert np.array_equal(p["ids_valid"], ids)
    assert np.array_equal(p["seg_start"], s0) and np.array_equal(p["seg_adapter"], s1)
    assert np.array_equal(p["perm"], g0)
    assert np.array_equal(p["group_start"], g1) and np.array_equal(p["group_adapter"], g2)


def test_hand_example():
    check([2, 2, -1, 0, 2, 0, 0, -1], 4)


def test_the_five_configs_ids():
    check(wl.tiny().ids, 4)
    rng = np.random.Generator(np.random.PCG64(1))
    check(rng.permutation(32), 32)
    check(np.repeat(rng.permutation(8), 512), 8)
    ids = wl.bounded_zipf_ids(rng, 256, 1000, 1.1)
    ids[rng.choice(256, 26, replace=False)] = -1
    check(ids, 1000)
    check(wl.full_set_batch().ids, 128)


@pytest.mark.parametrize("T,S", [(1, 1), (2, 3), (31, 5), (32, 5), (33, 70), (1023, 9), (1024, 2000),
                                 (1025, 17), (5000, 300), (32768, 1000)])
def test_random_ids(T, S):
    rng = np.random.Generator(np.random.PCG64(T * 31 + S))
    check(rng.integers(-1, S, size=T), S)
    runs = np.repeat(rng.integers(-1, S, size=T), rng.integers(1, 9, size=T))[:T]
    check(runs, S)


def test_extremes():
    check(np.full(777, -1), 3)
    check(np.full(777, 2), 3)
    check(np.arange(4096) % 65534, 65534)         # largest slot count, ids up to 65533


def test_empty_plan():
    p = gpu_plan(np.zeros(0, dtype=np.int32), 4)
    assert p["perm"].size == 0 and p["group_start"].tolist() == [0] and p["seg_start"].tolist() == [0]


def test_too_many_tokens_is_rejected():
    with pytest.raises(B.EdgeLoraError) as e:
        B.edgelora_plan_create(32769, 4)
    assert e.value.code == B.ERR_TOO_MANY_TOKENS
    import torch
    plan = B.edgelora_plan_create(16, 4)
    try:
        with pytest.raises(B.EdgeLoraError) as e:
            B.edgelora_plan_build(plan, torch.zeros(17, dtype=torch.int32, device="cuda"))
        assert e.value.code == B.ERR_TOO_MANY_TOKENS
    finally:
        B.edgelora_plan_destroy(plan)
