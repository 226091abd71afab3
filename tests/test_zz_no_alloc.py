"""edgelora_plan_build_static: the routing plan for hosts that may not allocate device memory.

A serving process that gave all of its device memory to its own arena at start-up, or that runs
the plan from a context where cudaMalloc is forbidden, still needs the routing plan.  The entry
point under test keeps the kernel's working arrays in an array built into the library and writes
only into buffers the caller passes.  Here it must reproduce, bit for bit, what the allocating
entry points (edgelora_plan_build + edgelora_plan_export) produce, on two calls in a row that
share the built-in array, the second with fewer tokens and different ids so that anything left
over from the first call would show.

This file sorts last on purpose: a run that stops at the first failure has then already been
through every other test.
"""
import numpy as np
import pytest

import oracle
from paper_2507_01438_b200 import binding as B

pytestmark = pytest.mark.gpu

KEYS = ("ids_valid", "perm", "group_start", "group_adapter", "seg_start", "seg_adapter")


def build_both(ids_np, n_slots):
    import torch
    T = len(ids_np)
    ids = torch.from_numpy(ids_np).cuda()
    # allocating path
    plan = B.edgelora_plan_create(max(T, 1), n_slots)
    try:
        B.edgelora_plan_build(plan, ids)
        want = B.edgelora_plan_export(plan, T)
    finally:
        B.edgelora_plan_destroy(plan)
    # non-allocating path: every buffer is the caller's, filled with a sentinel first
    out = {k: torch.full((T + 1,), -7, dtype=torch.int32, device="cuda") for k in KEYS}
    info = torch.full((4,), -7, dtype=torch.int32, device="cuda")
    rc = B.edgelora_plan_build_static(ids, n_slots, out["ids_valid"], out["perm"], out["group_start"],
                                      out["group_adapter"], out["seg_start"], out["seg_adapter"], info)
    assert rc == B.OK, B.strerror(rc)
    torch.cuda.synchronize()
    info = info.cpu().numpy()
    G, NS = int(info[0]), int(info[1])
    got = {k: v.cpu().numpy() for k, v in out.items()}
    sizes = {"ids_valid": T, "perm": T, "group_start": G + 1, "group_adapter": G,
             "seg_start": NS + 1, "seg_adapter": NS}
    return want, {k: got[k][:n] for k, n in sizes.items()}, info


def mixed_ids(seed, T, n_slots):
    rng = np.random.Generator(np.random.PCG64(seed))
    ids = rng.integers(-1, n_slots, size=T).astype(np.int32)
    runs = rng.integers(0, T, size=4)
    for r in runs:                                   # a few long runs, as in a prefill batch
        ids[r:r + 200] = rng.integers(0, n_slots)
    return ids


def test_static_plan_matches_allocating_plan_twice_in_a_row():
    first = mixed_ids(11, 3000, 97)
    second = mixed_ids(12, 517, 97)                  # fewer tokens, other ids: stale state would show
    second[5] = 1000                                 # out of range: must be reported, token -> -1
    for ids, bad in ((first, False), (second, True)):
        want, got, info = build_both(ids, 97)
        for k in KEYS:
            assert np.array_equal(want[k], got[k]), k
        assert info[3] == 0
        assert bool(info[2] & B.STATUS_BAD_ADAPTER_ID) == bad
        check_against_oracle(got, ids, 97)


def check_against_oracle(got, ids, n_slots):
    """The plan as the paper's grouping defines it (Section 3.4), from the CPU oracle."""
    valid = np.where((ids < -1) | (ids >= n_slots), -1, ids).astype(np.int32)
    seg_start, seg_adapter = oracle.segments(valid)
    perm, group_start, group_adapter = oracle.groups(valid, n_slots)
    assert np.array_equal(got["ids_valid"], valid)
    assert np.array_equal(got["seg_start"], seg_start) and np.array_equal(got["seg_adapter"], seg_adapter)
    assert np.array_equal(got["perm"], perm)
    assert np.array_equal(got["group_start"], group_start) and np.array_equal(got["group_adapter"], group_adapter)


def test_static_plan_at_its_size_limit():
    # T = the limit, once with alternating ids (as many runs as tokens: every fixed array is full)
    # and once as a single run; the second call must not allocate device memory.
    import torch
    T = B.PLAN_STATIC_MAX_TOKENS
    alternating = (np.arange(T) % 2).astype(np.int32) * 5
    one_run = np.full(T, 3, dtype=np.int32)
    want, got, info = build_both(alternating, 8)
    assert info[1] == T and info[0] == 2
    for k in KEYS:
        assert np.array_equal(want[k], got[k]), k
    check_against_oracle(got, alternating, 8)

    ids = torch.from_numpy(one_run).cuda()
    out = {k: torch.full((T + 1,), -7, dtype=torch.int32, device="cuda") for k in KEYS}
    info_t = torch.full((4,), -7, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    rc = B.edgelora_plan_build_static(ids, 8, out["ids_valid"], out["perm"], out["group_start"],
                                      out["group_adapter"], out["seg_start"], out["seg_adapter"], info_t)
    assert rc == B.OK
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before, "the non-allocating entry point took device memory"
    info = info_t.cpu().numpy()
    assert info.tolist() == [1, 1, 0, 0]
    got = {"ids_valid": out["ids_valid"][:T], "perm": out["perm"][:T], "group_start": out["group_start"][:2],
           "group_adapter": out["group_adapter"][:1], "seg_start": out["seg_start"][:2],
           "seg_adapter": out["seg_adapter"][:1]}
    check_against_oracle({k: v.cpu().numpy() for k, v in got.items()}, one_run, 8)


def test_static_plan_rejects_oversize_and_handles_empty():
    import torch
    T = B.PLAN_STATIC_MAX_TOKENS + 1
    z = torch.zeros(T + 1, dtype=torch.int32, device="cuda")
    info = torch.zeros(4, dtype=torch.int32, device="cuda")
    assert B.edgelora_plan_build_static(z[:T], 8, z, z, z, z, z, z, info) == B.ERR_TOO_MANY_TOKENS
    info.fill_(5)
    assert B.edgelora_plan_build_static(z[:0], 8, z, z, z, z, z, z, info) == B.OK
    torch.cuda.synchronize()
    assert info.cpu().tolist() == [0, 0, 0, 0]
