"""Pins for the routing oracle (segments and groups): hand example, brute force, invariants."""
import numpy as np
import pytest

import oracle
from helpers import golden


def test_hand_worked_routing():
    g = golden("hand_example_routing.json")
    ids = np.array(g["ids"], dtype=np.int32)
    start, adapter = oracle.segments(ids)
    assert start.tolist() == g["seg_start"] and adapter.tolist() == g["seg_adapter"]
    perm, gstart, gadapter = oracle.groups(ids, g["n_slots"])
    assert perm.tolist() == g["perm"]
    assert gstart.tolist() == g["group_start"] and gadapter.tolist() == g["group_adapter"]


def _brute_groups(ids):
    # O(T^2): position of token t = number of tokens that must come before it
    T = len(ids)
    perm = [0] * T
    for t in range(T):
        before = sum(1 for u in range(T) if ids[u] < ids[t] or (ids[u] == ids[t] and u < t))
        perm[before] = t
    return perm


@pytest.mark.parametrize("seed", range(6))
def test_groups_brute_force_and_invariants(seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    T = int(rng.integers(1, 40))
    S = int(rng.integers(1, 7))
    ids = rng.integers(-1, S, size=T).astype(np.int32)
    perm, gstart, gadapter = oracle.groups(ids, S)
    assert perm.tolist() == _brute_groups(ids.tolist())
    assert sorted(perm.tolist()) == list(range(T))                      # a permutation
    assert gstart[0] == 0 and gstart[-1] == T and np.all(np.diff(gstart) > 0)
    assert np.all(np.diff(gadapter) > 0)                                 # ascending, -1 first
    assert sorted(gadapter.tolist()) == sorted(set(ids.tolist()))
    for g in range(len(gadapter)):
        members = perm[gstart[g]:gstart[g + 1]]
        assert np.all(ids[members] == gadapter[g]) and np.all(np.diff(members) > 0)   # stable


@pytest.mark.parametrize("seed", range(6))
def test_segments_invariants(seed):
    rng = np.random.Generator(np.random.PCG64(100 + seed))
    T = int(rng.integers(1, 50))
    ids = np.repeat(rng.integers(-1, 3, size=T), rng.integers(1, 4, size=T))[:T].astype(np.int32)
    T = len(ids)
    start, adapter = oracle.segments(ids)
    assert start[0] == 0 and start[-1] == T and np.all(np.diff(start) > 0)
    rebuilt = np.concatenate([np.full(start[i + 1] - start[i], adapter[i]) for i in range(len(adapter))])
    assert np.array_equal(rebuilt, ids)                                  # covers [0, T)
    assert np.all(adapter[1:] != adapter[:-1])                           # runs are maximal


def test_same_id_reappearing_makes_a_new_segment_but_one_group():
    ids = np.array([1, 1, 0, 1], dtype=np.int32)
    start, adapter = oracle.segments(ids)
    assert start.tolist() == [0, 2, 3, 4] and adapter.tolist() == [1, 0, 1]
    perm, gstart, gadapter = oracle.groups(ids, 2)
    assert perm.tolist() == [2, 0, 1, 3] and gstart.tolist() == [0, 1, 4] and gadapter.tolist() == [0, 1]


def test_empty_and_rejects():
    start, adapter = oracle.segments(np.zeros(0, dtype=np.int32))
    assert start.tolist() == [0] and adapter.size == 0
    perm, gstart, gadapter = oracle.groups(np.zeros(0, dtype=np.int32), 3)
    assert perm.size == 0 and gstart.tolist() == [0] and gadapter.size == 0
    with pytest.raises(ValueError):
        oracle.groups(np.array([0, 3], dtype=np.int32), 3)
    with pytest.raises(ValueError):
        oracle.groups(np.array([-2], dtype=np.int32), 3)
