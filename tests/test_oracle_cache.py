"""Pins of the adapter-cache oracle (paper Sections 3.3 and 4.2) against facts that do not come
from it: the page-replacement results every operating-systems text gives for LRU, closed forms
for cyclic and repeated traces, and invariants."""
import numpy as np
import pytest

from oracle.cache import LFU, LRU, AdapterCache

# The reference string used by operating-systems textbooks to compare page replacement policies;
# with three frames least-recently-used replacement takes 12 faults, with four frames 8.
TEXTBOOK = [7, 0, 1, 2, 0, 3, 0, 4, 2, 3, 0, 3, 2, 1, 2, 0, 1, 7, 0, 1]


def run(cache, trace):
    return [cache.acquire(k) for k in trace]


@pytest.mark.parametrize("frames,faults", [(3, 12), (4, 8)])
def test_textbook_reference_string(frames, faults):
    c = AdapterCache(frames, LRU)
    run(c, TEXTBOOK)
    assert c.misses == faults and c.hits == len(TEXTBOOK) - faults
    assert c.evictions == faults - frames


def test_textbook_resident_sets_step_by_step():
    # the frame contents after each fault, as the same texts tabulate them for three frames
    c = AdapterCache(3, LRU)
    expect_after_fault = [{7}, {7, 0}, {7, 0, 1}, {2, 0, 1}, {2, 0, 3}, {4, 0, 3}, {4, 0, 2}, {4, 3, 2},
                          {0, 3, 2}, {1, 3, 2}, {1, 0, 2}, {1, 0, 7}]
    seen = []
    for k in TEXTBOOK:
        _, hit, _ = c.acquire(k)
        if not hit:
            seen.append(set(c.slot))
    assert seen == expect_after_fault


def test_cyclic_trace_one_more_key_than_blocks_never_hits_under_lru():
    n = 5
    c = AdapterCache(n, LRU)
    run(c, [i % (n + 1) for i in range(60)])
    assert c.hits == 0 and c.misses == 60 and c.evictions == 60 - n


def test_working_set_that_fits_misses_once_per_key():
    rng = np.random.Generator(np.random.PCG64(5))
    trace = rng.integers(0, 8, size=500).tolist()
    for policy in (LRU, LFU):
        c = AdapterCache(8, policy)
        run(c, trace)
        assert c.misses == len(set(trace)) and c.evictions == 0


def test_free_blocks_go_out_in_ascending_order_and_an_evicted_block_is_reused():
    c = AdapterCache(3, LRU)
    assert [c.acquire(k)[0] for k in (10, 11, 12)] == [0, 1, 2]
    block, hit, evicted = c.acquire(13)
    assert (block, hit, evicted) == (0, False, 10)      # 10 was the least recently used
    c.acquire(11)                                       # refresh 11: now 12 is the oldest
    assert c.acquire(14) == (2, False, 12)


def test_lfu_keeps_the_frequent_key_through_a_scan_lru_does_not():
    trace = [1, 1, 1, 1, 2, 3, 4, 5, 6, 1]
    lru, lfu = AdapterCache(3, LRU), AdapterCache(3, LFU)
    assert run(lru, trace)[-1][1] is False
    assert run(lfu, trace)[-1][1] is True
    # among equally rare keys LFU evicts the least recently used
    c = AdapterCache(2, LFU)
    run(c, [1, 2])
    assert c.acquire(3)[2] == 1


def test_pinned_keys_are_never_victims():
    c = AdapterCache(2, LRU)
    c.acquire(1, pin=True)
    c.acquire(2)
    assert c.acquire(3) == (1, False, 2)     # 1 is older but held by a request
    c.acquire(3, pin=True)
    with pytest.raises(RuntimeError):
        c.acquire(4)
    c.release(1)
    assert c.acquire(4) == (0, False, 1)


@pytest.mark.parametrize("policy", [LRU, LFU])
def test_invariants_on_a_power_law_trace(policy):
    rng = np.random.Generator(np.random.PCG64(9))
    w = 1.0 / np.arange(1, 201) ** 1.0
    trace = rng.choice(200, size=3000, p=w / w.sum()).tolist()
    c = AdapterCache(16, policy)
    for k in trace:
        block, hit, evicted = c.acquire(k)
        assert c.lookup(k) == block and 0 <= block < 16
        assert sorted(c.slot.values()) == sorted(set(c.slot.values()))      # one key per block
        assert c.resident() <= 16 and (evicted == -1 or c.lookup(evicted) == -1)
    assert c.hits + c.misses == len(trace) and c.evictions == c.misses - 16
    # a popular head makes the cache useful: far more hits than a uniform trace would give
    assert c.hits / len(trace) > 0.4


# ---------------------------------------------------------------- cache-aware selection (Algorithm 1)
from oracle.cache import select_adapter


def brute_force_choice(resident, scores, k):
    # every adapter ranked by hand; the answer is the best-scored resident one inside the top k,
    # else the best-scored overall
    ranked = []
    remaining = list(range(len(scores)))
    while remaining:
        best = remaining[0]
        for j in remaining:
            if scores[j] > scores[best]:
                best = j
        ranked.append(best)
        remaining.remove(best)
    inside = [a for a in ranked[:k] if a in resident]
    return inside[0] if inside else ranked[0]


def test_selection_with_k_one_is_the_argmax():
    rng = np.random.Generator(np.random.PCG64(2))
    c = AdapterCache(4)
    for _ in range(50):
        s = rng.random(20).astype(np.float32)
        a, _, _, _ = select_adapter(c, s, 1)
        assert a == int(np.argmax(s))


def test_selection_prefers_a_resident_adapter_inside_the_top_k_only():
    c = AdapterCache(2)
    c.acquire(5)
    c.acquire(9)
    s = np.zeros(12, dtype=np.float32)
    s[[3, 5, 9, 7]] = [0.9, 0.8, 0.7, 0.6]
    assert select_adapter(c, s, 1)[:3] == (3, 0, False)      # k = 1: top-1 loaded although 5 and 9 are resident
    c2 = AdapterCache(2)
    c2.acquire(5)
    c2.acquire(9)
    assert select_adapter(c2, s, 2)[:3] == (5, 0, True)       # 5 is the best resident one inside the top 2
    s[5] = 0.0
    assert select_adapter(c2, s, 2)[:3] == (9, 1, True)       # top 2 is now {3, 9}, and 9 is resident
    s[9] = 0.0
    assert select_adapter(c2, s, 2)[:3] == (3, 0, False)      # top 2 = {3, 7}: none resident, 3 is loaded over 5


@pytest.mark.parametrize("k", [1, 2, 3, 8])
def test_selection_against_brute_force(k):
    rng = np.random.Generator(np.random.PCG64(30 + k))
    c = AdapterCache(5)
    for _ in range(300):
        s = rng.random(24).astype(np.float32)
        if rng.random() < 0.3:
            s[rng.integers(0, 24, size=4)] = s[0]           # ties
        expect = brute_force_choice(set(c.slot), s.tolist(), k)
        was_resident = c.lookup(expect) >= 0
        a, block, hit, evicted = select_adapter(c, s, k)
        assert a == expect and hit == was_resident and c.lookup(a) == block
