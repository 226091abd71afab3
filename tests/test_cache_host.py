"""The library's adapter memory manager (host code behind the C ABI) against the oracle, decision
by decision: integer work, so block, hit flag and evicted key must be identical at every step.
Runs without a GPU: these entry points make no CUDA call."""
import numpy as np
import pytest

from oracle.cache import AdapterCache
from paper_2507_01438_b200 import binding as B


def power_law_trace(seed, n_keys, n, alpha=1.0):
    rng = np.random.Generator(np.random.PCG64(seed))
    w = 1.0 / np.arange(1, n_keys + 1) ** alpha
    order = rng.permutation(n_keys)                       # popular adapters are not neighbours
    return order[rng.choice(n_keys, size=n, p=w / w.sum())].tolist()


@pytest.mark.parametrize("policy", [B.CACHE_LRU, B.CACHE_LFU])
@pytest.mark.parametrize("n_blocks,n_keys,n", [(1, 5, 200), (4, 12, 600), (32, 1000, 5000), (100, 2000, 8000)])
def test_every_decision_matches_the_oracle(policy, n_blocks, n_keys, n):
    trace = power_law_trace(n_blocks * 7 + n_keys, n_keys, n)
    ref = AdapterCache(n_blocks, policy)
    c = B.edgelora_cache_create(n_blocks, policy)
    try:
        for step, k in enumerate(trace):
            assert B.edgelora_cache_acquire(c, k) == ref.acquire(k), f"step {step}, key {k}"
            if step % 97 == 0:
                probe = trace[(step * 31) % n]
                assert B.edgelora_cache_lookup(c, probe) == ref.lookup(probe)
        st = B.edgelora_cache_stats(c)
        assert st == {"hits": ref.hits, "misses": ref.misses, "evictions": ref.evictions, "resident": ref.resident()}
    finally:
        B.edgelora_cache_destroy(c)


@pytest.mark.parametrize("policy", [B.CACHE_LRU, B.CACHE_LFU])
def test_holds_of_running_requests_match_the_oracle(policy):
    # a serving loop: each step admits the adapters of up to three requests (held), and requests
    # admitted three steps earlier finish (released)
    rng = np.random.Generator(np.random.PCG64(21))
    trace = power_law_trace(3, 60, 900)
    ref = AdapterCache(12, policy)
    c = B.edgelora_cache_create(12, policy)
    held = []
    try:
        for i in range(0, len(trace), 3):
            batch = trace[i:i + int(rng.integers(1, 4))]
            for k in batch:
                assert B.edgelora_cache_acquire(c, k, pin=True) == ref.acquire(k, pin=True)
            held.append(batch)
            if len(held) > 3:
                for k in held.pop(0):
                    B.edgelora_cache_release(c, k)
                    ref.release(k)
        assert B.edgelora_cache_stats(c)["evictions"] == ref.evictions > 0
    finally:
        B.edgelora_cache_destroy(c)


def test_all_blocks_held_is_an_error_not_an_eviction():
    c = B.edgelora_cache_create(2, B.CACHE_LRU)
    try:
        B.edgelora_cache_acquire(c, 7, pin=True)
        B.edgelora_cache_acquire(c, 8, pin=True)
        with pytest.raises(B.EdgeLoraError) as e:
            B.edgelora_cache_acquire(c, 9)
        assert e.value.code == B.ERR_CACHE_FULL
        assert B.edgelora_cache_lookup(c, 7) == 0 and B.edgelora_cache_lookup(c, 8) == 1
        B.edgelora_cache_release(c, 7)
        assert B.edgelora_cache_acquire(c, 9) == (0, False, 7)
        with pytest.raises(B.EdgeLoraError):
            B.edgelora_cache_release(c, 7)            # gone
        with pytest.raises(B.EdgeLoraError):
            B.edgelora_cache_release(c, 9)            # resident but not held
    finally:
        B.edgelora_cache_destroy(c)


def test_argument_errors():
    with pytest.raises(B.EdgeLoraError):
        B.edgelora_cache_create(0)
    with pytest.raises(B.EdgeLoraError):
        B.edgelora_cache_create(4, 2)
    c = B.edgelora_cache_create(4)
    try:
        with pytest.raises(B.EdgeLoraError):
            B.edgelora_cache_acquire(c, -3)
    finally:
        B.edgelora_cache_destroy(c)


@pytest.mark.parametrize("k", [1, 3, 8, 500])
@pytest.mark.parametrize("policy", [B.CACHE_LRU, B.CACHE_LFU])
def test_cache_aware_selection_matches_the_oracle(policy, k):
    # router scores favour a few adapters per request (a sparse sigmoid output), with exact ties
    from oracle.cache import select_adapter
    rng = np.random.Generator(np.random.PCG64(50 + k))
    n = 300
    ref = AdapterCache(16, policy)
    c = B.edgelora_cache_create(16, policy)
    try:
        for step in range(800):
            s = (rng.random(n) * 0.05).astype(np.float32)
            hot = rng.choice(n, size=6, replace=False, p=None)
            s[hot] = rng.choice(np.array([0.5, 0.7, 0.9, 0.9], dtype=np.float32), size=6)
            assert B.edgelora_cache_select(c, s, k) == select_adapter(ref, s, k), f"step {step}"
        assert B.edgelora_cache_stats(c)["hits"] == ref.hits
    finally:
        B.edgelora_cache_destroy(c)


def test_prefill_before_serving():
    # Section 4.2: the cache starts full of (the caller's choice of) adapters, counters at zero
    keys = [41, 7, 19, 3]
    o = AdapterCache(6)
    c = B.edgelora_cache_create(6)
    try:
        assert B.edgelora_cache_prefill(c, keys).tolist() == o.prefill(keys) == [0, 1, 2, 3]
        assert B.edgelora_cache_stats(c) == {"hits": 0, "misses": 0, "evictions": 0, "resident": 4}
        for key in (7, 99, 41, 100, 101, 3):
            assert B.edgelora_cache_acquire(c, key) == o.acquire(key)
        st = B.edgelora_cache_stats(c)
        assert (st["hits"], st["misses"], st["evictions"]) == (o.hits, o.misses, o.evictions) == (3, 3, 1)
        with pytest.raises(B.EdgeLoraError):
            B.edgelora_cache_prefill(c, [1])                       # not empty any more
    finally:
        B.edgelora_cache_destroy(c)
