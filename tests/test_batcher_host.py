"""The native batcher (edgelora_batcher_*, host code of the library) against the CPU oracle: every
batch, every load, every clock value and every finished record must be identical.  No GPU needed.
"""
import numpy as np
import pytest

from oracle.batcher import Batcher as OracleBatcher
from oracle.cache import AdapterCache
from paper_2507_01438_b200 import binding as B
from paper_2507_01438_b200 import workloads as wl
from helpers import golden


def run_both(trace, n_slots, max_tokens, blocks, top_k, step_time):
    ob = OracleBatcher(n_slots, max_tokens, AdapterCache(blocks))
    cache = B.edgelora_cache_create(blocks)
    nb = B.edgelora_batcher_create(n_slots, max_tokens, top_k, cache)
    try:
        for i in range(len(trace.arrival)):
            ob.submit(i, trace.arrival[i], trace.in_len[i], trace.out_len[i], trace.candidates[i][:top_k])
            B.edgelora_batcher_submit(nb, i, trace.arrival[i], trace.in_len[i], trace.out_len[i],
                                      trace.candidates[i][:top_k])
        steps = 0
        while True:
            want = ob.next_batch()
            got = B.edgelora_batcher_next_batch(nb, max_tokens, n_slots)
            if want is None:
                assert got is None
                break
            assert got["now"] == want["now"] and got["n_decode"] == want["n_decode"]
            assert got["token_block"].tolist() == want["token_block"]
            assert got["token_slot"].tolist() == want["token_slot"]
            assert got["loads"] == [tuple(x) for x in want["loads"]]
            dt = step_time(want)
            ob.complete_step(dt)
            B.edgelora_batcher_complete_step(nb, dt)
            steps += 1
        fin = B.edgelora_batcher_finished(nb)
        assert fin["id"].tolist() == [r.rid for r in ob.done]
        assert fin["first_token"].tolist() == [r.first_token for r in ob.done]
        assert fin["finish"].tolist() == [r.finish for r in ob.done]
        assert fin["adapter"].tolist() == [r.adapter for r in ob.done]
        assert fin["hit"].tolist() == [int(r.hit) for r in ob.done]
        stats = B.edgelora_cache_stats(cache)
        assert (stats["hits"], stats["misses"]) == (ob.cache.hits, ob.cache.misses)
        return steps, len(ob.done)
    finally:
        B.edgelora_batcher_destroy(nb)
        B.edgelora_cache_destroy(cache)


def test_hand_worked_trace_through_the_library():
    g = golden("hand_example_batcher.json")
    t = wl.Trace(np.array([r["arrival"] for r in g["requests"]]), np.array([r["in_len"] for r in g["requests"]]),
                 np.array([r["out_len"] for r in g["requests"]]),
                 np.array([r["candidates"] for r in g["requests"]], dtype=np.int64))
    steps, done = run_both(t, g["n_slots"], g["max_batch_tokens"], g["cache_blocks"], 1, lambda b: g["step_seconds"])
    assert (steps, done) == (4, 3)


@pytest.mark.parametrize("n_slots,max_tokens,blocks,top_k,alpha,cv", [
    (1, 64, 2, 1, 1.0, 1.0), (5, 128, 4, 3, 1.0, 1.0), (20, 512, 20, 3, 0.5, 1.5), (50, 2112, 100, 3, 1.0, 2.0),
    (8, 16, 3, 2, 1.5, 1.25),
])
def test_power_law_traces(n_slots, max_tokens, blocks, top_k, alpha, cv):
    t = wl.serving_trace(seed=n_slots + blocks, n_adapters=200, alpha=alpha, rate=4.0, cv=cv, duration=40.0)
    step = lambda b: 0.003 + 2e-5 * len(b["token_block"]) + 0.001 * len(b["loads"])
    steps, done = run_both(t, n_slots, max_tokens, max(blocks, min(n_slots, 200)), top_k, step)
    assert done == len(t.arrival) and steps > 0


def test_argument_errors_and_stall():
    cache = B.edgelora_cache_create(1)
    nb = B.edgelora_batcher_create(2, 8, 1, cache)
    try:
        with pytest.raises(B.EdgeLoraError):
            B.edgelora_batcher_create(4, 3, 1, cache)                  # fewer tokens per step than slots
        with pytest.raises(B.EdgeLoraError):
            B.edgelora_batcher_submit(nb, 0, 0.0, 0, 1, [1])           # empty prompt
        B.edgelora_batcher_submit(nb, 0, 1.0, 4, 2, [1])
        with pytest.raises(B.EdgeLoraError):
            B.edgelora_batcher_submit(nb, 1, 0.5, 4, 2, [1])           # out of arrival order
        with pytest.raises(B.EdgeLoraError):
            B.edgelora_batcher_complete_step(nb, 1.0)                  # no step handed out
        got = B.edgelora_batcher_next_batch(nb, 8, 2)
        assert got["now"] == 1.0 and len(got["token_block"]) == 4     # the clock jumped to the arrival
        with pytest.raises(B.EdgeLoraError):
            B.edgelora_batcher_next_batch(nb, 8, 2)                    # the step is still open
    finally:
        B.edgelora_batcher_destroy(nb)
        B.edgelora_cache_destroy(cache)
