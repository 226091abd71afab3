"""Pins of the batcher oracle (oracle/batcher.py): a hand-worked trace, the closed form of a single
slot, invariants on random traces, the cut-and-continue rule for long prompts, and the wait in the
selection state when every cache block is held.  No GPU.
"""
import numpy as np
import pytest

from oracle.batcher import Batcher, metrics
from oracle.cache import AdapterCache
from paper_2507_01438_b200 import workloads as wl
from helpers import golden


def test_hand_worked_trace():
    g = golden("hand_example_batcher.json")
    b = Batcher(g["n_slots"], g["max_batch_tokens"], AdapterCache(g["cache_blocks"]))
    for r in g["requests"]:
        b.submit(r["id"], r["arrival"], r["in_len"], r["out_len"], r["candidates"])
    for want in g["steps"]:
        got = b.next_batch()
        assert got["now"] == want["now"]
        assert got["token_block"] == want["token_block"] and got["token_slot"] == want["token_slot"]
        assert got["n_decode"] == want["n_decode"]
        assert [list(x) for x in got["loads"]] == want["loads"]
        b.complete_step(g["step_seconds"])
    assert b.next_batch() is None
    assert [(r.rid, r.first_token, r.finish, r.hit) for r in b.done] == \
        [(f["id"], f["first_token"], f["finish"], f["hit"]) for f in g["finished"]]
    m = metrics(b.done)
    for k, v in g["metrics"].items():
        assert m[k] == pytest.approx(v, rel=1e-12)


def test_single_slot_is_sequential_service():
    # one slot, one step per prompt: a request starts when it has arrived and the one before it has
    # finished; its first token comes one step later, its last after out_len steps in all
    t = wl.serving_trace(seed=11, n_adapters=20, rate=0.4, duration=200.0, in_range=(8, 64), out_range=(1, 9))
    c = 0.25
    b = Batcher(1, 64, AdapterCache(4))
    for i in range(len(t.arrival)):
        b.submit(i, t.arrival[i], t.in_len[i], t.out_len[i], t.candidates[i])
    done = b.run(lambda batch: c)
    assert [r.rid for r in done] == list(range(len(t.arrival)))
    free_at = 0.0
    for r in done:
        start = max(r.arrival, free_at)
        assert r.first_token == pytest.approx(start + c, abs=1e-9)
        assert r.finish == pytest.approx(start + c * r.out_len, abs=1e-9)
        free_at = r.finish


def test_long_prompts_are_cut_at_the_token_budget():
    b = Batcher(2, 4, AdapterCache(2))
    b.submit(0, 0.0, 6, 1, [3])          # 6 prompt tokens, 4 per step at most
    b.submit(1, 0.0, 3, 2, [3])
    steps = []
    while True:
        got = b.next_batch()
        if got is None:
            break
        steps.append((got["token_slot"], got["n_decode"]))
        b.complete_step(1.0)
    # step 1: slot 0 takes the whole budget; step 2: its last 2 tokens, then 2 of slot 1's 3;
    # step 3: slot 1's last prompt token; step 4: slot 1 generates its second token
    assert steps == [([0, 0, 0, 0], 0), ([0, 0, 1, 1], 0), ([1], 0), ([1], 1)]
    assert [(r.rid, r.first_token, r.finish) for r in b.done] == [(0, 2.0, 2.0), (1, 3.0, 4.0)]


def test_a_request_waits_in_selection_while_every_block_is_held():
    b = Batcher(2, 16, AdapterCache(1))  # one block: two adapters cannot be resident together
    b.submit(0, 0.0, 4, 3, [5])
    b.submit(1, 0.0, 4, 1, [6])
    sizes = []
    while True:
        got = b.next_batch()
        if got is None:
            break
        sizes.append((len(got["token_block"]), got["loads"]))
        b.complete_step(1.0)
    # request 1 only starts (and loads adapter 6 into block 0) once request 0 has left
    assert sizes == [(4, [(5, 0)]), (1, []), (1, []), (4, [(6, 0)])]
    assert [(r.rid, r.first_token, r.finish, r.hit) for r in b.done] == [(0, 1.0, 3.0, False), (1, 4.0, 4.0, False)]


@pytest.mark.parametrize("n_slots,blocks,alpha", [(5, 8, 1.0), (20, 20, 0.5), (3, 40, 1.5)])
def test_invariants_on_random_traces(n_slots, blocks, alpha):
    t = wl.serving_trace(seed=n_slots, n_adapters=60, alpha=alpha, rate=3.0, cv=1.5, duration=60.0,
                         in_range=(8, 256), out_range=(8, 128))
    cache = AdapterCache(blocks)
    b = Batcher(n_slots, 512, cache)
    for i in range(len(t.arrival)):
        b.submit(i, t.arrival[i], t.in_len[i], t.out_len[i], t.candidates[i])
    held = {}
    tokens_of = {}
    last_now = 0.0
    while True:
        got = b.next_batch()
        if got is None:
            break
        assert got["now"] >= last_now
        last_now = got["now"]
        assert 1 <= len(got["token_block"]) <= 512 and got["n_decode"] <= n_slots
        assert got["token_slot"][:got["n_decode"]] == sorted(set(got["token_slot"][:got["n_decode"]]))
        for blk, s in zip(got["token_block"], got["token_slot"]):
            r = b.slots[s].req
            assert cache.lookup(r.adapter) == blk == r.block      # the held adapter never moved
            assert r.adapter in r.candidates
            tokens_of[r.rid] = tokens_of.get(r.rid, 0) + 1
        for key, blk in got["loads"]:
            assert cache.lookup(key) == blk
        b.complete_step(0.002 + 1e-5 * len(got["token_block"]))
    assert len(b.done) == len(t.arrival)
    for r in b.done:
        assert r.arrival < r.first_token <= r.finish
        assert tokens_of[r.rid] == r.in_len + r.out_len - 1         # the prompt, then one token per step
    m = metrics(b.done)
    assert 0.0 <= m["hit_rate"] <= 1.0 and m["requests"] == len(t.arrival)
    assert sum(cache.pins.values()) == 0                            # every hold was released


def test_trace_generator_statistics():
    t = wl.serving_trace(seed=3, rate=2.0, cv=1.5, duration=4000.0)
    gaps = np.diff(t.arrival)
    assert gaps.mean() == pytest.approx(0.5, rel=0.05)              # 1 / R
    assert gaps.std() / gaps.mean() == pytest.approx(1.5, rel=0.08)  # cv
    assert t.in_len.min() >= 8 and t.in_len.max() <= 256 and t.out_len.min() >= 8 and t.out_len.max() <= 128
    top = np.bincount(t.candidates[:, 0], minlength=100)
    assert np.sort(top)[::-1][0] / len(t.arrival) == pytest.approx(1.0 / np.sum(1.0 / np.arange(1, 101)), rel=0.15)
    assert all(len(set(c)) == len(c) for c in t.candidates)
