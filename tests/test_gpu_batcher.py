"""The request batcher driving the layer on the GPU: a short trace over more adapters than cache
blocks; every step loads what the batcher says, runs the batch through the layer with the batcher's
slot ids, and is checked against the layer oracle given the adapters by block as the pool stands at
that moment (paper Section 4 slot state machine + Section 3.2 / 3.3 + the batch LoRA layer of 3.4).
The batches themselves must be those of the batcher oracle."""
import numpy as np
import pytest

from oracle.batcher import Batcher as OracleBatcher
from oracle.cache import AdapterCache
from paper_2507_01438_b200 import binding as B
from paper_2507_01438_b200 import workloads as wl
from helpers import assert_parity, oracle_of
from gpu_helpers import from_dev_bf16, to_dev_bf16

pytestmark = pytest.mark.gpu


def test_a_trace_through_the_layer():
    import torch
    rng = np.random.Generator(np.random.PCG64(61))
    h_in, h_out, n_blocks, n_adapters, max_rank, n_slots, max_tokens, top_k = 384, 264, 4, 10, 16, 3, 96, 2
    W = wl.normal_bf16(rng, (h_out, h_in), 0.05)
    library = {k: wl.Adapter(wl.normal_bf16(rng, (r, h_in), 0.05), wl.normal_bf16(rng, (h_out, r), 0.05), 2.0)
               for k, r in enumerate(rng.choice([4, 8, 16], size=n_adapters))}
    trace = wl.serving_trace(seed=62, n_adapters=n_adapters, rate=20.0, duration=1.0, in_range=(8, 120),
                             out_range=(1, 6), top_k=top_k)
    assert 8 <= len(trace.arrival) <= 60
    pool = B.Pool(h_in, h_out, n_blocks, max_rank, max_tokens=max_tokens)
    cache = B.edgelora_cache_create(n_blocks)
    nb = B.edgelora_batcher_create(n_slots, max_tokens, top_k, cache)
    ob = OracleBatcher(n_slots, max_tokens, AdapterCache(n_blocks))
    Wd = to_dev_bf16(W)
    in_block = {}
    try:
        for i in range(len(trace.arrival)):
            B.edgelora_batcher_submit(nb, i, trace.arrival[i], trace.in_len[i], trace.out_len[i], trace.candidates[i])
            ob.submit(i, trace.arrival[i], trace.in_len[i], trace.out_len[i], trace.candidates[i])
        steps = checked = 0
        while True:
            got = B.edgelora_batcher_next_batch(nb, max_tokens, n_slots)
            want = ob.next_batch()
            if got is None:
                assert want is None
                break
            assert got["token_block"].tolist() == want["token_block"] and got["loads"] == [tuple(x) for x in want["loads"]]
            for key, block in got["loads"]:
                pool.load(block, library[key].A, library[key].B, library[key].scale)
                in_block[block] = key
            ids = got["token_block"].astype(np.int32)
            T = len(ids)
            if steps % 3 == 0 or got["loads"]:          # the layer on this step's batch, against the oracle
                x = wl.normal_bf16(rng, (T, h_in), 1.0)
                y = pool.linear(Wd, to_dev_bf16(x), torch.from_numpy(ids).cuda())
                batch = wl.Workload(f"step{steps}", h_in, h_out, n_blocks, max_rank, W, x, ids,
                                    {b: library[k] for b, k in in_block.items()})
                assert_parity(from_dev_bf16(y), oracle_of(batch), f"step {steps}")
                checked += 1
            dt = 0.01 + 1e-4 * T
            B.edgelora_batcher_complete_step(nb, dt)
            ob.complete_step(dt)
            steps += 1
        assert pool.status() == (0, 0) and checked >= 5
        fin = B.edgelora_batcher_finished(nb)
        assert len(fin["id"]) == len(trace.arrival)
        assert fin["finish"].tolist() == [r.finish for r in ob.done]
    finally:
        B.edgelora_batcher_destroy(nb)
        B.edgelora_cache_destroy(cache)
        pool.close()
