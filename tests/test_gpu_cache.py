"""The adapter memory manager driving a pool on the GPU: more adapters than blocks, every batch
admits its adapters (loads on a miss, into the block the manager names), runs the layer with
slot ids and is checked against the oracle, which is given the adapters by block as they stand
at that moment (paper Sections 3.3 / 4.2 with the batch LoRA layer of Section 3.4)."""
import numpy as np
import pytest

from oracle.cache import AdapterCache
from paper_2507_01438_b200 import binding as B
from paper_2507_01438_b200 import workloads as wl
from helpers import assert_parity, oracle_of
from gpu_helpers import from_dev_bf16, to_dev_bf16

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("policy", [B.CACHE_LRU, B.CACHE_LFU])
def test_batches_over_a_small_pool(policy):
    import torch
    rng = np.random.Generator(np.random.PCG64(40 + policy))
    h_in, h_out, n_blocks, n_adapters, max_rank = 512, 384, 4, 12, 16
    W = wl.normal_bf16(rng, (h_out, h_in), 0.05)
    library = {k: wl.Adapter(wl.normal_bf16(rng, (r, h_in), 0.05), wl.normal_bf16(rng, (h_out, r), 0.05), 2.0)
               for k, r in enumerate(rng.choice([4, 8, 16], size=n_adapters))}
    pool = B.Pool(h_in, h_out, n_blocks, max_rank, max_tokens=64)
    cache = B.edgelora_cache_create(n_blocks, policy)
    ref = AdapterCache(n_blocks, policy)
    in_block = {}                      # block -> adapter key, as the pool stands
    Wd = to_dev_bf16(W)
    weights = 1.0 / np.arange(1, n_adapters + 1)
    loads = 0
    try:
        for step in range(10):
            T = int(rng.integers(8, 64))
            keys = rng.choice(n_adapters, size=int(rng.integers(1, n_blocks + 1)), replace=False,
                              p=weights / weights.sum())
            for k in keys:
                block, hit, evicted = B.edgelora_cache_acquire(cache, int(k), pin=True)
                assert (block, hit, evicted) == ref.acquire(int(k), pin=True)
                if not hit:
                    pool.load(block, library[int(k)].A, library[int(k)].B, library[int(k)].scale)
                    in_block[block] = int(k)
                    loads += 1
            tok_keys = rng.choice(np.concatenate([keys, [-1]]), size=T)
            ids = np.array([B.edgelora_cache_lookup(cache, int(k)) if k >= 0 else -1 for k in tok_keys], dtype=np.int32)
            x = wl.normal_bf16(rng, (T, h_in), 1.0)
            y = pool.linear(Wd, to_dev_bf16(x), torch.from_numpy(ids).cuda())
            batch = wl.Workload(f"step{step}", h_in, h_out, n_blocks, max_rank, W, x, ids,
                                {b: library[k] for b, k in in_block.items()})
            assert_parity(from_dev_bf16(y), oracle_of(batch), f"step {step}")
            for k in keys:
                B.edgelora_cache_release(cache, int(k))
                ref.release(int(k))
        assert pool.status() == (0, 0)
        st = B.edgelora_cache_stats(cache)
        assert st["misses"] == loads and st["evictions"] == loads - n_blocks > 0
    finally:
        B.edgelora_cache_destroy(cache)
        pool.close()
