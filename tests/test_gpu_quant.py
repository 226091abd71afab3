"""Adapters loaded in Q8_0 (edgelora_pool_load_slot_q8): the layer's result against the Q8_0 layer
oracle, which decodes the blocks exactly; the pool's block holds the decoded values rounded to
bfloat16 (relative 2^-9 per weight, far inside the layer's tolerance), decode and prefill regime.
"""
import numpy as np
import pytest

from oracle.quant import lora_linear_q8
from paper_2507_01438_b200 import binding as B
from paper_2507_01438_b200 import workloads as wl
from helpers import assert_parity
from gpu_helpers import from_dev_bf16, to_dev_bf16

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("T,h_in,h_out,max_rank,ranks", [
    (40, 256, 264, 16, [16, 8, 5]), (300, 512, 384, 64, [64, 33, 32, 7]), (130, 1024, 256, 32, [32, 20])])
def test_q8_adapters_match_their_oracle(T, h_in, h_out, max_rank, ranks):
    import torch
    rng = np.random.Generator(np.random.PCG64(T + h_in))
    W = wl.normal_bf16(rng, (h_out, h_in), 0.05)
    x = wl.normal_bf16(rng, (T, h_in), 1.0)
    ids = rng.integers(-1, len(ranks), size=T).astype(np.int32)
    if T > 256:
        ids[40:200] = 1                                   # a long run as well
    adapters = {}
    pool = B.Pool(h_in, h_out, len(ranks), max_rank, max_tokens=T)
    try:
        for a, r in enumerate(ranks):
            A = (rng.standard_normal((r, h_in)) * 0.05).astype(np.float32)
            Bm = (rng.standard_normal((h_out, r)) * 0.05).astype(np.float32)
            adapters[a] = (wl.q8_0_encode(A), wl.q8_0_encode(Bm), r, 2.0)
            B.edgelora_pool_load_slot_q8(pool.handle, a, r, 2.0, adapters[a][0], adapters[a][1])
        y = pool.linear(to_dev_bf16(W), to_dev_bf16(x), torch.from_numpy(ids).cuda())
        assert pool.status() == (0, 0)
        assert_parity(from_dev_bf16(y), lora_linear_q8(W, x, ids, adapters), f"q8 T={T}")
        # a bfloat16 adapter reloaded into a slot that held a Q8_0 one, and back
        plain = wl.Adapter(wl.normal_bf16(rng, (ranks[0], h_in), 0.05), wl.normal_bf16(rng, (h_out, ranks[0]), 0.05), 1.0)
        pool.load(0, plain.A, plain.B, plain.scale)
        B.edgelora_pool_load_slot_q8(pool.handle, 0, ranks[0], 2.0, adapters[0][0], adapters[0][1])
        y2 = pool.linear(to_dev_bf16(W), to_dev_bf16(x), torch.from_numpy(ids).cuda())
        assert np.array_equal(from_dev_bf16(y2), from_dev_bf16(y))
    finally:
        pool.close()


def test_q8_argument_errors():
    pool = B.Pool(264, 256, 2, 16, max_tokens=16)         # 264 is not a multiple of 32
    try:
        with pytest.raises(B.EdgeLoraError) as e:
            B.edgelora_pool_load_slot_q8(pool.handle, 0, 8, 1.0, np.zeros((8, 9, 34), np.uint8), np.zeros((256, 1, 34), np.uint8))
        assert e.value.code == B.ERR_INVALID_ARG
    finally:
        pool.close()


@pytest.mark.parametrize("T,h_in,h_out,max_rank,ranks", [
    (40, 512, 264, 16, [16, 8, 5]), (200, 1024, 384, 64, [64, 33, 32, 7]), (256, 256, 256, 32, [32, 20, 1])])
def test_pool_that_keeps_A_in_q8(T, h_in, h_out, max_rank, ranks):
    # the pool stores A as Q8_0 blocks; the decode shrink decodes them as it streams them
    import torch
    rng = np.random.Generator(np.random.PCG64(T + h_out))
    W = wl.normal_bf16(rng, (h_out, h_in), 0.05)
    x = wl.normal_bf16(rng, (T, h_in), 1.0)
    ids = rng.integers(-1, len(ranks), size=T).astype(np.int32)
    adapters = {}
    pool = B.Pool(h_in, h_out, len(ranks), max_rank, max_tokens=512, flags=B.FLAG_A_Q8)
    try:
        for a, r in enumerate(ranks):
            A = (rng.standard_normal((r, h_in)) * 0.05).astype(np.float32)
            Bm = (rng.standard_normal((h_out, r)) * 0.05).astype(np.float32)
            adapters[a] = (wl.q8_0_encode(A), wl.q8_0_encode(Bm), r, 2.0)
            B.edgelora_pool_load_slot_q8(pool.handle, a, r, 2.0, adapters[a][0], adapters[a][1])
        Wd, idt = to_dev_bf16(W), torch.from_numpy(ids).cuda()
        y = pool.linear(Wd, to_dev_bf16(x), idt)
        assert pool.status() == (0, 0)
        assert_parity(from_dev_bf16(y), lora_linear_q8(W, x, ids, adapters), f"q8 pool T={T}")
        # reload a slot with another adapter of lower rank: the padding rows must be cleared
        A2 = (rng.standard_normal((1, h_in)) * 0.05).astype(np.float32)
        B2 = (rng.standard_normal((h_out, 1)) * 0.05).astype(np.float32)
        adapters[0] = (wl.q8_0_encode(A2), wl.q8_0_encode(B2), 1, 1.0)
        B.edgelora_pool_load_slot_q8(pool.handle, 0, 1, 1.0, adapters[0][0], adapters[0][1])
        y = pool.linear(Wd, to_dev_bf16(x), idt)
        assert_parity(from_dev_bf16(y), lora_linear_q8(W, x, ids, adapters), "after the reload")
        # what such a pool does not take
        with pytest.raises(B.EdgeLoraError) as e:
            B.edgelora_pool_load_slot(pool.handle, 1, 4, 1.0, np.zeros((4, h_in), np.uint16), np.zeros((h_out, 4), np.uint16))
        assert e.value.code == B.ERR_INVALID_ARG
        big = torch.zeros((300, h_in), dtype=torch.bfloat16, device="cuda")
        with pytest.raises(B.EdgeLoraError) as e:
            pool.linear(Wd, big, torch.zeros(300, dtype=torch.int32, device="cuda"))
        assert e.value.code == B.ERR_INVALID_ARG
    finally:
        pool.close()


def test_q8_pool_needs_a_width_of_256():
    with pytest.raises(B.EdgeLoraError) as e:
        B.Pool(320, 256, 2, 16, max_tokens=16, flags=B.FLAG_A_Q8)
    assert e.value.code == B.ERR_INVALID_ARG
