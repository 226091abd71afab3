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


# ------------------------------------------------------------------ base weights stored in Q8_0 / Q4_0
@pytest.mark.parametrize("fmt,code,encode", [("q8_0", B.WEIGHTS_Q8_0, wl.q8_0_encode), ("q4_0", B.WEIGHTS_Q4_0, wl.q4_0_encode)])
def test_base_weights_decode_is_bit_exact_and_feeds_the_layer(fmt, code, encode):
    # The decode kernel against the oracle's decode: d * code is exact in both, so after rounding to
    # bfloat16 the bits must agree.  Then the layer over the decoded W against the layer oracle.
    import torch
    from oracle.quant import weights_decode
    from gpu_helpers import to_dev_bf16, from_dev_bf16, make_pool
    from helpers import assert_parity, oracle_of
    from test_gpu_parity import random_workload
    w = random_workload(8800, 40, 512, 392, ranks=[16, 8, 12], max_rank=16)
    Wf = wl.bf16_bits_to_f32(w.W)
    blocks = encode(Wf)                                              # [h_out, h_in / 32, 34 or 18]
    want_bits = wl.f32_to_bf16_bits(weights_decode(fmt, blocks, w.h_in).astype(np.float32))
    Wq = torch.from_numpy(blocks).cuda()
    W = torch.zeros((w.h_out, w.h_in), dtype=torch.bfloat16, device="cuda")
    B.edgelora_weights_decode(code, Wq, w.h_out, w.h_in, W)
    torch.cuda.synchronize()
    got_bits = W.view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(got_bits, want_bits)
    w2 = wl.Workload(f"{fmt}_weights", w.h_in, w.h_out, w.n_slots, w.max_rank, want_bits, w.x, w.ids, w.adapters)
    pool = make_pool(w2, 64)
    try:
        y = pool.linear(W, to_dev_bf16(w2.x), torch.from_numpy(w2.ids).cuda())
        assert pool.status() == (0, 0)
        assert_parity(from_dev_bf16(y), oracle_of(w2), f"layer over W decoded from {fmt}")
    finally:
        pool.close()
    with pytest.raises(B.EdgeLoraError) as e:
        B.edgelora_weights_decode(7, Wq, w.h_out, w.h_in, W)
    assert e.value.code == B.ERR_INVALID_ARG
