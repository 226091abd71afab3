"""Pins of the Q8_0 oracle (oracle/quant.py): blocks written out by hand, the decode of the input
generator's encoder within the format's error bound, and the layer with Q8_0 adapters against the
bfloat16 layer oracle on adapters that both formats hold exactly.  No GPU.
"""
import numpy as np
import pytest

import oracle
from oracle.quant import lora_linear_q8, q8_0_decode
from paper_2507_01438_b200 import workloads as wl
from helpers import adapter_set, bits, golden


def test_hand_written_blocks():
    for case in golden("q8_0_blocks.json")["cases"]:
        blk = np.array(case["bytes"], dtype=np.uint8).reshape(1, 34)
        got = q8_0_decode(blk, 32)
        want = np.zeros(32)
        want[:len(case["values"])] = case["values"]
        assert np.allclose(got, want, rtol=1e-14, atol=0), case["what"]


def test_encoder_round_trip_is_within_half_a_step():
    rng = np.random.Generator(np.random.PCG64(8))
    v = (rng.standard_normal((5, 100)) * 0.02).astype(np.float32)
    blocks = wl.q8_0_encode(v)
    assert blocks.shape == (5, 4, 34)
    back = q8_0_decode(blocks, 100)
    d = np.abs(np.pad(v, ((0, 0), (0, 28))).reshape(5, 4, 32)).max(axis=-1) / 127.0
    step = np.repeat(d, 32, axis=1)[:, :100]
    assert np.all(np.abs(back - v) <= 0.5 * step * (1 + 2e-3) + 1e-12)   # half a step (+ the half-precision d)
    assert np.all(q8_0_decode(wl.q8_0_encode(np.zeros((2, 32), np.float32)), 32) == 0.0)
    # values that are multiples of a power-of-two step survive exactly
    exact = (rng.integers(-127, 128, size=(3, 64)) * 0.25).astype(np.float32)
    exact[:, 0], exact[:, 32] = 127 * 0.25, -127 * 0.25
    assert np.array_equal(q8_0_decode(wl.q8_0_encode(exact), 64), exact.astype(np.float64))


def test_layer_with_q8_adapters_equals_the_bf16_layer_on_values_both_formats_hold():
    # entries are small integers times 1/8: exact in bfloat16 and, with d = 1/8 (max |v| = 127/8), in Q8_0
    rng = np.random.Generator(np.random.PCG64(9))
    h_in, h_out, T = 64, 48, 9
    W = bits(rng.integers(-3, 4, size=(h_out, h_in)) * 0.5)
    x = bits(rng.integers(-2, 3, size=(T, h_in)) * 1.0)
    ids = np.array([0, 1, -1, 1, 0, 0, -1, 1, 1], dtype=np.int32)
    ad_bf16, ad_q8 = {}, {}
    for a, rank in ((0, 5), (1, 33)):
        A = rng.integers(-7, 8, size=(rank, h_in)) * 0.125
        Bm = rng.integers(-7, 8, size=(h_out, rank)) * 0.125
        A[:, 0::32] = 127 * 0.125                         # pins every block's scale to 1/8
        Bm[:, 0::32] = -127 * 0.125
        ad_bf16[a] = wl.Adapter(bits(A), bits(Bm), 0.5)
        ad_q8[a] = (wl.q8_0_encode(A), wl.q8_0_encode(Bm), rank, 0.5)
    want = oracle.lora_linear(W, x, ids, adapter_set(2, ad_bf16))
    got = lora_linear_q8(W, x, ids, ad_q8)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-12)
    base = oracle.lora_linear(W, x, np.full(T, -1, np.int32), adapter_set(2, {}))
    assert np.array_equal(got[ids < 0], base[ids < 0]) and not np.allclose(got[ids >= 0], base[ids >= 0])


# ------------------------------------------------------------------ base weights in Q4_0 / Q8_0
def test_q4_0_hand_written_block():
    from oracle.quant import q4_0_decode
    fx = golden("q4_0_block.json")
    blk = np.array(fx["block_bytes"], dtype=np.uint8).reshape(1, 18)
    assert np.array_equal(q4_0_decode(blk, 32), np.array(fx["values"], dtype=np.float64))
    # a shorter row takes the leading values only
    assert np.array_equal(q4_0_decode(blk, 20), np.array(fx["values"][:20], dtype=np.float64))


def test_q4_0_encoder_round_trip_is_within_half_a_step():
    from oracle.quant import q4_0_decode, weights_decode
    rng = np.random.Generator(np.random.PCG64(9))
    v = (rng.standard_normal((6, 128)) * 0.05).astype(np.float32)
    blocks = wl.q4_0_encode(v)
    assert blocks.shape == (6, 4, 18)
    back = q4_0_decode(blocks, 128)
    m = np.abs(v.reshape(6, 4, 32)).max(axis=-1)
    step = np.repeat(m / 8.0, 32, axis=1)
    # half a step, except at the end of the range opposite to the largest element (code 15 = +7 steps)
    assert np.all(np.abs(back - v) <= 1.0 * step * (1 + 2e-3) + 1e-12)
    inner = np.abs(v) <= 6.5 * step
    assert np.all(np.abs(back - v)[inner] <= 0.5 * step[inner] * (1 + 4e-3) + 1e-12)
    assert np.all(q4_0_decode(wl.q4_0_encode(np.zeros((2, 32), np.float32)), 32) == 0.0)
    # multiples of a power-of-two step with the extreme at -8 steps survive exactly
    exact = (rng.integers(-7, 8, size=(3, 64)) * 0.125).astype(np.float32)
    exact[:, 0], exact[:, 32] = -8 * 0.125, -8 * 0.125
    assert np.array_equal(q4_0_decode(wl.q4_0_encode(exact), 64), exact.astype(np.float64))
    assert np.array_equal(weights_decode("q4_0", wl.q4_0_encode(exact), 64), exact.astype(np.float64))
    exact8 = (rng.integers(-127, 128, size=(3, 64)) * 0.25).astype(np.float32)
    exact8[:, 0], exact8[:, 32] = 127 * 0.25, -127 * 0.25          # d = 1/4 exactly
    assert np.array_equal(weights_decode("q8_0", wl.q8_0_encode(exact8), 64), exact8.astype(np.float64))
