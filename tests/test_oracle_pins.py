"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle itself.

Each test is chosen so that a plausible slip in the oracle (dropped low-rank term, missing
scale, transposed A or B, wrong slot, wrong token order) makes at least one of them fail.
"""
import numpy as np
import pytest

import oracle
from paper_2507_01438_b200 import workloads as wl
from helpers import adapter_set, bits, golden, oracle_of


def _f64(b):
    return wl.bf16_bits_to_f32(b).astype(np.float64)


def _random_case(seed, T=7, h_in=12, h_out=9, ranks=(1, 3, 2), with_base_only=True):
    rng = np.random.Generator(np.random.PCG64(seed))
    W = wl.normal_bf16(rng, (h_out, h_in), 0.5)
    x = wl.normal_bf16(rng, (T, h_in), 1.0)
    s = oracle.AdapterSet(len(ranks))
    for a, r in enumerate(ranks):
        s.put(a, wl.normal_bf16(rng, (r, h_in), 0.5), wl.normal_bf16(rng, (h_out, r), 0.5),
              0.25 * (a + 1))
    lo = -1 if with_base_only else 0
    ids = rng.integers(lo, len(ranks), size=T).astype(np.int32)
    return W, x, ids, s


# ---------------------------------------------------------------- format
def test_bf16_widening_matches_format_definition():
    g = golden("bf16_patterns.json")
    s = oracle.AdapterSet(1)
    one = bits([[1.0]])
    for pat, val in g["patterns"].items():
        W = np.array([[int(pat, 16)]], dtype=np.uint16)
        y = oracle.lora_linear(W, one, np.array([-1], dtype=np.int32), s)
        assert y[0, 0] == val


# ---------------------------------------------------------------- hand-worked example
def test_hand_worked_example():
    g = golden("hand_example_lora.json")
    s = oracle.AdapterSet(2)
    for a, ad in g["adapters"].items():
        s.put(int(a), bits(ad["A"]), bits(ad["B"]), ad["scale"])
    y = oracle.lora_linear(bits(g["W"]), bits(g["x"]), np.array(g["ids"], dtype=np.int32), s)
    assert np.array_equal(y, np.array(g["y"], dtype=np.float64))


# ---------------------------------------------------------------- closed form: merged weight
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_single_adapter_batch_equals_merged_weight(seed):
    # Section 2.1: at inference B x A can be merged into W; a batch that uses one adapter
    # therefore equals (W + s B A) x, formed here by library matrix products in fp64.
    W, x, _, s = _random_case(seed, T=5, h_in=11, h_out=6, ranks=(3, 2))
    for a in (0, 1):
        ids = np.full(x.shape[0], a, dtype=np.int32)
        merged = _f64(W) + s.scale[a] * (_f64(s.B[a]) @ _f64(s.A[a]))
        expect = _f64(x) @ merged.T
        y = oracle.lora_linear(W, x, ids, s)
        np.testing.assert_allclose(y, expect, rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------- brute force vs library matmul
@pytest.mark.parametrize("seed", [3, 4, 5, 6])
def test_mixed_batch_against_numpy_fp64(seed):
    W, x, ids, s = _random_case(seed)
    y = oracle.lora_linear(W, x, ids, s)
    for t in range(x.shape[0]):
        e = _f64(W) @ _f64(x[t])
        a = int(ids[t])
        if a >= 0:
            e = e + s.scale[a] * (_f64(s.B[a]) @ (_f64(s.A[a]) @ _f64(x[t])))
        np.testing.assert_allclose(y[t], e, rtol=1e-12, atol=1e-13)


def test_low_rank_term_is_not_negligible_in_the_pins():
    # guards the pins themselves: with the low-rank term dropped the results differ visibly
    W, x, ids, s = _random_case(3, with_base_only=False)
    y = oracle.lora_linear(W, x, ids, s)
    base = oracle.lora_linear(W, x, np.full_like(ids, -1), s)
    assert np.abs(y - base).max() > 1e-2


# ---------------------------------------------------------------- invariants
def test_base_only_and_null_adapters_return_Wx_exactly():
    W, x, ids, s = _random_case(7, with_base_only=False)
    base = oracle.lora_linear(W, x, np.full_like(ids, -1), s)
    np.testing.assert_allclose(base, _f64(x) @ _f64(W).T, rtol=1e-12, atol=1e-13)
    # zero B
    z = oracle.AdapterSet(s.n_slots)
    for a in s.A:
        z.put(a, s.A[a], np.zeros_like(s.B[a]), s.scale[a])
    assert np.array_equal(oracle.lora_linear(W, x, ids, z), base)
    # zero scale
    z = oracle.AdapterSet(s.n_slots)
    for a in s.A:
        z.put(a, s.A[a], s.B[a], 0.0)
    assert np.array_equal(oracle.lora_linear(W, x, ids, z), base)
    # id -1 rows of a mixed batch are the base rows bit for bit
    mixed = ids.copy()
    mixed[::2] = -1
    y = oracle.lora_linear(W, x, mixed, s)
    assert np.array_equal(y[::2], base[::2])
    assert not np.array_equal(y[1::2], base[1::2])


def test_linear_in_x():
    # integers small enough that every product and sum is exact in fp64 and in bf16
    rng = np.random.Generator(np.random.PCG64(11))
    h_in, h_out, T = 6, 5, 4
    W = bits(rng.integers(-3, 4, size=(h_out, h_in)))
    s = oracle.AdapterSet(2)
    s.put(0, bits(rng.integers(-2, 3, size=(2, h_in))), bits(rng.integers(-2, 3, size=(h_out, 2))), 0.5)
    s.put(1, bits(rng.integers(-2, 3, size=(1, h_in))), bits(rng.integers(-2, 3, size=(h_out, 1))), 2.0)
    ids = np.array([0, 1, -1, 0], dtype=np.int32)
    x1 = rng.integers(-4, 5, size=(T, h_in))
    x2 = rng.integers(-4, 5, size=(T, h_in))
    f = lambda x: oracle.lora_linear(W, bits(x), ids, s)
    assert np.array_equal(f(2 * x1 + 3 * x2), 2 * f(x1) + 3 * f(x2))


def test_token_permutation_equivariance():
    W, x, ids, s = _random_case(8, T=9)
    p = np.random.Generator(np.random.PCG64(1)).permutation(x.shape[0])
    y = oracle.lora_linear(W, x, ids, s)
    yp = oracle.lora_linear(W, np.ascontiguousarray(x[p]), np.ascontiguousarray(ids[p]), s)
    assert np.array_equal(yp, y[p])


def test_slot_relabelling():
    W, x, ids, s = _random_case(9, with_base_only=True)
    swap = {0: 2, 1: 0, 2: 1}
    t = oracle.AdapterSet(3)
    for a, b in swap.items():
        t.put(b, s.A[a], s.B[a], s.scale[a])
    ids2 = np.array([swap[int(a)] if a >= 0 else -1 for a in ids], dtype=np.int32)
    assert np.array_equal(oracle.lora_linear(W, x, ids, s), oracle.lora_linear(W, x, ids2, t))


def test_rank_padding_with_zeros_changes_nothing():
    W, x, ids, s = _random_case(10, with_base_only=False)
    p = oracle.AdapterSet(s.n_slots)
    for a in s.A:
        r, h_in = s.A[a].shape
        A = np.zeros((r + 3, h_in), dtype=np.uint16)
        A[:r] = s.A[a]
        B = np.zeros((s.B[a].shape[0], r + 3), dtype=np.uint16)
        B[:, :r] = s.B[a]
        p.put(a, A, B, s.scale[a])
    assert np.array_equal(oracle.lora_linear(W, x, ids, s), oracle.lora_linear(W, x, ids, p))


def test_one_token_at_a_time_equals_the_batch():
    # Section 4.3: grouping tokens by adapter must equal handling every sample alone
    W, x, ids, s = _random_case(12)
    y = oracle.lora_linear(W, x, ids, s)
    for t in range(x.shape[0]):
        yt = oracle.lora_linear(W, x[t:t + 1].copy(), ids[t:t + 1].copy(), s)
        assert np.array_equal(yt[0], y[t])


def test_bad_ids_are_rejected():
    W, x, ids, s = _random_case(13)
    for bad in (-2, 3, 100):
        i = ids.copy()
        i[2] = bad
        with pytest.raises(ValueError):
            oracle.lora_linear(W, x, i, s)
    e = oracle.AdapterSet(4)          # slot 3 exists but is empty
    for a in s.A:
        e.put(a, s.A[a], s.B[a], s.scale[a])
    i = ids.copy()
    i[0] = 3
    with pytest.raises(ValueError):
        oracle.lora_linear(W, x, i, e)


def test_empty_batch():
    W, x, ids, s = _random_case(14)
    y = oracle.lora_linear(W, x[:0].copy(), ids[:0].copy(), s)
    assert y.shape == (0, W.shape[0])


# ---------------------------------------------------------------- projection form
@pytest.mark.parametrize("seed", [20, 21])
def test_projection_equals_y_times_v(seed):
    W, x, ids, s = _random_case(seed, T=8, h_in=10, h_out=7, ranks=(2, 4, 1))
    v = np.random.Generator(np.random.PCG64(seed)).standard_normal(W.shape[0])
    p = oracle.lora_projection(W, x, ids, s, v)
    np.testing.assert_allclose(p, oracle.lora_linear(W, x, ids, s) @ v, rtol=1e-11, atol=1e-12)


# ---------------------------------------------------------------- the task's first workload
def test_tiny_workload_against_numpy_fp64():
    w = wl.tiny()
    assert w.W.shape == (256, 256) and w.T == 16 and w.n_slots == 4
    assert set(np.unique(w.ids)).issubset({-1, 0, 1, 2, 3})
    y = oracle_of(w)
    Wd, xd = _f64(w.W), _f64(w.x)
    for t in range(w.T):
        e = Wd @ xd[t]
        a = int(w.ids[t])
        if a >= 0:
            ad = w.adapters[a]
            e = e + ad.scale * (_f64(ad.B) @ (_f64(ad.A) @ xd[t]))
        np.testing.assert_allclose(y[t], e, rtol=1e-11, atol=1e-13)
    # the low-rank term is a visible part of the output (a dropped adapter would fail parity)
    base = oracle.lora_linear(w.W, w.x, np.full_like(w.ids, -1), adapter_set(w.n_slots, w.adapters))
    rows = w.ids >= 0
    assert np.sqrt(np.mean((y[rows] - base[rows]) ** 2)) > 0.05 * np.sqrt(np.mean(y ** 2))
