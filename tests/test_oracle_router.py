"""Pins of the router-head oracle (paper Section 3.2: scores in [0, 1], one per adapter)."""
import math

import numpy as np

from oracle.router import router_scores
from paper_2507_01438_b200 import workloads as wl


def bf16(a):
    return wl.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def test_hand_computed_values():
    # logits ln 3, -ln 3, 0, 2 by construction: sigmoid gives 3/4, 1/4, 1/2, 1/(1+e^-2)
    h = bf16([[1.0, 2.0, 0.0, -1.0]])
    Wr = bf16([[0.0, 0.0, 5.0, 0.0], [0.0, 0.0, 0.0, 0.0], [0.0, 0.0, -7.0, 0.0], [1.0, 0.5, 0.0, 0.0]])
    bias = [math.log(3.0), -math.log(3.0), 0.0, 0.0]
    s = router_scores(Wr, bias, h)
    assert np.allclose(s[0], [0.75, 0.25, 0.5, 1.0 / (1.0 + math.exp(-2.0))], rtol=0, atol=1e-15)


def test_dot_product_orientation_and_bias():
    # W_r[j] picks component j of h: a transposed operand or a dropped bias fails
    h = bf16([[0.5, -1.5, 2.0], [3.0, 0.25, -0.75]])
    Wr = bf16(np.eye(3))
    bias = np.array([0.125, 0.0, -0.5])
    s = router_scores(Wr, bias, h)
    logits = np.log(s / (1.0 - s))
    assert np.allclose(logits, np.array([[0.625, -1.5, 1.5], [3.125, 0.25, -1.25]]), atol=1e-12)


def test_range_symmetry_and_saturation():
    rng = np.random.Generator(np.random.PCG64(1))
    Wr = wl.normal_bf16(rng, (50, 64), 1.0)
    h = wl.normal_bf16(rng, (7, 64), 1.0)
    s = router_scores(Wr, None, h)
    assert np.all(s > 0) and np.all(s < 1)
    neg = router_scores(Wr ^ np.uint16(0x8000), None, h)       # sign bit flipped: -W_r
    assert np.allclose(s + neg, 1.0, atol=1e-15)                # sigmoid(-v) = 1 - sigmoid(v)
    big = router_scores(bf16(np.full((1, 64), 100.0)), None, bf16(np.ones((1, 64))))
    assert big[0, 0] == 1.0 and np.isfinite(router_scores(bf16(np.full((1, 64), -100.0)), None, bf16(np.ones((1, 64))))[0, 0])
