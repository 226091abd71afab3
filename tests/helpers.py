"""Shared test helpers: the parity comparator and conversion of workloads to oracle inputs."""
import json
import os

import numpy as np

import oracle
from paper_2507_01438_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")

# Tolerance fixed by the benchmark spec (bf16 in, fp32 accumulate, bf16 out):
#   |y_gpu - y_ref| <= RTOL * |y_ref| + ATOL_RMS * rms(y_ref), rms over the compared block.
RTOL = 1e-2
ATOL_RMS = 1e-2


def golden(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return json.load(f)


def bits(a):
    """Small exactly-representable numbers -> bf16 bit patterns."""
    a = np.asarray(a, dtype=np.float32)
    b = wl.f32_to_bf16_bits(a)
    assert np.array_equal(wl.bf16_bits_to_f32(b), a), "value not exactly representable in bf16"
    return b


def adapter_set(n_slots, adapters) -> "oracle.AdapterSet":
    s = oracle.AdapterSet(n_slots)
    for a, ad in adapters.items():
        s.put(int(a), ad.A, ad.B, ad.scale)
    return s


def oracle_of(w: "wl.Workload", rows=None) -> np.ndarray:
    x, ids = w.x, w.ids
    if rows is not None:
        x = np.ascontiguousarray(x[rows])
        ids = np.ascontiguousarray(ids[rows])
    return oracle.lora_linear(w.W, x, ids, adapter_set(w.n_slots, w.adapters))


def parity_violations(y_test: np.ndarray, y_ref: np.ndarray):
    """Returns (n_bad, worst_ratio): elements outside the tolerance, and max err/allowed."""
    y_test = np.asarray(y_test, dtype=np.float64)
    y_ref = np.asarray(y_ref, dtype=np.float64)
    assert y_test.shape == y_ref.shape
    if y_ref.size == 0:
        return 0, 0.0
    rms = float(np.sqrt(np.mean(y_ref * y_ref)))
    allowed = RTOL * np.abs(y_ref) + ATOL_RMS * rms
    err = np.abs(y_test - y_ref)
    if rms == 0.0:
        return int(np.count_nonzero(err > 0)), float(err.max())
    bad = err > allowed
    return int(np.count_nonzero(bad)), float((err / allowed).max())


def assert_parity(y_test, y_ref, what=""):
    assert np.all(np.isfinite(np.asarray(y_test, dtype=np.float64))), f"{what}: non-finite output"
    n_bad, worst = parity_violations(y_test, y_ref)
    assert n_bad == 0, f"{what}: {n_bad} elements outside tolerance, worst err/allowed = {worst:.3f}"
