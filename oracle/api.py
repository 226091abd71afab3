"""ctypes marshalling for the C oracle (test infrastructure; see lora_oracle.c).

No arithmetic of the method happens here: arrays go in, fp64 / int32 arrays
come out.
"""
import ctypes
import os
from dataclasses import dataclass, field
from typing import Dict, Optional

import numpy as np

from . import build as _build

_LIB = None


def lib_path() -> str:
    return _build.build()


def _lib():
    global _LIB
    if _LIB is None:
        lib = ctypes.CDLL(lib_path())
        pp = ctypes.POINTER(ctypes.c_void_p)
        lib.oracle_lora_linear.restype = ctypes.c_int
        lib.oracle_lora_linear.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
            pp, pp, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        lib.oracle_lora_projection.restype = ctypes.c_int
        lib.oracle_lora_projection.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
            pp, pp, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        lib.oracle_segments.restype = ctypes.c_int32
        lib.oracle_segments.argtypes = [ctypes.c_void_p, ctypes.c_int32,
                                        ctypes.c_void_p, ctypes.c_void_p]
        lib.oracle_groups.restype = ctypes.c_int32
        lib.oracle_groups.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32,
                                      ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        _LIB = lib
    return _LIB


def num_threads() -> int:
    """Threads the OpenMP loops will use (affinity mask, capped by OMP_NUM_THREADS)."""
    n = len(os.sched_getaffinity(0))
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        try:
            n = min(n, int(env.split(",")[0]))
        except ValueError:
            pass
    return n


@dataclass
class AdapterSet:
    """Slot-indexed adapters as the oracle sees them: dense, unpadded bf16 bits.

    ``A[a]`` is uint16 [rank, h_in]; ``B[a]`` is uint16 [h_out, rank]; slots not
    present are empty.
    """
    n_slots: int
    A: Dict[int, np.ndarray] = field(default_factory=dict)
    B: Dict[int, np.ndarray] = field(default_factory=dict)
    scale: Dict[int, float] = field(default_factory=dict)

    def put(self, slot: int, A: np.ndarray, B: np.ndarray, scale: float) -> None:
        assert A.dtype == np.uint16 and B.dtype == np.uint16
        assert A.ndim == 2 and B.ndim == 2 and A.shape[0] == B.shape[1]
        self.A[slot] = np.ascontiguousarray(A)
        self.B[slot] = np.ascontiguousarray(B)
        self.scale[slot] = float(scale)

    def _tables(self):
        S = self.n_slots
        Ap = (ctypes.c_void_p * S)()
        Bp = (ctypes.c_void_p * S)()
        rank = np.zeros(S, dtype=np.int32)
        scale = np.zeros(S, dtype=np.float32)
        for a in self.A:
            Ap[a] = self.A[a].ctypes.data
            Bp[a] = self.B[a].ctypes.data
            rank[a] = self.A[a].shape[0]
            scale[a] = self.scale[a]
        return Ap, Bp, rank, scale


def _check(W, x, ids):
    assert W.dtype == np.uint16 and x.dtype == np.uint16 and ids.dtype == np.int32
    assert W.flags.c_contiguous and x.flags.c_contiguous and ids.flags.c_contiguous
    h_out, h_in = W.shape
    T = x.shape[0]
    assert x.shape == (T, h_in) and ids.shape == (T,)
    return T, h_in, h_out


def lora_linear(W: np.ndarray, x: np.ndarray, ids: np.ndarray,
                adapters: AdapterSet) -> np.ndarray:
    """fp64 [T, h_out] result of the per-token definition; raises on a bad id."""
    T, h_in, h_out = _check(W, x, ids)
    Ap, Bp, rank, scale = adapters._tables()
    for a in adapters.A:
        assert adapters.A[a].shape[1] == h_in and adapters.B[a].shape[0] == h_out
    y = np.empty((T, h_out), dtype=np.float64)
    rc = _lib().oracle_lora_linear(
        W.ctypes.data, x.ctypes.data, ids.ctypes.data, T, h_in, h_out,
        adapters.n_slots, Ap, Bp, rank.ctypes.data, scale.ctypes.data, y.ctypes.data)
    if rc != 0:
        raise ValueError("adapter id out of range or names an empty slot")
    return y


def lora_projection(W: np.ndarray, x: np.ndarray, ids: np.ndarray,
                    adapters: AdapterSet, v: np.ndarray) -> np.ndarray:
    """fp64 [T]: p[t] = sum_j v[j] * y[t][j], computed without forming y."""
    T, h_in, h_out = _check(W, x, ids)
    assert v.dtype == np.float64 and v.shape == (h_out,)
    Ap, Bp, rank, scale = adapters._tables()
    max_rank = max(1, int(rank.max()) if rank.size else 1)
    vW = np.empty(h_in, dtype=np.float64)
    vB = np.empty((adapters.n_slots, max_rank), dtype=np.float64)
    p = np.empty(T, dtype=np.float64)
    rc = _lib().oracle_lora_projection(
        W.ctypes.data, x.ctypes.data, ids.ctypes.data, T, h_in, h_out,
        adapters.n_slots, Ap, Bp, rank.ctypes.data, scale.ctypes.data,
        np.ascontiguousarray(v).ctypes.data, max_rank, vW.ctypes.data,
        vB.ctypes.data, p.ctypes.data)
    if rc != 0:
        raise ValueError("adapter id out of range or names an empty slot")
    return p


def segments(ids: np.ndarray):
    """(seg_start[n_seg+1], seg_adapter[n_seg]) -- maximal runs of equal id."""
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    T = ids.shape[0]
    start = np.empty(T + 1, dtype=np.int32)
    adapter = np.empty(max(T, 1), dtype=np.int32)
    n = _lib().oracle_segments(ids.ctypes.data, T, start.ctypes.data, adapter.ctypes.data)
    return start[: n + 1].copy(), adapter[:n].copy()


def groups(ids: np.ndarray, n_slots: int):
    """(perm[T], group_start[G+1], group_adapter[G]) -- ids ascending, -1 first, stable."""
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    T = ids.shape[0]
    perm = np.empty(max(T, 1), dtype=np.int32)
    start = np.empty(T + 2, dtype=np.int32)
    adapter = np.empty(max(T, 1), dtype=np.int32)
    n = _lib().oracle_groups(ids.ctypes.data, T, n_slots, perm.ctypes.data,
                             start.ctypes.data, adapter.ctypes.data)
    if n < 0:
        raise ValueError("adapter id out of range")
    return perm[:T].copy(), start[: n + 1].copy(), adapter[:n].copy()
