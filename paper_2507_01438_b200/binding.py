"""Python binding of the C-ABI library (``include/edgelora.h``): argument marshalling only.

Every function here has the name of the C entry point it calls.  Tensors are torch CUDA tensors
(used for device memory and streams only); the arithmetic all happens in the CUDA kernels of
``libedgelora.so``.  There is no CPU path: importing works anywhere, but creating a pool without
the compiled library or without a CUDA device raises.
"""
import ctypes
import os
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# EDGELORA_CHECKED=1 in the environment selects the checked build of the library (index tests in the
# kernels, guard zones around its device buffers; `python -m paper_2507_01438_b200.build --checked`)
LIB_PATH = os.path.join(_HERE, "libedgelora_checked.so" if os.environ.get("EDGELORA_CHECKED") == "1"
                        else "libedgelora.so")

OK = 0
ERR_INVALID_ARG, ERR_BAD_SLOT, ERR_RANK_TOO_LARGE, ERR_ARENA_TOO_SMALL = -1, -2, -3, -4
ERR_CUDA, ERR_BAD_ADAPTER_ID, ERR_SLOT_EMPTY, ERR_TIMEOUT, ERR_TOO_MANY_TOKENS = -5, -6, -7, -8, -9
ERR_CACHE_FULL, ERR_BOUNDS = -10, -11
STATUS_BAD_ADAPTER_ID, STATUS_SLOT_EMPTY, STATUS_TIMEOUT, STATUS_BOUNDS = 0x1, 0x2, 0x4, 0x8
OPT_REGIME, OPT_PROFILE, OPT_PDL, OPT_DECODE_SPLITS, OPT_SHRINK_ITEMS, OPT_WAIT_CYCLES = 1, 2, 3, 4, 5, 6
OPT_GATHER_SPLITS, OPT_GATHER_MIN_T, OPT_SHRINK_DEPTH, OPT_FUSED_DECODE = 7, 8, 9, 10
KERNEL_NAMES = ("plan", "shrink_small_decode", "shrink_tiles", "base_gemm")

EXPORTS = (
    "edgelora_pool_bytes_required", "edgelora_pool_create", "edgelora_pool_load_slot",
    "edgelora_pool_evict_slot", "edgelora_pool_wait_loads", "edgelora_lora_linear",
    "edgelora_lora_linear_host", "edgelora_plan_create", "edgelora_plan_destroy",
    "edgelora_plan_build", "edgelora_plan_export", "edgelora_lora_linear_planned",
    "edgelora_pool_plan", "edgelora_pool_sync_status", "edgelora_pool_set_option",
    "edgelora_pool_last_launch", "edgelora_pool_kernel_times", "edgelora_pool_destroy",
    "edgelora_strerror", "edgelora_plan_build_static", "edgelora_lora_linear_host_async",
    "edgelora_pool_host_sync", "edgelora_cache_create", "edgelora_cache_destroy", "edgelora_cache_acquire",
    "edgelora_cache_release", "edgelora_cache_lookup", "edgelora_cache_stats", "edgelora_cache_select",
    "edgelora_router_scores", "edgelora_plan_sync_status", "edgelora_pool_selftest_wait",
    "edgelora_siteset_create", "edgelora_siteset_destroy", "edgelora_siteset_run",
    "edgelora_siteset_run_host", "edgelora_siteset_plan",
    "edgelora_cache_prefill", "edgelora_pool_load_slot_q8", "edgelora_pool_load_slot_pinned", "edgelora_batcher_create", "edgelora_batcher_destroy", "edgelora_batcher_submit",
    "edgelora_batcher_next_batch", "edgelora_batcher_complete_step", "edgelora_batcher_finished",
    "edgelora_build_is_checked", "edgelora_check_guards", "edgelora_weights_decode",
)


class EdgeLoraError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {strerror(code)} ({code})")


class PoolConfig(ctypes.Structure):
    _fields_ = [("h_in", ctypes.c_int32), ("h_out", ctypes.c_int32), ("n_slots", ctypes.c_int32),
                ("max_rank", ctypes.c_int32), ("max_tokens", ctypes.c_int32),
                ("flags", ctypes.c_uint32), ("arena_dev", ctypes.c_void_p),
                ("arena_bytes", ctypes.c_size_t)]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libedgelora.so (built in-tree by ``python -m paper_2507_01438_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                           "`python -m paper_2507_01438_b200.build` (needs nvcc); there is no fallback")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, cp = ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER
    L.edgelora_pool_bytes_required.argtypes = [cp(PoolConfig), cp(ctypes.c_size_t)]
    L.edgelora_pool_create.argtypes = [cp(PoolConfig), cp(vp)]
    L.edgelora_pool_load_slot.argtypes = [vp, i32, i32, ctypes.c_float, vp, vp]
    L.edgelora_pool_evict_slot.argtypes = [vp, i32]
    L.edgelora_pool_load_slot_q8.argtypes = [vp, i32, i32, ctypes.c_float, vp, vp]
    L.edgelora_pool_load_slot_pinned.argtypes = [vp, i32, i32, ctypes.c_float, vp, vp]
    L.edgelora_pool_wait_loads.argtypes = [vp]
    L.edgelora_lora_linear.argtypes = [vp, vp, vp, vp, i32, vp, vp]
    L.edgelora_lora_linear_host.argtypes = [vp, vp, vp, vp, i32, vp, vp]
    L.edgelora_lora_linear_host_async.argtypes = [vp, vp, vp, vp, i32, vp, vp]
    L.edgelora_pool_host_sync.argtypes = [vp]
    i64 = ctypes.c_int64
    L.edgelora_cache_create.argtypes = [i32, i32, cp(vp)]
    L.edgelora_cache_destroy.argtypes = [vp]
    L.edgelora_cache_acquire.argtypes = [vp, i64, i32, cp(i32), cp(i32), cp(i64)]
    L.edgelora_cache_release.argtypes = [vp, i64]
    L.edgelora_cache_prefill.argtypes = [vp, vp, i32, vp]
    L.edgelora_router_scores.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp]
    L.edgelora_cache_select.argtypes = [vp, vp, i32, i32, i32, cp(i64), cp(i32), cp(i32), cp(i64)]
    L.edgelora_cache_lookup.argtypes = [vp, i64, cp(i32)]
    L.edgelora_cache_stats.argtypes = [vp, cp(i64), cp(i64), cp(i64), cp(i32)]
    f64 = ctypes.c_double
    L.edgelora_batcher_create.argtypes = [i32, i32, i32, vp, cp(vp)]
    L.edgelora_batcher_destroy.argtypes = [vp]
    L.edgelora_batcher_submit.argtypes = [vp, i64, f64, i32, i32, vp]
    L.edgelora_batcher_next_batch.argtypes = [vp, i32, vp, vp, cp(i32), cp(i32), vp, vp, cp(i32), cp(f64)]
    L.edgelora_batcher_complete_step.argtypes = [vp, f64]
    L.edgelora_batcher_finished.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, cp(i32)]
    L.edgelora_plan_create.argtypes = [i32, i32, cp(vp)]
    L.edgelora_plan_destroy.argtypes = [vp]
    L.edgelora_plan_build.argtypes = [vp, vp, i32, vp]
    L.edgelora_plan_export.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp]
    L.edgelora_lora_linear_planned.argtypes = [vp, vp, vp, vp, i32, vp, vp]
    L.edgelora_plan_build_static.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
    L.edgelora_pool_plan.argtypes = [vp, cp(vp)]
    L.edgelora_siteset_create.argtypes = [i32, cp(vp), cp(vp), cp(i32), i32, i32, cp(vp)]
    L.edgelora_siteset_destroy.argtypes = [vp]
    L.edgelora_siteset_run.argtypes = [vp, cp(vp), vp, i32, cp(vp), vp]
    L.edgelora_siteset_run_host.argtypes = [vp, cp(vp), vp, i32, cp(vp), vp]
    L.edgelora_siteset_plan.argtypes = [vp, cp(vp)]
    L.edgelora_plan_sync_status.argtypes = [vp, vp, cp(ctypes.c_uint32)]
    L.edgelora_pool_selftest_wait.argtypes = [vp, vp]
    L.edgelora_build_is_checked.argtypes = []
    L.edgelora_weights_decode.argtypes = [i32, vp, i32, i32, vp, vp]
    L.edgelora_check_guards.argtypes = []
    L.edgelora_pool_sync_status.argtypes = [vp, cp(ctypes.c_uint32)]
    L.edgelora_pool_set_option.argtypes = [vp, i32, i32]
    L.edgelora_pool_last_launch.argtypes = [vp, vp]
    L.edgelora_pool_kernel_times.argtypes = [vp, vp, vp, i32]
    L.edgelora_pool_destroy.argtypes = [vp]
    L.edgelora_strerror.argtypes = [ctypes.c_int]
    L.edgelora_strerror.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name != "edgelora_strerror":
            getattr(L, name).restype = ctypes.c_int
    _lib = L
    return L


def strerror(code: int) -> str:
    return lib().edgelora_strerror(code).decode()


def _check(rc: int, what: str) -> None:
    if rc != OK:
        raise EdgeLoraError(rc, what)


def _stream_ptr(stream) -> int:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream) if hasattr(stream, "cuda_stream") else int(stream)


def _dev_ptr(t, dtype_bytes: int, what: str) -> int:
    assert t.is_cuda and t.is_contiguous() and t.element_size() == dtype_bytes, what
    return t.data_ptr()


def edgelora_pool_bytes_required(h_in, h_out, n_slots, max_rank) -> int:
    cfg = PoolConfig(h_in, h_out, n_slots, max_rank, 0, 0, None, 0)
    out = ctypes.c_size_t(0)
    _check(lib().edgelora_pool_bytes_required(ctypes.byref(cfg), ctypes.byref(out)), "pool_bytes_required")
    return out.value


FLAG_A_Q8 = 1


def edgelora_pool_create(h_in, h_out, n_slots, max_rank, max_tokens=0, arena=None, flags=0) -> int:
    """Returns the opaque pool handle.  ``arena`` may be a torch CUDA tensor lent for the slot blocks."""
    cfg = PoolConfig(h_in, h_out, n_slots, max_rank, max_tokens, flags,
                     arena.data_ptr() if arena is not None else None,
                     arena.numel() * arena.element_size() if arena is not None else 0)
    out = ctypes.c_void_p()
    _check(lib().edgelora_pool_create(ctypes.byref(cfg), ctypes.byref(out)), "pool_create")
    return out.value


def edgelora_pool_load_slot(pool, slot: int, rank: int, scale: float, A: np.ndarray, B: np.ndarray) -> None:
    """A: uint16 [rank, h_in], B: uint16 [h_out, rank] (bf16 bit patterns, host memory)."""
    A = np.ascontiguousarray(A, dtype=np.uint16)
    B = np.ascontiguousarray(B, dtype=np.uint16)
    _check(lib().edgelora_pool_load_slot(pool, slot, rank, scale, A.ctypes.data, B.ctypes.data), "pool_load_slot")


def edgelora_pool_load_slot_pinned(pool, slot: int, rank: int, scale: float, A_pinned, B_pinned) -> int:
    """A_pinned / B_pinned: page-locked CPU tensors (int16 view of bf16) in the block layout; they
    must stay alive until the load has landed.  Returns the C return code."""
    return lib().edgelora_pool_load_slot_pinned(pool, slot, rank, scale, A_pinned.data_ptr(), B_pinned.data_ptr())


def edgelora_pool_load_slot_q8(pool, slot: int, rank: int, scale: float, A_q8: np.ndarray, B_q8: np.ndarray) -> None:
    """A_q8: uint8 [rank, h_in / 32, 34], B_q8: uint8 [h_out, ceil(rank / 32), 34] (Q8_0 blocks, host)."""
    A_q8 = np.ascontiguousarray(A_q8, dtype=np.uint8)
    B_q8 = np.ascontiguousarray(B_q8, dtype=np.uint8)
    _check(lib().edgelora_pool_load_slot_q8(pool, slot, rank, scale, A_q8.ctypes.data, B_q8.ctypes.data),
           "pool_load_slot_q8")


def edgelora_pool_evict_slot(pool, slot: int) -> None:
    _check(lib().edgelora_pool_evict_slot(pool, slot), "pool_evict_slot")


def edgelora_pool_wait_loads(pool) -> None:
    _check(lib().edgelora_pool_wait_loads(pool), "pool_wait_loads")


def edgelora_lora_linear(pool, W, x, adapter_id, y, stream=None) -> None:
    """W [h_out,h_in], x [T,h_in], y [T,h_out]: torch bf16 CUDA tensors; adapter_id: int32 [T]."""
    T = int(x.shape[0])
    _check(lib().edgelora_lora_linear(pool, _dev_ptr(W, 2, "W"), _dev_ptr(x, 2, "x") if T else None,
                                      _dev_ptr(adapter_id, 4, "ids") if T else None, T,
                                      _dev_ptr(y, 2, "y") if T else None, _stream_ptr(stream)),
           "lora_linear")


def edgelora_lora_linear_planned(pool, plan, W, x, y, stream=None) -> None:
    T = int(x.shape[0])
    _check(lib().edgelora_lora_linear_planned(pool, plan, _dev_ptr(W, 2, "W"), _dev_ptr(x, 2, "x"), T,
                                              _dev_ptr(y, 2, "y"), _stream_ptr(stream)),
           "lora_linear_planned")


def edgelora_lora_linear_host(pool, W, x_host: np.ndarray, ids_host: np.ndarray, y_host: np.ndarray,
                              stream=None) -> None:
    """Host buffers in and out (numpy uint16 / int32); W stays a device tensor."""
    assert x_host.dtype == np.uint16 and ids_host.dtype == np.int32 and y_host.dtype == np.uint16
    assert x_host.flags.c_contiguous and ids_host.flags.c_contiguous and y_host.flags.c_contiguous
    T = int(x_host.shape[0])
    _check(lib().edgelora_lora_linear_host(pool, _dev_ptr(W, 2, "W"), x_host.ctypes.data,
                                           ids_host.ctypes.data, T, y_host.ctypes.data,
                                           _stream_ptr(stream)), "lora_linear_host")


def edgelora_lora_linear_host_async(pool, W, x_host, ids_host, y_host, stream=None) -> None:
    """Pipelined host-buffer call; the arguments are page-locked CPU tensors (torch, pin_memory) or
    numpy arrays of uint16 / int32 / uint16 and must stay alive until ``edgelora_pool_host_sync``."""
    def ptr(a):
        return a.data_ptr() if hasattr(a, "data_ptr") else a.ctypes.data
    T = int(x_host.shape[0])
    _check(lib().edgelora_lora_linear_host_async(pool, _dev_ptr(W, 2, "W"), ptr(x_host), ptr(ids_host), T,
                                                 ptr(y_host), _stream_ptr(stream)), "lora_linear_host_async")


def edgelora_pool_host_sync(pool) -> None:
    _check(lib().edgelora_pool_host_sync(pool), "pool_host_sync")


def edgelora_plan_create(max_tokens: int, n_slots: int) -> int:
    out = ctypes.c_void_p()
    _check(lib().edgelora_plan_create(max_tokens, n_slots, ctypes.byref(out)), "plan_create")
    return out.value


def edgelora_plan_destroy(plan) -> None:
    _check(lib().edgelora_plan_destroy(plan), "plan_destroy")


def edgelora_plan_build(plan, adapter_id, stream=None) -> None:
    T = int(adapter_id.shape[0])
    _check(lib().edgelora_plan_build(plan, _dev_ptr(adapter_id, 4, "ids") if T else None, T,
                                     _stream_ptr(stream)), "plan_build")


def edgelora_plan_export(plan, T: int, stream=None) -> dict:
    """Host copies of the last built plan, trimmed to their true lengths."""
    n = max(T, 1)
    arr = {k: np.zeros(n + 1, dtype=np.int32) for k in
           ("ids_valid", "perm", "group_start", "group_adapter", "seg_start", "seg_adapter")}
    counts = np.zeros(2, dtype=np.int32)
    _check(lib().edgelora_plan_export(plan, _stream_ptr(stream), arr["ids_valid"].ctypes.data,
                                      arr["perm"].ctypes.data, arr["group_start"].ctypes.data,
                                      arr["group_adapter"].ctypes.data, arr["seg_start"].ctypes.data,
                                      arr["seg_adapter"].ctypes.data, counts.ctypes.data), "plan_export")
    G, NS = int(counts[0]), int(counts[1])
    return {"ids_valid": arr["ids_valid"][:T].copy(), "perm": arr["perm"][:T].copy(),
            "group_start": arr["group_start"][:G + 1].copy(), "group_adapter": arr["group_adapter"][:G].copy(),
            "seg_start": arr["seg_start"][:NS + 1].copy(), "seg_adapter": arr["seg_adapter"][:NS].copy()}


PLAN_STATIC_MAX_TOKENS = 4096


def edgelora_plan_build_static(adapter_id, n_slots: int, ids_valid, perm, group_start, group_adapter,
                               seg_start, seg_adapter, info, stream=None) -> int:
    """The plan builder for callers that cannot allocate device memory (see the header): every
    array is a caller-owned int32 CUDA tensor ([T] or [T+1]; info is [4]).  Returns the C return
    code instead of raising, so that callers can test the size limit."""
    T = int(adapter_id.shape[0])
    ptr = (lambda t: _dev_ptr(t, 4, "int32 array")) if T else (lambda t: None)
    return lib().edgelora_plan_build_static(ptr(adapter_id), T, n_slots, ptr(ids_valid), ptr(perm),
                                            ptr(group_start), ptr(group_adapter), ptr(seg_start),
                                            ptr(seg_adapter), _dev_ptr(info, 4, "info"),
                                            _stream_ptr(stream))


def _ptr_array(ptrs):
    return (ctypes.c_void_p * len(ptrs))(*[ctypes.c_void_p(p) if p else None for p in ptrs])


def edgelora_siteset_create(pools, Ws, input_of_site, n_inputs: int, max_tokens: int) -> int:
    """pools: pool handles, Ws: bf16 CUDA tensors [h_out, h_in] (kept alive by the caller)."""
    n = len(pools)
    idx = (ctypes.c_int32 * n)(*[int(i) for i in input_of_site])
    out = ctypes.c_void_p()
    _check(lib().edgelora_siteset_create(n, _ptr_array(list(pools)), _ptr_array([_dev_ptr(W, 2, "W") for W in Ws]),
                                         idx, n_inputs, max_tokens, ctypes.byref(out)), "siteset_create")
    return out.value


def edgelora_siteset_destroy(s) -> None:
    _check(lib().edgelora_siteset_destroy(s), "siteset_destroy")


def edgelora_siteset_run(s, xs, adapter_id, ys, stream=None) -> None:
    """xs: one bf16 CUDA tensor per input, ys: one per site, adapter_id: int32 CUDA tensor [T]."""
    T = int(adapter_id.shape[0])
    _check(lib().edgelora_siteset_run(s, _ptr_array([_dev_ptr(x, 2, "x") for x in xs]),
                                      _dev_ptr(adapter_id, 4, "ids") if T else None, T,
                                      _ptr_array([_dev_ptr(y, 2, "y") for y in ys]), _stream_ptr(stream)),
           "siteset_run")


def edgelora_siteset_run_host(s, xs_host, ids_host, ys_host, stream=None) -> None:
    """Host buffers (pinned torch CPU tensors or numpy arrays); ys_host entries may be None."""
    def ptr(a):
        return None if a is None else (a.data_ptr() if hasattr(a, "data_ptr") else a.ctypes.data)
    T = int(ids_host.shape[0])
    _check(lib().edgelora_siteset_run_host(s, _ptr_array([ptr(x) for x in xs_host]), ptr(ids_host), T,
                                           _ptr_array([ptr(y) for y in ys_host]), _stream_ptr(stream)),
           "siteset_run_host")


def edgelora_siteset_plan(s) -> int:
    out = ctypes.c_void_p()
    _check(lib().edgelora_siteset_plan(s, ctypes.byref(out)), "siteset_plan")
    return out.value


def edgelora_pool_plan(pool) -> int:
    out = ctypes.c_void_p()
    _check(lib().edgelora_pool_plan(pool, ctypes.byref(out)), "pool_plan")
    return out.value


def edgelora_pool_sync_status(pool):
    """Returns (return code, status bits); does not raise on device-detected conditions."""
    bits = ctypes.c_uint32(0)
    rc = lib().edgelora_pool_sync_status(pool, ctypes.byref(bits))
    if rc == ERR_CUDA or rc == ERR_INVALID_ARG:
        raise EdgeLoraError(rc, "pool_sync_status")
    return rc, bits.value


def edgelora_plan_sync_status(plan, stream=None):
    """Returns (return code, status bits) of a plan built with edgelora_plan_build; clears the bits."""
    bits = ctypes.c_uint32(0)
    rc = lib().edgelora_plan_sync_status(plan, _stream_ptr(stream), ctypes.byref(bits))
    if rc == ERR_CUDA or rc == ERR_INVALID_ARG:
        raise EdgeLoraError(rc, "plan_sync_status")
    return rc, bits.value


WEIGHTS_Q8_0, WEIGHTS_Q4_0 = 0, 1


def edgelora_weights_decode(fmt: int, W_blocks, h_out: int, h_in: int, W, stream=None) -> None:
    """W_blocks: torch uint8 CUDA tensor [h_out, h_in / 32, 34 or 18]; W: torch bf16 CUDA tensor [h_out, h_in]."""
    _check(lib().edgelora_weights_decode(fmt, W_blocks.data_ptr(), h_out, h_in, _dev_ptr(W, 2, "W"),
                                         _stream_ptr(stream)), "weights_decode")


def edgelora_build_is_checked() -> bool:
    return bool(lib().edgelora_build_is_checked())


def edgelora_check_guards() -> int:
    """EDGELORA_OK, or ERR_BOUNDS when something wrote outside one of the library's device buffers
    (checked build; the normal build has no guard zones and always answers OK)."""
    return lib().edgelora_check_guards()


def edgelora_pool_selftest_wait(pool, stream=None) -> int:
    """Returns the C return code (INVALID_ARG unless the pool's wait limit was lowered first)."""
    return lib().edgelora_pool_selftest_wait(pool, _stream_ptr(stream))


def edgelora_pool_set_option(pool, option: int, value: int) -> None:
    _check(lib().edgelora_pool_set_option(pool, option, value), "pool_set_option")


def edgelora_pool_last_launch(pool) -> dict:
    info = np.zeros(8, dtype=np.int64)
    _check(lib().edgelora_pool_last_launch(pool, info.ctypes.data), "pool_last_launch")
    return {"launches": int(info[0]), "regime": {1: "decode", 2: "prefill"}.get(int(info[1]), "none"),
            "gemm_grid": int(info[2]), "split_k": int(info[3]), "stages": int(info[4]),
            "n_tile": int(info[5]), "total_launches": int(info[6])}


def edgelora_pool_kernel_times(pool, reset: bool = True) -> dict:
    ms = np.zeros(5, dtype=np.float64)
    n = np.zeros(5, dtype=np.int64)
    _check(lib().edgelora_pool_kernel_times(pool, ms.ctypes.data, n.ctypes.data, 1 if reset else 0),
           "pool_kernel_times")
    return {k: {"ms": float(ms[i]), "launches": int(n[i])} for i, k in enumerate(KERNEL_NAMES)}


def edgelora_pool_destroy(pool) -> None:
    _check(lib().edgelora_pool_destroy(pool), "pool_destroy")


CACHE_LRU, CACHE_LFU = 0, 1
ERR_CACHE_FULL = -10


def edgelora_cache_create(n_blocks: int, policy: int = CACHE_LRU) -> int:
    out = ctypes.c_void_p()
    _check(lib().edgelora_cache_create(n_blocks, policy, ctypes.byref(out)), "cache_create")
    return out.value


def edgelora_cache_destroy(cache) -> None:
    _check(lib().edgelora_cache_destroy(cache), "cache_destroy")


def edgelora_cache_acquire(cache, key: int, pin: bool = False):
    """Returns (block, hit, evicted key or -1)."""
    slot, hit, ev = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int64()
    _check(lib().edgelora_cache_acquire(cache, key, 1 if pin else 0, ctypes.byref(slot), ctypes.byref(hit),
                                        ctypes.byref(ev)), "cache_acquire")
    return slot.value, bool(hit.value), ev.value


def edgelora_cache_select(cache, scores: np.ndarray, k: int, pin: bool = False):
    """Returns (adapter, block, hit, evicted key or -1); scores is a float32 numpy array."""
    assert scores.dtype == np.float32 and scores.flags.c_contiguous
    key, slot, hit, ev = ctypes.c_int64(), ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int64()
    _check(lib().edgelora_cache_select(cache, scores.ctypes.data, int(scores.shape[0]), k, 1 if pin else 0,
                                       ctypes.byref(key), ctypes.byref(slot), ctypes.byref(hit), ctypes.byref(ev)),
           "cache_select")
    return key.value, slot.value, bool(hit.value), ev.value


def edgelora_router_scores(Wr, bias, h, scores=None, stream=None):
    """Wr [n, hidden], h [B, hidden] bf16 device tensors, bias [n] float32 device tensor or None."""
    import torch
    n, hidden = int(Wr.shape[0]), int(Wr.shape[1])
    Bn = int(h.shape[0])
    if scores is None:
        scores = torch.empty((Bn, n), dtype=torch.float32, device=Wr.device)
    _check(lib().edgelora_router_scores(_dev_ptr(Wr, 2, "Wr"), bias.data_ptr() if bias is not None else None,
                                        _dev_ptr(h, 2, "h") if Bn else None, Bn, n, hidden, scores.data_ptr(),
                                        _stream_ptr(stream)), "router_scores")
    return scores


def edgelora_cache_prefill(cache, keys) -> np.ndarray:
    """Makes `keys` resident in an empty cache before serving starts; returns their blocks."""
    k = np.ascontiguousarray(keys, dtype=np.int64)
    blocks = np.zeros(len(k), dtype=np.int32)
    _check(lib().edgelora_cache_prefill(cache, k.ctypes.data, len(k), blocks.ctypes.data), "cache_prefill")
    return blocks


def edgelora_cache_release(cache, key: int) -> None:
    _check(lib().edgelora_cache_release(cache, key), "cache_release")


def edgelora_cache_lookup(cache, key: int) -> int:
    slot = ctypes.c_int32()
    _check(lib().edgelora_cache_lookup(cache, key, ctypes.byref(slot)), "cache_lookup")
    return slot.value


def edgelora_cache_stats(cache) -> dict:
    h, m, e, r = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int32()
    _check(lib().edgelora_cache_stats(cache, ctypes.byref(h), ctypes.byref(m), ctypes.byref(e), ctypes.byref(r)),
           "cache_stats")
    return {"hits": h.value, "misses": m.value, "evictions": e.value, "resident": r.value}


class Pool:
    """Small convenience wrapper: owns a pool handle and loads a workload's adapters."""

    def __init__(self, h_in, h_out, n_slots, max_rank, max_tokens=0, arena=None, flags=0):
        self.handle = edgelora_pool_create(h_in, h_out, n_slots, max_rank, max_tokens, arena, flags)
        self.h_in, self.h_out, self.n_slots, self.max_rank = h_in, h_out, n_slots, max_rank
        self._arena = arena

    def load(self, slot, A, B, scale):
        edgelora_pool_load_slot(self.handle, slot, int(A.shape[0]), float(scale), A, B)

    def load_all(self, adapters: dict):
        for slot, ad in adapters.items():
            self.load(int(slot), ad.A, ad.B, ad.scale)
        edgelora_pool_wait_loads(self.handle)

    def linear(self, W, x, ids, y=None, stream=None):
        import torch
        if y is None:
            y = torch.empty((x.shape[0], self.h_out), dtype=torch.bfloat16, device=x.device)
        edgelora_lora_linear(self.handle, W, x, ids, y, stream)
        return y

    def status(self):
        return edgelora_pool_sync_status(self.handle)

    def close(self):
        if self.handle:
            edgelora_pool_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def edgelora_batcher_create(n_slots: int, max_batch_tokens: int, top_k: int, cache) -> int:
    out = ctypes.c_void_p()
    _check(lib().edgelora_batcher_create(n_slots, max_batch_tokens, top_k, cache, ctypes.byref(out)),
           "batcher_create")
    return out.value


def edgelora_batcher_destroy(batcher) -> None:
    _check(lib().edgelora_batcher_destroy(batcher), "batcher_destroy")


def edgelora_batcher_submit(batcher, request_id: int, arrival: float, in_len: int, out_len: int, candidates) -> None:
    c = np.ascontiguousarray(candidates, dtype=np.int64)
    _check(lib().edgelora_batcher_submit(batcher, request_id, float(arrival), int(in_len), int(out_len),
                                         c.ctypes.data), "batcher_submit")


def edgelora_batcher_next_batch(batcher, max_batch_tokens: int, n_slots: int):
    """None when every request is finished, else a dict: now, token_block, token_slot, n_decode, loads."""
    tb = np.zeros(max_batch_tokens, dtype=np.int32)
    ts = np.zeros(max_batch_tokens, dtype=np.int32)
    lk = np.zeros(n_slots, dtype=np.int64)
    lb = np.zeros(n_slots, dtype=np.int32)
    n, nd, nl, now = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32(), ctypes.c_double()
    rc = lib().edgelora_batcher_next_batch(batcher, max_batch_tokens, tb.ctypes.data, ts.ctypes.data,
                                           ctypes.byref(n), ctypes.byref(nd), lk.ctypes.data, lb.ctypes.data,
                                           ctypes.byref(nl), ctypes.byref(now))
    if rc < 0:
        raise EdgeLoraError(rc, "batcher_next_batch")
    if rc == 0:
        return None
    return {"now": now.value, "token_block": tb[:n.value], "token_slot": ts[:n.value], "n_decode": nd.value,
            "loads": [(int(k), int(b)) for k, b in zip(lk[:nl.value], lb[:nl.value])]}


def edgelora_batcher_complete_step(batcher, seconds: float) -> None:
    _check(lib().edgelora_batcher_complete_step(batcher, float(seconds)), "batcher_complete_step")


def edgelora_batcher_finished(batcher) -> dict:
    n = ctypes.c_int32()
    _check(lib().edgelora_batcher_finished(batcher, 0, None, None, None, None, None, None, ctypes.byref(n)),
           "batcher_finished")
    k = n.value
    out = {"id": np.zeros(k, np.int64), "arrival": np.zeros(k), "first_token": np.zeros(k),
           "finish": np.zeros(k), "adapter": np.zeros(k, np.int64), "hit": np.zeros(k, np.int32)}
    if k:
        _check(lib().edgelora_batcher_finished(batcher, k, out["id"].ctypes.data, out["arrival"].ctypes.data,
                                               out["first_token"].ctypes.data, out["finish"].ctypes.data,
                                               out["adapter"].ctypes.data, out["hit"].ctypes.data,
                                               ctypes.byref(n)), "batcher_finished")
    return out
