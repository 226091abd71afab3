"""Helpers for the GPU parity tests: move workloads to the device and run them through the C ABI."""
import numpy as np

from paper_2507_01438_b200 import binding as B
from paper_2507_01438_b200 import workloads as wl


SENTINEL = 0x7FA5   # bfloat16 bits of a NaN payload that no result takes


def to_dev_bf16(bits: np.ndarray):
    import torch
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def from_dev_bf16(t) -> np.ndarray:
    import torch
    return wl.bf16_bits_to_f32(t.view(torch.int16).cpu().numpy().view(np.uint16))


def make_pool(w: "wl.Workload", max_tokens=0) -> "B.Pool":
    pool = B.Pool(w.h_in, w.h_out, w.n_slots, w.max_rank, max_tokens=max_tokens or max(w.T, 1))
    pool.load_all(w.adapters)
    return pool


def run_gpu(w: "wl.Workload", regime: int = 0, pool=None, return_plan=False, options=None):
    """Runs the layer once; returns y as fp32 numpy [T, h_out] (and the exported plan)."""
    import torch
    own = pool is None
    if own:
        pool = make_pool(w)
    try:
        B.edgelora_pool_set_option(pool.handle, B.OPT_REGIME, regime)
        for opt, value in (options or {}).items():
            B.edgelora_pool_set_option(pool.handle, opt, value)
        W = to_dev_bf16(w.W)
        x = to_dev_bf16(w.x)
        ids = torch.from_numpy(w.ids).cuda()
        # y sits between two sentinel rows (a bit pattern no result takes): writes outside y show there
        framed = torch.full((w.T + 2, w.h_out), float("nan"), dtype=torch.bfloat16, device="cuda")
        framed[0].view(torch.int16).fill_(SENTINEL)
        framed[-1].view(torch.int16).fill_(SENTINEL)
        y = framed[1:w.T + 1]
        B.edgelora_lora_linear(pool.handle, W, x, ids, y)
        rc, bits = pool.status()
        assert rc == 0 and bits == 0, f"status rc={rc} bits={bits:#x}"
        edges = framed[[0, -1]].view(torch.int16).cpu().numpy()
        assert (edges == SENTINEL).all(), "the rows in front of or behind y were written"
        assert B.edgelora_check_guards() == B.OK       # guard zones of the library's buffers (checked build)
        out = from_dev_bf16(y)
        if return_plan:
            plan = B.edgelora_plan_export(B.edgelora_pool_plan(pool.handle), w.T)
            return out, plan
        return out
    finally:
        if own:
            pool.close()
