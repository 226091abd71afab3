"""Small decode batches in one launch (shrink teams inside the base product's grid), through the C ABI
against the CPU oracle: the same cases with the one-launch path on and off, the number of launches
each takes, chains of calls whose input is the previous call's output under every launch mode, and
the status bits of the one-launch path.
"""
import numpy as np
import pytest

from paper_2507_01438_b200 import binding as B
from paper_2507_01438_b200 import workloads as wl
from helpers import assert_parity, oracle_of
from gpu_helpers import from_dev_bf16, make_pool, run_gpu, to_dev_bf16
from test_gpu_parity import check_plan, random_workload

pytestmark = pytest.mark.gpu

SHAPES = [
    (32, 4096, 4096, 16, [16, 8, 16, 12, 16, 3, 16, 16]),   # the q_proj decode shape: 4 K splits, 128 CTAs + spare
    (24, 2048, 1024, 64, [64, 40, 8, 33, 64]),              # 8 K splits, rank 64: eight row groups per token
    (64, 2048, 1024, 16, [16, 8, 3, 16, 12, 16]),           # the largest batch of the path
    (1, 1024, 512, 16, [16, 5]),                            # one token
    (7, 520, 264, 8, [8, 3, 1]),                            # h_in not a multiple of a K step, ragged row tile
    (33, 8192, 2048, 32, [32, 24, 8, 16]),                  # long rows: several K steps per warp and item
]


@pytest.mark.parametrize("fused", [1, 0])
@pytest.mark.parametrize("T,h_in,h_out,max_rank,ranks", SHAPES)
def test_one_launch_and_two_launch_paths_match_the_oracle(T, h_in, h_out, max_rank, ranks, fused):
    w = random_workload(7000 + T + h_out, T, h_in, h_out, ranks=ranks, max_rank=max_rank)
    pool = make_pool(w, 64)
    try:
        y, plan = run_gpu(w, 1, pool=pool, return_plan=True, options={B.OPT_FUSED_DECODE: fused})
        info = B.edgelora_pool_last_launch(pool.handle)
        assert_parity(y, oracle_of(w), f"decode T={T} {h_in}->{h_out} fused={fused}")
        check_plan(plan, w.ids, w.n_slots)
        if not fused:
            assert info["launches"] == 2
        elif info["launches"] == 1:
            # run it again on the same pool: the arrival counters must be back at zero
            y2 = run_gpu(w, 1, pool=pool, options={B.OPT_FUSED_DECODE: 1})
            assert np.array_equal(y, y2)
    finally:
        pool.close()


def test_q_proj_shape_takes_one_launch():
    w = random_workload(7100, 32, 4096, 4096, ranks=[16] * 8, max_rank=16)
    pool = make_pool(w, 64)
    try:
        run_gpu(w, 1, pool=pool)
        assert B.edgelora_pool_last_launch(pool.handle)["launches"] == 1
    finally:
        pool.close()


@pytest.mark.parametrize("pdl", [0, 1, 2])
def test_chain_of_dependent_calls(pdl):
    # y of call i is x of call i + 1 (h_in == h_out), issued back to back without synchronising:
    # with EDGELORA_OPT_PDL = 0 and 1 the library must order the calls itself.  (Mode 2 is for
    # independent calls: there the chain is synchronised between the calls.)
    import torch
    h = 1024
    base = random_workload(7200, 48, h, h, ranks=[16, 8, 16, 4], max_rank=16)
    W = wl.normal_bf16(np.random.Generator(np.random.PCG64(1)), (h, h), 0.03)
    w0 = wl.Workload("chain", h, h, base.n_slots, base.max_rank, W, base.x, base.ids, base.adapters)
    pool = make_pool(w0, 64)
    try:
        B.edgelora_pool_set_option(pool.handle, B.OPT_REGIME, 1)
        B.edgelora_pool_set_option(pool.handle, B.OPT_PDL, pdl)
        Wd = to_dev_bf16(W)
        ids = torch.from_numpy(w0.ids).cuda()
        bufs = [to_dev_bf16(w0.x)] + [torch.zeros((w0.T, h), dtype=torch.bfloat16, device="cuda") for _ in range(4)]
        torch.cuda.synchronize()
        for i in range(4):
            B.edgelora_lora_linear(pool.handle, Wd, bufs[i], ids, bufs[i + 1])
            if pdl == 2:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        assert pool.status() == (0, 0)
        x = w0.x
        for i in range(4):
            wi = wl.Workload(f"chain{i}", h, h, w0.n_slots, w0.max_rank, W, x, w0.ids, w0.adapters)
            got = bufs[i + 1].view(torch.int16).cpu().numpy().view(np.uint16)
            assert_parity(wl.bf16_bits_to_f32(got), oracle_of(wi), f"call {i} of the chain, pdl={pdl}")
            x = got                      # the next call read exactly these bits
    finally:
        pool.close()


def test_status_bits_of_the_one_launch_path():
    import torch
    w = random_workload(7300, 20, 1024, 768, ranks=[16, 0, 8], max_rank=16)   # slot 1 is empty
    ids = w.ids.copy()
    ids[3], ids[5], ids[11] = 1, 9, -4           # an empty slot and two ids outside [-1, 3)
    pool = make_pool(w, 64)
    try:
        B.edgelora_pool_set_option(pool.handle, B.OPT_REGIME, 1)
        y = torch.zeros((w.T, w.h_out), dtype=torch.bfloat16, device="cuda")
        B.edgelora_lora_linear(pool.handle, to_dev_bf16(w.W), to_dev_bf16(w.x), torch.from_numpy(ids).cuda(), y)
        rc, bits = pool.status()
        assert bits == (B.STATUS_BAD_ADAPTER_ID | B.STATUS_SLOT_EMPTY)
        valid = np.where((ids < -1) | (ids >= 3) | (ids == 1), -1, ids).astype(np.int32)
        ref = wl.Workload("fallback", w.h_in, w.h_out, w.n_slots, w.max_rank, w.W, w.x, valid, w.adapters)
        assert_parity(from_dev_bf16(y), oracle_of(ref), "bad ids and empty slots fall back to the base product")
    finally:
        pool.close()
