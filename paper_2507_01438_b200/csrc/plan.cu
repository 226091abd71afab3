// Routing plan (paper Section 3.4: requests needing the same adapter form a u-batch; Section 4.3:
// adapter ids are mapped to sample indices, results return to their original positions).
//
// One CTA turns adapter_id[T] into
//   ids_valid   the ids with out-of-range values replaced by -1 (status bit raised),
//   segments    maximal runs of equal id in token order,
//   groups      tokens ordered by (id, token): ids ascending with -1 first, token order kept,
//   short lists the groups restricted to tokens the gather-by-token shrink handles,
//   sgmv tiles  in batches above kDecodeMaxT tokens, for runs of >= kSegMin tokens on a real
//               adapter: 128-token tiles of the run (work list of the segment shrink).
// The order is produced by a bitonic sort of the unique keys ((id + 1) << 16 | token) in shared
// memory, so it is exact and the same on every run.
#include "internal.cuh"
#include "launch.cuh"
#include "ptx.cuh"

namespace edgelora {

constexpr int kPlanThreads = 1024;

// In-place exclusive prefix sum of data[0..n) by the whole CTA; returns the total.
__device__ int block_exclusive_scan(int32_t *data, int n, int *warp_sums) {
  const int tid = threadIdx.x;
  const int per = (n + kPlanThreads - 1) / kPlanThreads;
  const int lo = min(n, tid * per), hi = min(n, lo + per);
  int local = 0;
  for (int i = lo; i < hi; ++i) local += data[i];
  // inclusive scan of `local` across the CTA
  int incl = local;
  const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    int v = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += v;
  }
  if (lane == 31) warp_sums[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = warp_sums[lane];
    int wi = w;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      int v = __shfl_up_sync(0xffffffffu, wi, d);
      if (lane >= d) wi += v;
    }
    warp_sums[lane] = wi - w;  // exclusive prefix of the warp totals
    if (lane == 31) warp_sums[32] = wi;
  }
  __syncthreads();
  int run = warp_sums[warp] + incl - local;
  for (int i = lo; i < hi; ++i) {
    int v = data[i];
    data[i] = run;
    run += v;
  }
  const int total = warp_sums[32];
  __syncthreads();
  return total;
}

__global__ void __launch_bounds__(kPlanThreads)
plan_kernel(const int32_t *__restrict__ ids, int32_t T, int32_t n_slots, PlanView pv, int32_t npow2) {
  extern __shared__ uint32_t keys[];
  __shared__ int warp_sums[33];
  const int tid = threadIdx.x;

  ptx::pdl_launch_dependents();
  ptx::pdl_wait_prior_grids();  // earlier kernels on the stream may still read the plan arrays

  // 1. validate, build keys
  bool bad = false;
  for (int i = tid; i < npow2; i += kPlanThreads) {
    uint32_t key = 0xFFFFFFFFu;
    if (i < T) {
      int32_t a = ids[i];
      if (a < -1 || a >= n_slots) {
        a = -1;
        bad = true;
      }
      pv.ids_valid[i] = a;
      key = (static_cast<uint32_t>(a + 1) << 16) | static_cast<uint32_t>(i);
    }
    keys[i] = key;
  }
  if (bad) atomicOr(pv.status, EDGELORA_STATUS_BAD_ADAPTER_ID);
  __syncthreads();

  // 2. bitonic sort, ascending
  for (int k = 2; k <= npow2; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int i = tid; i < npow2; i += kPlanThreads) {
        const int ixj = i ^ j;
        if (ixj > i) {
          const uint32_t a = keys[i], b = keys[ixj];
          const bool up = (i & k) == 0;
          if ((a > b) == up) {
            keys[i] = b;
            keys[ixj] = a;
          }
        }
      }
      __syncthreads();
    }
  }

  // 3. segments
  for (int t = tid; t < T; t += kPlanThreads)
    pv.scratch[t] = (t == 0 || pv.ids_valid[t] != pv.ids_valid[t - 1]) ? 1 : 0;
  __syncthreads();
  const int n_segs = block_exclusive_scan(pv.scratch, T, warp_sums);
  for (int t = tid; t < T; t += kPlanThreads) {
    const bool head = (t == 0 || pv.ids_valid[t] != pv.ids_valid[t - 1]);
    const int s = pv.scratch[t] + (head ? 1 : 0) - 1;
    pv.tok_seg[t] = s;
    if (head) {
      pv.seg_start[s] = t;
      pv.seg_adapter[s] = pv.ids_valid[t];
    }
  }
  if (tid == 0) {
    pv.seg_start[n_segs] = T;
    pv.counts[1] = n_segs;
  }
  __syncthreads();

  // 4. groups
  for (int i = tid; i < T; i += kPlanThreads) {
    pv.perm[i] = static_cast<int32_t>(keys[i] & 0xFFFFu);
    pv.scratch[i] = (i == 0 || (keys[i] >> 16) != (keys[i - 1] >> 16)) ? 1 : 0;
  }
  __syncthreads();
  const int n_groups = block_exclusive_scan(pv.scratch, T, warp_sums);
  for (int i = tid; i < T; i += kPlanThreads) {
    if (i == 0 || (keys[i] >> 16) != (keys[i - 1] >> 16)) {
      const int g = pv.scratch[i];
      pv.group_start[g] = i;
      pv.group_adapter[g] = static_cast<int32_t>(keys[i] >> 16) - 1;
    }
  }
  const int has_base = (keys[0] >> 16) == 0 ? 1 : 0;  // the group of id -1 sorts first
  for (int i = tid; i < T; i += kPlanThreads) {
    const uint32_t id1 = keys[i] >> 16;
    if (id1 != 0 && (i == 0 || id1 != (keys[i - 1] >> 16)))
      pv.lg_adapter[pv.scratch[i] - has_base] = static_cast<int32_t>(id1) - 1;
  }
  if (tid == 0) {
    pv.group_start[n_groups] = T;
    pv.counts[0] = n_groups;
    pv.counts[4] = n_groups - has_base;
    pv.counts[5] = 0;
  }
  __syncthreads();

  // 4b. the same groups restricted to "short" tokens: every token of a small batch, otherwise
  // the tokens of runs shorter than kSegMin (long runs go to the segment shrink)
  const bool all_short = T <= kDecodeMaxT;
  for (int i = tid; i < T; i += kPlanThreads) {
    const int t = static_cast<int>(keys[i] & 0xFFFFu);
    const int s = pv.tok_seg[t];
    pv.scratch[i] = (all_short || (pv.seg_start[s + 1] - pv.seg_start[s]) < kSegMin) ? 1 : 0;
  }
  __syncthreads();
  const int n_short = block_exclusive_scan(pv.scratch, T, warp_sums);
  for (int i = tid; i < T; i += kPlanThreads) {
    const int t = static_cast<int>(keys[i] & 0xFFFFu);
    const int s = pv.tok_seg[t];
    if (all_short || (pv.seg_start[s + 1] - pv.seg_start[s]) < kSegMin) pv.perm_short[pv.scratch[i]] = t;
  }
  for (int g = tid; g < n_groups; g += kPlanThreads) pv.gs_short[g] = pv.scratch[pv.group_start[g]];
  if (tid == 0) {
    pv.gs_short[n_groups] = n_short;
    pv.counts[3] = n_short;
  }
  __syncthreads();

  // 5. 128-token tiles of the long runs (segment shrink work list)
  for (int s = tid; s < n_segs; s += kPlanThreads) {
    const int len = pv.seg_start[s + 1] - pv.seg_start[s];
    pv.scratch[s] =
        (!all_short && pv.seg_adapter[s] >= 0 && len >= kSegMin) ? (len + kTileM - 1) / kTileM : 0;
  }
  __syncthreads();
  const int n_tiles = block_exclusive_scan(pv.scratch, n_segs, warp_sums);
  for (int s = tid; s < n_segs; s += kPlanThreads) {
    const int t0 = pv.seg_start[s];
    const int len = pv.seg_start[s + 1] - t0;
    if (!all_short && pv.seg_adapter[s] >= 0 && len >= kSegMin) {
      int tile = pv.scratch[s];
      for (int o = 0; o < len; o += kTileM, ++tile) {
        if (tile < pv.max_sgmv_tiles) {
          pv.sgmv_tiles[4 * tile + 0] = t0 + o;
          pv.sgmv_tiles[4 * tile + 1] = min(kTileM, len - o);
          pv.sgmv_tiles[4 * tile + 2] = pv.seg_adapter[s];
          pv.sgmv_tiles[4 * tile + 3] = 0;
        }
      }
    }
  }
  if (tid == 0) pv.counts[2] = min(n_tiles, pv.max_sgmv_tiles);

  // 6. the distinct ids >= 0 inside every 128-token tile, in order of first appearance (the LoRA
  // K blocks of that tile in the base-product kernel).  One warp per tile; lane l holds the ids
  // of tokens l, l + 32, l + 64, l + 96 of the tile.
  {
    const int lane = tid & 31, warp = tid >> 5;
    const int n_mt = (T + kTileM - 1) / kTileM;
    for (int m = warp; m < n_mt; m += kPlanThreads / 32) {
      int32_t id[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int t = m * kTileM + q * 32 + lane;
        id[q] = t < T ? pv.ids_valid[t] : -1;
      }
      const int32_t id0 = __shfl_sync(0xffffffffu, id[0], 0);
      bool same = true;
#pragma unroll
      for (int q = 0; q < 4; ++q) same = same && (id[q] == id0);
      if (__all_sync(0xffffffffu, same)) {  // the usual prefill tile: one run
        if (lane == 0) {
          pv.mt_count[m] = id0 >= 0 ? 1 : 0;
          pv.mt_list[m * kTileM] = id0;
        }
        continue;
      }
      bool first[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) first[q] = id[q] >= 0;
#pragma unroll
      for (int qq = 0; qq < 4; ++qq) {
        for (int src = 0; src < 32; ++src) {
          const int32_t v = __shfl_sync(0xffffffffu, id[qq], src);
          const int pos = qq * 32 + src;
#pragma unroll
          for (int q = 0; q < 4; ++q)
            if (pos < q * 32 + lane && v == id[q]) first[q] = false;
        }
      }
      int base = 0;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint32_t b = __ballot_sync(0xffffffffu, first[q]);
        if (first[q]) pv.mt_list[m * kTileM + base + __popc(b & ((1u << lane) - 1u))] = id[q];
        base += __popc(b);
      }
      if (lane == 0) pv.mt_count[m] = base;
    }
  }
}

void launch_plan(const int32_t *ids, int32_t T, int32_t n_slots, const PlanView &pv, bool pdl,
                 cudaStream_t stream) {
  int npow2 = 32;
  while (npow2 < T) npow2 <<= 1;
  launch_ex(plan_kernel, dim3(1), dim3(kPlanThreads), static_cast<size_t>(npow2) * 4, stream, pdl, 1,
            ids, T, n_slots, pv, npow2);
}

void init_plan_kernel() {
  cudaFuncSetAttribute(plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                       kMaxTokensLimit * 4);
}

}  // namespace edgelora
