// Routing plan (paper Section 3.4: requests needing the same adapter form a u-batch; Section 4.3:
// adapter ids are mapped to sample indices, results return to their original positions).
//
// One CTA turns adapter_id[T] into
//   ids_valid   the ids with out-of-range values replaced by -1 (status bit raised),
//   segments    maximal runs of equal id in token order,
//   groups      tokens ordered by (id, token): ids ascending with -1 first, token order kept,
//   short lists the groups restricted to tokens the gather-by-token shrink handles,
//   sgmv tiles  in batches above kDecodeMaxT tokens, for runs of >= kSegMin tokens on a real
//               adapter: 128-token tiles of the run (work list of the segment shrink),
//   tile lists  the distinct ids >= 0 inside every 128-token tile (the LoRA K blocks of that tile).
// Tokens of one run stay together in the group order, so the runs are sorted, not the tokens: a
// bitonic sort of the unique keys ((id + 1) << 16 | run index) in shared memory, exact and the
// same on every launch.  Prefix sums run in rounds of one element per thread (warp shuffles plus
// one shared-memory stage), so nothing but the outputs goes through global memory.
#include "internal.cuh"
#include "launch.cuh"
#include "ptx.cuh"

namespace edgelora {

constexpr int kPlanThreads = 1024;

// Exclusive prefix sum over i in [0, n) of value(i), one element per thread per round;
// consume(i, prefix) is called for every i.  Returns the total.  `wt` is shared memory [34].
template <typename Value, typename Consume>
__device__ __forceinline__ int scan_rounds(int n, int *wt, Value value, Consume consume) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int base = 0;
  for (int i0 = 0; i0 < n; i0 += kPlanThreads) {
    const int i = i0 + tid;
    const int v = i < n ? value(i) : 0;
    int incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int o = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += o;
    }
    if (lane == 31) wt[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      const int w = wt[lane];
      int wi = w;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, wi, d);
        if (lane >= d) wi += o;
      }
      wt[lane] = wi - w;
      if (lane == 31) wt[32] = wi;
    }
    __syncthreads();
    if (i < n) consume(i, base + wt[warp] + incl - v);
    base += wt[32];
    __syncthreads();
  }
  return base;
}

__global__ void __launch_bounds__(kPlanThreads)
plan_kernel(const int32_t *__restrict__ ids, int32_t T, int32_t n_slots, PlanView pv) {
  extern __shared__ uint32_t keys[];  // one key per run, padded to a power of two
  __shared__ int wt[34];
  const int tid = threadIdx.x;

  ptx::pdl_launch_dependents();
  ptx::pdl_wait_prior_grids();  // earlier kernels on the stream may still read the plan arrays

  // 1. validate
  bool bad = false;
  for (int t = tid; t < T; t += kPlanThreads) {
    int32_t a = ids[t];
    if (a < -1 || a >= n_slots) {
      a = -1;
      bad = true;
    }
    pv.ids_valid[t] = a;
  }
  if (__syncthreads_or(bad ? 1 : 0) && tid == 0) atomicOr(pv.status, EDGELORA_STATUS_BAD_ADAPTER_ID);

  // 2. segments = maximal runs of equal id in token order
  auto is_head = [&](int t) { return (t == 0 || pv.ids_valid[t] != pv.ids_valid[t - 1]) ? 1 : 0; };
  const int n_segs = scan_rounds(
      T, wt, is_head, [&](int t, int before) {
        const int head = is_head(t);
        const int s = before + head - 1;
        pv.tok_seg[t] = s;
        if (head) {
          pv.seg_start[s] = t;
          pv.seg_adapter[s] = pv.ids_valid[t];
        }
      });
  if (tid == 0) {
    pv.seg_start[n_segs] = T;
    pv.counts[1] = n_segs;
  }
  __syncthreads();

  // 3. runs ordered by (id, run index): -1 first, token order kept (runs are in token order)
  int npow2 = 32;
  while (npow2 < n_segs) npow2 <<= 1;
  for (int i = tid; i < npow2; i += kPlanThreads)
    keys[i] = i < n_segs ? ((static_cast<uint32_t>(pv.seg_adapter[i] + 1) << 16) | static_cast<uint32_t>(i))
                         : 0xFFFFFFFFu;
  __syncthreads();
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

  // 4. groups: the runs in sorted order, concatenated.  out_start[j] (in pv.scratch) is where the
  // j-th sorted run begins in perm; inv (borrowing pv.mt_list until step 8) maps a run to j.
  int32_t *out_start = pv.scratch, *inv = pv.mt_list, *gidx = pv.perm_short;  // gidx: until step 6
  auto run_of = [&](int j) { return static_cast<int>(keys[j] & 0xFFFFu); };
  auto run_len = [&](int j) {
    const int s = run_of(j);
    return pv.seg_start[s + 1] - pv.seg_start[s];
  };
  scan_rounds(n_segs, wt, run_len, [&](int j, int before) {
    out_start[j] = before;
    inv[run_of(j)] = j;
  });
  for (int t = tid; t < T; t += kPlanThreads) {
    const int s = pv.tok_seg[t];
    const int pos = out_start[inv[s]] + (t - pv.seg_start[s]);
    if (EL_CHECK(pv.status, s >= 0 && s < n_segs && pos >= 0 && pos < T, 30)) pv.perm[pos] = t;
  }
  auto is_ghead = [&](int j) { return (j == 0 || (keys[j] >> 16) != (keys[j - 1] >> 16)) ? 1 : 0; };
  const int has_base = (n_segs > 0 && (keys[0] >> 16) == 0) ? 1 : 0;  // the group of id -1 sorts first
  const int n_groups = scan_rounds(n_segs, wt, is_ghead, [&](int j, int before) {
    const int head = is_ghead(j);
    const int g = before + head - 1;
    gidx[j] = g;
    if (head) {
      const int32_t a = static_cast<int32_t>(keys[j] >> 16) - 1;
      pv.group_start[g] = out_start[j];
      pv.group_adapter[g] = a;
      if (a >= 0) pv.lg_adapter[g - has_base] = a;
    }
  });
  if (tid == 0) {
    pv.group_start[n_groups] = T;
    pv.counts[0] = n_groups;
    pv.counts[4] = n_groups - has_base;
    pv.counts[5] = 0;
  }

  // 5. the same groups restricted to "short" tokens: every token of a small batch, otherwise the
  // tokens of runs shorter than kSegMin (long runs go to the segment shrink).  sstart[j] replaces
  // out_start[j] in pv.scratch.
  const bool all_short = T <= kDecodeMaxT;
  auto short_len = [&](int j) {
    const int len = run_len(j);
    return (all_short || len < kSegMin) ? len : 0;
  };
  const int n_short = scan_rounds(n_segs, wt, short_len, [&](int j, int before) {
    out_start[j] = before;
    if (is_ghead(j)) pv.gs_short[gidx[j]] = before;
  });
  // 6. (gidx is dead from here: perm_short takes its final content)
  for (int t = tid; t < T; t += kPlanThreads) {
    const int s = pv.tok_seg[t];
    const int len = pv.seg_start[s + 1] - pv.seg_start[s];
    const int pos = out_start[inv[s]] + (t - pv.seg_start[s]);
    if ((all_short || len < kSegMin) && EL_CHECK(pv.status, pos >= 0 && pos < T, 31)) pv.perm_short[pos] = t;
  }
  if (tid == 0) {
    pv.gs_short[n_groups] = n_short;
    pv.counts[3] = n_short;
  }

  // 7. 128-token tiles of the long runs (segment shrink work list), in token order
  auto run_tiles = [&](int s) {
    const int len = pv.seg_start[s + 1] - pv.seg_start[s];
    return (!all_short && pv.seg_adapter[s] >= 0 && len >= kSegMin) ? (len + kTileM - 1) / kTileM : 0;
  };
  const int n_tiles = scan_rounds(n_segs, wt, run_tiles, [&](int s, int before) {
    const int t0 = pv.seg_start[s];
    const int len = pv.seg_start[s + 1] - t0;
    const int nt = run_tiles(s);
    for (int i = 0; i < nt; ++i) {
      const int tile = before + i;
      if (tile < pv.max_sgmv_tiles) {
        pv.sgmv_tiles[4 * tile + 0] = t0 + i * kTileM;
        pv.sgmv_tiles[4 * tile + 1] = min(kTileM, len - i * kTileM);
        pv.sgmv_tiles[4 * tile + 2] = pv.seg_adapter[s];
        pv.sgmv_tiles[4 * tile + 3] = 0;
      }
    }
  });
  if (tid == 0) pv.counts[2] = min(n_tiles, pv.max_sgmv_tiles);
  __syncthreads();  // inv (in pv.mt_list) is dead from here

  // 8. the distinct ids >= 0 inside every 128-token tile, in order of first appearance (the LoRA
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
  int npow2 = 32;  // the number of runs is only known on the device: size for the worst case
  while (npow2 < T) npow2 <<= 1;
  launch_ex(plan_kernel, dim3(1), dim3(kPlanThreads), static_cast<size_t>(npow2) * 4, stream, pdl, 1,
            ids, T, n_slots, pv);
}

void init_plan_kernel() {
  cudaFuncSetAttribute(plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                       kMaxTokensLimit * 4);
}

}  // namespace edgelora
