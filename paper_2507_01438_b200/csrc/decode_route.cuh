// Routing helpers shared by the kernels that derive a decode batch's u-batches (paper Section 3.4)
// from the caller's ids inside the kernel: a CTA-wide prefix sum and the publication of the routing
// plan in its canonical form (the form the plan kernel writes for larger batches).
#pragma once
#include "internal.cuh"
#include "ptx.cuh"

namespace edgelora {

// Exclusive prefix sum of one int per thread over the first 256 threads of the CTA; `total` gets
// the sum.  Every thread of the CTA calls it (it synchronises the CTA); threads from 256 on pass 0
// and ignore the result.  wt: shared memory, 9 ints.
__device__ __forceinline__ int block_scan_256(int v, int *wt, int &total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int o = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += o;
  }
  if (lane == 31 && warp < 8) wt[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const int w = lane < 8 ? wt[lane] : 0;
    int wi = w;
#pragma unroll
    for (int d = 1; d < 8; d <<= 1) {
      const int o = __shfl_up_sync(0xffffffffu, wi, d);
      if (lane >= d) wi += o;
    }
    if (lane < 8) wt[lane] = wi - w;
    if (lane == 7) wt[8] = wi;
  }
  __syncthreads();
  const int res = wt[warp < 8 ? warp : 8] + incl - v;
  total = wt[8];
  __syncthreads();
  return res;
}

// Writes the routing plan of a batch of T <= 256 tokens in canonical order (ids ascending, -1
// first; segments in token order).  Called by every thread of one CTA; thread t < T passes the
// validated id `a` of token t (-1 = no adapter), the others -1.  s_id[256] holds those ids already;
// s_cnt[256] and s_wt[9] are scratch.  Everything is worked out in shared memory and registers
// first; the stores come after griddepcontrol.wait (earlier kernels on the stream may still read the
// plan).
__device__ __forceinline__ void publish_decode_plan(const PlanView &pv, int a, int T, int any_bad, int KS,
                                                    const int32_t *s_id, int32_t *s_cnt, int *s_wt) {
  const int tid = threadIdx.x;
  const uint32_t key = (static_cast<uint32_t>(a + 1) << 16) | static_cast<uint32_t>(tid);
  int rp = 0;
  if (tid < T)
    for (int u = 0; u < T; ++u)
      rp += (((static_cast<uint32_t>(s_id[u] + 1) << 16) | static_cast<uint32_t>(u)) < key) ? 1 : 0;
  __syncthreads();  // every thread is done with s_cnt as a counter
  if (tid < T) s_cnt[rp] = tid;  // s_cnt now holds the tokens in canonical order
  __syncthreads();
  int ida = -2, tok = 0;
  bool head = false;
  if (tid < T) {
    tok = s_cnt[tid];
    ida = s_id[tok];
    head = tid == 0 || s_id[s_cnt[tid - 1]] != ida;
  }
  int n_groups;
  const int gi = block_scan_256(head ? 1 : 0, s_wt, n_groups);
  const int has_base = (T > 0 && s_id[s_cnt[0]] < 0) ? 1 : 0;
  const bool shead = tid < T && (tid == 0 || s_id[tid - 1] != a);
  int n_segs;
  const int si = block_scan_256(shead ? 1 : 0, s_wt, n_segs);

  ptx::pdl_wait_prior_grids();
  if (any_bad && tid == 0) atomicOr(pv.status, EDGELORA_STATUS_BAD_ADAPTER_ID);
  if (tid < T) {
    pv.ids_valid[tid] = a;
    pv.perm[tid] = tok;
    pv.perm_short[tid] = tok;
    if (head) {
      pv.group_start[gi] = tid;
      pv.gs_short[gi] = tid;
      pv.group_adapter[gi] = ida;
      if (ida >= 0) pv.lg_adapter[gi - has_base] = ida;
    }
    pv.tok_seg[tid] = si + (shead ? 1 : 0) - 1;
    if (shead) {
      pv.seg_start[si] = tid;
      pv.seg_adapter[si] = a;
    }
  }
  if (tid == 0) {
    pv.group_start[n_groups] = T;
    pv.gs_short[n_groups] = T;
    pv.seg_start[n_segs] = T;
    pv.counts[0] = n_groups;
    pv.counts[1] = n_segs;
    pv.counts[2] = 0;
    pv.counts[3] = T;
    pv.counts[4] = n_groups - has_base;
    pv.counts[5] = KS;
  }
}

}  // namespace edgelora
