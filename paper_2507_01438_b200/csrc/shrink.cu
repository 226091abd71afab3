// Gather-by-token shrink (BGMV): z[t] = s_a * A_a x[t] for tokens scattered across adapters
// (paper Section 2.1 for A: r x h_in; Section 4.3: tokens that share an adapter are handled as one
// sub-batch so the adapter is fetched once).
//
// One CTA per (group, rank row i): it streams row i of A_a once from HBM with 128-bit loads and
// dots it against the x rows of up to eight tokens of the group at a time; partial sums are
// reduced with warp shuffles and a small shared-memory stage.  It walks the plan's "short" token
// lists: in large batches tokens that belong to long runs are left to the segment shrink.
#include "internal.cuh"
#include "launch.cuh"
#include "ptx.cuh"

namespace edgelora {

constexpr int kBgmvThreads = 256;
constexpr int kBgmvTok = 8;

__device__ __forceinline__ float dot8(const uint4 &a, const uint4 &b) {
  float s = ptx::bf16_lo(a.x) * ptx::bf16_lo(b.x);
  s = fmaf(ptx::bf16_hi(a.x), ptx::bf16_hi(b.x), s);
  s = fmaf(ptx::bf16_lo(a.y), ptx::bf16_lo(b.y), s);
  s = fmaf(ptx::bf16_hi(a.y), ptx::bf16_hi(b.y), s);
  s = fmaf(ptx::bf16_lo(a.z), ptx::bf16_lo(b.z), s);
  s = fmaf(ptx::bf16_hi(a.z), ptx::bf16_hi(b.z), s);
  s = fmaf(ptx::bf16_lo(a.w), ptx::bf16_lo(b.w), s);
  s = fmaf(ptx::bf16_hi(a.w), ptx::bf16_hi(b.w), s);
  return s;
}

__global__ void __launch_bounds__(kBgmvThreads)
bgmv_shrink_kernel(const uint16_t *__restrict__ x, const uint16_t *__restrict__ A_pool,
                   const SlotRow *__restrict__ slots, PlanView pv, float *__restrict__ zws,
                   int32_t T, int32_t h_in, int32_t R_pad, int32_t zsplits, int32_t max_tokens,
                   uint32_t *status) {
  __shared__ float red[kBgmvThreads / 32][kBgmvTok];
  __shared__ int32_t tok[kBgmvTok];

  ptx::pdl_launch_dependents();
  ptx::pdl_wait_prior_grids();  // the plan comes from the previous kernel

  const int g = blockIdx.x / R_pad;
  const int i = blockIdx.x % R_pad;
  if (g >= pv.counts[0]) return;
  const int a = pv.group_adapter[g];
  if (a < 0) return;
  const SlotRow row = slots[a];
  const int g0 = pv.gs_short[g], g1 = pv.gs_short[g + 1];
  if (row.rank <= 0) {
    if (threadIdx.x == 0 && i == 0) atomicOr(status, EDGELORA_STATUS_SLOT_EMPTY);
    return;
  }
  const bool live_row = i < row.rank;
  const uint4 *Arow =
      reinterpret_cast<const uint4 *>(A_pool + (static_cast<size_t>(a) * R_pad + i) * h_in);
  const int n8 = h_in >> 3;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const size_t zsplit_stride = static_cast<size_t>(max_tokens) * R_pad;

  for (int base = g0; base < g1; base += kBgmvTok) {
    const int n_tok = min(kBgmvTok, g1 - base);
    __syncthreads();
    if (threadIdx.x < n_tok) tok[threadIdx.x] = pv.perm_short[base + threadIdx.x];
    __syncthreads();

    if (!live_row) {  // padding rows of the block: z is defined as zero there
      for (int q = threadIdx.x; q < n_tok * zsplits; q += kBgmvThreads)
        zws[(q / n_tok) * zsplit_stride + static_cast<size_t>(tok[q % n_tok]) * R_pad + i] = 0.f;
      continue;
    }

    float acc[kBgmvTok];
#pragma unroll
    for (int q = 0; q < kBgmvTok; ++q) acc[q] = 0.f;
    for (int k = threadIdx.x; k < n8; k += kBgmvThreads) {
      const uint4 av = __ldg(Arow + k);
#pragma unroll
      for (int q = 0; q < kBgmvTok; ++q) {
        if (q < n_tok) {
          const uint4 xv =
              __ldg(reinterpret_cast<const uint4 *>(x + static_cast<size_t>(tok[q]) * h_in) + k);
          acc[q] += dot8(av, xv);
        }
      }
    }
#pragma unroll
    for (int q = 0; q < kBgmvTok; ++q) {
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) acc[q] += __shfl_xor_sync(0xffffffffu, acc[q], d);
      if (lane == 0) red[warp][q] = acc[q];
    }
    __syncthreads();
    if (threadIdx.x < n_tok) {
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < kBgmvThreads / 32; ++w) s += red[w][threadIdx.x];
      const size_t off = static_cast<size_t>(tok[threadIdx.x]) * R_pad + i;
      zws[off] = row.scale * s;
      for (int sp = 1; sp < zsplits; ++sp) zws[sp * zsplit_stride + off] = 0.f;
    }
  }
}

void launch_bgmv_shrink(const uint16_t *x, const uint16_t *A_pool, const SlotRow *slots,
                        const PlanView &pv, float *zws, int32_t T, int32_t h_in, int32_t R_pad,
                        int32_t n_slots, int32_t zsplits, int32_t max_tokens, uint32_t *status,
                        bool pdl, cudaStream_t stream) {
  const int max_groups = (T < n_slots + 1) ? T : n_slots + 1;
  launch_ex(bgmv_shrink_kernel, dim3(max_groups * R_pad), dim3(kBgmvThreads), 0, stream, pdl, 1, x,
            A_pool, slots, pv, zws, T, h_in, R_pad, zsplits, max_tokens, status);
}

}  // namespace edgelora

namespace edgelora {

// ---------------------------------------------------------------------------------------------
// Decode shrink with the routing folded in (batches of at most 256 tokens).
//
// A decode step is a few microseconds long, so a separate routing launch would cost as much as
// the arithmetic.  Here every CTA derives the u-batches (paper Section 3.4) from the ids itself, in
// shared memory, and then takes its share of the work items (group, K chunk).  An item streams the
// live rows of A_a over its K chunk once from HBM with 16-byte cp.async copies into a private
// shared-memory ring (two K steps of eight rows ahead per lane), and dots them with the x rows of
// up to four tokens of the group at a time (a group's tokens are cut into blocks of eight, each
// block an item of its own, so that a popular adapter does not serialise on one CTA); lanes are
// reduced by shuffles, K sub-ranges of one item by a small shared-memory stage.  Partial sums go
// to zws[chunk][token][row]; whichever item finishes a group last adds the chunks in a fixed
// order into the final plane zws[kMaxZSplits] that the base-product kernel reads.  The last CTA also
// writes the routing plan in its canonical form for the base-product kernel and for export.

constexpr int kDsTok = 4;

__device__ __forceinline__ void unpack8(const uint4 &v, float (&f)[8]) {
  f[0] = ptx::bf16_lo(v.x); f[1] = ptx::bf16_hi(v.x);
  f[2] = ptx::bf16_lo(v.y); f[3] = ptx::bf16_hi(v.y);
  f[4] = ptx::bf16_lo(v.z); f[5] = ptx::bf16_hi(v.z);
  f[6] = ptx::bf16_lo(v.w); f[7] = ptx::bf16_hi(v.w);
}

// Exclusive prefix sum of one int per thread over the 256-thread CTA; `total` gets the sum.
__device__ __forceinline__ int block_scan_256(int v, int *wt /* smem[9] */, int &total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int o = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += o;
  }
  if (lane == 31) wt[warp] = incl;
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
  const int res = wt[warp] + incl - v;
  total = wt[8];
  __syncthreads();
  return res;
}

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ptx::smem_u32(smem_dst)), "l"(gmem_src)
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

constexpr int kRingSlots = 8 + kDsTok;  // 16-byte slots of one lane in one ring stage: 8 A rows + x rows

// Eight rows of A against NT token rows of x over the K steps step0, step0 + dstep, ... < step1;
// one K step is 256 elements, lane l owns elements [8 l, 8 l + 8) of it.  Every lane prefetches
// its own operands DEPTH - 1 steps ahead into its private slots of a shared-memory ring with
// cp.async, so that many 16-byte requests per lane are in flight without holding registers.
template <int NT, int DEPTH>
__device__ __forceinline__ void shrink_rows8(const uint4 *__restrict__ A0, size_t row_u4,
                                             const uint4 *const (&xr)[kDsTok], int step0, int step1,
                                             int dstep, int n_u4, int lane, uint4 *ring /* this thread's slot 0 */,
                                             float (&acc)[8 * kDsTok]) {
  constexpr int kStageStride = kRingSlots * kShrinkThreads;  // uint4 between stages
  auto issue = [&](int step, int stage) {
    const int k = step * 32 + lane;
    if (step < step1 && k < n_u4) {
      uint4 *dst = ring + stage * kStageStride;
#pragma unroll
      for (int r = 0; r < 8; ++r) cp_async16(dst + r * kShrinkThreads, A0 + r * row_u4 + k);
#pragma unroll
      for (int q = 0; q < NT; ++q) cp_async16(dst + (8 + q) * kShrinkThreads, xr[q] + k);
    }
    cp_async_commit();  // an empty group keeps the group count uniform
  };
#pragma unroll
  for (int d = 0; d < DEPTH - 1; ++d) issue(step0 + d * dstep, d);
  int stage = 0;
  for (int step = step0; step < step1; step += dstep) {
    int pre = stage + DEPTH - 1;
    if (pre >= DEPTH) pre -= DEPTH;
    issue(step + (DEPTH - 1) * dstep, pre);
    cp_async_wait<DEPTH - 1>();
    const int k = step * 32 + lane;
    if (k < n_u4) {
      const uint4 *src = ring + stage * kStageStride;
      float xf[NT][8];
#pragma unroll
      for (int q = 0; q < NT; ++q) unpack8(src[(8 + q) * kShrinkThreads], xf[q]);
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        float af[8];
        unpack8(src[r * kShrinkThreads], af);
#pragma unroll
        for (int q = 0; q < NT; ++q)
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[r * kDsTok + q] = fmaf(af[e], xf[q][e], acc[r * kDsTok + q]);
      }
    }
    if (++stage == DEPTH) stage = 0;
  }
  cp_async_wait<0>();
}

constexpr int kDsDepth = 3;      // ring stages
constexpr int kDsBlockTok = 8;   // tokens of one group handled by one work item (two passes of four)
constexpr size_t kDsRingBytes = static_cast<size_t>(kDsDepth) * kRingSlots * kShrinkThreads * 16;

__global__ void __launch_bounds__(kShrinkThreads)
decode_shrink_kernel(const int32_t *__restrict__ ids, const uint16_t *__restrict__ x,
                     const uint16_t *__restrict__ A_pool, const SlotRow *__restrict__ slots,
                     PlanView pv, float *__restrict__ zws, int32_t *__restrict__ group_counters,
                     int32_t T, int32_t h_in, int32_t R_pad, int32_t n_slots, int32_t max_tokens,
                     int32_t target_items, uint32_t *status) {
  extern __shared__ uint4 s_ring[];    // [depth][slot][thread]
  __shared__ int32_t s_id[256];        // validated id of each token
  __shared__ int32_t s_grp[256];       // group (in order of first appearance) of a group's first token
  __shared__ int32_t s_gadapter[256];  // adapter of each group
  __shared__ int32_t s_gstart[257];    // token list boundaries
  __shared__ int32_t s_gtok[256];      // tokens ordered by (group, token)
  __shared__ int32_t s_cnt[256];
  __shared__ int32_t s_bgrp[256];      // token blocks: group and first position in s_gtok
  __shared__ int32_t s_btok[256];
  __shared__ int s_wt[9];
  __shared__ float s_red[8][32];
  __shared__ int s_last;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  ptx::pdl_launch_dependents();

  // ---- routing, in shared memory (reads only the caller's ids)
  int a = -1;
  bool bad = false;
  if (tid < T) {
    a = ids[tid];
    if (a < -1 || a >= n_slots) {
      a = -1;
      bad = true;
    }
  }
  s_id[tid] = a;
  s_cnt[tid] = 0;
  __syncthreads();
  int pos = 0, first = tid;
  if (a >= 0) {
    for (int u = 0; u < tid; ++u) {
      if (s_id[u] == a) {
        if (pos == 0) first = u;
        ++pos;
      }
    }
  }
  const bool leader = a >= 0 && pos == 0;
  int G;
  const int g = block_scan_256(leader ? 1 : 0, s_wt, G);
  if (leader) {
    s_grp[tid] = g;
    s_gadapter[g] = a;
  }
  __syncthreads();
  int mygrp = -1;
  if (a >= 0) {
    mygrp = s_grp[first];
    atomicAdd(&s_cnt[mygrp], 1);
  }
  __syncthreads();
  int tot;
  const int n_mine = tid < G ? s_cnt[tid] : 0;
  const int gs = block_scan_256(n_mine, s_wt, tot);
  if (tid < G) s_gstart[tid] = gs;
  if (tid == 0) s_gstart[G] = tot;
  // token blocks of at most kDsBlockTok tokens
  const int nb_mine = (n_mine + kDsBlockTok - 1) / kDsBlockTok;
  int NB;
  const int b0 = block_scan_256(nb_mine, s_wt, NB);
  for (int b = 0; b < nb_mine; ++b) {
    s_bgrp[b0 + b] = tid;
    s_btok[b0 + b] = gs + b * kDsBlockTok;
  }
  __syncthreads();
  if (mygrp >= 0) s_gtok[s_gstart[mygrp] + pos] = tid;
  const int any_bad = __syncthreads_or(bad ? 1 : 0);

  // K chunks: enough items to occupy the machine, but an item keeps at least about 128 KB of A
  // (below that the extra pass that adds the chunks costs more than it saves) and one K step per
  // warp sub-range.
  const int n_ksteps = (h_in + 255) >> 8;
  const int ksubs_nominal = 64 / R_pad;  // 4, 2, 1 for a rank stride of 16, 32, 64
  int KS = (target_items + max(NB, 1) - 1) / max(NB, 1);
  KS = min(KS, max(1, (R_pad * h_in * 2) >> 17));
  KS = max(1, min(min(KS, kMaxZSplits), n_ksteps / ksubs_nominal));
  const int spc = (n_ksteps + KS - 1) / KS;
  KS = (n_ksteps + spc - 1) / spc;

  ptx::pdl_wait_prior_grids();  // earlier kernels may still read the plan and z

  // ---- the last CTA publishes the plan in canonical order (ids ascending, -1 first)
  if (blockIdx.x == gridDim.x - 1) {
    if (any_bad && tid == 0) atomicOr(pv.status, EDGELORA_STATUS_BAD_ADAPTER_ID);
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
    }
    const bool shead = tid < T && (tid == 0 || s_id[tid - 1] != a);
    int n_segs;
    const int si = block_scan_256(shead ? 1 : 0, s_wt, n_segs);
    if (tid < T) {
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

  // ---- work items (token block of a group, K chunk)
  const int n_items = NB * KS;
  const int n_u4 = h_in >> 3;
  const size_t zplane = static_cast<size_t>(max_tokens) * R_pad;
  uint4 *my_ring = s_ring + tid;
  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
    const int bi = item / KS, c = item - bi * KS;
    const int gi = s_bgrp[bi];
    const int ad = s_gadapter[gi];
    const SlotRow row = slots[ad];
    const int t0 = s_btok[bi], g_end = s_gstart[gi + 1];
    const int t1 = min(t0 + kDsBlockTok, g_end);
    if (row.rank <= 0) {
      if (tid == 0 && c == 0 && t0 == s_gstart[gi]) atomicOr(status, EDGELORA_STATUS_SLOT_EMPTY);
      continue;
    }
    const int n_rg = (row.rank + 7) >> 3;  // live groups of eight rows
    int rg_p2 = 1;
    while (rg_p2 < n_rg) rg_p2 <<= 1;
    const int ksubs = 8 / rg_p2;
    const int rg = warp % rg_p2, ksub = warp / rg_p2;
    const int step0 = c * spc, step1 = min(n_ksteps, step0 + spc);
    const uint4 *A0 =
        reinterpret_cast<const uint4 *>(A_pool + (static_cast<size_t>(ad) * R_pad + rg * 8) * h_in);
    for (int tb = t0; tb < t1; tb += kDsTok) {
      const int nt = min(kDsTok, t1 - tb);
      float acc[8 * kDsTok];
#pragma unroll
      for (int i = 0; i < 8 * kDsTok; ++i) acc[i] = 0.f;
      if (rg < n_rg) {
        const uint4 *xr[kDsTok];
#pragma unroll
        for (int q = 0; q < kDsTok; ++q)
          xr[q] = reinterpret_cast<const uint4 *>(x + static_cast<size_t>(s_gtok[tb + min(q, nt - 1)]) * h_in);
        const size_t row_u4 = static_cast<size_t>(n_u4);
        if (nt == 1) shrink_rows8<1, kDsDepth>(A0, row_u4, xr, step0 + ksub, step1, ksubs, n_u4, lane, my_ring, acc);
        else if (nt == 2) shrink_rows8<2, kDsDepth>(A0, row_u4, xr, step0 + ksub, step1, ksubs, n_u4, lane, my_ring, acc);
        else if (nt == 3) shrink_rows8<3, kDsDepth>(A0, row_u4, xr, step0 + ksub, step1, ksubs, n_u4, lane, my_ring, acc);
        else shrink_rows8<4, kDsDepth>(A0, row_u4, xr, step0 + ksub, step1, ksubs, n_u4, lane, my_ring, acc);
      }
      // lane L ends with the sum over lanes of value L (= row L / 4, token L % 4)
#pragma unroll
      for (int off = 16, cnt = 16; off >= 1; off >>= 1, cnt >>= 1) {
        const bool upper = (lane & off) != 0;
#pragma unroll
        for (int i = 0; i < cnt; ++i) {
          const float send = upper ? acc[i] : acc[i + cnt];
          const float keep = upper ? acc[i + cnt] : acc[i];
          acc[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
        }
      }
      float v = acc[0];
      if (ksubs > 1) {
        s_red[warp][lane] = v;
        __syncthreads();
        if (ksub == 0)
          for (int j = 1; j < ksubs; ++j) v += s_red[warp + j * rg_p2][lane];
        __syncthreads();
      }
      const int q = lane & 3, r = rg * 8 + (lane >> 2);
      if (ksub == 0 && rg < n_rg && q < nt)
        zws[(KS > 1 ? c : kMaxZSplits) * zplane + static_cast<size_t>(s_gtok[tb + q]) * R_pad + r] =
            row.scale * v;
    }
    if (KS > 1) {
      // The item that completes a group adds the K chunks in order into the final plane (it never
      // waits for the others).
      const int gt0 = s_gstart[gi];
      const int arrivals = KS * ((g_end - gt0 + kDsBlockTok - 1) / kDsBlockTok);
      __threadfence();
      __syncthreads();
      if (tid == 0) {
        const int old = atomicAdd(&group_counters[gi], 1);
        s_last = (old == arrivals - 1) ? 1 : 0;
        if (s_last) group_counters[gi] = 0;  // ready for the next launch
      }
      __syncthreads();
      if (s_last) {
        __threadfence();
        const int live = n_rg * 8;
        for (int idx = tid; idx < (g_end - gt0) * live; idx += kShrinkThreads) {
          const int q = idx / live, r = idx - q * live;
          const size_t off = static_cast<size_t>(s_gtok[gt0 + q]) * R_pad + r;
          float part[kMaxZSplits];
#pragma unroll
          for (int sp = 0; sp < kMaxZSplits; ++sp) part[sp] = sp < KS ? __ldcg(zws + sp * zplane + off) : 0.f;
          float sum = 0.f;
#pragma unroll
          for (int sp = 0; sp < kMaxZSplits; ++sp) sum += part[sp];
          zws[kMaxZSplits * zplane + off] = sum;
        }
      }
    }
  }
}

void launch_decode_shrink(const int32_t *ids, const uint16_t *x, const uint16_t *A_pool,
                          const SlotRow *slots, const PlanView &pv, float *zws,
                          int32_t *group_counters, int32_t T, int32_t h_in, int32_t R_pad,
                          int32_t n_slots, int32_t max_tokens, int32_t target_items, int32_t grid,
                          uint32_t *status, bool pdl, cudaStream_t stream) {
  static bool configured = false;  // per process; the attribute is per function and device-wide
  if (!configured) {
    cudaFuncSetAttribute(decode_shrink_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         static_cast<int>(kDsRingBytes));
    configured = true;
  }
  launch_ex(decode_shrink_kernel, dim3(grid), dim3(kShrinkThreads), kDsRingBytes, stream, pdl, 1, ids, x, A_pool,
            slots, pv, zws, group_counters, T, h_in, R_pad, n_slots, max_tokens, target_items, status);
}

}  // namespace edgelora
