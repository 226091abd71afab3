// Shrink for small decode batches: z[t] = s_a * A_a x[t] for tokens scattered across adapters
// (paper Section 2.1 for A: r x h_in; Section 4.3: tokens that share an adapter are handled as one
// sub-batch so the adapter is fetched once), with the routing derived inside the kernel so that a
// step of a few microseconds needs no routing launch.  Larger batches take the tensor-core gather
// tiles of the tile kernel (gemm.cu).
#include <cuda_fp16.h>

#include "decode_route.cuh"
#include "internal.cuh"
#include "launch.cuh"
#include "ptx.cuh"

namespace edgelora {

// ---------------------------------------------------------------------------------------------
// Decode shrink with the routing folded in (batches of at most 256 tokens).
//
// A decode step is a few microseconds long, so a separate routing launch would cost as much as
// the arithmetic.  Here every CTA derives the u-batches (paper Section 3.4) from the ids itself, in
// shared memory, and then takes its share of the work items (group, K chunk).  An item streams the
// live rows of A_a over its K chunk once from HBM with TMA copies into a private shared-memory
// ring (three K steps of eight rows ahead per warp), and dots them with the x rows of
// up to four tokens of the group at a time (a group's tokens are cut into blocks of eight, each
// block an item of its own, so that a popular adapter does not serialise on one CTA); lanes are
// reduced by shuffles.  Items belong to single warps, which run independently so that the fixed
// latencies of one overlap the streaming of the others.  Partial sums go to
// zws[chunk][token][row]; whichever warp finishes a (group, eight rows) last adds the chunks in a
// fixed order into the final plane zws[kMaxZSplits] that the base-product kernel reads.  The last CTA also
// writes the routing plan in its canonical form for the base-product kernel and for export.

constexpr int kDsTok = 4;

__device__ __forceinline__ void unpack8(const uint4 &v, float (&f)[8]) {
  f[0] = ptx::bf16_lo(v.x); f[1] = ptx::bf16_hi(v.x);
  f[2] = ptx::bf16_lo(v.y); f[3] = ptx::bf16_hi(v.y);
  f[4] = ptx::bf16_lo(v.z); f[5] = ptx::bf16_hi(v.z);
  f[6] = ptx::bf16_lo(v.w); f[7] = ptx::bf16_hi(v.w);
}

constexpr int kDsMaxDepth = 5;                      // ring stages per warp: up to 5, or 2 for small batches
constexpr int kDsRowBytes = kShrinkStepElems * 2;   // 512: one row segment of one K step
constexpr int kDsStageBytes = (8 + kDsTok) * kDsRowBytes;  // 8 rows of A, then up to 4 rows of x

// Eight rows of A against NT token rows of x over the K steps [step0, step1).  One K step is 256
// elements; lane l owns elements [8 l, 8 l + 8) of it.  The warp's lane 0 keeps kDsDepth - 1 steps
// in flight with TMA copies (one box of 8 x 512 bytes of A and one 512-byte row of x per token)
// into the warp's private ring; columns past h_in arrive as zeros.  `phase` holds one parity bit
// per ring stage and lives across calls.  Returns false if a wait gave up.
// The ring's bytes are those of kDsDepth stages with four x rows; with fewer x rows a stage is
// shorter, and with one token five stages fit where four did: a third more bytes in flight for the
// items that dominate a many-adapter batch (the stream is bound by latency times bytes in flight).
template <int NT, int kDsDepth>
struct RingShape {
  static constexpr int kStage = (8 + NT) * kDsRowBytes;
  static constexpr int kDepth = (kDsDepth * kDsStageBytes) / kStage > kDsMaxDepth ? kDsMaxDepth
                                                                                  : (kDsDepth * kDsStageBytes) / kStage;
};
// kQ8: the A rows are kept in Q8_0 (paper Section 5.1: per 32 values a half-precision scale d and 32
// signed bytes q, value d * q), in the pool as two planes per slot: the bytes [R_pad][h_in] and the
// scales [R_pad][h_in / 32].  A K step of 256 values is then 256 bytes + 8 scales per row: two boxes
// per step (8 x 256 bytes at the start of the stage, 8 x 16 bytes behind them), and lane l decodes the
// eight values it owns (one aligned 8-byte load, block l / 4) on the fly: sum_e q_e x_e in fp32,
// times d once.  17/32 of the bytes of the bfloat16 rows.
constexpr int kQ8QBytes = kShrinkStepElems;            // 256 bytes of q per row and step
constexpr int kQ8DBytes = (kShrinkStepElems / 32) * 2;  // 16 bytes of scales per row and step
// signed byte i of w as a float: the byte with its sign bit flipped is q + 128, placed in the
// mantissa of 2^23 it reads 2^23 + 128 + q
__device__ __forceinline__ float s8_to_float(uint32_t w_flipped, int i) {
  return __uint_as_float(__byte_perm(w_flipped, 0x4B000000u, 0x7440u + i)) - 8388736.0f;
}
template <int NT, int kDsDepthCfg, bool kQ8>
__device__ __forceinline__ bool shrink_rows8(const CUtensorMap *tmap_a, const CUtensorMap *tmap_d,
                                             const CUtensorMap *tmap_x,
                                             int32_t slot, int32_t row0, const int32_t (&tok)[kDsTok],
                                             int step0, int step1, int stride, uint8_t *ring, uint64_t *bars,
                                             uint32_t &phase, int lane, float (&acc)[8 * kDsTok]) {
  constexpr int kDsDepth = RingShape<NT, kDsDepthCfg>::kDepth;
  constexpr int kStage = RingShape<NT, kDsDepthCfg>::kStage;
  auto issue = [&](int step, int stage) {
    if (lane == 0 && step < step1) {
      uint8_t *dst = ring + stage * kStage;
      ptx::mbar_arrive_expect_tx_relaxed(&bars[stage],
                                         (kQ8 ? 8 * (kQ8QBytes + kQ8DBytes) : 8 * kDsRowBytes) + NT * kDsRowBytes);
      ptx::tma_load_3d(dst, tmap_a, &bars[stage], step * (kQ8 ? kQ8QBytes / 2 : kShrinkStepElems), row0, slot);
      if (kQ8) ptx::tma_load_3d(dst + 8 * kQ8QBytes, tmap_d, &bars[stage], step * (kShrinkStepElems / 32), row0, slot);
#pragma unroll
      for (int q = 0; q < NT; ++q)
        ptx::tma_load_2d(dst + (8 + q) * kDsRowBytes, tmap_x, &bars[stage], step * kShrinkStepElems, tok[q]);
    }
  };
#pragma unroll
  for (int d = 0; d < kDsDepth - 1; ++d) issue(step0 + d * stride, d);
  int stage = 0;
  for (int step = step0; step < step1; step += stride) {
    __syncwarp();  // every lane has finished reading the stage that is refilled next
    issue(step + (kDsDepth - 1) * stride, (stage + kDsDepth - 1) % kDsDepth);
    if (!ptx::mbar_wait(&bars[stage], (phase >> stage) & 1u)) return false;
    phase ^= 1u << stage;
    const uint4 *src = reinterpret_cast<const uint4 *>(ring + stage * kStage) + lane;
    float xf[NT][8];
#pragma unroll
    for (int q = 0; q < NT; ++q) unpack8(src[(8 + q) * (kDsRowBytes / 16)], xf[q]);
    if (kQ8) {
      const uint8_t *st = ring + stage * kStage;
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        const uint2 qq = *reinterpret_cast<const uint2 *>(st + r * kQ8QBytes + lane * 8);
        const float d = __half2float(__ushort_as_half(
            *reinterpret_cast<const unsigned short *>(st + 8 * kQ8QBytes + r * kQ8DBytes + (lane >> 2) * 2)));
        const uint32_t w0 = qq.x ^ 0x80808080u, w1 = qq.y ^ 0x80808080u;
        float qf[8];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          qf[e] = s8_to_float(w0, e);
          qf[4 + e] = s8_to_float(w1, e);
        }
#pragma unroll
        for (int q = 0; q < NT; ++q) {
          float part = 0.f;
#pragma unroll
          for (int e = 0; e < 8; ++e) part = fmaf(qf[e], xf[q][e], part);
          acc[r * kDsTok + q] = fmaf(d, part, acc[r * kDsTok + q]);
        }
      }
    } else {
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        float af[8];
        unpack8(src[r * (kDsRowBytes / 16)], af);
#pragma unroll
        for (int q = 0; q < NT; ++q)
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[r * kDsTok + q] = fmaf(af[e], xf[q][e], acc[r * kDsTok + q]);
      }
    }
    if (++stage == kDsDepth) stage = 0;
  }
  return true;
}

constexpr int kDsBlockTok = kDsTok;  // tokens of one group handled by one work item (one pass)
constexpr int kDsTicket = kDecodeMaxT * 8;  // index of the work-item ticket counter in group_counters

__device__ __forceinline__ int atomic_add_acq_rel(int32_t *p, int v) {
  int old;
  asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
  return old;
}
constexpr size_t ds_ring_bytes(int depth) {
  return static_cast<size_t>(kShrinkThreads / 32) * depth * kDsStageBytes + 1024;
}

// kDsDepth = 4 fills an SM's shared memory (large batches: bandwidth); kDsDepth = 2 leaves room
// for a CTA of the base-product kernel beside it (small batches: the two kernels overlap).
template <int kDsDepth, bool kQ8>
__global__ void __launch_bounds__(kShrinkThreads, 2)  // <= 128 registers: fits beside the base-product CTAs
decode_shrink_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_d,
                     const __grid_constant__ CUtensorMap tmap_x,
                     const int32_t *__restrict__ ids, const SlotRow *__restrict__ slots,
                     PlanView pv, float *__restrict__ zws, int32_t *__restrict__ group_counters,
                     int32_t T, int32_t h_in, int32_t R_pad, int32_t n_slots, int32_t max_tokens,
                     int32_t target_items, int32_t late_ticket, uint32_t *status) {
  extern __shared__ uint8_t s_ring_raw[];  // [warp][stage][8 A rows + 4 x rows][512 bytes]
  __shared__ uint64_t s_bars[kShrinkThreads / 32][kDsMaxDepth];
  __shared__ __align__(16) int32_t s_id[256];  // validated id of each token
  __shared__ int32_t s_grp[256];       // group (in order of first appearance) of a group's first token
  __shared__ int32_t s_gadapter[256];  // adapter of each group
  __shared__ int32_t s_gstart[257];    // token list boundaries
  __shared__ int32_t s_gtok[256];      // tokens ordered by (group, token)
  __shared__ int32_t s_cnt[256];
  __shared__ int32_t s_bgrp[256];      // token blocks: group and first position in s_gtok
  __shared__ int32_t s_btok[256];
  __shared__ int32_t s_grank[256];     // rank and scale of each group's slot
  __shared__ float s_gscale[256];
  __shared__ int s_wt[9];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  ptx::pdl_launch_dependents();
  if (tid == 0) {
    ptx::prefetch_tensormap(&tmap_a);
    ptx::prefetch_tensormap(&tmap_x);
  }
  if (lane < kDsMaxDepth) {  // every warp sets up its own ring barriers
    ptx::mbar_init(&s_bars[warp][lane], 1);
    ptx::fence_barrier_init();
  }

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
  SlotRow myrow = {0, 0.f, 0, 0};
  if (a >= 0) myrow = slots[a];  // in flight during the duplicate scan below
  s_id[tid] = a;
  s_cnt[tid] = 0;
  __syncthreads();
  int pos = 0, first = tid;
  if (a >= 0) {  // earlier tokens on the same adapter, four ids per shared-memory load
    auto see = [&](int id, int u) {
      if (id == a) {
        if (pos == 0) first = u;
        ++pos;
      }
    };
    const int full = tid & ~3;
    for (int u = 0; u < full; u += 4) {
      const int4 w = *reinterpret_cast<const int4 *>(&s_id[u]);
      see(w.x, u);
      see(w.y, u + 1);
      see(w.z, u + 2);
      see(w.w, u + 3);
    }
    for (int u = full; u < tid; ++u) see(s_id[u], u);
  }
  const bool leader = a >= 0 && pos == 0;
  int G;
  const int g = block_scan_256(leader ? 1 : 0, s_wt, G);
  if (leader) {
    s_grp[tid] = g;
    s_gadapter[g] = a;
    s_grank[g] = myrow.rank;
    s_gscale[g] = myrow.scale;
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

  // Work items are per warp: (token block, K chunk, group of eight rank rows).  K chunks: enough
  // items for every warp of the grid, but a chunk keeps at least four K steps (1024 elements)
  // unless h_in is shorter, so that the ring's ramp-up is amortised.
  const int n_ksteps = (h_in + 255) >> 8;
  const int n_rgn = R_pad >> 3;  // row groups of the rank stride: 2, 4 or 8
  int KS = (target_items + max(NB * n_rgn, 1) - 1) / max(NB * n_rgn, 1);
  KS = max(1, min(min(KS, kMaxZSplits), n_ksteps / 4));
  const int spc = (n_ksteps + KS - 1) / KS;
  KS = (n_ksteps + spc - 1) / spc;

  // Earlier kernels on the stream may still read the plan and z, so every write to them below comes
  // after griddepcontrol.wait; the operand loads (the pool and x are not written by this library's
  // kernels) start before it.
  const bool publisher = blockIdx.x == gridDim.x - 1;

  // ---- the last CTA publishes the plan in canonical order (ids ascending, -1 first): everything
  // is worked out in shared memory and registers first, the stores come after the wait
  if (publisher) publish_decode_plan(pv, a, T, any_bad, KS, s_id, s_cnt, s_wt);

  // ---- per-warp work items, no CTA-wide synchronisation from here on
  const int n_items = NB * KS * n_rgn;
  const size_t zplane = static_cast<size_t>(max_tokens) * R_pad;
  uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(s_ring_raw) + 127) & ~uintptr_t(127)) +
                  static_cast<size_t>(warp) * kDsDepth * kDsStageBytes;
  uint64_t *bars = s_bars[warp];
  uint32_t phase = 0;
  bool ok = true, waited = publisher;
  // Items are drawn from a ticket counter so that warps stay busy whatever the items cost; the
  // next ticket is drawn before the current item is processed.  The very last draw of the launch
  // (item number n_items + warps - 1) puts the counter back to zero.
  // (the publishing CTA takes no items: nothing that the next kernel waits for queues behind it)
  const int warps_total = (gridDim.x - 1) * (kShrinkThreads / 32);
  int32_t *ticket = group_counters + kDsTicket;
  int item = publisher ? n_items : blockIdx.x * (kShrinkThreads / 32) + warp;  // first round is static
  // The warp that completes a (group, row group) adds the K chunks in order into the final plane;
  // it never waits for the others.  (Run at the end of the item, with the ring drained: its
  // release is a fence, and a fence behind copies in flight waits for them too - putting it off
  // into the next item's ramp-up measured slower.)
  int pend_gi = -1, pend_rg = 0, pend_gt0 = 0, pend_gend = 0;
  auto finalize = [&]() {
    if (pend_gi < 0) return;
    const int arrivals = KS * ((pend_gend - pend_gt0 + kDsBlockTok - 1) / kDsBlockTok);
    __syncwarp();  // the lanes' z stores happen before lane 0's release
    int old = 0;
    if (lane == 0) old = atomic_add_acq_rel(&group_counters[pend_gi * 8 + pend_rg], 1);
    old = __shfl_sync(0xffffffffu, old, 0);
    if (old == arrivals - 1) {
      if (lane == 0) group_counters[pend_gi * 8 + pend_rg] = 0;  // ready for the next launch
      for (int idx = lane; idx < (pend_gend - pend_gt0) * 8; idx += 32) {
        const int tq = idx >> 3;
        const size_t off = static_cast<size_t>(s_gtok[pend_gt0 + tq]) * R_pad + pend_rg * 8 + (idx & 7);
        float part[kMaxZSplits];
#pragma unroll
        for (int sp = 0; sp < kMaxZSplits; ++sp) part[sp] = sp < KS ? __ldcg(zws + sp * zplane + off) : 0.f;
        float sum = 0.f;
#pragma unroll
        for (int sp = 0; sp < kMaxZSplits; ++sp) sum += part[sp];
        zws[kMaxZSplits * zplane + off] = sum;
      }
    }
    pend_gi = -1;
  };
  // When this launch may start under the kernels of the call before it (late_ticket), another
  // instance of this kernel can still be running, and the counter is theirs until this warp's
  // dependency wait has returned: the draw then comes after the wait, at the end of the item.
  const bool use_tickets = n_items > warps_total;  // otherwise the static first round is everything
  auto draw = [&]() {
    if (!use_tickets) return n_items;
    if (!waited) {
      ptx::pdl_wait_prior_grids();
      waited = true;
    }
    int n = 0;
    if (lane == 0) n = warps_total + atomicAdd(ticket, 1);
    return __shfl_sync(0xffffffffu, n, 0);
  };
  while (ok && item < n_items) {
    int next = 0;
    if (!late_ticket) {
      if (lane == 0 && use_tickets) next = warps_total + atomicAdd(ticket, 1);
      next = use_tickets ? __shfl_sync(0xffffffffu, next, 0) : n_items;
    }
    const int cur = item;
    // consecutive items are the K chunks of one (token block, row group), and chunk c takes the K
    // steps c, c + KS, c + 2 KS, ...: warps that run side by side fetch neighbouring 512-byte
    // pieces of the same rows at about the same time
    const int c = cur % KS;
    const int br = cur / KS;
    const int bi = br / n_rgn, rg = br - bi * n_rgn;
    const int gi = s_bgrp[bi];
    const int ad = s_gadapter[gi];
    const int rank = s_grank[gi];
    const float scale = s_gscale[gi];
    const int gt0 = s_gstart[gi], g_end = s_gstart[gi + 1];
    const int t0 = s_btok[bi], t1 = min(t0 + kDsBlockTok, g_end);
    if (rank <= 0) {
      if (lane == 0 && c == 0 && rg == 0 && t0 == gt0) atomicOr(status, EDGELORA_STATUS_SLOT_EMPTY);
      item = late_ticket ? draw() : next;
      continue;
    }
    const int n_rg = (rank + 7) >> 3;  // live groups of eight rows
    if (rg >= n_rg) {  // rows past the rank are zero padding: nothing to do
      item = late_ticket ? draw() : next;
      continue;
    }
    const int step0 = c, step1 = n_ksteps;
    const int q = lane & 3, r = rg * 8 + (lane >> 2);
    for (int tb = t0; ok && tb < t1; tb += kDsTok) {
      const int nt = min(kDsTok, t1 - tb);
      float acc[8 * kDsTok];
#pragma unroll
      for (int i = 0; i < 8 * kDsTok; ++i) acc[i] = 0.f;
      int32_t tok[kDsTok];
#pragma unroll
      for (int qq = 0; qq < kDsTok; ++qq) tok[qq] = s_gtok[tb + min(qq, nt - 1)];
      if (nt == 1) ok = shrink_rows8<1, kDsDepth, kQ8>(&tmap_a, &tmap_d, &tmap_x, ad, rg * 8, tok, step0, step1, KS, ring, bars, phase, lane, acc);
      else if (nt == 2) ok = shrink_rows8<2, kDsDepth, kQ8>(&tmap_a, &tmap_d, &tmap_x, ad, rg * 8, tok, step0, step1, KS, ring, bars, phase, lane, acc);
      else if (nt == 3) ok = shrink_rows8<3, kDsDepth, kQ8>(&tmap_a, &tmap_d, &tmap_x, ad, rg * 8, tok, step0, step1, KS, ring, bars, phase, lane, acc);
      else ok = shrink_rows8<4, kDsDepth, kQ8>(&tmap_a, &tmap_d, &tmap_x, ad, rg * 8, tok, step0, step1, KS, ring, bars, phase, lane, acc);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
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
      if (!waited) {  // first write of this warp to memory that earlier kernels may read
        ptx::pdl_wait_prior_grids();
        waited = true;
      }
      if (q < nt && EL_CHECK(status, s_gtok[tb + q] >= 0 && s_gtok[tb + q] < max_tokens && ad >= 0 && ad < n_slots, 20))
        zws[(KS > 1 ? c : kMaxZSplits) * zplane + static_cast<size_t>(s_gtok[tb + q]) * R_pad + r] =
            scale * acc[0];
    }
    if (!ok) break;
    item = late_ticket ? draw() : next;
    if (KS > 1) {
      pend_gi = gi;
      pend_rg = rg;
      pend_gt0 = gt0;
      pend_gend = g_end;
      finalize();
    }
  }
  // Every warp stops at its first ticket >= n_items, so exactly n_items - (first round) + warps
  // draws happen; the one that drew the last ticket resets the counter for the next launch.
  if (lane == 0 && ok && !publisher && use_tickets) {
    const int first_round = min(n_items, warps_total);
    const int last_ticket = warps_total + (n_items - first_round) + first_round - 1;
    if (item == last_ticket) *ticket = 0;
  }
  if (!ok && lane == 0) atomicOr(status, EDGELORA_STATUS_TIMEOUT);
}

// The shared-memory limit is an attribute of (function, device): set for the current device, by
// edgelora_pool_create, so that every device a pool lives on is configured.
cudaError_t shrink_set_smem_limit() {
  cudaError_t e = cudaSuccess;
  const int b4 = static_cast<int>(ds_ring_bytes(4)), b2 = static_cast<int>(ds_ring_bytes(2));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_shrink_kernel<4, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, b4);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_shrink_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, b2);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_shrink_kernel<4, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, b4);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_shrink_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, b2);
  return e;
}

cudaError_t launch_decode_shrink(const CUtensorMap &tmap_a, const CUtensorMap &tmap_d, const CUtensorMap &tmap_x,
                                 const int32_t *ids, const SlotRow *slots, const PlanView &pv,
                                 float *zws, int32_t *group_counters, int32_t T, int32_t h_in,
                                 int32_t R_pad, int32_t n_slots, int32_t max_tokens,
                                 int32_t target_items, int32_t grid, uint32_t *status, bool pdl, bool a_q8,
                                 int32_t depth, cudaStream_t stream) {
  const int32_t late_ticket = pdl ? 1 : 0;  // pdl here = this launch may start under the call before it
#define EDGELORA_SHRINK(D, Q)                                                                                     \
  launch_ex(decode_shrink_kernel<D, Q>, dim3(grid), dim3(kShrinkThreads), ds_ring_bytes(D), stream, pdl, 1, tmap_a, \
            tmap_d, tmap_x, ids, slots, pv, zws, group_counters, T, h_in, R_pad, n_slots, max_tokens, target_items,        \
            late_ticket, status)
  if (depth == 2) return a_q8 ? EDGELORA_SHRINK(2, true) : EDGELORA_SHRINK(2, false);
  return a_q8 ? EDGELORA_SHRINK(4, true) : EDGELORA_SHRINK(4, false);
#undef EDGELORA_SHRINK
}

}  // namespace edgelora
