// tcgen05 / TMEM / TMA bf16 GEMM for batch LoRA inference (paper Section 3.4): the base product
// W [x_0 .. x_n] batched over every token, with the low-rank expand B_a z folded into the same
// accumulator so that y is written once.
//
// D[128 x BN] (fp32, in tensor memory) = R[128 x K] * C[BN x K]^T, both operands K-major bf16 in
// 128-byte-swizzled shared-memory tiles of 64 K elements ("K blocks"), multiplied by tcgen05.mma
// issued from one thread.  A tile's K blocks are the K blocks of h_in followed by one "LoRA
// K block" per adapter the tile touches: its operands are B_a (fetched by TMA, zero-filled beyond
// the rank stride) and the tokens' z rounded to bf16, masked to the tokens of that adapter and
// written into the operand tile by four builder warps.  Modes (GemmParams::mode):
//
//   prefill  R = 128 tokens of x,  C = BN rows of W;  LoRA blocks: R = masked z, C = B_a rows.
//            Persistent over tiles, two TMEM accumulators so the epilogue of one tile overlaps the
//            main loop of the next.  Epilogue: y = bf16(D).
//   decode   R = 128 rows of W,    C = all tokens (N = T rounded up); LoRA blocks: R = B_a rows,
//            C = masked z.  W is streamed once; K and the LoRA groups are split across CTAs so
//            every SM pulls from HBM.  The K splits of one row tile form a thread-block cluster:
//            after the main loop every CTA sends its fp32 partial tile, column block by column
//            block, into the shared memory of the CTA that owns those tokens (distributed shared
//            memory), and each owner adds the partials in a fixed order and writes its part of y.
//   sgmv     R = 128 tokens of one run, C = A_a (N = rank stride): the segment shrink
//            z = s_a A_a x for long runs, tile list from the plan.  No LoRA blocks.
//
// Warp roles: warp 0 issues TMA, warp 1 owns TMEM and issues the MMAs, warps 2..5 are the
// epilogue (each reads the 32 TMEM lanes of its quadrant), warps 6..9 build the z operand.
// Every mbarrier wait is bounded; on a timeout the status word gets EDGELORA_STATUS_TIMEOUT and
// all roles leave their loops.
#include <cstdio>
#include <cstdlib>

#include "decode_route.cuh"
#include "internal.cuh"
#include "launch.cuh"
#include "ptx.cuh"

namespace edgelora {

struct TileCoord {
  int32_t row_r;   // first row of the R operand tile
  int32_t row_c;   // first row of the C operand tile
  int32_t slot;    // sgmv: slot whose A block is the C operand
  int32_t kb0, kb1;
  int32_t split;
  int32_t nrows;   // sgmv: tokens of the tile that belong to the run
  int32_t mtile;   // prefill: token tile; decode: W row tile
  // gather tiles of a shrink job: R = the A blocks of `ng` consecutive LoRA groups stacked (R_pad rows
  // each), C = the rows of x of those groups' tokens, fetched one by one
  int32_t kind;    // 0 regular, 1 gather
  int32_t g0, ng;  // first group (index into the plan's group arrays) and number of groups
  int32_t tok0, ntok;  // the groups' tokens: perm_short[tok0 .. tok0 + ntok)
  int32_t gtile;   // index of the gather tile (its arrival counter)
};

// K splits of the gather tiles when the host leaves the choice to the device (it does not know
// how many adapters a batch touches): the split count up to 8 whose (tile, split) items fill whole
// waves of the grid best, each split keeping at least four K blocks.
__device__ __forceinline__ int32_t gather_splits(const GemmParams &p, int32_t n_gt, int32_t grid) {
  if (p.splits > 0) return p.splits;
  int32_t best = 1;
  float best_eff = 0.f;
  for (int32_t sp = 1; sp <= 8 && p.kb_total / sp >= 4; ++sp) {
    if ((sp - 1) * ((p.kb_total + sp - 1) / sp) >= p.kb_total) continue;  // every split needs a K block
    const int32_t items = n_gt * sp, waves = (items + grid - 1) / grid;
    const float eff = waves > 0 ? static_cast<float>(items) / static_cast<float>(waves * grid) : 0.f;
    if (eff > best_eff + 0.02f) {
      best_eff = eff;
      best = sp;
    }
  }
  return best;
}
// LoRA groups (ids >= 0) of the batch per gather tile, and the number of gather tiles.
__device__ __forceinline__ int32_t gather_tiles(const GemmParams &p) {
  if (!p.gather) return 0;
  const int32_t per = kTileM / p.R_pad;
  return (p.counts[4] + per - 1) / per;
}

// Prefill jobs: tiles are dealt round-robin to the CTAs of the persistent grid, so when the tile count
// is not a multiple of the grid the CTAs from (count % grid) on get one tile fewer.  The tiles of the
// first token tile go to those CTAs: in a serving batch the first token tile holds the decode tokens
// (one token per generating request, many adapters, so many LoRA K blocks), and its tiles are the
// longest of the launch.  Returns how many tiles are placed that way (tile_coord says where).
// Only for launches of a site set (heavy_first).
__device__ __forceinline__ int32_t heavy_slots(const GemmParams &p, int32_t grid) {
  const int32_t total = p.n_mtiles * p.n_ntiles, rem = total % grid;
  if (p.mode != kModePrefill || !p.heavy_first || p.n_mtiles < 2 || total <= grid || rem == 0) return 0;
  return min(p.n_ntiles, grid - rem);
}

__device__ __forceinline__ int32_t total_tiles(const GemmParams &p) {
  if (p.mode == kModePrefill) return p.n_mtiles * p.n_ntiles;
  if (p.mode == kModeDecode) return p.n_mtiles * p.splits;
  const int32_t n_gt = gather_tiles(p);
  return p.counts[2] * max(p.splits, 1) + n_gt * gather_splits(p, n_gt, gridDim.x);
}

__device__ __forceinline__ TileCoord tile_coord(const GemmParams &p, int32_t tile) {
  TileCoord c;
  c.slot = 0;
  c.nrows = kTileM;
  c.kind = 0;
  c.g0 = c.ng = c.tok0 = c.ntok = c.gtile = 0;
  int32_t kb_per = p.kb_per;
  if (p.mode == kModePrefill) {
    int m, n;
    const int32_t H = heavy_slots(p, gridDim.x);
    const int32_t rem = (p.n_mtiles * p.n_ntiles) % static_cast<int32_t>(gridDim.x);
    if (H > 0) {
      // Position `tile` is step tile / grid of CTA tile % grid.  The tile (0, j) sits on CTA rem + j, at
      // the step at which the sweep over the other tiles (column by column, below) is at column j, so
      // that the W tile it needs is the one the launch is reading anyway.  pos(j) grows with j: the
      // number of placed tiles in front of a position is found by bisection.
      const int32_t grid = static_cast<int32_t>(gridDim.x);
      const int32_t last_step = (p.n_mtiles * p.n_ntiles) / grid - 1;  // last step of a CTA with a tile fewer
      auto pos = [&](int32_t j) { return min(last_step, (j * (p.n_mtiles - 1)) / grid) * grid + rem + j; };
      int32_t lo = 0, hi = H;
      while (lo < hi) {
        const int32_t mid = (lo + hi) >> 1;
        if (pos(mid) < tile) lo = mid + 1;
        else hi = mid;
      }
      if (lo < H && pos(lo) == tile) {
        m = 0;
        n = lo;
      } else {  // the other tiles in their usual order, the H placed ones taken out
        const int32_t u = tile - lo;
        if (u < H * (p.n_mtiles - 1)) {
          n = u / (p.n_mtiles - 1);
          m = 1 + u % (p.n_mtiles - 1);
        } else {
          const int32_t o = u + H;
          n = o / p.n_mtiles;
          m = o % p.n_mtiles;
        }
      }
    } else {
      m = tile % p.n_mtiles;
      n = tile / p.n_mtiles;
    }
    c.row_r = m * kTileM;
    c.row_c = n * p.BN;
    c.split = 0;
    c.mtile = m;
  } else if (p.mode == kModeDecode) {
    const int m = tile / p.splits;  // the splits of a row tile are consecutive CTAs: one cluster
    c.split = tile - m * p.splits;
    c.row_r = m * kTileM;
    c.row_c = 0;
    c.mtile = m;
  } else {
    const int n_t = p.counts[2];
    const int n_seg_items = n_t * max(p.splits, 1);
    c.row_c = 0;
    c.mtile = 0;
    if (tile < n_seg_items) {
      const int st = tile % n_t;
      c.split = tile / n_t;
      c.row_r = p.sgmv_tiles[4 * st + 0];
      c.nrows = p.sgmv_tiles[4 * st + 1];
      c.slot = p.sgmv_tiles[4 * st + 2];
      if (!EL_CHECK(p.status, c.row_r >= 0 && c.nrows >= 0 && c.row_r + c.nrows <= p.T && c.slot >= 0 && c.slot < p.n_slots, 4)) {
        c.row_r = 0;  // a tile of no rows: computed, nothing written
        c.nrows = 0;
        c.slot = 0;
      }
    } else {
      const int n_gt = gather_tiles(p);
      const int gsp = gather_splits(p, n_gt, gridDim.x);
      const int g = tile - n_seg_items;
      const int per = kTileM / p.R_pad;
      const int n_groups = p.counts[0], n_lg = p.counts[4];
      c.kind = 1;
      c.gtile = g % n_gt;
      c.split = g / n_gt;
      c.g0 = (n_groups - n_lg) + c.gtile * per;  // the group of id -1, when there is one, comes first
      c.ng = min(per, n_groups - c.g0);
      c.tok0 = p.gs_short[c.g0];
      c.ntok = p.gs_short[c.g0 + c.ng] - c.tok0;
      c.row_r = 0;
      kb_per = (p.kb_total + gsp - 1) / gsp;
    }
  }
  c.kb0 = c.split * kb_per;
  c.kb1 = min(p.kb_total, c.kb0 + kb_per);
  if (c.kb1 < c.kb0) c.kb1 = c.kb0;
  return c;
}
// Passes over a tile: a gather tile with more tokens than one pass holds takes several.
__device__ __forceinline__ int32_t tile_passes(const GemmParams &p, const TileCoord &c) {
  return c.kind == 1 ? (c.ntok + p.gN - 1) / p.gN : 1;
}

// decode: first W row of the tile this CTA works on
__device__ __forceinline__ int32_t tc_row0(const GemmParams &p, int32_t bid) {
  return bid / p.splits * kTileM;
}

// The LoRA K blocks of a tile: entries [e0, e1) step `de` of `list`.  Entries whose slot is
// empty are skipped by every role alike (they all read the same slot table).
struct LoraList {
  const int32_t *list;
  int32_t e0, e1, de;
};
__device__ __forceinline__ LoraList lora_list(const GemmParams &p, const TileCoord &tc,
                                              const int32_t *s_lg, const volatile int32_t *s_nlg) {
  LoraList l;
  if (p.mode == kModePrefill) {
    l.list = p.mt_list + tc.mtile * kTileM;
    l.e0 = 0;
    l.e1 = p.mt_count[tc.mtile];
    l.de = 1;
  } else if (p.mode == kModeDecode) {
    l.list = s_lg;    // built by this CTA from the ids (see the builder warps)
    l.e0 = tc.split;  // the groups are dealt round-robin to the K splits of a row tile
    l.e1 = *s_nlg;
    l.de = p.splits;
  } else {
    l.list = nullptr;
    l.e0 = l.e1 = 0;
    l.de = 1;
  }
  return l;
}

__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
// Barrier over every thread of every CTA of the cluster (a hardware barrier: all of them reach it,
// on the time-out paths too, because no role loop is unbounded).
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_cta_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the same shared-memory offset in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void st_cluster_f32x4(uint32_t addr, float a, float b, float c, float d) {
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d)
               : "memory");
}

// z of token t as packed bf16 (eight 16-byte chunks; chunks at or past the rank stride are zero):
// the partial planes are added in order, values at or past the true rank forced to zero.
__device__ __forceinline__ void load_z_packed(const GemmParams &p, int32_t t, int32_t rank,
                                              uint4 (&out)[8]) {
  if (!EL_CHECK(p.status, rank <= p.R_pad && t >= 0 && t < p.max_tokens, 3)) {
    rank = 0;  // all zeros, read from row 0
    t = 0;
  }
  const int nch = p.R_pad >> 3;
  const float *zt = p.zws + static_cast<size_t>(t) * p.R_pad;
  const size_t plane = static_cast<size_t>(p.max_tokens) * p.R_pad;
#pragma unroll
  for (int c0 = 0; c0 < 8; c0 += 4) {
    float acc[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) acc[i] = 0.f;
    if (c0 < nch) {
      for (int sp = 0; sp < p.zsplits; ++sp) {
        const float4 *zp = reinterpret_cast<const float4 *>(zt + sp * plane) + 2 * c0;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          if (c0 + c < nch) {
            const float4 u = __ldcg(zp + 2 * c), w = __ldcg(zp + 2 * c + 1);
            acc[c * 8 + 0] += u.x; acc[c * 8 + 1] += u.y; acc[c * 8 + 2] += u.z; acc[c * 8 + 3] += u.w;
            acc[c * 8 + 4] += w.x; acc[c * 8 + 5] += w.y; acc[c * 8 + 6] += w.z; acc[c * 8 + 7] += w.w;
          }
        }
      }
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
#define EL(i) (((c0 + c) * 8 + (i)) < rank ? acc[c * 8 + (i)] : 0.f)
      out[c0 + c].x = ptx::pack_bf16x2(EL(0), EL(1));
      out[c0 + c].y = ptx::pack_bf16x2(EL(2), EL(3));
      out[c0 + c].z = ptx::pack_bf16x2(EL(4), EL(5));
      out[c0 + c].w = ptx::pack_bf16x2(EL(6), EL(7));
#undef EL
    }
  }
}

// The copies of one pass over a gather tile, K blocks [kb0, kb1).  A K block needs one copy per
// group of the tile (its A block, R_pad rows of the R operand) and one per token quad (four rows of
// x into the C operand).  A TMA copy is issued from a warp's uniform datapath, one lane after the
// other at roughly a hundred cycles each, so the copies of a K block are dealt out to kGatherParts
// warps (the producer warp is part 0 and also posts the byte count; the four builder warps, idle
// during shrink tiles, are parts 1..4): copy i goes to part i % kGatherParts, lane i / kGatherParts.
// The parts other than the producer follow it the way the builder warps follow it through LoRA
// K blocks: the producer announces a free stage on the stage's "go" barrier, every other part
// waits for that, issues its copies and arrives on the stage's "z full" barrier, which the MMA
// warp waits for beside the byte count.  (Waiting on the stage's empty barrier directly would not
// do: a part that has nothing to copy for a while can get several ring revolutions ahead, and a
// parity wait cannot tell revolutions apart.)  A copy that lands before the byte count is posted
// only drives the barrier's transaction count below zero for a moment.
constexpr int kGatherParts = 5;
__device__ __forceinline__ bool gather_pass_copies(const GemmParams &jp, const TileCoord &tc, int32_t t0,
                                                   const CUtensorMap *ma, const CUtensorMap *mg, uint8_t *smem,
                                                   uint32_t stage_bytes, uint64_t *full_bar, uint64_t *empty_bar,
                                                   uint64_t *zgo_bar, uint64_t *zfull_bar,
                                                   volatile uint32_t *abort_flag, uint32_t nstages, long long wl,
                                                   int part, int lane, uint32_t &stage, uint32_t &phase,
                                                   uint32_t &gophase) {
  const uint32_t r_bytes = kTileM * kBlockK * 2;
  const uint32_t a_bytes = static_cast<uint32_t>(jp.R_pad) * kBlockK * 2;
  const int32_t n = min(jp.gN, tc.ntok - t0);
  const int32_t n_quads = (n + 3) >> 2;
  // live groups of the tile (an empty slot has no A block to fetch), for the byte count
  int32_t slot_l = -1;
  if (lane < tc.ng) {
    const int32_t a = jp.group_adapter[tc.g0 + lane];
    if (a >= 0 && jp.slots[a].rank > 0) slot_l = a;
  }
  const uint32_t live_mask = __ballot_sync(0xffffffffu, slot_l >= 0);
  const uint32_t tx = __popc(live_mask) * a_bytes + static_cast<uint32_t>(n_quads) * 4 * kBlockK * 2;
  // this lane's copy
  const int32_t item = part + kGatherParts * lane;
  int32_t my_slot = -1, my_quad = -1, tok[4] = {0, 0, 0, 0};
  const int32_t slot_of_item = __shfl_sync(0xffffffffu, slot_l, item < tc.ng ? item : 0);
  if (item < tc.ng) {
    my_slot = slot_of_item;
  } else {
    if (item - tc.ng < n_quads) {
      my_quad = item - tc.ng;
#pragma unroll
      for (int i = 0; i < 4; ++i)  // rows past the pass's last token repeat it (they land in unused columns)
      {
        tok[i] = jp.perm_short[tc.tok0 + t0 + min(my_quad * 4 + i, n - 1)];
        if (!EL_CHECK(jp.status, tok[i] >= 0 && tok[i] < jp.T, 5)) tok[i] = 0;
      }
    }
  }
  for (int32_t kb = tc.kb0; kb < tc.kb1; ++kb) {
    int got = 1;
    if (lane == 0) {
      if (part == 0)
        got = (ptx::mbar_wait(&empty_bar[stage], phase ^ 1, wl) && !*abort_flag) ? 1 : 0;
      else
        got = (ptx::mbar_wait(&zgo_bar[stage], (gophase >> stage) & 1u, wl) && !*abort_flag) ? 1 : 0;
    }
    if (!__shfl_sync(0xffffffffu, got, 0)) return false;
    gophase ^= 1u << stage;
    uint8_t *sr = smem + static_cast<size_t>(stage) * stage_bytes;
    if (part == 0 && lane == 0) {
      ptx::mbar_arrive(&zgo_bar[stage]);
      ptx::mbar_arrive_expect_tx(&full_bar[stage], tx);
    }
    if (my_slot >= 0)
      ptx::tma_load_2d(sr + static_cast<size_t>(item) * a_bytes, ma, &full_bar[stage], kb * kBlockK,
                       my_slot * jp.R_pad);
    if (my_quad >= 0)
      ptx::tma_gather4_2d(sr + r_bytes + static_cast<size_t>(my_quad) * (4 * kBlockK * 2), mg, &full_bar[stage],
                          kb * kBlockK, tok[0], tok[1], tok[2], tok[3]);
    if (part != 0) {
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&zfull_bar[stage]);
    }
    if (++stage == nstages) {
      stage = 0;
      phase ^= 1;
    }
  }
  return true;
}

__device__ __forceinline__ int32_t ld_acquire_gpu(const int32_t *ptr) {
  int32_t v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
  return v;
}

// Fused decode launches (batches of at most 64 tokens): z[t] = s_a A_a x[t] on the CUDA cores, by
// "teams" of four warps: the four builder warps of every CTA of the decode job (idle there, because
// the expand is added by the owners of the cluster reduction) and two teams in every spare CTA.
// A team item is (token, eight rank rows, K chunk): chunk c covers the K steps c, c + ks, ... of 256
// elements; warp w of the team takes every fourth of them, lane l the elements [8 l, 8 l + 8) of a
// step (one 16-byte load of x and eight of A in flight per lane).  The four warps' sums meet in
// shared memory and are added in a fixed order; the partial result goes to plane c of f.z, and the
// expand adds the planes in order.  Rows at or past the rank are never read by the expand and are
// not written.  s_tid / s_trank / s_tscale: the tokens' validated ids, ranks and scales in shared
// memory; s_red: 48 floats; bar_id: a named barrier of the team's 128 threads.
template <int kBarId>
__device__ __forceinline__ void shrink_team_items(const GemmParams &p, const FusedDecode &f, int team, int n_teams,
                                                  int wt, int lane, const int32_t *s_tid, const int32_t *s_trank,
                                                  const float *s_tscale, float *s_red, bool &waited) {
  const int n_ksteps = (p.h_in + kShrinkStepElems - 1) / kShrinkStepElems;
  const int n_rgn = p.R_pad >> 3, KS = f.ks;
  const int n_items = p.T * n_rgn * KS;
  const size_t zplane = static_cast<size_t>(p.max_tokens) * p.R_pad;
  const int row_u4 = p.h_in >> 3;  // 16-byte pieces of a row (h_in is a multiple of 8)
  int par = 0;
  for (int item = team; item < n_items; item += n_teams) {
    const int c = item % KS, tr = item / KS;
    const int t = tr / n_rgn, rg = tr - t * n_rgn;
    const int at = s_tid[t], rank = s_trank[t];
    if (at < 0) continue;
    if (rank <= 0) {
      if (wt == 0 && lane == 0 && c == 0 && rg == 0) atomicOr(p.status, EDGELORA_STATUS_SLOT_EMPTY);
      continue;
    }
    if (rg * 8 >= rank) continue;  // zero padding of the block
    const uint4 *Arow =
        reinterpret_cast<const uint4 *>(f.A_pool + (static_cast<size_t>(at) * p.R_pad + rg * 8) * p.h_in);
    const uint4 *xrow = reinterpret_cast<const uint4 *>(f.x + static_cast<size_t>(t) * p.h_in);
    float acc[8];
#pragma unroll
    for (int r = 0; r < 8; ++r) acc[r] = 0.f;
    for (int s0 = c + KS * wt; s0 < n_ksteps; s0 += 4 * KS) {
      const int k0 = s0 * 32 + lane;
      if (k0 >= row_u4) continue;
      uint4 av[8];
      const uint4 xv = __ldcg(xrow + k0);
#pragma unroll
      for (int r = 0; r < 8; ++r) av[r] = __ldg(Arow + static_cast<size_t>(r) * row_u4 + k0);
      const float xf[8] = {ptx::bf16_lo(xv.x), ptx::bf16_hi(xv.x), ptx::bf16_lo(xv.y), ptx::bf16_hi(xv.y),
                           ptx::bf16_lo(xv.z), ptx::bf16_hi(xv.z), ptx::bf16_lo(xv.w), ptx::bf16_hi(xv.w)};
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        float v = acc[r];
        v = fmaf(ptx::bf16_lo(av[r].x), xf[0], v);
        v = fmaf(ptx::bf16_hi(av[r].x), xf[1], v);
        v = fmaf(ptx::bf16_lo(av[r].y), xf[2], v);
        v = fmaf(ptx::bf16_hi(av[r].y), xf[3], v);
        v = fmaf(ptx::bf16_lo(av[r].z), xf[4], v);
        v = fmaf(ptx::bf16_hi(av[r].z), xf[5], v);
        v = fmaf(ptx::bf16_lo(av[r].w), xf[6], v);
        v = fmaf(ptx::bf16_hi(av[r].w), xf[7], v);
        acc[r] = v;
      }
    }
    float out = 0.f;
#pragma unroll
    for (int r = 0; r < 8; ++r) {
      float v = acc[r];
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
      if (lane == r) out = v;
    }
    // buffer `par` is written again two items later, behind the next item's barrier, which warp 0
    // reaches only after it has read this item's sums
    if (wt > 0 && lane < 8) s_red[(par * 3 + wt - 1) * 8 + lane] = out;
    named_bar_sync(kBarId, 128);
    if (wt == 0) {
      if (!waited) {  // first write of this team to memory that earlier kernels may read
        ptx::pdl_wait_prior_grids();
        waited = true;
      }
      if (lane < 8) {
        const float sum = ((out + s_red[(par * 3 + 0) * 8 + lane]) + s_red[(par * 3 + 1) * 8 + lane]) +
                          s_red[(par * 3 + 2) * 8 + lane];
        f.z[c * zplane + static_cast<size_t>(t) * p.R_pad + rg * 8 + lane] = s_tscale[t] * sum;
      }
    }
    par ^= 1;
  }
  if (wt == 0) {
    __syncwarp();  // the lanes' z stores happen before lane 0's release
    if (lane == 0) {
      ptx::pdl_wait_prior_grids();  // the counters belong to the kernel before this one until it is done
      __threadfence();
      atomicAdd(f.sync, 1);
    }
  }
}

// A spare CTA of a fused decode launch: two shrink teams (warps 0..3 and 4..7); the first spare CTA
// also publishes the routing plan.
__device__ __forceinline__ void fused_shrink_cta(const GemmParams &p, const FusedDecode &f, uint8_t *smem, int n_teams) {
  int32_t *s_id = reinterpret_cast<int32_t *>(smem);  // [256] validated ids
  int32_t *s_cnt = s_id + 256;                        // [256] scratch of the plan publication
  int32_t *s_rank = s_cnt + 256;                      // [256]
  float *s_scale = reinterpret_cast<float *>(s_rank + 256);  // [256]
  float *s_red = s_scale + 256;                              // [2][48]
  int *s_wt = reinterpret_cast<int *>(s_red + 96);           // [9]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  ptx::pdl_launch_dependents();
  int a = -1;
  bool bad = false;
  if (tid < p.T) {
    a = p.ids[tid];
    if (a < -1 || a >= p.n_slots) {
      a = -1;
      bad = true;
    }
  }
  SlotRow row = {0, 0.f, 0, 0};
  if (a >= 0) row = p.slots[a];
  if (tid < 256) {
    s_id[tid] = a;
    s_rank[tid] = row.rank;
    s_scale[tid] = row.scale;
  }
  const int any_bad = __syncthreads_or(bad ? 1 : 0);
  bool waited = false;
  if (f.x_wait) {
    ptx::pdl_wait_prior_grids();
    waited = true;
  }
  if (warp < 4)
    shrink_team_items<2>(p, f, static_cast<int>(blockIdx.x) * 2, n_teams, warp, lane, s_id, s_rank, s_scale, s_red,
                         waited);
  else if (warp < 8)
    shrink_team_items<3>(p, f, static_cast<int>(blockIdx.x) * 2 + 1, n_teams, warp - 4, lane, s_id, s_rank, s_scale,
                         s_red + 48, waited);
  if (blockIdx.x == 0) publish_decode_plan(f.pv, a, p.T, any_bad, f.ks, s_id, s_cnt, s_wt);
}

// kMinBlocks = 2 caps the registers so that two CTAs share an SM (small decode tiles); with 1 the
// builder keeps both of its z rows in registers without spilling.  kShrink = false compiles the
// kernel without the shrink jobs (segment and gather tiles, second job) and without the staged y
// stores: the decode-mode launches, which need none of them, keep a smaller kernel.
// kFused: a decode launch whose first f.n_ctas CTAs are shrink CTAs (fused_shrink_cta); the job's
// own CTAs are numbered from there.
template <int kMinBlocks, bool kShrink, bool kFused>
__global__ void __launch_bounds__(kGemmThreads, kMinBlocks)
lora_gemm_kernel(const __grid_constant__ CUtensorMap tmap_r, const __grid_constant__ CUtensorMap tmap_c,
                 const __grid_constant__ CUtensorMap tmap_b, const GemmParams p,
                 const __grid_constant__ CUtensorMap tmap_r2, const __grid_constant__ CUtensorMap tmap_c2,
                 const __grid_constant__ CUtensorMap tmap_g2, const GemmParams p2,
                 const __grid_constant__ CUtensorMap tmap_y, const FusedDecode f) {
  extern __shared__ uint8_t smem_raw[];
  // tiles need 1024-byte alignment for the 128-byte swizzle
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int32_t cta0 = kFused ? f.n_ctas : 0;  // whole clusters: the cluster ranks of the others are unchanged
  const int32_t ngrid0 = static_cast<int32_t>(gridDim.x) - cta0;
  if (kFused && static_cast<int32_t>(blockIdx.x) < cta0) {
    fused_shrink_cta(p, f, smem, 2 * cta0 + ngrid0);
    return;
  }
  const int32_t bid = static_cast<int32_t>(blockIdx.x) - cta0, ngrid = ngrid0;
  const uint32_t r_bytes = kTileM * kBlockK * 2;              // 16 KB
  const uint32_t c_bytes = static_cast<uint32_t>(p.BN) * kBlockK * 2;
  // the ring is laid out for the first job: its C region holds ring_rows rows
  const uint32_t stage_bytes = r_bytes + static_cast<uint32_t>(p.ring_rows) * kBlockK * 2;
  // Second job (optional): the segment shrink of ANOTHER linear site as extra tiles of this
  // persistent grid, after the first job's tiles.  Its tile list comes from a plan on the device, so
  // the host passes an upper bound (p2.n_mtiles) and every role stops at the true count, which it
  // reads after the dependency wait.  Its N tile is never wider than the first job's.
  const bool has2 = kShrink && p2.mode == kModeSgmv;
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + static_cast<size_t>(p.stages) * stage_bytes);
  uint64_t *full_bar = bars;                      // [stages]  TMA -> MMA
  uint64_t *empty_bar = bars + kMaxStages;        // [stages]  MMA -> TMA
  uint64_t *zfull_bar = bars + 2 * kMaxStages;    // [stages]  builder -> MMA (LoRA K blocks)
  uint64_t *zgo_bar = bars + 3 * kMaxStages;      // [stages]  TMA warp -> builder (stage is free)
  uint64_t *tfull_bar = bars + 4 * kMaxStages;    // [2]       MMA -> epilogue
  uint64_t *tempty_bar = tfull_bar + 2;           // [2]       epilogue -> MMA
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(tempty_bar + 2);
  volatile uint32_t *abort_flag = tmem_slot + 1;
  // decode extras, 512 bytes after the barriers: the batch's adapter list derived from the ids
  // by the builder warps
  uint8_t *extra = reinterpret_cast<uint8_t *>(bars) + 512;
  volatile int32_t *s_nlg = reinterpret_cast<volatile int32_t *>(extra + 64);
  uint64_t *lg_bar = reinterpret_cast<uint64_t *>(extra + 72);              // builder -> TMA, MMA
  int32_t *s_lg = reinterpret_cast<int32_t *>(extra + 128);                 // [256] ids ascending
  int32_t *s_vid = reinterpret_cast<int32_t *>(extra + 1152);               // [256] validated ids
  uint8_t *s_head = extra + 2176;                                           // [256]
  uint32_t *s_key = reinterpret_cast<uint32_t *>(extra + 2432);             // [256] sort keys
  volatile int32_t *s_last = reinterpret_cast<volatile int32_t *>(extra + 80);  // gather tiles: last arriver
  uint64_t *ep_bar = reinterpret_cast<uint64_t *>(extra + 88);              // rendezvous of the epilogue warps
  uint8_t *y_stage = reinterpret_cast<uint8_t *>(bars) + 4096;              // prefill epilogue: 4 x 4 KB, 1024-aligned
  uint8_t *b_stage = y_stage;  // fused decode: B_a rows of the owner's tokens, then their z (never both uses at once)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long wl = p.wait_cycles;  // limit of every bounded wait below
  // LoRA K blocks: prefill always; decode unless the batch is small enough for the expand to be
  // added by the owners of the cluster reduction (then z is needed only at the very end and the
  // whole main loop overlaps the shrink kernel)
  const bool has_lora = p.mode == kModePrefill || (p.mode == kModeDecode && !p.expand_in_reduce);

  if (threadIdx.x == 0) {
    ptx::prefetch_tensormap(&tmap_r);
    ptx::prefetch_tensormap(&tmap_c);
    if (has_lora) ptx::prefetch_tensormap(&tmap_b);
    if (has2) {
      ptx::prefetch_tensormap(&tmap_r2);
      ptx::prefetch_tensormap(&tmap_c2);
      if (p2.gather) ptx::prefetch_tensormap(&tmap_g2);
    }
    if (kShrink && p.mode == kModeSgmv && p.gather) ptx::prefetch_tensormap(&tmap_b);
    if (kShrink && p.y_tma) ptx::prefetch_tensormap(&tmap_y);
    for (int s = 0; s < p.stages; ++s) {
      ptx::mbar_init(&full_bar[s], 1);
      ptx::mbar_init(&empty_bar[s], 1);
      ptx::mbar_init(&zfull_bar[s], 4);  // one arrival per builder warp
      ptx::mbar_init(&zgo_bar[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&tfull_bar[i], 1);
      ptx::mbar_init(&tempty_bar[i], 4);  // one arrival per epilogue warp
    }
    ptx::mbar_init(lg_bar, 1);
    ptx::mbar_init(ep_bar, 4);  // one arrival per epilogue warp
    *abort_flag = 0;
    *s_nlg = 0;
    ptx::fence_barrier_init();
    if (kFused && f.x_wait) {
      // W is not written by any kernel of this library: this thread (lane 0 of the producer warp, which
      // has just initialised the barriers) requests the W tiles of the first ring revolution at once,
      // before the tensor-memory allocation and the CTA-wide barrier; the producer adds the x tiles
      // after its dependency wait
      const TileCoord tc0 = tile_coord(p, bid);
      const int32_t npre = min(p.stages, tc0.kb1 - tc0.kb0);
      for (int32_t i = 0; i < npre; ++i) {
        ptx::mbar_arrive_expect_tx(&full_bar[i], r_bytes + c_bytes);
        ptx::tma_load_2d(smem + static_cast<size_t>(i) * stage_bytes, &tmap_r, &full_bar[i], (tc0.kb0 + i) * kBlockK,
                         tc0.row_r);
      }
    }
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, static_cast<uint32_t>(p.tmem_cols));
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  // Every CTA of this grid now holds its tensor memory, so a dependent grid may start to launch.
  ptx::pdl_launch_dependents();

  if (p.mode == kModeSgmv) ptx::pdl_wait_prior_grids();  // tile list comes from the plan kernel
  const int32_t n_tiles0 = total_tiles(p);
  // Where the second job's tiles go.  Positions continue after the first job's, round-robin over the
  // CTAs, so the first of them fall on the CTAs that got one tile fewer (or none).  Those CTAs are free
  // for about a tile's time: they take fill_rounds of the second job's tiles each before the others
  // get any (the positions of the others are holes in those rounds); the CTAs that took the first
  // token tile's tiles, which are longer, sit out the first round (n_hole).
  const int32_t n_hole = has2 ? heavy_slots(p, gridDim.x) : 0;
  const int32_t rem0 = (has2 && p.mode == kModePrefill) ? n_tiles0 % ngrid : 0;
  const int32_t n_short = rem0 > 0 ? ngrid - rem0 : 0;
  const int32_t fill = max(1, p.fill_rounds);
  const int32_t n_tiles = n_tiles0 + (has2 ? p2.n_mtiles + (n_short > 0 ? n_short + (fill - 1) * ngrid : 0) : 0);
  const uint32_t nstages = static_cast<uint32_t>(p.stages);
  // Every role walks the same tile sequence: tiles below n_tiles0 belong to the first job; for the
  // others the true count of the second job is read once (after griddepcontrol.wait: the plan may
  // come from a kernel this one was allowed to start under) and the walk ends at it.
  int32_t n2_true = -1;
  auto second_job_tile = [&](int32_t tile) -> int32_t {  // local tile index, -2 = a hole, -1 = stop
    const int32_t q = tile - n_tiles0;
    int32_t local;
    if (n_short == 0) {
      local = q;
    } else if (q < n_short) {
      if (q < n_hole) return -2;
      local = q - n_hole;
    } else {
      const int32_t q2 = q - n_short, round = q2 / ngrid + 1, c = q2 % ngrid;
      if (round < fill) {
        if (c < rem0) return -2;
        local = (n_short - n_hole) + (round - 1) * n_short + (c - rem0);
      } else {
        local = (n_short - n_hole) + (fill - 1) * n_short + (round - fill) * ngrid + c;
      }
    }
    if (n2_true < 0) {
      ptx::pdl_wait_prior_grids();
      n2_true = total_tiles(p2);
    }
    return local < n2_true ? local : -1;
  };

  bool fused_z_ok = true;  // fused launches: set by the epilogue warps' wait for the shrink teams
  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    // The whole warp walks the loop (state stays uniform); lane 0 waits and issues the tile loads,
    // and for gather tiles every lane issues its share of the one-row loads.
    {
      uint32_t stage = 0, phase = 0, unused_go = 0;
      bool ok = true, waited = p.mode == kModeSgmv, x_waited = false;
      auto wait_empty = [&]() {  // lane 0 polls, the warp learns the result
        int got = 1;
        if (lane == 0) got = (ptx::mbar_wait(&empty_bar[stage], phase ^ 1, wl) && !*abort_flag) ? 1 : 0;
        return __shfl_sync(0xffffffffu, got, 0) != 0;
      };
      auto advance = [&]() {
        if (++stage == nstages) {
          stage = 0;
          phase ^= 1;
        }
      };
      for (int32_t tile = bid; ok && tile < n_tiles; tile += ngrid) {
        const bool second = tile >= n_tiles0;
        int32_t local = tile;
        if (second && (local = second_job_tile(tile)) < 0) {
          if (local == -2) continue;
          break;
        }
        const GemmParams &jp = second ? p2 : p;
        const CUtensorMap *mr = second ? &tmap_r2 : &tmap_r, *mc = second ? &tmap_c2 : &tmap_c;
        const TileCoord tc = tile_coord(jp, local);
        if (kShrink && tc.kind == 1) {
          // gather tile: this warp is part 0 of the copies (see gather_pass_copies)
          const CUtensorMap *mg = second ? &tmap_g2 : &tmap_b;
          for (int32_t t0 = 0; ok && t0 < tc.ntok; t0 += jp.gN)
            ok = gather_pass_copies(jp, tc, t0, mc, mg, smem, stage_bytes, full_bar, empty_bar, zgo_bar, zfull_bar,
                                    abort_flag, nstages, wl, 0, lane, stage, phase, unused_go);
          continue;
        }
        const uint32_t tx_bytes = r_bytes + static_cast<uint32_t>(jp.BN) * kBlockK * 2;
        int32_t kb_first = tc.kb0;
        if (kFused && f.x_wait && !x_waited) {
          // x may be an output of the kernel before this one, W is not: the W tiles of the first ring
          // revolution were requested in the prologue (with the bytes of both tiles announced), the x
          // tiles follow the dependency wait
          const int32_t npre = min(static_cast<int32_t>(nstages), tc.kb1 - tc.kb0);  // the ring is empty: no waits
          ptx::pdl_wait_prior_grids();
          if (lane == 0)
            for (int32_t i = 0; i < npre; ++i)
              ptx::tma_load_2d(smem + static_cast<size_t>(i) * stage_bytes + r_bytes, mc, &full_bar[i],
                               (tc.kb0 + i) * kBlockK, tc.row_c);
          for (int32_t i = 0; i < npre; ++i) advance();
          kb_first += npre;
          x_waited = true;
        }
        for (int32_t kb = kb_first; kb < tc.kb1; ++kb) {
          if (!wait_empty()) {
            ok = false;
            break;
          }
          if (lane == 0) {
            uint8_t *sr = smem + static_cast<size_t>(stage) * stage_bytes;
            ptx::mbar_arrive_expect_tx(&full_bar[stage], tx_bytes);
            ptx::tma_load_2d(sr, mr, &full_bar[stage], kb * kBlockK, tc.row_r);
            if (jp.mode == kModeSgmv)
              ptx::tma_load_2d(sr + r_bytes, mc, &full_bar[stage], kb * kBlockK, tc.slot * jp.R_pad);
            else
              ptx::tma_load_2d(sr + r_bytes, mc, &full_bar[stage], kb * kBlockK, tc.row_c);
          }
          advance();
        }
        if (!ok || !has_lora || second) continue;
        if (!waited) {
          if (p.mode == kModeDecode) {  // the builder warps derive the adapter list from the ids
            int got = 1;
            if (lane == 0) got = ptx::mbar_wait(lg_bar, 0, wl) ? 1 : 0;
            if (!__shfl_sync(0xffffffffu, got, 0)) {
              ok = false;
              break;
            }
          } else {                      // the tile lists come from the plan kernel
            ptx::pdl_wait_prior_grids();
          }
          waited = true;
        }
        const LoraList ll = lora_list(p, tc, s_lg, s_nlg);
        for (int32_t e = ll.e0; e < ll.e1; e += ll.de) {
          const int32_t a = ll.list[e];
          if (!EL_CHECK(p.status, a >= 0 && a < p.n_slots, 1)) continue;
          if (p.mode != kModeDecode && p.slots[a].rank <= 0) continue;
          if (!wait_empty()) {
            ok = false;
            break;
          }
          if (lane == 0) {
            // The stage is free: let the builder write its half (it follows this warp, never the
            // stage barriers directly, so it cannot run ahead of the ring).
            ptx::mbar_arrive(&zgo_bar[stage]);
            uint8_t *sr = smem + static_cast<size_t>(stage) * stage_bytes;
            if (p.mode == kModePrefill) {  // C operand: rows [row_c, row_c + BN) of B_a
              ptx::mbar_arrive_expect_tx(&full_bar[stage], c_bytes);
              ptx::tma_load_3d(sr + r_bytes, &tmap_b, &full_bar[stage], 0, tc.row_c, a);
            } else {                       // R operand: rows [row_r, row_r + 128) of B_a
              ptx::mbar_arrive_expect_tx(&full_bar[stage], r_bytes);
              ptx::tma_load_3d(sr, &tmap_b, &full_bar[stage], 0, tc.row_r, a);
            }
          }
          advance();
        }
      }
      if (!ok && lane == 0) {
        *abort_flag = 1;
        atomicOr(p.status, EDGELORA_STATUS_TIMEOUT);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const int lora_ksteps = p.R_pad / kUmmaK;
      uint32_t stage = 0, phase = 0, zphase = 0;  // zphase: one parity bit per stage
      bool ok = true, waited = p.mode == kModeSgmv;
      int32_t it = 0;
      for (int32_t tile = bid; ok && tile < n_tiles; tile += ngrid) {
        const bool second = tile >= n_tiles0;
        int32_t local = tile;
        if (second && (local = second_job_tile(tile)) < 0) {
          if (local == -2) continue;
          break;
        }
        const GemmParams &jp = second ? p2 : p;
        const TileCoord tc = tile_coord(jp, local);
        const int32_t n_pass = tile_passes(jp, tc);
        uint32_t acc = 0, tmem_d = tmem_base;
        for (int32_t pass = 0; ok && pass < n_pass; ++pass, ++it) {
          // UMMA N: the job's N tile, or for a gather pass its token count rounded up to 16
          const uint32_t n_cols = (kShrink && tc.kind == 1)
                                      ? static_cast<uint32_t>((min(jp.gN, tc.ntok - pass * jp.gN) + 15) & ~15)
                                      : static_cast<uint32_t>(jp.BN);
          const uint32_t idesc = ptx::umma_idesc_bf16(kTileM, n_cols);
          acc = (p.n_acc == 2) ? (it & 1) : 0;
          const uint32_t use = (p.n_acc == 2) ? (it >> 1) : it;
          if (!ptx::mbar_wait(&tempty_bar[acc], (use & 1) ^ 1, wl) || *abort_flag) {
            ok = false;
            break;
          }
          ptx::tc_fence_after_sync();
          tmem_d = tmem_base + acc * static_cast<uint32_t>(p.acc_cols);
          for (int32_t kb = tc.kb0; kb < tc.kb1; ++kb) {
            if (!ptx::mbar_wait(&full_bar[stage], phase, wl) || *abort_flag) {
              ok = false;
              break;
            }
            if (kShrink && tc.kind == 1) {  // the other parts of the tile's copies have been through this stage
              if (!ptx::mbar_wait(&zfull_bar[stage], (zphase >> stage) & 1u, wl)) {
                ok = false;
                break;
              }
              zphase ^= 1u << stage;
            }
            ptx::tc_fence_after_sync();
            const uint32_t sr = ptx::smem_u32(smem + static_cast<size_t>(stage) * stage_bytes);
            const uint64_t da = ptx::umma_desc_k128(sr);
            const uint64_t db = ptx::umma_desc_k128(sr + r_bytes);
#pragma unroll
            for (int k = 0; k < kBlockK / kUmmaK; ++k) {
              // advancing 16 bf16 along K inside the swizzled row = 32 bytes = 2 descriptor units
              ptx::umma_bf16(tmem_d, da + 2 * k, db + 2 * k, idesc, (kb > tc.kb0 || k > 0) ? 1u : 0u);
            }
            ptx::umma_commit(&empty_bar[stage]);  // frees the smem stage once these MMAs are done
            if (++stage == nstages) {
              stage = 0;
              phase ^= 1;
            }
          }
          if (!ok) break;
          // a gather pass is complete here; other tiles go on with their LoRA K blocks below
          if (kShrink && tc.kind == 1) ptx::umma_commit(&tfull_bar[acc]);
        }
        if (!ok) break;
        if (kShrink && tc.kind == 1) continue;
        const uint32_t idesc = ptx::umma_idesc_bf16(kTileM, static_cast<uint32_t>(jp.BN));
        if (!ok) break;
        if (has_lora && !second) {
          if (!waited) {
            if (p.mode == kModeDecode) {
              if (!ptx::mbar_wait(lg_bar, 0, wl)) {
                ok = false;
                break;
              }
            } else {
              ptx::pdl_wait_prior_grids();
            }
            waited = true;
          }
          const LoraList ll = lora_list(p, tc, s_lg, s_nlg);
          for (int32_t e = ll.e0; e < ll.e1; e += ll.de) {
            const int32_t a = ll.list[e];
            if (!EL_CHECK(p.status, a >= 0 && a < p.n_slots, 1)) continue;
            if (p.mode != kModeDecode && p.slots[a].rank <= 0) continue;
            if (!ptx::mbar_wait(&full_bar[stage], phase, wl) ||
                !ptx::mbar_wait(&zfull_bar[stage], (zphase >> stage) & 1u, wl) || *abort_flag) {
              ok = false;
              break;
            }
            zphase ^= 1u << stage;
            ptx::tc_fence_after_sync();
            const uint32_t sr = ptx::smem_u32(smem + static_cast<size_t>(stage) * stage_bytes);
            const uint64_t da = ptx::umma_desc_k128(sr);
            const uint64_t db = ptx::umma_desc_k128(sr + r_bytes);
            // the whole z operand is there (rows of tokens on other adapters are zero), so one
            // MMA per 16 rank columns covers every token: an MMA costs about the same whatever
            // its N, and the issuing thread is what bounds a LoRA K block
            for (int k = 0; k < lora_ksteps; ++k) ptx::umma_bf16(tmem_d, da + 2 * k, db + 2 * k, idesc, 1u);
            ptx::umma_commit(&empty_bar[stage]);
            if (++stage == nstages) {
              stage = 0;
              phase ^= 1;
            }
          }
          if (!ok) break;
        }
        ptx::umma_commit(&tfull_bar[acc]);  // accumulator complete
      }
      if (!ok) {
        *abort_flag = 1;
        atomicOr(p.status, EDGELORA_STATUS_TIMEOUT);
      }
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int quad = warp & 3;                      // TMEM lanes [32*quad, 32*quad+32)
    const int row_in_tile = quad * 32 + lane;
    const bool clustered = p.mode == kModeDecode && p.splits > 1;
    if (kFused && clustered && f.b_stage) {
      // This CTA will finish tokens [rank * cols_per, ...) of its row tile: the B_a rows they need (the
      // tile's 128 rows of the token's adapter, contiguous in the pool) are copied into shared memory
      // now, one bulk copy per token, while the main loop runs (the ids are the caller's input, the
      // pool is not written by this kernel).  One warp per token; cols_per <= 16.
      const int cols_per = p.BN / p.splits;
      const int t0 = static_cast<int>(cluster_cta_rank()) * cols_per;
      const uint32_t tok_bytes = kTileM * p.R_pad * 2;
      const uint32_t copy_bytes = static_cast<uint32_t>(min(kTileM, p.h_out - tc_row0(p, bid)) * p.R_pad * 2);
      int32_t a_of[4];
      uint32_t my_bytes = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int cl = quad + 4 * i;
        int32_t a = -1, rank = 0;
        if (cl < cols_per && t0 + cl < p.T) {
          a = p.ids[t0 + cl];
          if (a < 0 || a >= p.n_slots) a = -1;
          if (a >= 0) rank = p.slots[a].rank;
        }
        if (rank <= 0) a = -1;
        a_of[i] = a;
        if (cl < cols_per && lane == 0) {  // kept for the expand at the end
          s_vid[cl] = a;
          s_lg[cl] = rank;
        }
        if (a >= 0) my_bytes += copy_bytes;
      }
      if (lane == 0) {
        ptx::mbar_arrive_expect_tx(ep_bar, my_bytes);
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (a_of[i] >= 0)
            ptx::bulk_load_1d(b_stage + static_cast<size_t>(quad + 4 * i) * tok_bytes,
                              p.B_pool + (static_cast<size_t>(a_of[i]) * p.h_out + tc_row0(p, bid)) * p.R_pad,
                              copy_bytes, ep_bar);
      }
    } else if (clustered && p.expand_in_reduce) {
      // This CTA will finish tokens [rank * cols_per, ...) of its row tile; pull the B_a rows they
      // need into L2 now (the ids are the caller's input, the pool is not written by the shrink).
      const int cols_per = p.BN / p.splits;
      const int t0 = static_cast<int>(cluster_cta_rank()) * cols_per;
      for (int cl = quad; cl < cols_per; cl += 4) {  // one warp per token
        int32_t a = -1, rank = 0;
        if (t0 + cl < p.T) {
          a = p.ids[t0 + cl];
          if (a < 0 || a >= p.n_slots) a = -1;
          if (a >= 0) rank = p.slots[a].rank;
        }
        if (lane == 0) {  // kept for the expand at the end
          s_vid[cl] = rank > 0 ? a : -1;
          s_lg[cl] = rank;
        }
        if (t0 + cl < p.T) {
          if (a >= 0 && a < p.n_slots) {
            const uint8_t *rows = reinterpret_cast<const uint8_t *>(
                p.B_pool + (static_cast<size_t>(a) * p.h_out + tc_row0(p, bid)) * p.R_pad);
            const int bytes = min(kTileM, p.h_out - tc_row0(p, bid)) * p.R_pad * 2;  // this tile's rows, contiguous
            for (int off = lane * 128; off < bytes; off += 32 * 128)
              asm volatile("prefetch.global.L2 [%0];" ::"l"(rows + off));
          }
        }
      }
    }
    if (kFused && clustered) {
      // z comes from the shrink teams of this grid (every CTA of the launch is resident, so all of them
      // run).  These warps have nothing to do until the accumulator is complete: bounded wait for the
      // teams' arrival counter now, then this thread's share of the owner's z (tokens x R_pad floats,
      // at most 128 16-byte pieces; the K chunks' planes added in order) goes to shared memory, behind
      // the staged B_a rows.
      const int cols_per = p.BN / p.splits, etid = threadIdx.x - 64;
      const int my_rank = static_cast<int>(cluster_cta_rank());
      // the counter belongs to the kernel before this one (another launch of this pool, which leaves it
      // at zero) until that kernel is done
      ptx::pdl_wait_prior_grids();
      // one thread of the CTA polls; the named barrier of the four warps passes its acquire on
      if (warp == 2 && lane == 0) {
        int got = 1;
        const long long t_start = clock64();
        while (ld_acquire_gpu(f.sync) < 2 * cta0 + ngrid) {
          if (clock64() - t_start > wl) {
            got = 0;
            break;
          }
        }
        if (!got) atomicOr(p.status, EDGELORA_STATUS_TIMEOUT);
        *s_last = got;  // (the gather tiles' flag: unused in this launch)
      }
      named_bar_sync(1, 128);
      fused_z_ok = *s_last != 0;
      const int tok = my_rank * cols_per + etid / (p.R_pad >> 2);
      if (f.b_stage && fused_z_ok && etid < cols_per * (p.R_pad >> 2)) {
        float4 z_mine = make_float4(0.f, 0.f, 0.f, 0.f);
        if (tok < p.T) {
          const size_t zplane4 = static_cast<size_t>(p.max_tokens) * p.R_pad / 4;
          const float4 *zp = reinterpret_cast<const float4 *>(f.z) +
                             static_cast<size_t>(my_rank) * cols_per * (p.R_pad >> 2) + etid;
          z_mine = __ldcg(zp);
          for (int sp = 1; sp < f.ks; ++sp) {
            const float4 w = __ldcg(zp + sp * zplane4);
            z_mine.x += w.x; z_mine.y += w.y; z_mine.z += w.z; z_mine.w += w.w;
          }
        }
        // read by the expand, behind two cluster barriers
        reinterpret_cast<float4 *>(b_stage + static_cast<size_t>(cols_per) * kTileM * p.R_pad * 2)[etid] = z_mine;
      }
    }
    // Earlier kernels may still read y, and z comes from the shrink kernel.  With the expand in
    // the reduction both matter only at the very end, so that wait moves there.
    if (!(clustered && p.expand_in_reduce)) ptx::pdl_wait_prior_grids();
    bool ok = true;
    int32_t it = 0;
    uint32_t ep_phase = 0;
    for (int32_t tile = bid; ok && tile < n_tiles; tile += ngrid) {
      const bool second = tile >= n_tiles0;
      int32_t local = tile;
      if (second && (local = second_job_tile(tile)) < 0) {
        if (local == -2) continue;
        break;
      }
      const GemmParams &jp = second ? p2 : p;
      const TileCoord tc = tile_coord(jp, local);
      if (kShrink && tc.kind == 1) {
        // ---- gather tile: accumulator row m = (group m / R_pad of the tile, rank row m % R_pad),
        // column c = token perm_short[tok0 + pass * gN + c].  This thread writes z of its rank row
        // for the tokens of its group, scaled by s_a, into the partial plane of the tile's K split.
        const int32_t gi = row_in_tile / jp.R_pad, r = row_in_tile % jp.R_pad;
        int32_t c_lo = 0, c_hi = 0;  // this row's tokens, as positions inside the tile's token list
        float scale = 0.f;
        bool live = false;
        if (gi < tc.ng) {
          const int32_t a = jp.group_adapter[tc.g0 + gi];
          const SlotRow row = jp.slots[a];
          live = row.rank > 0;
          scale = row.scale;
          c_lo = jp.gs_short[tc.g0 + gi] - tc.tok0;
          c_hi = jp.gs_short[tc.g0 + gi + 1] - tc.tok0;
          if (!live && r == 0 && tc.split == 0 && c_hi > c_lo) atomicOr(jp.status, EDGELORA_STATUS_SLOT_EMPTY);
        }
        const size_t plane = static_cast<size_t>(jp.max_tokens) * jp.R_pad;
        float *zsplit = jp.zws_out + static_cast<size_t>(tc.split) * plane;
        const int32_t n_pass = tile_passes(jp, tc);
        for (int32_t pass = 0; ok && pass < n_pass; ++pass, ++it) {
          const uint32_t acc = (p.n_acc == 2) ? (it & 1) : 0;
          const uint32_t use = (p.n_acc == 2) ? (it >> 1) : it;
          if (!(ptx::mbar_wait(&tfull_bar[acc], use & 1, wl) && !*abort_flag)) {
            ok = false;
            *abort_flag = 1;
            break;
          }
          ptx::tc_fence_after_sync();
          const int32_t t0 = pass * jp.gN, n = min(jp.gN, tc.ntok - t0);
          int32_t tok[8];  // lane l keeps the tokens of columns l, l + 32, ...
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const int c = q * 32 + lane;
            tok[q] = c < n ? jp.perm_short[tc.tok0 + t0 + c] : 0;
            if (!EL_CHECK(jp.status, tok[q] >= 0 && tok[q] < jp.max_tokens, 6)) tok[q] = 0;
          }
          const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) +
                                 acc * static_cast<uint32_t>(p.acc_cols);
          const int32_t n16 = (n + 15) & ~15;
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const int32_t c0 = q * 32;
            if (c0 < n16) {  // uniform over the warp
              float v[32];
              if (n16 - c0 >= 32) {
                ptx::tmem_ld_32x32(taddr + c0, v);
              } else {
                float h[16];
                ptx::tmem_ld_32x16(taddr + c0, h);
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                  v[i] = h[i];
                  v[i + 16] = 0.f;
                }
              }
#pragma unroll
              for (int jj = 0; jj < 32; ++jj) {
                const int32_t t = __shfl_sync(0xffffffffu, tok[q], jj);
                const int32_t c = t0 + c0 + jj;  // position inside the tile's token list
                if (live && c >= c_lo && c < c_hi && c0 + jj < n)
                  zsplit[static_cast<size_t>(t) * jp.R_pad + r] = scale * v[jj];
              }
            }
          }
          ptx::tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&tempty_bar[acc]);
        }
        if (!ok) break;
        if (jp.finalize) {
          // Whichever K split of this tile arrives last adds the splits, in order, into the final
          // plane (the one the base-product kernel reads); nobody waits for another CTA.  The four
          // epilogue warps meet on a barrier with a bounded wait, like every wait of this kernel.
          auto ep_sync = [&]() {
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ep_bar);
            const bool met = ptx::mbar_wait(ep_bar, ep_phase, wl);
            ep_phase ^= 1u;
            __syncwarp();
            return met;
          };
          const int32_t n_gt = gather_tiles(jp);
          const int32_t gsp = gather_splits(jp, n_gt, gridDim.x);
          __threadfence();                 // this thread's z stores, before the arrival below
          if (!ep_sync()) {
            ok = false;
            break;
          }
          if (threadIdx.x == 64) {
            const int32_t old = atomicAdd(&jp.tile_counters[tc.gtile], 1);
            *s_last = (old == gsp - 1) ? 1 : 0;
            if (old == gsp - 1) jp.tile_counters[tc.gtile] = 0;  // ready for the next launch
          }
          if (!ep_sync()) {
            ok = false;
            break;
          }
          if (*s_last) {
            __threadfence();
            if (live) {
              float *zfinal = jp.zws_out + static_cast<size_t>(kMaxZSplits) * plane;
              for (int32_t c = c_lo; c < c_hi; ++c) {
                const size_t off = static_cast<size_t>(jp.perm_short[tc.tok0 + c]) * jp.R_pad + r;
                float sum = 0.f;
                for (int32_t sp = 0; sp < gsp; ++sp) sum += __ldcg(jp.zws_out + sp * plane + off);
                zfinal[off] = sum;
              }
            }
          }
          if (!ep_sync()) {                // s_last is reused by the next tile
            ok = false;
            break;
          }
        }
        continue;
      }
      const uint32_t acc = (p.n_acc == 2) ? (it & 1) : 0;
      const uint32_t use = (p.n_acc == 2) ? (it >> 1) : it;
      ++it;
      const int32_t row = tc.row_r + row_in_tile;
      float scale = 0.f;
      if (jp.mode == kModeSgmv) scale = jp.slots[tc.slot].scale;

      const bool got = ptx::mbar_wait(&tfull_bar[acc], use & 1, wl) && !*abort_flag;
      if (!got) {
        ok = false;
        *abort_flag = 1;
        break;
      }
      if (clustered) break;  // the accumulator is read after the cluster barrier below
      ptx::tc_fence_after_sync();
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) +
                             acc * static_cast<uint32_t>(p.acc_cols);  // accumulators are spaced for the first job
      for (int32_t c0 = 0; got && c0 < jp.BN; c0 += 32) {
        float v[32];
        if (jp.BN - c0 >= 32) {
          ptx::tmem_ld_32x32(taddr + c0, v);
        } else {  // sgmv with a rank stride of 16: only 16 columns exist
          float h[16];
          ptx::tmem_ld_32x16(taddr + c0, h);
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            v[i] = h[i];
            v[i + 16] = 0.f;
          }
        }
        if (kShrink && jp.mode == kModePrefill && jp.y_tma) {
          // row = token, columns = output features row_c + c0 + [0, 32).  The warp's 32 rows x 64
          // columns go to its shared-memory stage as bf16 (rows of 128 bytes, 16-byte chunks
          // swizzled by the row so that the lanes' stores spread over the banks) and leave with one
          // TMA store: whole 128-byte lines to memory instead of 32 scattered pieces per
          // instruction; rows and columns outside y are dropped by the copy.
          uint8_t *my_stage = y_stage + quad * (32 * 128);
          const int half = (c0 >> 5) & 1;  // which 64 bytes of the stage row
          if (half == 0) {                 // the previous store of this warp has read the stage
            if (lane == 0) ptx::bulk_wait_group_read0();
            __syncwarp();
          }
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint4 o;
            o.x = ptx::pack_bf16x2(v[8 * q + 0], v[8 * q + 1]);
            o.y = ptx::pack_bf16x2(v[8 * q + 2], v[8 * q + 3]);
            o.z = ptx::pack_bf16x2(v[8 * q + 4], v[8 * q + 5]);
            o.w = ptx::pack_bf16x2(v[8 * q + 6], v[8 * q + 7]);
            const int chunk = half * 4 + q;
            *reinterpret_cast<uint4 *>(my_stage + lane * 128 + ((chunk ^ (lane & 7)) << 4)) = o;
          }
          if (half == 1 || c0 + 32 >= jp.BN) {
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
              ptx::tma_store_2d(&tmap_y, my_stage, tc.row_c + (c0 & ~63), tc.row_r + quad * 32);
              ptx::bulk_commit_group();
            }
          }
        } else if (jp.mode == kModePrefill) {
          // row = token, columns = output features row_c + c0 + [0, 32)
          if (row < jp.T) {
            uint16_t *yrow = jp.y + static_cast<size_t>(row) * jp.h_out;
#pragma unroll
            for (int q = 0; q < 32; q += 8) {
              const int j = tc.row_c + c0 + q;
              if (j < jp.h_out) {  // h_out is a multiple of 8: a group of 8 is all in or all out
                uint4 o;
                o.x = ptx::pack_bf16x2(v[q + 0], v[q + 1]);
                o.y = ptx::pack_bf16x2(v[q + 2], v[q + 3]);
                o.z = ptx::pack_bf16x2(v[q + 4], v[q + 5]);
                o.w = ptx::pack_bf16x2(v[q + 6], v[q + 7]);
                *reinterpret_cast<uint4 *>(yrow + j) = o;
              }
            }
          }
        } else if (jp.mode == kModeDecode) {
          // single K split: row = W row j, columns = tokens c0 + [0, 32), straight to y
          if (row < jp.h_out) {
#pragma unroll
            for (int jj = 0; jj < 32; ++jj) {
              const int t = c0 + jj;
              if (t < jp.T)
                jp.y[static_cast<size_t>(t) * jp.h_out + row] =
                    static_cast<uint16_t>(ptx::pack_bf16x2(v[jj], 0.f) & 0xFFFFu);
            }
          }
        } else {
          // sgmv: row = token of the run, columns = rank index; z partial = scale * acc
          if (row_in_tile < tc.nrows) {
            float *zrow = jp.zws_out + (static_cast<size_t>(tc.split) * jp.max_tokens + row) * jp.R_pad + c0;
            const int nc = min(32, jp.BN - c0);
            for (int q = 0; q < nc; q += 4)
              *reinterpret_cast<float4 *>(zrow + q) =
                  make_float4(scale * v[q], scale * v[q + 1], scale * v[q + 2], scale * v[q + 3]);
          }
        }
      }
      if (got) {
        // all TMEM reads of this warp are complete (tcgen05.wait::ld inside the loads)
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&tempty_bar[acc]);
      }

    }
    if (!ok && lane == 0) {
      *abort_flag = 1;
      atomicOr(p.status, EDGELORA_STATUS_TIMEOUT);
    }
  } else if (kFused) {
    // ------------------------------------------------------------ shrink team (warps 6..9)
    const int btid = threadIdx.x - 192;  // 0..127
    int32_t *s_tid = reinterpret_cast<int32_t *>(s_key) + 64;  // s_key is free: no LoRA K blocks in this launch
    int32_t *s_trank = s_tid + 64;
    float *s_tscale = reinterpret_cast<float *>(s_trank + 64);
    if (btid < 64) {
      int32_t a = -1;
      if (btid < p.T) {
        a = p.ids[btid];
        if (a < 0 || a >= p.n_slots) a = -1;
      }
      SlotRow row = {0, 0.f, 0, 0};
      if (a >= 0) row = p.slots[a];
      s_tid[btid] = a;
      s_trank[btid] = row.rank;
      s_tscale[btid] = row.scale;
    }
    named_bar_sync(2, 128);
    bool waited = false;
    if (f.x_wait) {
      ptx::pdl_wait_prior_grids();
      waited = true;
    }
    shrink_team_items<2>(p, f, 2 * cta0 + bid, 2 * cta0 + ngrid, warp - 6, lane, s_tid, s_trank, s_tscale,
                         reinterpret_cast<float *>(s_key), waited);
  } else if (has_lora || has2 || (kShrink && p.mode == kModeSgmv && p.gather)) {
    // ------------------------------------------------------------ z operand builder (warps 6..9)
    // (and, during gather tiles, parts 1..4 of the tile's copies)
    const int btid = threadIdx.x - 192;  // 0..127
    const int bwarp = warp - 6;
    const int nch = p.R_pad >> 3;        // 16-byte chunks of one operand row that the MMAs read
    uint32_t count = 0;                  // K blocks so far: stage = count % stages
    uint32_t gophase = 0;                // one parity bit per stage for zgo_bar
    bool ok = true, waited = false;
    // a shrink tile (of the second job, or of a first job that is a shrink job): gather tiles take
    // this warp's part of the copies, segment tiles only move the ring on
    auto shrink_tile = [&](const GemmParams &jp, int32_t local, const CUtensorMap *ma, const CUtensorMap *mg) {
      const TileCoord t2 = tile_coord(jp, local);
      if (t2.kind != 1) {
        count += static_cast<uint32_t>(t2.kb1 - t2.kb0);
        return true;
      }
      for (int32_t t0 = 0; t0 < t2.ntok; t0 += jp.gN) {
        uint32_t stage = count % nstages, phase = (count / nstages) & 1u;
        if (!gather_pass_copies(jp, t2, t0, ma, mg, smem, stage_bytes, full_bar, empty_bar, zgo_bar, zfull_bar,
                                abort_flag, nstages, wl, 1 + bwarp, lane, stage, phase, gophase))
          return false;
        count += static_cast<uint32_t>(t2.kb1 - t2.kb0);
      }
      return true;
    };
    if (has_lora && p.mode == kModeDecode) {
      // The batch's adapters (paper Section 3.4: one u-batch per adapter), distinct and ascending,
      // straight from the caller's ids so that the B_a tiles can be fetched before the shrink
      // kernel has finished.  Thread b looks after tokens b and b + 128.
      // Keys (id << 8 | token) of the tokens that carry an adapter are sorted (bitonic, BN keys);
      // the first key of every id that names a loaded slot joins the list.
      const int nk = p.BN;  // a power of two, 32..256
      for (int t = btid; t < 256; t += 128) {
        int32_t a = -1;
        if (t < p.T) {
          a = p.ids[t];
          if (a < -1 || a >= p.n_slots) a = -1;
        }
        s_vid[t] = a;
        s_key[t] = a >= 0 ? ((static_cast<uint32_t>(a) << 8) | static_cast<uint32_t>(t)) : 0xFFFFFFFFu;
      }
      named_bar_sync(2, 128);
      for (int k = 2; k <= nk; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
          for (int i = btid; i < nk; i += 128) {
            const int ixj = i ^ j;
            if (ixj > i) {
              const uint32_t ka = s_key[i], kb = s_key[ixj];
              if ((ka > kb) == ((i & k) == 0)) {
                s_key[i] = kb;
                s_key[ixj] = ka;
              }
            }
          }
          named_bar_sync(2, 128);
        }
      }
      for (int i = btid; i < nk; i += 128) {
        const uint32_t key = s_key[i];
        bool head = key != 0xFFFFFFFFu && (i == 0 || (s_key[i - 1] >> 8) != (key >> 8));
        if (head) head = p.slots[key >> 8].rank > 0;  // empty slots stay base-only (the shrink flags them)
        s_head[i] = head ? 1 : 0;
      }
      named_bar_sync(2, 128);
      if (bwarp == 0) {  // 32 lanes x 8 consecutive keys: positions by a warp prefix sum
        int c = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) c += (lane * 8 + q < nk) ? s_head[lane * 8 + q] : 0;
        int incl = c;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const int o = __shfl_up_sync(0xffffffffu, incl, d);
          if (lane >= d) incl += o;
        }
        int pos = incl - c;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const int i = lane * 8 + q;
          if (i < nk && s_head[i]) s_lg[pos++] = static_cast<int32_t>(s_key[i] >> 8);
        }
        if (lane == 31) *s_nlg = incl;
      }
      named_bar_sync(2, 128);
      if (btid == 0) ptx::mbar_arrive(lg_bar);
    }
    for (int32_t tile = bid; ok && tile < n_tiles; tile += ngrid) {
      if (kShrink && tile >= n_tiles0) {  // a tile of the second job: no LoRA blocks
        const int32_t local = second_job_tile(tile);
        if (local == -2) continue;
        if (local < 0) break;
        ok = shrink_tile(p2, local, &tmap_c2, &tmap_g2);
        continue;
      }
      if (kShrink && p.mode == kModeSgmv) {  // the first job is a shrink job
        ok = shrink_tile(p, tile, &tmap_c, &tmap_b);
        continue;
      }
      const TileCoord tc = tile_coord(p, tile);
      count += static_cast<uint32_t>(tc.kb1 - tc.kb0);
      if (!has_lora) continue;
      if (!waited) {  // z (and in prefill the tile lists) come from the kernels before this one
        ptx::pdl_wait_prior_grids();
        waited = true;
      }
      const LoraList ll = lora_list(p, tc, s_lg, s_nlg);
      const int tok0 = (p.mode == kModePrefill) ? tc.row_r : 0;
      const uint32_t region = (p.mode == kModePrefill) ? 0u : r_bytes;
      // The ids of this thread's rows do not change over the tile's LoRA blocks, so their z is
      // fetched once per tile (while the base K blocks stream) and kept as packed bf16.
      int32_t id_lo = -1, id_hi = -1;
      if (p.mode == kModeDecode) {
        id_lo = s_vid[btid];
        if (kMinBlocks == 1) id_hi = s_vid[btid + 128];  // the two-per-SM variant runs with BN <= 128
      } else if (tok0 + btid < p.T) {
        id_lo = p.ids_valid[tok0 + btid];
        if (!EL_CHECK(p.status, id_lo >= -1 && id_lo < p.n_slots, 2)) id_lo = -1;
      }
      uint4 z_lo[8], z_hi[8];
      if (ll.e0 < ll.e1) {
        if (id_lo >= 0) load_z_packed(p, tok0 + btid, p.slots[id_lo].rank, z_lo);
        if (kMinBlocks == 1 && id_hi >= 0) load_z_packed(p, tok0 + btid + 128, p.slots[id_hi].rank, z_hi);
      }
      for (int32_t e = ll.e0; e < ll.e1; e += ll.de) {
        const int32_t a = ll.list[e];
        if (!EL_CHECK(p.status, a >= 0 && a < p.n_slots, 1)) continue;
        if (p.mode != kModeDecode && p.slots[a].rank <= 0) continue;
        const uint32_t stage = count % nstages;
        ++count;
        if (!ptx::mbar_wait(&zgo_bar[stage], (gophase >> stage) & 1u, wl) || *abort_flag) {
          ok = false;
          break;
        }
        gophase ^= 1u << stage;
        uint8_t *dst = smem + static_cast<size_t>(stage) * stage_bytes + region;
        // 128-byte swizzle: the 16-byte chunk index is XORed with the row index modulo 8.
        // Every token row the MMAs read is written: z of the tokens on this adapter, zeros for
        // the others (prefill: the tile's 128 rows; decode: rows btid and btid + 128 below BN).
        const bool m_lo = id_lo == a, m_hi = id_hi == a;
        const bool w_lo = p.mode == kModePrefill || btid < p.BN;
        const bool w_hi = kMinBlocks == 1 && p.mode == kModeDecode && btid + 128 < p.BN;
        if (w_lo) {
          uint8_t *drow = dst + btid * 128;
#pragma unroll
          for (int c = 0; c < 8; ++c)
            if (c < nch)
              *reinterpret_cast<uint4 *>(drow + ((c ^ (btid & 7)) << 4)) =
                  m_lo ? z_lo[c] : make_uint4(0u, 0u, 0u, 0u);
        }
        if (w_hi) {
          uint8_t *drow = dst + (btid + 128) * 128;
#pragma unroll
          for (int c = 0; c < 8; ++c)
            if (c < nch)
              *reinterpret_cast<uint4 *>(drow + ((c ^ (btid & 7)) << 4)) =
                  m_hi ? z_hi[c] : make_uint4(0u, 0u, 0u, 0u);
        }
        fence_proxy_async_smem();  // make the generic-proxy writes visible to the tensor core
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&zfull_bar[stage]);
      }
    }
    if (!ok && lane == 0) {
      *abort_flag = 1;
      atomicOr(p.status, EDGELORA_STATUS_TIMEOUT);
    }
  }

  if (p.mode == kModeDecode && p.splits > 1) {
    // ---------------------------------------------------------- split-K reduction in the cluster
    // CTA `rank` of the cluster owns tokens [rank * cols_per, (rank + 1) * cols_per).  Its buffer
    // buf[src split][token][row] overlays the operand ring, which is idle once every CTA of the
    // cluster is past its main loop (first barrier).
    const bool epi = warp >= 2 && warp < 6;
    const int quad = warp & 3, row_in_tile = quad * 32 + lane, etid = threadIdx.x - 64;
    const uint32_t my_rank = cluster_cta_rank();
    const int cols_per = p.BN / p.splits;  // a power of two (BN and splits are)
    const int shift = 31 - __clz(cols_per);
    // Large batches: the builder warps (6..9, the same four lane quadrants) send every other
    // 32-token block, and all ten warps sum.  The epilogue warps have waited for the accumulator;
    // the barrier below passes that on to the others.
    const bool wide = !p.expand_in_reduce;
    const bool sender = epi || (wide && warp >= 6);
    const int c_first = (wide && warp >= 6) ? 32 : 0, c_step = wide ? 64 : 32;
    const bool have_acc = sender && !*abort_flag;  // this CTA's accumulator is complete (tfull waited)
    const bool z_ok = fused_z_ok;  // fused launches: the wait for the shrink teams ended in time
    float4 *z_stage = reinterpret_cast<float4 *>(b_stage + static_cast<size_t>(cols_per) * kTileM * p.R_pad * 2);
    // The partial tiles land in the operand ring, which is idle once every CTA of the cluster is past
    // its main loop: hence the first barrier.  A fused launch with room to spare (b_stage == 2) has a
    // buffer of its own behind the staged rows instead, and sends at once.
    const bool own_buf = kFused && f.b_stage == 2;
    uint8_t *red = own_buf ? b_stage + ((static_cast<size_t>(cols_per) * (kTileM * p.R_pad * 2 + p.R_pad * 4) + 1023) &
                                        ~static_cast<size_t>(1023))
                           : smem;
    __syncwarp();
    if (!own_buf) cluster_sync_all();
    if (have_acc) {
      ptx::tc_fence_after_sync();
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
      const uint32_t local = ptx::smem_u32(red) +
                             ((my_rank * cols_per) * kTileM + row_in_tile) * 4u;
      const uint32_t qpo = static_cast<uint32_t>(cols_per) >> 2;  // token quads per owner
      for (int32_t c0 = c_first; c0 < p.BN; c0 += c_step) {
        float v[32];
        ptx::tmem_ld_32x32(taddr + c0, v);
        if (p.expand_in_reduce && !(kFused && f.b_stage)) {  // buf[src][token][row]
#pragma unroll
          for (int jj = 0; jj < 32; ++jj) {
            const int col = c0 + jj;
            const uint32_t owner = static_cast<uint32_t>(col >> shift);
            const uint32_t off = static_cast<uint32_t>(col & (cols_per - 1)) * kTileM * 4u;
            st_cluster_f32(map_to_cta(local + off, owner), v[jj]);  // a warp writes 128 bytes in a row
          }
        } else {  // buf[src][token quad][row][4 tokens]: 16-byte stores, a warp writes 512 bytes in a row
#pragma unroll
          for (int g4 = 0; g4 < 8; ++g4) {
            const int col = c0 + g4 * 4;
            const uint32_t owner = static_cast<uint32_t>(col >> shift);
            const uint32_t quad_i = static_cast<uint32_t>(col & (cols_per - 1)) >> 2;
            const uint32_t addr = ptx::smem_u32(red) + ((my_rank * qpo + quad_i) * kTileM + row_in_tile) * 16u;
            st_cluster_f32x4(map_to_cta(addr, owner), v[g4 * 4], v[g4 * 4 + 1], v[g4 * 4 + 2], v[g4 * 4 + 3]);
          }
        }
      }
    }
    __syncwarp();
    cluster_sync_all();
    if (epi || wide) {
      const float *buf = reinterpret_cast<const float *>(red);
      const int n_units = cols_per * 32;  // unit = (token, 4 adjacent W rows)
      const int row0 = bid / p.splits * kTileM;
      auto sum_partials = [&](int cl, int r4) {
        float4 acc4 = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int sp = 0; sp < p.splits; ++sp) {
          const float4 w = *reinterpret_cast<const float4 *>(buf + ((sp * cols_per + cl) * kTileM + r4));
          acc4.x += w.x; acc4.y += w.y; acc4.z += w.z; acc4.w += w.w;
        }
        return acc4;
      };
      auto store4 = [&](int t, int j, const float4 &v) {
        uint2 o;
        o.x = ptx::pack_bf16x2(v.x, v.y);
        o.y = ptx::pack_bf16x2(v.z, v.w);
        *reinterpret_cast<uint2 *>(p.y + static_cast<size_t>(t) * p.h_out + j) = o;
      };
      if (!p.expand_in_reduce) {
        // unit = (token quad, W row): the splits' partial sums are 16 bytes each, lanes take
        // adjacent rows, so a warp writes 64 bytes in a row of y per token
        const int qpo = cols_per >> 2;
        const float4 *buf4 = reinterpret_cast<const float4 *>(red);
        ptx::pdl_wait_prior_grids();  // warps 0 and 1 have not waited yet; earlier kernels may read y
        for (int u = threadIdx.x; u < qpo * kTileM; u += kGemmThreads) {
          const int qd = u >> 7, r = u & (kTileM - 1);
          const int t0 = static_cast<int>(my_rank) * cols_per + qd * 4, j = row0 + r;
          if (t0 >= p.T || j >= p.h_out) continue;
          float4 a4 = make_float4(0.f, 0.f, 0.f, 0.f);
          for (int sp = 0; sp < p.splits; ++sp) {
            const float4 w = buf4[(sp * qpo + qd) * kTileM + r];
            a4.x += w.x; a4.y += w.y; a4.z += w.z; a4.w += w.w;
          }
          const float o[4] = {a4.x, a4.y, a4.z, a4.w};
#pragma unroll
          for (int i = 0; i < 4; ++i)
            if (t0 + i < p.T)
              p.y[static_cast<size_t>(t0 + i) * p.h_out + j] =
                  static_cast<uint16_t>(ptx::pack_bf16x2(o[i], 0.f) & 0xFFFFu);
        }
      } else if (kFused && f.b_stage) {
        // Small batches, one launch: unit = (token quad, W row), as above, and everything the expand
        // needs is in shared memory by now: B_a[row][0..R_pad) of each token's adapter (lanes take
        // adjacent rows: 32-byte pieces side by side) and the tokens' z (the same for every lane).
        const int qpo = cols_per >> 2;
        const float4 *buf4 = reinterpret_cast<const float4 *>(red);
        const int n_units = qpo * kTileM;  // at most 4 per thread (cols_per <= 16)
        const int nch = p.R_pad >> 3;
        ptx::pdl_wait_prior_grids();  // earlier kernels may still read y
        bool b_ok = true;
        {
          int got = 1;
          if (lane == 0) got = ptx::mbar_wait(ep_bar, 0, wl) ? 1 : 0;  // the staged B_a rows
          if (!__shfl_sync(0xffffffffu, got, 0)) {
            if (lane == 0) atomicOr(p.status, EDGELORA_STATUS_TIMEOUT);
            b_ok = false;
          }
        }
        const int r = etid & 127, j = row0 + r;
        // This code runs once per launch: kept as rolled loops, because what it costs is fetching its
        // instructions, not executing them (fully unrolled it took 2.9 us instead of about 1 us).
#pragma unroll 1
        for (int u = etid; u < n_units && j < p.h_out; u += 128) {
          const int qd = u >> 7;
          float4 a4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
          for (int sp = 0; sp < p.splits; ++sp) {
            const float4 w = buf4[(sp * qpo + qd) * kTileM + r];
            a4.x += w.x; a4.y += w.y; a4.z += w.z; a4.w += w.w;
          }
          const int t0q = static_cast<int>(my_rank) * cols_per + qd * 4;
#pragma unroll 1
          for (int k = 0; k < 4; ++k) {
            const int cl = qd * 4 + k;
            const int32_t a = (z_ok && b_ok) ? s_vid[cl] : -1, rank = s_lg[cl];
            float add = k == 0 ? a4.x : k == 1 ? a4.y : k == 2 ? a4.z : a4.w;
            if (a >= 0) {
              const uint4 *Brow =
                  reinterpret_cast<const uint4 *>(b_stage + static_cast<size_t>(cl) * kTileM * p.R_pad * 2) + r * nch;
              const float4 *zt = z_stage + cl * (p.R_pad >> 2);
#pragma unroll 1
              for (int c = 0; c < nch && c * 8 < rank; ++c) {
                const uint4 bb = Brow[c];
                const float4 u0 = zt[2 * c], u1 = zt[2 * c + 1];
                add = fmaf(ptx::bf16_lo(bb.x), u0.x, add);
                add = fmaf(ptx::bf16_hi(bb.x), u0.y, add);
                add = fmaf(ptx::bf16_lo(bb.y), u0.z, add);
                add = fmaf(ptx::bf16_hi(bb.y), u0.w, add);
                add = fmaf(ptx::bf16_lo(bb.z), u1.x, add);
                add = fmaf(ptx::bf16_hi(bb.z), u1.y, add);
                add = fmaf(ptx::bf16_lo(bb.w), u1.z, add);
                add = fmaf(ptx::bf16_hi(bb.w), u1.w, add);
              }
            }
            if (t0q + k < p.T)
              p.y[static_cast<size_t>(t0q + k) * p.h_out + j] =
                  static_cast<uint16_t>(ptx::pack_bf16x2(add, 0.f) & 0xFFFFu);
          }
        }
        if (lane == 0) {
          // this warp is past its wait for the shrink teams: the last such warp of the grid puts both
          // counters back to zero for the next launch
          if (atomicAdd(f.sync + 1, 1) == ngrid * 4 - 1) {
            f.sync[0] = 0;
            f.sync[1] = 0;
          }
        }
      } else {
        // Small batches: wait for the shrink kernel (and for earlier readers of y), then per unit add the
        // splits' partial sums, fetch z and the B_a rows in one round trip, add B_a[j..j+3][0..r) . z[t]
        // in fp32 (z carries s_a) and write y.  A rolled loop over the units (at most 4 per thread:
        // cols_per <= 16): this code runs once per launch, and what it costs is mostly the fetching
        // of its instructions.
        ptx::pdl_wait_prior_grids();
        const int nch = p.R_pad >> 3;
        const int n_zp = kFused ? f.ks : 1;
        const size_t zplane4 = static_cast<size_t>(p.max_tokens) * p.R_pad / 4;
        auto load_z4 = [&](const float4 *ptr) {
          float4 v = __ldcg(ptr);
          for (int sp = 1; sp < n_zp; ++sp) {
            const float4 w = __ldcg(ptr + sp * zplane4);
            v.x += w.x; v.y += w.y; v.z += w.z; v.w += w.w;
          }
          return v;
        };
#pragma unroll 1
        for (int u = etid; u < n_units; u += 128) {
          const int cl = u >> 5, r4 = (u & 31) << 2;
          const int t = static_cast<int>(my_rank) * cols_per + cl, j = row0 + r4;
          if (t >= p.T || j >= p.h_out) continue;
          float4 acc4 = sum_partials(cl, r4);
          const int32_t a = z_ok ? s_vid[cl] : -1, rank = s_lg[cl];  // stored by the epilogue warps at the start
          if (a >= 0) {
            const uint4 *Brow = reinterpret_cast<const uint4 *>(
                p.B_pool + (static_cast<size_t>(a) * p.h_out + j) * p.R_pad);
            const float4 *zt = reinterpret_cast<const float4 *>((kFused ? f.z : p.zws) + static_cast<size_t>(t) * p.R_pad);
            float add[4] = {0.f, 0.f, 0.f, 0.f};
            for (int c0 = 0; c0 < nch && c0 * 8 < rank; c0 += 2) {
              uint4 b[2][4];
              float4 z4[2][2];
#pragma unroll
              for (int cc = 0; cc < 2; ++cc) {  // two chunks of 8 rank values: 12 loads in flight
                const int c = c0 + cc;
                const bool on = c < nch && c * 8 < rank;
#pragma unroll
                for (int r = 0; r < 4; ++r) b[cc][r] = on ? __ldg(Brow + r * nch + c) : make_uint4(0u, 0u, 0u, 0u);
                z4[cc][0] = on ? load_z4(zt + 2 * c) : make_float4(0.f, 0.f, 0.f, 0.f);
                z4[cc][1] = on ? load_z4(zt + 2 * c + 1) : make_float4(0.f, 0.f, 0.f, 0.f);
              }
#pragma unroll
              for (int cc = 0; cc < 2; ++cc) {
                const float4 u0 = z4[cc][0], u1 = z4[cc][1];
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                  const uint4 bb = b[cc][r];
                  float s4 = add[r];
                  s4 = fmaf(ptx::bf16_lo(bb.x), u0.x, s4);
                  s4 = fmaf(ptx::bf16_hi(bb.x), u0.y, s4);
                  s4 = fmaf(ptx::bf16_lo(bb.y), u0.z, s4);
                  s4 = fmaf(ptx::bf16_hi(bb.y), u0.w, s4);
                  s4 = fmaf(ptx::bf16_lo(bb.z), u1.x, s4);
                  s4 = fmaf(ptx::bf16_hi(bb.z), u1.y, s4);
                  s4 = fmaf(ptx::bf16_lo(bb.w), u1.z, s4);
                  s4 = fmaf(ptx::bf16_hi(bb.w), u1.w, s4);
                  add[r] = s4;
                }
              }
            }
            acc4.x += add[0]; acc4.y += add[1]; acc4.z += add[2]; acc4.w += add[3];
          }
          store4(t, j, acc4);
        }
        if (kFused && lane == 0) {
          // this warp is past its wait for the shrink teams: the last such warp of the grid puts both
          // counters back to zero for the next launch
          if (atomicAdd(f.sync + 1, 1) == ngrid * 4 - 1) {
            f.sync[0] = 0;
            f.sync[1] = 0;
          }
        }
      }
    }
  }

  if (kShrink && p.y_tma && warp >= 2 && warp < 6 && lane == 0) ptx::bulk_wait_group0();  // this warp's y stores
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, static_cast<uint32_t>(p.tmem_cols));
  }
}

// A GemmParams that stands for "no second job".
static GemmParams no_job() {
  GemmParams none{};
  none.mode = -1;
  return none;
}
static FusedDecode not_fused() {
  FusedDecode f{};
  return f;
}

cudaError_t gemm_set_smem_limit(size_t smem_bytes) {
  cudaError_t e = cudaSuccess;
  const int bytes = static_cast<int>(smem_bytes);
#define EDGELORA_SMEM(MB, SH, FU)                                                                               \
  if (e == cudaSuccess)                                                                                         \
    e = cudaFuncSetAttribute(lora_gemm_kernel<MB, SH, FU>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  EDGELORA_SMEM(1, true, false)
  EDGELORA_SMEM(2, true, false)
  EDGELORA_SMEM(1, false, false)
  EDGELORA_SMEM(2, false, false)
  EDGELORA_SMEM(1, false, true)
#undef EDGELORA_SMEM
  return e;
}

cudaError_t launch_gemm(const CUtensorMap &tmap_row, const CUtensorMap &tmap_col,
                        const CUtensorMap &tmap_b, const GemmParams &p, int32_t grid,
                        size_t smem_bytes, bool pdl, cudaStream_t stream, const CUtensorMap *tmap_y) {
  return launch_gemm2(tmap_row, tmap_col, tmap_b, p, tmap_row, tmap_col, tmap_b, no_job(), grid, smem_bytes,
                      pdl, stream, tmap_y);
}

static bool two_per_sm(size_t smem_bytes, int32_t BN, int32_t acc_cols) {
  return smem_bytes * 2 <= 225 * 1024 && BN <= 128 && acc_cols <= 128;
}

// With a second job: p2.mode == kModeSgmv (a shrink job: segment tiles and, with p2.gather, gather
// tiles; tmap_g2 is then the one-row map of its x), p2.n_mtiles = upper bound on its tiles,
// p2.BN and p2.gN <= p.ring_rows and p.acc_cols, and p is a prefill-mode job.
cudaError_t launch_gemm2(const CUtensorMap &tmap_row, const CUtensorMap &tmap_col,
                         const CUtensorMap &tmap_b, const GemmParams &p, const CUtensorMap &tmap_row2,
                         const CUtensorMap &tmap_col2, const CUtensorMap &tmap_g2, const GemmParams &p2,
                         int32_t grid, size_t smem_bytes, bool pdl, cudaStream_t stream,
                         const CUtensorMap *tmap_y) {
  const CUtensorMap &my = tmap_y ? *tmap_y : tmap_row;  // unused unless p.y_tma
  const int cluster = (p.mode == kModeDecode && p.splits > 1) ? p.splits : 1;
  const bool two = two_per_sm(smem_bytes, p.BN, p.acc_cols);        // two CTAs fit an SM
  const bool lean = p.mode == kModeDecode && p2.mode != kModeSgmv;  // no shrink job, plain y stores
#define EDGELORA_LAUNCH(MB, SH)                                                                                    \
  launch_ex(lora_gemm_kernel<MB, SH, false>, dim3(grid), dim3(kGemmThreads), smem_bytes, stream, pdl, cluster,      \
            tmap_row, tmap_col, tmap_b, p, tmap_row2, tmap_col2, tmap_g2, p2, my, not_fused())
  if (two) return lean ? EDGELORA_LAUNCH(2, false) : EDGELORA_LAUNCH(2, true);
  return lean ? EDGELORA_LAUNCH(1, false) : EDGELORA_LAUNCH(1, true);
#undef EDGELORA_LAUNCH
}

cudaError_t launch_gemm_fused(const CUtensorMap &tmap_row, const CUtensorMap &tmap_col, const GemmParams &p,
                              const FusedDecode &f, size_t smem_bytes, bool pdl, cudaStream_t stream) {
  const int32_t grid = f.n_ctas + p.n_mtiles * p.splits;
  return launch_ex(lora_gemm_kernel<1, false, true>, dim3(grid), dim3(kGemmThreads), smem_bytes, stream, pdl, p.splits,
                   tmap_row, tmap_col, tmap_row, p, tmap_row, tmap_col, tmap_row, no_job(), tmap_row, f);
}

int32_t gemm_fused_max_ctas(int32_t cluster, size_t smem_bytes) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(cluster) * 64);
  cfg.blockDim = dim3(kGemmThreads);
  cfg.dynamicSmemBytes = smem_bytes;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = static_cast<unsigned>(cluster);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  const cudaError_t e = cudaOccupancyMaxActiveClusters(&n, lora_gemm_kernel<1, false, true>, &cfg);
  if (getenv("EDGELORA_LOG"))
    fprintf(stderr, "edgelora: one-launch decode, clusters of %d, %zu bytes of shared memory: %s, %d clusters fit\n",
            cluster, smem_bytes, cudaGetErrorString(e), n);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return n * cluster;
}

}  // namespace edgelora
