// tcgen05 / TMEM / TMA bf16 GEMM for the dense contractions of batch LoRA inference
// (paper Section 3.4: the base product W [x_0 .. x_n] is batched over every token of the batch).
//
// D[128 x BN] (fp32, in tensor memory) = R[128 x K] * C[BN x K]^T, both operands K-major bf16,
// fetched by TMA into 128-byte-swizzled shared-memory tiles and multiplied by tcgen05.mma issued
// from one thread.  The same kernel serves three uses, chosen by GemmParams::mode:
//
//   prefill  R = 128 tokens of x,  C = BN rows of W.  Epilogue: y = bf16(D + B_a z) per token
//            (expand fused, y written once).  Persistent over tiles, two TMEM accumulators so the
//            epilogue of one tile overlaps the main loop of the next.
//   decode   R = 128 rows of W,    C = all tokens (N = T rounded up).  W is streamed once; K is
//            split across CTAs so every SM pulls from HBM; fp32 partials go to a workspace that
//            the combine kernel reduces.
//   sgmv     R = 128 tokens of one run, C = A_a (N = rank stride): the segment shrink
//            z = s_a A_a x for long runs, tile list from the plan.
//
// Warp roles: warp 0 issues TMA, warp 1 owns TMEM and issues the MMAs, warps 2..5 are the
// epilogue (each reads the 32 TMEM lanes of its quadrant).  Every mbarrier wait is bounded; on a
// timeout the status word gets EDGELORA_STATUS_TIMEOUT and all roles leave their loops.
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
};

__device__ __forceinline__ int32_t total_tiles(const GemmParams &p) {
  if (p.mode == kModePrefill) return p.n_mtiles * p.n_ntiles;
  if (p.mode == kModeDecode) return p.n_mtiles * p.splits;
  return p.counts[2] * p.splits;
}

__device__ __forceinline__ TileCoord tile_coord(const GemmParams &p, int32_t tile) {
  TileCoord c;
  c.slot = 0;
  c.nrows = kTileM;
  if (p.mode == kModePrefill) {
    const int m = tile % p.n_mtiles, n = tile / p.n_mtiles;
    c.row_r = m * kTileM;
    c.row_c = n * p.BN;
    c.split = 0;
  } else if (p.mode == kModeDecode) {
    const int m = tile % p.n_mtiles;
    c.split = tile / p.n_mtiles;
    c.row_r = m * kTileM;
    c.row_c = 0;
  } else {
    const int n_t = p.counts[2];
    const int st = tile % n_t;
    c.split = tile / n_t;
    c.row_r = p.sgmv_tiles[4 * st + 0];
    c.nrows = p.sgmv_tiles[4 * st + 1];
    c.slot = p.sgmv_tiles[4 * st + 2];
    c.row_c = 0;
  }
  c.kb0 = c.split * p.kb_per;
  c.kb1 = min(p.kb_total, c.kb0 + p.kb_per);
  return c;
}

// ---- epilogues: each thread owns one accumulator row (TMEM lane) and NC consecutive columns ----

// prefill: row = token, columns = output features n0 + c0 + [0, NC)
template <int NC>
__device__ __forceinline__ void epilogue_prefill_chunk(const GemmParams &p, float (&acc)[NC],
                                                       int32_t t, bool valid, int32_t a,
                                                       int32_t rank, const float (&z)[64],
                                                       int32_t col0) {
  if (a >= 0 && rank > 0) {
    const uint16_t *Bbase = p.B_pool + (static_cast<size_t>(a) * p.h_out) * p.R_pad;
#pragma unroll
    for (int jj = 0; jj < NC; ++jj) {
      const int j = col0 + jj;
      if (j < p.h_out) {
        const uint4 *Brow = reinterpret_cast<const uint4 *>(Bbase + static_cast<size_t>(j) * p.R_pad);
        float s = 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          if (c * 8 < rank) {
            const uint4 b = __ldg(Brow + c);
            s = fmaf(ptx::bf16_lo(b.x), z[c * 8 + 0], s);
            s = fmaf(ptx::bf16_hi(b.x), z[c * 8 + 1], s);
            s = fmaf(ptx::bf16_lo(b.y), z[c * 8 + 2], s);
            s = fmaf(ptx::bf16_hi(b.y), z[c * 8 + 3], s);
            s = fmaf(ptx::bf16_lo(b.z), z[c * 8 + 4], s);
            s = fmaf(ptx::bf16_hi(b.z), z[c * 8 + 5], s);
            s = fmaf(ptx::bf16_lo(b.w), z[c * 8 + 6], s);
            s = fmaf(ptx::bf16_hi(b.w), z[c * 8 + 7], s);
          }
        }
        acc[jj] += s;
      }
    }
  }
  if (valid) {
    uint16_t *yrow = p.y + static_cast<size_t>(t) * p.h_out;
#pragma unroll
    for (int q = 0; q < NC; q += 8) {
      const int j = col0 + q;
      if (j < p.h_out) {  // h_out is a multiple of 8, so a group of 8 is all in or all out
        uint4 o;
        o.x = ptx::pack_bf16x2(acc[q + 0], acc[q + 1]);
        o.y = ptx::pack_bf16x2(acc[q + 2], acc[q + 3]);
        o.z = ptx::pack_bf16x2(acc[q + 4], acc[q + 5]);
        o.w = ptx::pack_bf16x2(acc[q + 6], acc[q + 7]);
        *reinterpret_cast<uint4 *>(yrow + j) = o;
      }
    }
  }
}

// decode: row = W row j, columns = tokens c0 + [0, NC); partial sums to ws[split][t][j]
template <int NC>
__device__ __forceinline__ void epilogue_decode_chunk(const GemmParams &p, const float (&acc)[NC],
                                                      int32_t j, int32_t split, int32_t c0) {
  if (j >= p.h_out) return;
  float *base = p.ws + (static_cast<size_t>(split) * p.T) * p.h_out + j;
#pragma unroll
  for (int jj = 0; jj < NC; ++jj) {
    const int t = c0 + jj;
    if (t < p.T) base[static_cast<size_t>(t) * p.h_out] = acc[jj];
  }
}

// sgmv: row = token of the run, columns = rank index; z partial = scale * acc
template <int NC>
__device__ __forceinline__ void epilogue_sgmv_chunk(const GemmParams &p, const float (&acc)[NC],
                                                    int32_t t, bool valid, float scale,
                                                    int32_t split, int32_t c0) {
  if (!valid) return;
  float *zrow = p.zws_out + (static_cast<size_t>(split) * p.max_tokens + t) * p.R_pad + c0;
#pragma unroll
  for (int q = 0; q < NC; q += 4) {
    float4 o = make_float4(scale * acc[q], scale * acc[q + 1], scale * acc[q + 2], scale * acc[q + 3]);
    *reinterpret_cast<float4 *>(zrow + q) = o;
  }
}

__global__ void __launch_bounds__(kGemmThreads, 1)
lora_gemm_kernel(const __grid_constant__ CUtensorMap tmap_r, const __grid_constant__ CUtensorMap tmap_c,
                 const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  // tiles need 1024-byte alignment for the 128-byte swizzle
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t r_bytes = kTileM * kBlockK * 2;              // 16 KB
  const uint32_t c_bytes = static_cast<uint32_t>(p.BN) * kBlockK * 2;
  const uint32_t stage_bytes = r_bytes + c_bytes;
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + static_cast<size_t>(p.stages) * stage_bytes);
  uint64_t *full_bar = bars;                      // [stages]  TMA -> MMA
  uint64_t *empty_bar = bars + kMaxStages;        // [stages]  MMA -> TMA
  uint64_t *tfull_bar = bars + 2 * kMaxStages;    // [2]       MMA -> epilogue
  uint64_t *tempty_bar = tfull_bar + 2;           // [2]       epilogue -> MMA
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(tempty_bar + 2);
  volatile uint32_t *abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    ptx::prefetch_tensormap(&tmap_r);
    ptx::prefetch_tensormap(&tmap_c);
    for (int s = 0; s < p.stages; ++s) {
      ptx::mbar_init(&full_bar[s], 1);
      ptx::mbar_init(&empty_bar[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&tfull_bar[i], 1);
      ptx::mbar_init(&tempty_bar[i], 4);  // one arrival per epilogue warp
    }
    *abort_flag = 0;
    ptx::fence_barrier_init();
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
  const int32_t n_tiles = total_tiles(p);

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      for (int32_t tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x) {
        const TileCoord tc = tile_coord(p, tile);
        for (int32_t kb = tc.kb0; kb < tc.kb1; ++kb) {
          if (!ptx::mbar_wait(&empty_bar[stage], phase ^ 1) || *abort_flag) {
            ok = false;
            break;
          }
          uint8_t *sr = smem + static_cast<size_t>(stage) * stage_bytes;
          ptx::mbar_arrive_expect_tx(&full_bar[stage], stage_bytes);
          ptx::tma_load_2d(sr, &tmap_r, &full_bar[stage], kb * kBlockK, tc.row_r);
          if (p.mode == kModeSgmv)
            ptx::tma_load_3d(sr + r_bytes, &tmap_c, &full_bar[stage], kb * kBlockK, 0, tc.slot);
          else
            ptx::tma_load_2d(sr + r_bytes, &tmap_c, &full_bar[stage], kb * kBlockK, tc.row_c);
          if (++stage == static_cast<uint32_t>(p.stages)) {
            stage = 0;
            phase ^= 1;
          }
        }
      }
      if (!ok) {
        *abort_flag = 1;
        atomicOr(p.status, EDGELORA_STATUS_TIMEOUT);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = ptx::umma_idesc_bf16(kTileM, static_cast<uint32_t>(p.BN));
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      int32_t it = 0;
      for (int32_t tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x, ++it) {
        const TileCoord tc = tile_coord(p, tile);
        const uint32_t acc = (p.n_acc == 2) ? (it & 1) : 0;
        const uint32_t use = (p.n_acc == 2) ? (it >> 1) : it;
        if (!ptx::mbar_wait(&tempty_bar[acc], (use & 1) ^ 1) || *abort_flag) {
          ok = false;
          break;
        }
        ptx::tc_fence_after_sync();
        const uint32_t tmem_d = tmem_base + acc * static_cast<uint32_t>(p.BN);
        for (int32_t kb = tc.kb0; kb < tc.kb1; ++kb) {
          if (!ptx::mbar_wait(&full_bar[stage], phase) || *abort_flag) {
            ok = false;
            break;
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
          if (++stage == static_cast<uint32_t>(p.stages)) {
            stage = 0;
            phase ^= 1;
          }
        }
        if (!ok) break;
        ptx::umma_commit(&tfull_bar[acc]);  // accumulator complete
      }
      if (!ok) {
        *abort_flag = 1;
        atomicOr(p.status, EDGELORA_STATUS_TIMEOUT);
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int quad = warp & 3;                      // TMEM lanes [32*quad, 32*quad+32)
    const int row_in_tile = quad * 32 + lane;
    ptx::pdl_wait_prior_grids();                    // z / plan / workspace owners have finished
    bool ok = true;
    int32_t it = 0;
    for (int32_t tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x, ++it) {
      const TileCoord tc = tile_coord(p, tile);
      const uint32_t acc = (p.n_acc == 2) ? (it & 1) : 0;
      const uint32_t use = (p.n_acc == 2) ? (it >> 1) : it;

      // per-row state that does not need the accumulator
      int32_t a = -1, rank = 0;
      float scale = 0.f;
      bool valid = false;
      float z[64];
      const int32_t row = tc.row_r + row_in_tile;
      if (p.mode == kModePrefill) {
        valid = row < p.T;
        if (valid) a = p.ids_valid[row];
        if (a >= 0) rank = p.slots[a].rank;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          if (c * 8 < rank) {
            float4 lo = make_float4(0.f, 0.f, 0.f, 0.f), hi = lo;
            for (int sp = 0; sp < p.zsplits; ++sp) {
              const float4 *zp = reinterpret_cast<const float4 *>(
                  p.zws + (static_cast<size_t>(sp) * p.max_tokens + row) * p.R_pad + c * 8);
              const float4 u = zp[0], v = zp[1];
              lo.x += u.x; lo.y += u.y; lo.z += u.z; lo.w += u.w;
              hi.x += v.x; hi.y += v.y; hi.z += v.z; hi.w += v.w;
            }
            z[c * 8 + 0] = lo.x; z[c * 8 + 1] = lo.y; z[c * 8 + 2] = lo.z; z[c * 8 + 3] = lo.w;
            z[c * 8 + 4] = hi.x; z[c * 8 + 5] = hi.y; z[c * 8 + 6] = hi.z; z[c * 8 + 7] = hi.w;
          } else {
#pragma unroll
            for (int q = 0; q < 8; ++q) z[c * 8 + q] = 0.f;
          }
        }
      } else if (p.mode == kModeSgmv) {
        valid = row_in_tile < tc.nrows;
        scale = p.slots[tc.slot].scale;
      }

      if (!ptx::mbar_wait(&tfull_bar[acc], use & 1) || *abort_flag) {
        ok = false;
        break;
      }
      ptx::tc_fence_after_sync();
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) +
                             acc * static_cast<uint32_t>(p.BN);
      for (int32_t c0 = 0; c0 < p.BN; c0 += 32) {
        if (p.BN - c0 >= 32) {
          float v[32];
          ptx::tmem_ld_32x32(taddr + c0, v);
          if (p.mode == kModePrefill)
            epilogue_prefill_chunk<32>(p, v, row, valid, a, rank, z, tc.row_c + c0);
          else if (p.mode == kModeDecode)
            epilogue_decode_chunk<32>(p, v, row, tc.split, c0);
          else
            epilogue_sgmv_chunk<32>(p, v, row, valid, scale, tc.split, c0);
        } else {
          float v[16];
          ptx::tmem_ld_32x16(taddr + c0, v);
          if (p.mode == kModePrefill)
            epilogue_prefill_chunk<16>(p, v, row, valid, a, rank, z, tc.row_c + c0);
          else if (p.mode == kModeDecode)
            epilogue_decode_chunk<16>(p, v, row, tc.split, c0);
          else
            epilogue_sgmv_chunk<16>(p, v, row, valid, scale, tc.split, c0);
        }
      }
      // all TMEM reads of this warp are complete (tcgen05.wait::ld inside the loads)
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&tempty_bar[acc]);
    }
    if (!ok && lane == 0) {
      *abort_flag = 1;
      atomicOr(p.status, EDGELORA_STATUS_TIMEOUT);
    }
  }

  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, static_cast<uint32_t>(p.tmem_cols));
  }
}

cudaError_t gemm_set_smem_limit(size_t smem_bytes) {
  return cudaFuncSetAttribute(lora_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              static_cast<int>(smem_bytes));
}

cudaError_t launch_gemm(const CUtensorMap &tmap_row, const CUtensorMap &tmap_col,
                        const GemmParams &p, int32_t grid, size_t smem_bytes, bool pdl,
                        cudaStream_t stream) {
  return launch_ex(lora_gemm_kernel, dim3(grid), dim3(kGemmThreads), smem_bytes, stream, pdl,
                   tmap_row, tmap_col, p);
}

}  // namespace edgelora
