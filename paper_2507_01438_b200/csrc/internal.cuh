// Structures shared by the kernels and the host launcher of the batch LoRA library.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/edgelora.h"

namespace edgelora {

constexpr int kTileM = 128;        // UMMA M: rows of the TMEM accumulator (one per lane)
constexpr int kBlockK = 64;        // bf16 elements per K block = one 128-byte swizzled row
constexpr int kUmmaK = 16;         // K of one tcgen05.mma for 16-bit inputs
constexpr int kMaxStages = 12;
constexpr int kSegMin = 32;        // prefill: runs at least this long go through the segment shrink
constexpr int kDecodeMaxT = 256;   // decode regime: all tokens are one UMMA N tile
constexpr int kMaxTokensLimit = 32768;
constexpr int kGemmThreads = 320;  // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue, warps 6..9 z operand
constexpr int kMaxZSplits = 16;    // partial z planes (K splits of the shrink); plane 16 = summed z
constexpr int kShrinkThreads = 256;
constexpr int kShrinkStepElems = 256;  // K elements of one shrink step (512 bytes of a row)

// Checked build: EL_CHECK(status, cond, site) is `cond`, and when it is false raises
// EDGELORA_STATUS_BOUNDS in the status word and records `site` (a number naming the test) in the
// word after it, first failure only; the caller skips the access.  In the normal build it is `true`
// and costs nothing.  Every role of a kernel evaluates the same tests on the same data, so a skipped
// K block is skipped by all of them.
#ifdef EDGELORA_CHECKED
__device__ __forceinline__ bool el_check_fail(uint32_t *status, uint32_t site) {
  atomicOr(status, EDGELORA_STATUS_BOUNDS);
  atomicCAS(status + 1, 0u, site);
  return false;
}
#define EL_CHECK(status, cond, site) ((cond) ? true : ::edgelora::el_check_fail((status), (site)))
#else
#define EL_CHECK(status, cond, site) (true)
#endif

// One row of the slot table (paper Section 3.3: one fixed block per resident adapter).
struct SlotRow {
  int32_t rank;        // 0 = empty
  float scale;         // s_a
  int32_t generation;  // bumped on every load / evict
  int32_t pad;
};

// Device arrays of a routing plan.
struct PlanView {
  int32_t *ids_valid;      // [maxT]   id, or -1 where the caller's id was out of range
  int32_t *perm;           // [maxT]   tokens ordered by (id, token)
  int32_t *group_start;    // [maxT+1]
  int32_t *group_adapter;  // [maxT]
  int32_t *seg_start;      // [maxT+1]
  int32_t *seg_adapter;    // [maxT]
  int32_t *tok_seg;        // [maxT]   segment index of each token
  int32_t *perm_short;     // [maxT]   perm restricted to tokens the gather-by-token shrink handles
  int32_t *gs_short;       // [maxT+1] group boundaries inside perm_short
  int32_t *sgmv_tiles;     // [max_sgmv_tiles][4] {first token, tokens, slot, 0}
  int32_t *scratch;        // [maxT+1]
  int32_t *lg_adapter;     // [maxT]   distinct ids >= 0 of the batch, ascending (the LoRA groups)
  int32_t *mt_count;       // [maxT/128+1] distinct ids >= 0 inside each 128-token tile
  int32_t *mt_list;        // [ceil(maxT/128)*128] those ids, tile m at [128 m, 128 m + mt_count[m])
  int32_t *counts;         // [8]  0: n_groups, 1: n_segments, 2: n_sgmv_tiles, 3: short tokens,
                           //      4: LoRA groups, 5: K chunks used by the decode shrink
  uint32_t *status;        // device status word of the plan
  int32_t max_sgmv_tiles;
};

enum GemmMode : int32_t { kModePrefill = 0, kModeDecode = 1, kModeSgmv = 2 };

struct GemmParams {
  int32_t mode;
  int32_t T, h_in, h_out;
  int32_t BN;          // UMMA N = rows of the column-operand tile (multiple of 16, <= 256)
  int32_t stages;      // TMA pipeline depth
  int32_t n_acc;       // TMEM accumulator buffers (1 or 2)
  int32_t tmem_cols;   // power of two >= n_acc * acc_cols, >= 32
  int32_t ring_rows;   // rows of the C region of a ring stage (>= BN; wider when gather passes need it)
  int32_t acc_cols;    // TMEM columns between the accumulators (>= BN, >= gN)
  int32_t y_tma;       // prefill: y leaves through a shared-memory stage and TMA stores (needs the y map)
  int32_t fill_rounds; // prefill with a second job: how many of that job's tiles a CTA with a tile fewer (or none)
                       // takes before the other CTAs get any: about (K blocks of a tile) / (K blocks of such an item)
  int32_t heavy_first; // prefill: the first token tile holds the batch's decode tokens (many LoRA K blocks per
                       // output tile): its tiles go to the CTAs that get one tile fewer (see heavy_slots)
  int32_t kb_total;    // K blocks of 64 covering h_in
  int32_t kb_per;      // K blocks per split
  int32_t splits;
  int32_t n_mtiles;    // prefill: token tiles; decode: W row tiles
  int32_t n_ntiles;    // prefill: W row tiles of BN
  int32_t R_pad;       // slot block rank stride
  int32_t zsplits;     // partial z planes the consumer sums
  int32_t expand_in_reduce;  // decode, small batches: B_a z is added by the owners of the cluster
                             // reduction on the CUDA cores instead of by LoRA K blocks
  int32_t max_tokens;  // row stride of the z / plan workspaces
  long long wait_cycles;  // limit of the bounded in-kernel waits, in SM clock cycles
  // shrink jobs (mode sgmv): gather tiles for the tokens the segment tiles do not cover
  int32_t gather;      // 1: the job also has gather tiles (stacked A rows x gathered token rows)
  int32_t finalize;    // 1: whoever completes a gather tile last adds its K splits into the final z plane
  int32_t gN;          // most token rows of one gather pass (multiple of 16, <= rows of the ring's C region)
  const int32_t *perm_short;     // plan: tokens ordered by (id, token), short runs only
  const int32_t *gs_short;       // plan: group boundaries inside perm_short
  const int32_t *group_adapter;  // plan: adapter of each group (-1 first when present)
  int32_t *tile_counters;        // [>= gather tiles] arrivals per gather tile, zero between launches
  const int32_t *ids_valid;
  const int32_t *ids;       // decode: the caller's ids (validated again inside the kernel)
  int32_t n_slots;
  const SlotRow *slots;
  const uint16_t *B_pool;   // [S][h_out][R_pad]
  const float *zws;         // [zsplits][max_tokens][R_pad]   (read by the prefill epilogue)
  float *zws_out;           // same buffer, written by the segment shrink
  uint16_t *y;              // [T][h_out]
  const int32_t *sgmv_tiles;
  const int32_t *counts;
  const int32_t *mt_count;    // prefill: per 128-token tile
  const int32_t *mt_list;
  uint32_t *status;
};

// Small decode batches in one launch (paper Section 3.4, both LoRA products and the base product of
// one layer call): the first n_ctas CTAs of the tile kernel's grid compute z = s_a A_a x on the CUDA
// cores while the others stream W; the owners of the cluster reduction wait (bounded) for the
// shrink CTAs' arrival counter before they add B_a z.
struct FusedDecode {
  int32_t n_ctas;          // 0 = not fused; otherwise a multiple of the cluster size
  int32_t ks;              // K chunks of the shrink = partial z planes the expand adds, in order
  int32_t x_wait;          // 1: x may be an output of the kernel before this one: wait before reading it
  int32_t b_stage;         // 1: the launch's shared memory has room, behind the ring and the barriers, for the
                           // B_a rows (tokens per owner x 128 rows x R_pad) and z of an owner's tokens;
                           // 2: also for the buffer of the cluster reduction
  const uint16_t *A_pool;  // [S][R_pad][h_in]
  const uint16_t *x;       // [T][h_in]
  float *z;                // [ks][max_tokens][R_pad]
  int32_t *sync;           // [2] {shrink CTAs done, expand warps past their wait}; zero between launches
  PlanView pv;             // published by the first shrink CTA
};

// kernels (defined in plan.cu, shrink.cu, gemm.cu)
void launch_plan(const int32_t *ids, int32_t T, int32_t n_slots, const PlanView &pv, bool pdl,
                 cudaStream_t stream);
void init_plan_kernel();
cudaError_t launch_gemm(const CUtensorMap &tmap_row, const CUtensorMap &tmap_col,
                        const CUtensorMap &tmap_b, const GemmParams &p, int32_t grid,
                        size_t smem_bytes, bool pdl, cudaStream_t stream, const CUtensorMap *tmap_y = nullptr);
cudaError_t launch_gemm2(const CUtensorMap &tmap_row, const CUtensorMap &tmap_col,
                         const CUtensorMap &tmap_b, const GemmParams &p, const CUtensorMap &tmap_row2,
                         const CUtensorMap &tmap_col2, const CUtensorMap &tmap_g2, const GemmParams &p2,
                         int32_t grid, size_t smem_bytes, bool pdl, cudaStream_t stream,
                         const CUtensorMap *tmap_y = nullptr);
// Decode job with the shrink in the same grid: grid = f.n_ctas + p.n_mtiles * p.splits CTAs.
cudaError_t launch_gemm_fused(const CUtensorMap &tmap_row, const CUtensorMap &tmap_col, const GemmParams &p,
                              const FusedDecode &f, size_t smem_bytes, bool pdl, cudaStream_t stream);
// How many CTAs of such a launch (in whole clusters) can be resident at once on the current device.
int32_t gemm_fused_max_ctas(int32_t cluster, size_t smem_bytes);
constexpr int kYStageBytes = 4 * 32 * 128;  // prefill epilogue: per epilogue warp 32 rows x 64 bf16
cudaError_t gemm_set_smem_limit(size_t smem_bytes);
cudaError_t shrink_set_smem_limit();
cudaError_t launch_q8_to_block(const uint8_t *A_q8, const uint8_t *B_q8, uint16_t *A_blk, uint16_t *B_blk,
                               int32_t rank, int32_t R_pad, int32_t h_in, int32_t h_out, int32_t sms,
                               cudaStream_t stream);
void set_last_cuda_error(cudaError_t e, const char *what);
cudaError_t launch_wait_selftest(uint32_t *status, long long wait_cycles, cudaStream_t stream);
cudaError_t launch_decode_shrink(const CUtensorMap &tmap_a, const CUtensorMap &tmap_d, const CUtensorMap &tmap_x,
                                 const int32_t *ids, const SlotRow *slots, const PlanView &pv,
                                 float *zws, int32_t *group_counters, int32_t T, int32_t h_in,
                                 int32_t R_pad, int32_t n_slots, int32_t max_tokens,
                                 int32_t target_items, int32_t grid, uint32_t *status, bool pdl, bool a_q8,
                                 int32_t depth, cudaStream_t stream);

}  // namespace edgelora
