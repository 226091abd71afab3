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
  launch_ex(bgmv_shrink_kernel, dim3(max_groups * R_pad), dim3(kBgmvThreads), 0, stream, pdl, x,
            A_pool, slots, pv, zws, T, h_in, R_pad, zsplits, max_tokens, status);
}

}  // namespace edgelora
