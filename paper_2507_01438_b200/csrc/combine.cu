// Decode combine: y[t] = bf16( sum_split partial[split][t] + B_a z[t] )   (paper Section 3.4: the
// results of the pre-trained part and of the LoRA part are combined and returned to the token's
// own position).  The split-K partials of the base product are summed in a fixed order, the
// expand B_a z (z already carries s_a) is added, and y is written once.
//
// One CTA per (token, 512 output columns); a thread owns two adjacent columns, so the rows of
// B_a it reads are contiguous across the warp and y is stored as packed bf16 pairs.
#include "internal.cuh"
#include "launch.cuh"
#include "ptx.cuh"

namespace edgelora {

constexpr int kCombineThreads = 256;

__global__ void __launch_bounds__(kCombineThreads)
decode_combine_kernel(const float *__restrict__ ws, int32_t splits, const float *__restrict__ zws,
                      int32_t zsplits, int32_t max_tokens, const uint16_t *__restrict__ B_pool,
                      const SlotRow *__restrict__ slots, const int32_t *__restrict__ ids_valid,
                      uint16_t *__restrict__ y, int32_t T, int32_t h_out, int32_t R_pad) {
  __shared__ float zs[64];
  ptx::pdl_launch_dependents();
  ptx::pdl_wait_prior_grids();

  const int t = blockIdx.y;
  const int j = 2 * (blockIdx.x * kCombineThreads + threadIdx.x);
  const int a = ids_valid[t];
  const int rank = (a >= 0) ? slots[a].rank : 0;
  if (threadIdx.x < 64) {
    float s = 0.f;
    if (static_cast<int>(threadIdx.x) < rank)
      for (int sp = 0; sp < zsplits; ++sp)
        s += zws[(static_cast<size_t>(sp) * max_tokens + t) * R_pad + threadIdx.x];
    zs[threadIdx.x] = s;
  }
  __syncthreads();
  if (j >= h_out) return;

  float y0 = 0.f, y1 = 0.f;
  for (int sp = 0; sp < splits; ++sp) {
    const float2 v = *reinterpret_cast<const float2 *>(ws + (static_cast<size_t>(sp) * T + t) * h_out + j);
    y0 += v.x;
    y1 += v.y;
  }
  if (rank > 0) {
    const uint4 *B0 = reinterpret_cast<const uint4 *>(B_pool + (static_cast<size_t>(a) * h_out + j) * R_pad);
    const uint4 *B1 = B0 + (R_pad >> 3);
    float s0 = 0.f, s1 = 0.f;
    for (int c = 0; c * 8 < rank; ++c) {
      const uint4 b0 = __ldg(B0 + c), b1 = __ldg(B1 + c);
      const float *zc = zs + c * 8;
      s0 = fmaf(ptx::bf16_lo(b0.x), zc[0], s0); s0 = fmaf(ptx::bf16_hi(b0.x), zc[1], s0);
      s0 = fmaf(ptx::bf16_lo(b0.y), zc[2], s0); s0 = fmaf(ptx::bf16_hi(b0.y), zc[3], s0);
      s0 = fmaf(ptx::bf16_lo(b0.z), zc[4], s0); s0 = fmaf(ptx::bf16_hi(b0.z), zc[5], s0);
      s0 = fmaf(ptx::bf16_lo(b0.w), zc[6], s0); s0 = fmaf(ptx::bf16_hi(b0.w), zc[7], s0);
      s1 = fmaf(ptx::bf16_lo(b1.x), zc[0], s1); s1 = fmaf(ptx::bf16_hi(b1.x), zc[1], s1);
      s1 = fmaf(ptx::bf16_lo(b1.y), zc[2], s1); s1 = fmaf(ptx::bf16_hi(b1.y), zc[3], s1);
      s1 = fmaf(ptx::bf16_lo(b1.z), zc[4], s1); s1 = fmaf(ptx::bf16_hi(b1.z), zc[5], s1);
      s1 = fmaf(ptx::bf16_lo(b1.w), zc[6], s1); s1 = fmaf(ptx::bf16_hi(b1.w), zc[7], s1);
    }
    y0 += s0;
    y1 += s1;
  }
  *reinterpret_cast<uint32_t *>(y + static_cast<size_t>(t) * h_out + j) = ptx::pack_bf16x2(y0, y1);
}

void launch_decode_combine(const float *ws, int32_t splits, const float *zws, int32_t zsplits,
                           int32_t max_tokens, const uint16_t *B_pool, const SlotRow *slots,
                           const int32_t *ids_valid, uint16_t *y, int32_t T, int32_t h_out,
                           int32_t R_pad, bool pdl, cudaStream_t stream) {
  dim3 grid((h_out + 2 * kCombineThreads - 1) / (2 * kCombineThreads), T);
  launch_ex(decode_combine_kernel, grid, dim3(kCombineThreads), 0, stream, pdl, ws, splits, zws,
            zsplits, max_tokens, B_pool, slots, ids_valid, y, T, h_out, R_pad);
}

}  // namespace edgelora
