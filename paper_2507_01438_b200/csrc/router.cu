// Scoring head of the adapter router (paper Section 3.2: one score in [0, 1] per adapter for a
// prompt; Section 5.1: a classification head on the base model): scores[b][j] =
// sigmoid(W_r[j] . h[b] + bias[j]).  One pass over W_r ([n][hidden] bf16, 8-16 MB for the paper's
// 1000-2000 adapters) is all the memory traffic there is, so this is a streaming kernel: a warp
// owns a row of W_r, reads it once with 16-byte loads (512 contiguous bytes per warp and step) and
// dots it with up to eight prompts' hidden states at a time, which sit in shared memory; lanes are
// reduced by shuffles.  fp32 accumulation, fp32 scores.
#include "internal.cuh"
#include "launch.cuh"
#include "ptx.cuh"

#include <algorithm>
#include <mutex>

namespace edgelora {

constexpr int kRouterThreads = 256;
constexpr int kRouterReq = 8;  // prompts per pass over a row
constexpr int kRouterUnroll = 8;

__global__ void __launch_bounds__(kRouterThreads)
router_scores_kernel(const uint16_t *__restrict__ Wr, const float *__restrict__ bias,
                     const uint16_t *__restrict__ h, int32_t B, int32_t n, int32_t hidden,
                     float *__restrict__ scores) {
  extern __shared__ uint4 s_h[];  // [min(B, 8)][hidden / 8]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n8 = hidden >> 3;
  ptx::pdl_launch_dependents();
  ptx::pdl_wait_prior_grids();  // h comes from earlier work on the stream
  for (int b0 = 0; b0 < B; b0 += kRouterReq) {
    const int nb = min(kRouterReq, B - b0);
    __syncthreads();
    for (int i = threadIdx.x; i < nb * n8; i += kRouterThreads)
      s_h[i] = __ldg(reinterpret_cast<const uint4 *>(h + static_cast<size_t>(b0) * hidden) + i);
    __syncthreads();
    for (int j = blockIdx.x * (kRouterThreads / 32) + warp; j < n; j += gridDim.x * (kRouterThreads / 32)) {
      const uint4 *row = reinterpret_cast<const uint4 *>(Wr + static_cast<size_t>(j) * hidden);
      float acc[kRouterReq];
#pragma unroll
      for (int q = 0; q < kRouterReq; ++q) acc[q] = 0.f;
      // kRouterUnroll loads of 16 bytes per lane in flight: a row is a few KB, so what matters is
      // how many requests a warp has outstanding, not how fast it adds
      for (int k0 = lane; k0 < n8; k0 += 32 * kRouterUnroll) {
        uint4 wv[kRouterUnroll];
#pragma unroll
        for (int u = 0; u < kRouterUnroll; ++u)
          wv[u] = (k0 + 32 * u < n8) ? __ldg(row + k0 + 32 * u) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int u = 0; u < kRouterUnroll; ++u) {
          const int k = k0 + 32 * u;
          if (k >= n8) break;
          const uint4 w = wv[u];
          const float w0 = ptx::bf16_lo(w.x), w1 = ptx::bf16_hi(w.x), w2 = ptx::bf16_lo(w.y), w3 = ptx::bf16_hi(w.y);
          const float w4 = ptx::bf16_lo(w.z), w5 = ptx::bf16_hi(w.z), w6 = ptx::bf16_lo(w.w), w7 = ptx::bf16_hi(w.w);
#pragma unroll
          for (int q = 0; q < kRouterReq; ++q) {
            if (q < nb) {
              const uint4 x = s_h[q * n8 + k];
              float s = acc[q];
              s = fmaf(w0, ptx::bf16_lo(x.x), s); s = fmaf(w1, ptx::bf16_hi(x.x), s);
              s = fmaf(w2, ptx::bf16_lo(x.y), s); s = fmaf(w3, ptx::bf16_hi(x.y), s);
              s = fmaf(w4, ptx::bf16_lo(x.z), s); s = fmaf(w5, ptx::bf16_hi(x.z), s);
              s = fmaf(w6, ptx::bf16_lo(x.w), s); s = fmaf(w7, ptx::bf16_hi(x.w), s);
              acc[q] = s;
            }
          }
        }
      }
#pragma unroll
      for (int q = 0; q < kRouterReq; ++q)
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) acc[q] += __shfl_xor_sync(0xffffffffu, acc[q], d);
      if (lane < nb) {
        float v = 0.f;
#pragma unroll
        for (int q = 0; q < kRouterReq; ++q)
          if (q == lane) v = acc[q];
        if (bias) v += bias[j];
        // sigmoid without overflow on either side
        const float e = __expf(-fabsf(v));
        const float s = v >= 0.f ? 1.f / (1.f + e) : e / (1.f + e);
        scores[static_cast<size_t>(b0 + lane) * n + j] = s;
      }
    }
  }
}

}  // namespace edgelora

extern "C" int edgelora_router_scores(const void *Wr_dev, const float *bias_dev, const void *h_dev, int32_t B,
                                      int32_t n, int32_t hidden, float *scores_dev, void *stream) {
  using namespace edgelora;
  if (B < 0 || n < 1 || hidden < 8 || (hidden & 7) || hidden > 8192) return EDGELORA_ERR_INVALID_ARG;
  if (B == 0) return EDGELORA_OK;
  if (!Wr_dev || !h_dev || !scores_dev) return EDGELORA_ERR_INVALID_ARG;
  // the shared-memory limit is an attribute of (function, device): kept per device
  static std::mutex mu;
  static int sms_of[64] = {0};  // 0 = this device is not configured yet
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
    cudaGetLastError();
    return EDGELORA_ERR_CUDA;
  }
  {
    std::lock_guard<std::mutex> lock(mu);
    if (sms_of[dev] == 0) {
      if (cudaFuncSetAttribute(router_scores_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               kRouterReq * 8192 * 2) != cudaSuccess ||
          cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
        cudaGetLastError();
        return EDGELORA_ERR_CUDA;
      }
      sms_of[dev] = sms;
    }
    sms = sms_of[dev];
  }
  const int warps = kRouterThreads / 32;
  const int grid = std::max(1, std::min((n + warps - 1) / warps, sms * 4));
  const size_t smem = static_cast<size_t>(std::min(B, kRouterReq)) * hidden * 2;
  cudaError_t e = launch_ex(router_scores_kernel, dim3(grid), dim3(kRouterThreads), smem,
                            static_cast<cudaStream_t>(stream), false, 1, static_cast<const uint16_t *>(Wr_dev),
                            bias_dev, static_cast<const uint16_t *>(h_dev), B, n, hidden, scores_dev);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return EDGELORA_ERR_CUDA;
  }
  return EDGELORA_OK;
}
