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
constexpr int kRouterReq = 8;      // prompts per pass over a row
constexpr int kRouterUnroll = 16;  // 16-byte loads per lane in flight: a whole row of 4096 values

// A warp asks for (the first 8 KB of) its first row before the prompts are staged in shared memory, so
// that the rows are on their way while the CTA synchronises: the kernel is a few microseconds long and
// what it waits for is the first round trip to HBM.  Up to eight prompts share a pass over W_r; the
// loop over them is rolled (the row stays in registers), because code that runs once or twice per
// launch costs its instruction fetch: lane q ends up with the score of prompt b0 + q.
__global__ void __launch_bounds__(kRouterThreads)
router_scores_kernel(const uint16_t *__restrict__ Wr, const float *__restrict__ bias,
                     const uint16_t *__restrict__ h, int32_t B, int32_t n, int32_t hidden,
                     float *__restrict__ scores) {
  extern __shared__ uint4 s_h[];  // [min(B, 8)][hidden / 8]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n8 = hidden >> 3;
  const int j_first = blockIdx.x * (kRouterThreads / 32) + warp, j_step = gridDim.x * (kRouterThreads / 32);
  ptx::pdl_launch_dependents();
  auto load_chunk = [&](int j, int k0, uint4 (&wv)[kRouterUnroll]) {
    const uint4 *row = reinterpret_cast<const uint4 *>(Wr + static_cast<size_t>(j) * hidden);
#pragma unroll
    for (int u = 0; u < kRouterUnroll; ++u)
      wv[u] = (k0 + 32 * u < n8) ? __ldg(row + k0 + 32 * u) : make_uint4(0u, 0u, 0u, 0u);
  };
  uint4 wv[kRouterUnroll];
  if (j_first < n) load_chunk(j_first, lane, wv);  // W_r is not written by anything on the stream
  ptx::pdl_wait_prior_grids();                      // h comes from earlier work on the stream
  for (int b0 = 0; b0 < B; b0 += kRouterReq) {
    const int nb = min(kRouterReq, B - b0);
    __syncthreads();
    for (int i = threadIdx.x; i < nb * n8; i += kRouterThreads)
      s_h[i] = __ldg(reinterpret_cast<const uint4 *>(h + static_cast<size_t>(b0) * hidden) + i);
    __syncthreads();
    for (int j = j_first; j < n; j += j_step) {
      float v = 0.f;  // lane q: W_r[j] . h[b0 + q]
      for (int k0 = lane; k0 < n8; k0 += 32 * kRouterUnroll) {
        if (!(b0 == 0 && j == j_first && k0 == lane)) load_chunk(j, k0, wv);  // the first chunk is already here
#pragma unroll 1
        for (int q = 0; q < nb; ++q) {
          const uint4 *hq = s_h + q * n8 + k0;
          float s = 0.f;
#pragma unroll
          for (int u = 0; u < kRouterUnroll; ++u) {
            if (k0 + 32 * u < n8) {  // (values past the row are zero: nothing to add)
              const uint4 w = wv[u], x = hq[32 * u];
              s = fmaf(ptx::bf16_lo(w.x), ptx::bf16_lo(x.x), s); s = fmaf(ptx::bf16_hi(w.x), ptx::bf16_hi(x.x), s);
              s = fmaf(ptx::bf16_lo(w.y), ptx::bf16_lo(x.y), s); s = fmaf(ptx::bf16_hi(w.y), ptx::bf16_hi(x.y), s);
              s = fmaf(ptx::bf16_lo(w.z), ptx::bf16_lo(x.z), s); s = fmaf(ptx::bf16_hi(w.z), ptx::bf16_hi(x.z), s);
              s = fmaf(ptx::bf16_lo(w.w), ptx::bf16_lo(x.w), s); s = fmaf(ptx::bf16_hi(w.w), ptx::bf16_hi(x.w), s);
            }
          }
#pragma unroll
          for (int d = 16; d > 0; d >>= 1) s += __shfl_xor_sync(0xffffffffu, s, d);
          if (lane == q) v += s;
        }
      }
      if (lane < nb) {
        if (bias) v += bias[j];
        // sigmoid without overflow on either side
        const float e = __expf(-fabsf(v));
        const float sg = v >= 0.f ? 1.f / (1.f + e) : e / (1.f + e);
        scores[static_cast<size_t>(b0 + lane) * n + j] = sg;
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
