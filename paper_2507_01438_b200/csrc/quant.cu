// Q8_0 adapters (paper Section 5.1: "All LoRA adapters are quantized using the Q8_0 format").
// Q8_0 is the published ggml block format: 32 consecutive values of a row share one half-precision
// scale d and are stored as signed bytes q; the value is d * q.  A block is 34 bytes: d (2 bytes,
// little endian), then q[32].
//
// The kernel here turns an adapter that arrived in this format into the pool's block layout
// (A padded to [R_pad][h_in], B to [h_out][R_pad], bfloat16, padding zero): the host-to-device copy
// moves the 8-bit form (about half the bytes), the conversion happens on the device, on the pool's
// side stream, and the layer kernels read the block as they read any other.
#include <cuda_fp16.h>

#include <algorithm>

#include "internal.cuh"
#include "ptx.cuh"

namespace edgelora {

constexpr int kQ8Block = 32;
constexpr int kQ8Bytes = 34;

__device__ __forceinline__ float q8_value(const uint8_t *row_blocks, int32_t k) {
  const uint8_t *blk = row_blocks + static_cast<size_t>(k / kQ8Block) * kQ8Bytes;
  const __half d = __ushort_as_half(static_cast<unsigned short>(blk[0] | (blk[1] << 8)));
  const int q = static_cast<int8_t>(blk[2 + (k % kQ8Block)]);
  return __half2float(d) * static_cast<float>(q);
}

// A_q8: [rank][h_in / 32] blocks; B_q8: [h_out][ceil(rank / 32)] blocks.  One thread per output pair.
__global__ void __launch_bounds__(256)
q8_to_block_kernel(const uint8_t *__restrict__ A_q8, const uint8_t *__restrict__ B_q8, uint16_t *__restrict__ A_blk,
                   uint16_t *__restrict__ B_blk, int32_t rank, int32_t R_pad, int32_t h_in, int32_t h_out) {
  // (A_q8 == nullptr: only B is converted, for pools that keep A in Q8_0)
  const size_t a_pairs = A_q8 ? static_cast<size_t>(R_pad) * h_in / 2 : 0, b_pairs = static_cast<size_t>(h_out) * R_pad / 2;
  const size_t a_row_bytes = static_cast<size_t>(h_in / kQ8Block) * kQ8Bytes;
  const size_t b_row_bytes = static_cast<size_t>((rank + kQ8Block - 1) / kQ8Block) * kQ8Bytes;
  for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < a_pairs + b_pairs;
       i += static_cast<size_t>(gridDim.x) * blockDim.x) {
    float lo = 0.f, hi = 0.f;
    uint32_t *dst;
    if (i < a_pairs) {
      const int32_t r = static_cast<int32_t>((2 * i) / h_in), k = static_cast<int32_t>((2 * i) % h_in);
      if (r < rank) {
        lo = q8_value(A_q8 + r * a_row_bytes, k);
        hi = q8_value(A_q8 + r * a_row_bytes, k + 1);
      }
      dst = reinterpret_cast<uint32_t *>(A_blk) + i;
    } else {
      const size_t e = 2 * (i - a_pairs);
      const int32_t j = static_cast<int32_t>(e / R_pad), c = static_cast<int32_t>(e % R_pad);
      if (c < rank) lo = q8_value(B_q8 + j * b_row_bytes, c);
      if (c + 1 < rank) hi = q8_value(B_q8 + j * b_row_bytes, c + 1);
      dst = reinterpret_cast<uint32_t *>(B_blk) + (i - a_pairs);
    }
    *dst = ptx::pack_bf16x2(lo, hi);
  }
}

// Base weights stored in a block format (paper Section 5.1, model table: base models in Q8_0 or
// Q4_0).  Q4_0 is the published ggml format of 18 bytes per 32 consecutive values of a row: a
// half-precision scale d, then 16 bytes; byte j holds value j in its low four bits and value j + 16
// in its high four bits, each as an unsigned code c with value d * (c - 8).  One thread decodes one
// block into 32 bfloat16 values (round to nearest even; d * code is exact in fp32).
template <int kFormat>  // 0: Q8_0, 1: Q4_0
__global__ void __launch_bounds__(256)
weights_decode_kernel(const uint8_t *__restrict__ Wq, uint16_t *__restrict__ W, size_t n_blocks) {
  constexpr int kBytes = kFormat == 0 ? kQ8Bytes : 18;
  for (size_t b = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; b < n_blocks;
       b += static_cast<size_t>(gridDim.x) * blockDim.x) {
    const uint8_t *blk = Wq + b * kBytes;
    const float d = __half2float(__ushort_as_half(static_cast<unsigned short>(blk[0] | (blk[1] << 8))));
    float v[32];
    if (kFormat == 0) {
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = d * static_cast<float>(static_cast<int8_t>(blk[2 + i]));
    } else {
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const int byte = blk[2 + j];
        v[j] = d * static_cast<float>((byte & 0xF) - 8);
        v[j + 16] = d * static_cast<float>((byte >> 4) - 8);
      }
    }
    uint4 *dst = reinterpret_cast<uint4 *>(W + b * 32);  // blocks follow one another along the rows
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      uint4 o;
      o.x = ptx::pack_bf16x2(v[8 * q + 0], v[8 * q + 1]);
      o.y = ptx::pack_bf16x2(v[8 * q + 2], v[8 * q + 3]);
      o.z = ptx::pack_bf16x2(v[8 * q + 4], v[8 * q + 5]);
      o.w = ptx::pack_bf16x2(v[8 * q + 6], v[8 * q + 7]);
      dst[q] = o;
    }
  }
}

cudaError_t launch_weights_decode(int32_t format, const uint8_t *Wq, uint16_t *W, size_t n_blocks, cudaStream_t stream) {
  const int grid = static_cast<int>(std::min<size_t>((n_blocks + 255) / 256, 148 * 8));
  if (format == 0)
    weights_decode_kernel<0><<<grid, 256, 0, stream>>>(Wq, W, n_blocks);
  else
    weights_decode_kernel<1><<<grid, 256, 0, stream>>>(Wq, W, n_blocks);
  return cudaGetLastError();
}

cudaError_t launch_q8_to_block(const uint8_t *A_q8, const uint8_t *B_q8, uint16_t *A_blk, uint16_t *B_blk,
                               int32_t rank, int32_t R_pad, int32_t h_in, int32_t h_out, int32_t sms,
                               cudaStream_t stream) {
  q8_to_block_kernel<<<sms * 4, 256, 0, stream>>>(A_q8, B_q8, A_blk, B_blk, rank, R_pad, h_in, h_out);
  return cudaGetLastError();
}

}  // namespace edgelora

extern "C" int edgelora_weights_decode(int32_t format, const void *W_blocks_dev, int32_t h_out, int32_t h_in,
                                       uint16_t *W_dev, void *stream) {
  if ((format != EDGELORA_WEIGHTS_Q8_0 && format != EDGELORA_WEIGHTS_Q4_0) || !W_blocks_dev || !W_dev || h_out <= 0 ||
      h_in <= 0 || h_in % 32 != 0)
    return EDGELORA_ERR_INVALID_ARG;
  const size_t n_blocks = static_cast<size_t>(h_out) * (h_in / 32);
  const cudaError_t e = edgelora::launch_weights_decode(format, static_cast<const uint8_t *>(W_blocks_dev), W_dev, n_blocks,
                                                        static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) {
    edgelora::set_last_cuda_error(e, "weights_decode_kernel");
    return EDGELORA_ERR_CUDA;
  }
  return EDGELORA_OK;
}
