// Routing plan for callers that must not allocate: the plan kernel's working arrays live in a
// file-scope device array instead of memory obtained at run time.  Everything else (the kernel,
// the meaning of the outputs) is shared with edgelora_plan_build / edgelora_plan_export.
#include <cuda_runtime.h>

#include <mutex>

#include "internal.cuh"

using namespace edgelora;

namespace {

constexpr int kStaticMaxTokens = EDGELORA_PLAN_STATIC_MAX_TOKENS;
constexpr int kStaticMaxTiles = kStaticMaxTokens / kSegMin + 8;
constexpr int kStaticTokenTiles = (kStaticMaxTokens + kTileM - 1) / kTileM;
// tok_seg, perm_short, lg_adapter: T each; gs_short, scratch: T + 1 each; segment tile list;
// per-token-tile adapter lists; counts[8]; status[4]
constexpr int kStaticInts = 3 * kStaticMaxTokens + 2 * (kStaticMaxTokens + 1) + 4 * kStaticMaxTiles +
                            (kStaticTokenTiles + 1) + kStaticTokenTiles * kTileM + 8 + 4;
constexpr int kMaxDevices = 64;

// Held by every GPU that loads the library, until the process exits (about 100 KB).
static __device__ __align__(256) int32_t g_plan_scratch[kStaticInts];

std::mutex g_mutex;
int32_t *g_scratch_addr[kMaxDevices] = {nullptr};  // device address of g_plan_scratch, per device

// The array's name is only a handle in host code; the address a kernel can use has to be asked
// for, once per device, with that device current.
int32_t *scratch_for_current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_scratch_addr[dev]) {
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_plan_scratch) != cudaSuccess || !ptr) {
      cudaGetLastError();
      return nullptr;
    }
    init_plan_kernel();
    g_scratch_addr[dev] = static_cast<int32_t *>(ptr);
  }
  return g_scratch_addr[dev];
}

}  // namespace

extern "C" int edgelora_plan_build_static(const int32_t *adapter_id_dev, int32_t T, int32_t n_slots,
                                          int32_t *ids_valid_dev, int32_t *perm_dev,
                                          int32_t *group_start_dev, int32_t *group_adapter_dev,
                                          int32_t *seg_start_dev, int32_t *seg_adapter_dev,
                                          int32_t *info_dev, void *stream) {
  if (T < 0 || n_slots < 1 || n_slots > 65534 || !info_dev) return EDGELORA_ERR_INVALID_ARG;
  if (T > kStaticMaxTokens) return EDGELORA_ERR_TOO_MANY_TOKENS;
  if (T > 0 && (!adapter_id_dev || !ids_valid_dev || !perm_dev || !group_start_dev ||
                !group_adapter_dev || !seg_start_dev || !seg_adapter_dev))
    return EDGELORA_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (T == 0) {
    if (cudaMemsetAsync(info_dev, 0, 4 * sizeof(int32_t), s) != cudaSuccess) return EDGELORA_ERR_CUDA;
    return EDGELORA_OK;
  }
  int32_t *q = scratch_for_current_device();
  if (!q) return EDGELORA_ERR_CUDA;

  PlanView pv{};
  pv.ids_valid = ids_valid_dev;
  pv.perm = perm_dev;
  pv.group_start = group_start_dev;
  pv.group_adapter = group_adapter_dev;
  pv.seg_start = seg_start_dev;
  pv.seg_adapter = seg_adapter_dev;
  pv.tok_seg = q; q += kStaticMaxTokens;
  pv.perm_short = q; q += kStaticMaxTokens;
  pv.gs_short = q; q += kStaticMaxTokens + 1;
  pv.scratch = q; q += kStaticMaxTokens + 1;
  pv.sgmv_tiles = q; q += 4 * kStaticMaxTiles;
  pv.lg_adapter = q; q += kStaticMaxTokens;
  pv.mt_count = q; q += kStaticTokenTiles + 1;
  pv.mt_list = q; q += kStaticTokenTiles * kTileM;
  pv.counts = q; q += 8;
  pv.status = reinterpret_cast<uint32_t *>(q);
  pv.max_sgmv_tiles = kStaticMaxTiles;

  // The array keeps what the previous call left: the status word must start at zero; every other
  // word the kernel reads it has written earlier in the same launch.
  if (cudaMemsetAsync(pv.status, 0, sizeof(uint32_t), s) != cudaSuccess) return EDGELORA_ERR_CUDA;
  launch_plan(adapter_id_dev, T, n_slots, pv, false, s);
  if (cudaGetLastError() != cudaSuccess) return EDGELORA_ERR_CUDA;
  // info = {n_groups, n_segments, status bits, 0}
  if (cudaMemcpyAsync(info_dev, pv.counts, 2 * sizeof(int32_t), cudaMemcpyDeviceToDevice, s) != cudaSuccess ||
      cudaMemcpyAsync(info_dev + 2, pv.status, sizeof(int32_t), cudaMemcpyDeviceToDevice, s) != cudaSuccess ||
      cudaMemsetAsync(info_dev + 3, 0, sizeof(int32_t), s) != cudaSuccess)
    return EDGELORA_ERR_CUDA;
  return EDGELORA_OK;
}
