// Private to the library: the pool and plan objects behind the opaque handles of the C ABI, shared
// by the files that implement the host side (pool.cu, siteset.cu).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <utility>
#include <vector>

#include "internal.cuh"
#include "ptx.cuh"

namespace edgelora {

constexpr int kStagingBuffers = 4;

// text behind EDGELORA_ERR_CUDA for edgelora_strerror (per thread)
extern thread_local char g_last_error[256];
void set_last_cuda_error(cudaError_t e, const char *what);

struct TmapKey {
  const void *base;
  uint64_t d0, d1, d2;
  uint32_t b1, b0;  // box rows, box columns (64 => 128-byte swizzle, otherwise no swizzle)
  uint64_t s1, s2;  // byte strides of dimensions 1 and 2 (0 = dense)
  bool operator==(const TmapKey &o) const {
    return base == o.base && d0 == o.d0 && d1 == o.d1 && d2 == o.d2 && b1 == o.b1 && b0 == o.b0 && s1 == o.s1 &&
           s2 == o.s2;
  }
};
struct TmapEntry {
  TmapKey key;
  CUtensorMap map;
};

struct StagingBuf {
  uint8_t *host = nullptr;  // pinned: [A padded][B padded][SlotRow]
  cudaEvent_t done = nullptr;
  bool in_flight = false;
};

struct ProfRec {
  int kernel;
  cudaEvent_t start, stop;
};

}  // namespace edgelora

struct edgelora_plan {
  using PlanView = edgelora::PlanView;
  int32_t max_tokens = 0, n_slots = 0, last_T = 0;
  void *block = nullptr;
  PlanView pv{};
};

struct edgelora_pool {
  using SlotRow = edgelora::SlotRow;
  using StagingBuf = edgelora::StagingBuf;
  using TmapEntry = edgelora::TmapEntry;
  using ProfRec = edgelora::ProfRec;
  edgelora_pool_config cfg{};
  int R_pad = 0, device = 0, sms = 0;
  bool owns_arena = false, a_q8 = false;  // a_q8: the A blocks are kept in Q8_0 (EDGELORA_FLAG_A_Q8)
  uint8_t *arena = nullptr;
  uint8_t *q8_dev = nullptr;  // device scratch for one adapter in Q8_0 form (first use of load_slot_q8)
  uint16_t *A_pool = nullptr, *B_pool = nullptr;
  size_t a_block = 0, b_block = 0;  // elements per slot
  SlotRow *slots_dev = nullptr;
  std::vector<SlotRow> slots_host;
  StagingBuf staging[edgelora::kStagingBuffers];
  int next_staging = 0;
  cudaStream_t side = nullptr;
  cudaEvent_t load_ev = nullptr, use_ev = nullptr;
  uint64_t load_seq = 0;
  std::vector<std::pair<cudaStream_t, uint64_t>> load_waited;  // per stream: last load it waited for
  bool use_recorded = false;
  edgelora_plan *plan = nullptr;
  float *zws = nullptr;
  int32_t *group_counters = nullptr;
  int opt_decode_splits = 0, opt_shrink_items = 0, opt_gather_splits = 0, opt_gather_min_t = 256, opt_shrink_depth = 0;
  uint32_t *status_dev = nullptr;
  std::vector<TmapEntry> tmaps;
  size_t tmap_next = 0;
  int opt_regime = 0, opt_profile = 0, opt_pdl = 1, opt_fused_decode = 1;
  uint64_t fused_key = 0;  // launch shape the occupancy answer below belongs to
  int fused_max_ctas = 0;
  long long wait_cycles = edgelora::ptx::kWaitLimitCycles;
  int64_t last_info[8] = {0};
  int64_t total_launches = 0;
  // profiling
  std::vector<ProfRec> prof;
  size_t prof_used = 0;
  double prof_ms[5] = {0};
  int64_t prof_n[5] = {0};
  // host-buffer entry point
  uint16_t *hx = nullptr, *hy = nullptr, *dx = nullptr, *dy = nullptr;
  int32_t *hids = nullptr, *dids = nullptr;
  // pipelined host-buffer path: two sets of device mirrors, two copy streams, events per set
  uint16_t *pdx[2] = {nullptr, nullptr}, *pdy[2] = {nullptr, nullptr};
  int32_t *pdids[2] = {nullptr, nullptr};
  cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;
  cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_done[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr};
  uint64_t host_calls = 0;
};


namespace edgelora {

// What the next site of a set hands to this site's base-product launch: its segment shrink runs as
// extra tiles of the same persistent kernel (sites are independent, so the tensor cores never
// wait for a shrink of their own).
struct NextShrink {
  edgelora_pool *pool = nullptr;
  const uint16_t *x = nullptr;
};

// The layer (see pool.cu).  `skip_shrink`: this site's shrinks were already issued (as part of the
// previous site's launches); `next`: issue the next site's shrinks along with this site's kernels;
// `independent`: the call reads nothing the previous call on the stream writes, so its first
// kernel may start under that call's tail.
int lora_linear_impl(edgelora_pool *p, edgelora_plan *plan, const int32_t *ids_dev, const void *W_dev,
                     const void *x_dev, int32_t T, void *y_dev, cudaStream_t stream,
                     bool skip_shrink = false, const NextShrink *next = nullptr, bool independent = false);

}  // namespace edgelora
