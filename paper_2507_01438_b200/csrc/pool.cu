// Host side of the C ABI: the adapter pool (slot blocks + slot table in HBM, pinned staging,
// side-stream loads), the routing-plan objects and the launcher of the batched layer.
// Paper Section 3.3 / 4.2 (pre-allocated pool of fixed blocks, reuse after eviction) and
// Section 3.4 / 4.3 (batch LoRA inference).
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <utility>
#include <vector>

#include "guard.h"
#include "pool.h"

using namespace edgelora;

namespace edgelora {
thread_local char g_last_error[256] = "";
void set_last_cuda_error(cudaError_t e, const char *what) {
  snprintf(g_last_error, sizeof g_last_error, "%s: %s", what, cudaGetErrorString(e));
  if (getenv("EDGELORA_LOG")) fprintf(stderr, "[edgelora] CUDA error: %s\n", g_last_error);
}
}  // namespace edgelora

namespace {

constexpr int kTmapCache = 32;
constexpr int kProfEvents = 8192;
constexpr size_t kSmemBudget = 220 * 1024;
constexpr int kMaxDecodeSplits = 8;  // K splits of a row tile form one (portable-size) cluster

#define CUDA_TRY(expr)                                   \
  do {                                                   \
    cudaError_t _e = (expr);                             \
    if (_e != cudaSuccess) {                             \
      set_last_cuda_error(_e, #expr);                    \
      return EDGELORA_ERR_CUDA;                          \
    }                                                    \
  } while (0)

inline int round_up(int v, int m) { return (v + m - 1) / m * m; }
inline int pad_rank(int r) { return r <= 16 ? 16 : (r <= 32 ? 32 : 64); }

// ---- cuTensorMapEncodeTiled through the runtime's driver entry point (no link to libcuda) ----
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 row-major [d2][d1][d0] (d2 == 0 => 2D), box = {box_cols, box_rows, 1}; out-of-range
// elements read as zero.  box_cols == 64: the 128-byte-swizzled operand tiles of the GEMM;
// otherwise (the shrink's row segments) no swizzle.
int encode_tmap(CUtensorMap *out, const void *base, uint64_t d0, uint64_t d1, uint64_t d2,
                uint32_t box_rows, uint32_t box_cols, uint64_t s1 = 0, uint64_t s2 = 0) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return EDGELORA_ERR_CUDA;
  const cuuint32_t rank = d2 ? 3 : 2;
  cuuint64_t dims[3] = {d0, d1, d2 ? d2 : 1};
  cuuint64_t strides[2] = {s1 ? s1 : d0 * 2, s2 ? s2 : d0 * d1 * 2};
  cuuint32_t box[3] = {box_cols, box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void *>(base), dims,
                  strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  box_cols == static_cast<uint32_t>(kBlockK) ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(g_last_error, sizeof g_last_error, "cuTensorMapEncodeTiled failed (%d)", (int)r);
    return EDGELORA_ERR_CUDA;
  }
  return EDGELORA_OK;
}

}  // namespace

namespace {

// The descriptor is copied out: a later miss of the same call may reuse the cache entry it came
// from (the cache is a ring), and the launch takes its descriptors by value anyway.
int get_tmap(edgelora_pool *p, CUtensorMap *out, const void *base, uint64_t d0, uint64_t d1,
             uint64_t d2, uint32_t box_rows, uint32_t box_cols = kBlockK, uint64_t s1 = 0, uint64_t s2 = 0) {
  TmapKey key{base, d0, d1, d2, box_rows, box_cols, s1, s2};
  for (auto &e : p->tmaps)
    if (e.key == key) {
      *out = e.map;
      return EDGELORA_OK;
    }
  TmapEntry e;
  e.key = key;
  int rc = encode_tmap(&e.map, base, d0, d1, d2, box_rows, box_cols, s1, s2);
  if (rc != EDGELORA_OK) return rc;
  *out = e.map;
  if (p->tmaps.size() < static_cast<size_t>(kTmapCache)) {
    p->tmaps.push_back(e);
  } else {
    p->tmaps[p->tmap_next] = e;
    p->tmap_next = (p->tmap_next + 1) % kTmapCache;
  }
  return EDGELORA_OK;
}

bool stream_capturing(cudaStream_t s) {
  cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(s, &st) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  return st != cudaStreamCaptureStatusNone;
}

struct ProfScope {
  edgelora_pool *p;
  cudaStream_t s;
  ProfRec *rec = nullptr;
  ProfScope(edgelora_pool *pool, int kernel, cudaStream_t stream) : p(pool), s(stream) {
    if (p->opt_profile && p->prof_used < p->prof.size() && !stream_capturing(s)) {
      rec = &p->prof[p->prof_used++];
      rec->kernel = kernel;
      cudaEventRecord(rec->start, s);
    }
  }
  ~ProfScope() {
    if (rec) cudaEventRecord(rec->stop, s);
  }
};

int check_cfg(const edgelora_pool_config *c) {
  if (!c) return EDGELORA_ERR_INVALID_ARG;
  if (c->h_in < 8 || c->h_out < 8 || (c->h_in % 8) || (c->h_out % 8)) return EDGELORA_ERR_INVALID_ARG;
  if (c->n_slots < 1 || c->n_slots > 65534) return EDGELORA_ERR_INVALID_ARG;
  if ((c->flags & EDGELORA_FLAG_A_Q8) && (c->h_in % 256)) return EDGELORA_ERR_INVALID_ARG;
  if (c->max_rank < 1) return EDGELORA_ERR_INVALID_ARG;
  if (c->max_rank > 64) return EDGELORA_ERR_RANK_TOO_LARGE;
  if (c->max_tokens < 0 || c->max_tokens > kMaxTokensLimit) return EDGELORA_ERR_TOO_MANY_TOKENS;
  return EDGELORA_OK;
}

size_t arena_bytes_for(const edgelora_pool_config *c) {
  const size_t R = pad_rank(c->max_rank);
  // A: bfloat16 rows, or Q8_0 rows of 34 bytes per 32 values; B: bfloat16
  const size_t a_row = (c->flags & EDGELORA_FLAG_A_Q8) ? static_cast<size_t>(c->h_in) / 32 * 34
                                                       : static_cast<size_t>(c->h_in) * 2;
  const size_t per_slot = R * a_row + 2 * R * static_cast<size_t>(c->h_out);
  return per_slot * c->n_slots;
}

int plan_alloc(edgelora_plan *pl) {
  const size_t mt = pl->max_tokens;
  const int max_tiles = pl->max_tokens / kSegMin + 8;
  // ids_valid, perm, group_adapter, seg_adapter, tok_seg, perm_short: mt each;
  // group_start, seg_start, gs_short, scratch: mt + 1 each; tiles; counts; status
  // lg_adapter: mt; mt_count: n_mt + 1; mt_list: n_mt * 128
  const size_t n_mt = (mt + kTileM - 1) / kTileM;
  const size_t ints = 7 * mt + 4 * (mt + 1) + 4 * static_cast<size_t>(max_tiles) + (n_mt + 1) +
                      n_mt * kTileM + 8 + 4;
  CUDA_TRY(el_malloc(&pl->block, ints * 4));
  CUDA_TRY(cudaMemset(pl->block, 0, ints * 4));
  int32_t *q = static_cast<int32_t *>(pl->block);
  PlanView &v = pl->pv;
  v.ids_valid = q; q += mt;
  v.perm = q; q += mt;
  v.group_adapter = q; q += mt;
  v.seg_adapter = q; q += mt;
  v.tok_seg = q; q += mt;
  v.perm_short = q; q += mt;
  v.group_start = q; q += mt + 1;
  v.seg_start = q; q += mt + 1;
  v.gs_short = q; q += mt + 1;
  v.scratch = q; q += mt + 1;
  v.sgmv_tiles = q; q += 4 * static_cast<size_t>(max_tiles);
  v.lg_adapter = q; q += mt;
  v.mt_count = q; q += n_mt + 1;
  v.mt_list = q; q += n_mt * kTileM;
  v.counts = q; q += 8;
  v.status = reinterpret_cast<uint32_t *>(q);
  v.max_sgmv_tiles = max_tiles;
  return EDGELORA_OK;
}

}  // namespace

extern "C" {

const char *edgelora_strerror(int code) {
  switch (code) {
    case EDGELORA_OK: return "ok";
    case EDGELORA_ERR_INVALID_ARG: return "invalid argument";
    case EDGELORA_ERR_BAD_SLOT: return "slot index out of range";
    case EDGELORA_ERR_RANK_TOO_LARGE: return "adapter rank exceeds the pool's max_rank (or 64)";
    case EDGELORA_ERR_ARENA_TOO_SMALL: return "caller arena smaller than edgelora_pool_bytes_required";
    case EDGELORA_ERR_CUDA: return g_last_error[0] ? g_last_error : "CUDA error";
    case EDGELORA_ERR_BAD_ADAPTER_ID: return "an adapter id outside [-1, n_slots) was seen (token computed base-only)";
    case EDGELORA_ERR_SLOT_EMPTY: return "an adapter id named an empty slot (token computed base-only)";
    case EDGELORA_ERR_TIMEOUT: return "a bounded in-kernel wait gave up";
    case EDGELORA_ERR_BOUNDS:
      return "checked build: a kernel met an index outside its array, or a guard zone around a device buffer was overwritten";
    case EDGELORA_ERR_TOO_MANY_TOKENS: return "T exceeds max_tokens (or max_tokens exceeds 32768)";
    case EDGELORA_ERR_CACHE_FULL: return "every block of the adapter cache is held by a running request";
    default: return "unknown error";
  }
}

int edgelora_pool_bytes_required(const edgelora_pool_config *cfg, size_t *bytes_out) {
  int rc = check_cfg(cfg);
  if (rc != EDGELORA_OK) return rc;
  if (!bytes_out) return EDGELORA_ERR_INVALID_ARG;
  *bytes_out = arena_bytes_for(cfg);
  return EDGELORA_OK;
}

int edgelora_plan_create(int32_t max_tokens, int32_t n_slots, edgelora_plan_t **plan_out) {
  if (!plan_out || n_slots < 1 || n_slots > 65534) return EDGELORA_ERR_INVALID_ARG;
  if (max_tokens == 0) max_tokens = 8192;
  if (max_tokens < 0 || max_tokens > kMaxTokensLimit) return EDGELORA_ERR_TOO_MANY_TOKENS;
  edgelora_plan *pl = new (std::nothrow) edgelora_plan();
  if (!pl) return EDGELORA_ERR_INVALID_ARG;
  pl->max_tokens = max_tokens;
  pl->n_slots = n_slots;
  int rc = plan_alloc(pl);
  if (rc != EDGELORA_OK) {
    if (pl->block) el_free(pl->block);
    delete pl;
    return rc;
  }
  init_plan_kernel();
  *plan_out = pl;
  return EDGELORA_OK;
}

int edgelora_plan_destroy(edgelora_plan_t *plan) {
  if (!plan) return EDGELORA_ERR_INVALID_ARG;
  cudaDeviceSynchronize();
  if (plan->block) el_free(plan->block);
  delete plan;
  return EDGELORA_OK;
}

int edgelora_plan_build(edgelora_plan_t *plan, const int32_t *ids_dev, int32_t T, void *stream) {
  if (!plan || T < 0 || (T > 0 && !ids_dev)) return EDGELORA_ERR_INVALID_ARG;
  if (T > plan->max_tokens) return EDGELORA_ERR_TOO_MANY_TOKENS;
  plan->last_T = T;
  if (T == 0) return EDGELORA_OK;
  launch_plan(ids_dev, T, plan->n_slots, plan->pv, false, static_cast<cudaStream_t>(stream));
  CUDA_TRY(cudaGetLastError());
  return EDGELORA_OK;
}

int edgelora_plan_export(edgelora_plan_t *plan, void *stream, int32_t *ids_valid, int32_t *perm,
                         int32_t *group_start, int32_t *group_adapter, int32_t *seg_start,
                         int32_t *seg_adapter, int32_t counts_out[2]) {
  if (!plan) return EDGELORA_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  CUDA_TRY(cudaStreamSynchronize(s));
  const int T = plan->last_T;
  int32_t counts[8] = {0};
  if (T > 0) CUDA_TRY(cudaMemcpy(counts, plan->pv.counts, sizeof counts, cudaMemcpyDeviceToHost));
  const int G = counts[0], NS = counts[1];
  auto get = [&](int32_t *dst, const int32_t *src, int n) -> cudaError_t {
    if (!dst || n <= 0) return cudaSuccess;
    return cudaMemcpy(dst, src, static_cast<size_t>(n) * 4, cudaMemcpyDeviceToHost);
  };
  CUDA_TRY(get(ids_valid, plan->pv.ids_valid, T));
  CUDA_TRY(get(perm, plan->pv.perm, T));
  CUDA_TRY(get(group_adapter, plan->pv.group_adapter, G));
  CUDA_TRY(get(seg_adapter, plan->pv.seg_adapter, NS));
  if (T > 0) {
    CUDA_TRY(get(group_start, plan->pv.group_start, G + 1));
    CUDA_TRY(get(seg_start, plan->pv.seg_start, NS + 1));
  } else {
    if (group_start) group_start[0] = 0;
    if (seg_start) seg_start[0] = 0;
  }
  if (counts_out) {
    counts_out[0] = G;
    counts_out[1] = NS;
  }
  return EDGELORA_OK;
}

int edgelora_pool_create(const edgelora_pool_config *cfg, edgelora_pool_t **pool_out) {
  int rc = check_cfg(cfg);
  if (rc != EDGELORA_OK) return rc;
  if (!pool_out) return EDGELORA_ERR_INVALID_ARG;
  const size_t need = arena_bytes_for(cfg);
  if (cfg->arena_dev) {
    if (cfg->arena_bytes < need) return EDGELORA_ERR_ARENA_TOO_SMALL;
    if (reinterpret_cast<uintptr_t>(cfg->arena_dev) % 256) return EDGELORA_ERR_INVALID_ARG;
  }
  int dev = 0;
  CUDA_TRY(cudaGetDevice(&dev));
  cudaDeviceProp prop;
  CUDA_TRY(cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10) {
    snprintf(g_last_error, sizeof g_last_error, "device is sm_%d%d; this library is built for sm_100a only",
             prop.major, prop.minor);
    return EDGELORA_ERR_CUDA;
  }
  if (!get_encode_fn()) {
    snprintf(g_last_error, sizeof g_last_error, "cuTensorMapEncodeTiled not available from the driver");
    return EDGELORA_ERR_CUDA;
  }

  edgelora_pool *p = new (std::nothrow) edgelora_pool();
  if (!p) return EDGELORA_ERR_INVALID_ARG;
  p->cfg = *cfg;
  if (p->cfg.max_tokens == 0) p->cfg.max_tokens = 8192;
  p->R_pad = pad_rank(cfg->max_rank);
  p->device = dev;
  p->sms = prop.multiProcessorCount;
  p->a_q8 = (cfg->flags & EDGELORA_FLAG_A_Q8) != 0;
  // elements (2 bytes each) of a slot's A and B blocks; Q8_0 rows are 17 such elements per 32 values
  p->a_block = p->a_q8 ? static_cast<size_t>(p->R_pad) * (cfg->h_in / 32) * 17 : static_cast<size_t>(p->R_pad) * cfg->h_in;
  p->b_block = static_cast<size_t>(cfg->h_out) * p->R_pad;
  p->slots_host.assign(cfg->n_slots, SlotRow{0, 0.f, 0, 0});
  p->tmaps.reserve(kTmapCache);

#define POOL_TRY(expr)                         \
  do {                                         \
    cudaError_t _e = (expr);                   \
    if (_e != cudaSuccess) {                   \
      set_last_cuda_error(_e, #expr);          \
      edgelora_pool_destroy(p);                \
      return EDGELORA_ERR_CUDA;                \
    }                                          \
  } while (0)

  if (cfg->arena_dev) {
    p->arena = static_cast<uint8_t *>(cfg->arena_dev);
  } else {
    POOL_TRY(el_malloc(&p->arena, need));
    p->owns_arena = true;
  }
  p->A_pool = reinterpret_cast<uint16_t *>(p->arena);
  p->B_pool = p->A_pool + p->a_block * cfg->n_slots;
  POOL_TRY(el_malloc(&p->slots_dev, sizeof(SlotRow) * cfg->n_slots));
  POOL_TRY(cudaMemset(p->slots_dev, 0, sizeof(SlotRow) * cfg->n_slots));
  POOL_TRY(el_malloc(&p->status_dev, 16));
  POOL_TRY(cudaMemset(p->status_dev, 0, 16));
  // room for a block in its own layout or, for Q8_0 loads, A and B as 8-bit blocks (+ alignment)
  const size_t b_q8_bytes = static_cast<size_t>(cfg->h_out) * ((p->R_pad + 31) / 32) * 34;
  const size_t stage_bytes = p->a_block * 2 + 16 + std::max(p->b_block * 2, b_q8_bytes) + sizeof(SlotRow);
  for (auto &sb : p->staging) {
    POOL_TRY(cudaMallocHost(&sb.host, stage_bytes));
    POOL_TRY(cudaEventCreateWithFlags(&sb.done, cudaEventDisableTiming));
  }
  POOL_TRY(cudaStreamCreateWithFlags(&p->side, cudaStreamNonBlocking));
  POOL_TRY(cudaEventCreateWithFlags(&p->load_ev, cudaEventDisableTiming));
  POOL_TRY(cudaEventCreateWithFlags(&p->use_ev, cudaEventDisableTiming));
  // partial planes [0, kMaxZSplits) plus the final plane of the decode shrink
  POOL_TRY(el_malloc(&p->zws, sizeof(float) * (kMaxZSplits + 1) * static_cast<size_t>(p->cfg.max_tokens) * p->R_pad));
  POOL_TRY(el_malloc(&p->group_counters, sizeof(int32_t) * (kDecodeMaxT * 8 + 32)));
  POOL_TRY(cudaMemset(p->group_counters, 0, sizeof(int32_t) * (kDecodeMaxT * 8 + 32)));
  POOL_TRY(gemm_set_smem_limit(kSmemBudget));
  POOL_TRY(shrink_set_smem_limit());
  rc = edgelora_plan_create(p->cfg.max_tokens, cfg->n_slots, &p->plan);
  if (rc != EDGELORA_OK) {
    edgelora_pool_destroy(p);
    return rc;
  }
#undef POOL_TRY
  *pool_out = p;
  return EDGELORA_OK;
}

int edgelora_pool_destroy(edgelora_pool_t *p) {
  if (!p) return EDGELORA_ERR_INVALID_ARG;
  cudaDeviceSynchronize();
  if (p->plan) edgelora_plan_destroy(p->plan);
  if (p->owns_arena && p->arena) el_free(p->arena);
  if (p->slots_dev) el_free(p->slots_dev);
  if (p->status_dev) el_free(p->status_dev);
  for (auto &sb : p->staging) {
    if (sb.host) cudaFreeHost(sb.host);
    if (sb.done) cudaEventDestroy(sb.done);
  }
  if (p->side) cudaStreamDestroy(p->side);
  if (p->load_ev) cudaEventDestroy(p->load_ev);
  if (p->use_ev) cudaEventDestroy(p->use_ev);
  if (p->zws) el_free(p->zws);
  if (p->q8_dev) el_free(p->q8_dev);
  if (p->group_counters) el_free(p->group_counters);
  for (auto &r : p->prof) {
    cudaEventDestroy(r.start);
    cudaEventDestroy(r.stop);
  }
  if (p->hx) cudaFreeHost(p->hx);
  if (p->hy) cudaFreeHost(p->hy);
  if (p->hids) cudaFreeHost(p->hids);
  if (p->dx) el_free(p->dx);
  if (p->dy) el_free(p->dy);
  if (p->dids) el_free(p->dids);
  for (int b = 0; b < 2; ++b) {
    if (p->pdx[b]) el_free(p->pdx[b]);
    if (p->pdy[b]) el_free(p->pdy[b]);
    if (p->pdids[b]) el_free(p->pdids[b]);
    if (p->ev_in[b]) cudaEventDestroy(p->ev_in[b]);
    if (p->ev_done[b]) cudaEventDestroy(p->ev_done[b]);
    if (p->ev_out[b]) cudaEventDestroy(p->ev_out[b]);
  }
  if (p->h2d_stream) cudaStreamDestroy(p->h2d_stream);
  if (p->d2h_stream) cudaStreamDestroy(p->d2h_stream);
  cudaGetLastError();
  delete p;
  return EDGELORA_OK;
}

// where the slot-table row sits in a staging buffer: behind the largest payload
static size_t slot_row_offset(const edgelora_pool *p) {
  const size_t b_q8_bytes = static_cast<size_t>(p->cfg.h_out) * ((p->R_pad + 31) / 32) * 34;
  return p->a_block * 2 + 16 + std::max(p->b_block * 2, b_q8_bytes);
}

static int stage_and_copy(edgelora_pool *p, int32_t slot, int32_t rank, float scale,
                          const uint16_t *A_host, const uint16_t *B_host) {
  if (p->a_q8 && rank > 0) return EDGELORA_ERR_INVALID_ARG;  // this pool takes Q8_0 adapters only
  StagingBuf &sb = p->staging[p->next_staging];
  p->next_staging = (p->next_staging + 1) % kStagingBuffers;
  if (sb.in_flight) {
    CUDA_TRY(cudaEventSynchronize(sb.done));
    sb.in_flight = false;
  }
  const int h_in = p->cfg.h_in, h_out = p->cfg.h_out, R = p->R_pad;
  uint16_t *sa = reinterpret_cast<uint16_t *>(sb.host);
  uint16_t *sbp = sa + p->a_block;
  SlotRow *srow = reinterpret_cast<SlotRow *>(sb.host + slot_row_offset(p));
  SlotRow &mirror = p->slots_host[slot];
  mirror.rank = rank;
  mirror.scale = scale;
  mirror.generation += 1;
  *srow = mirror;
  // order against the last layer call that may still read this pool
  if (p->use_recorded) CUDA_TRY(cudaStreamWaitEvent(p->side, p->use_ev, 0));
  if (rank > 0) {
    // A: rows [rank, R) are zero; B: columns [rank, R) are zero
    memcpy(sa, A_host, static_cast<size_t>(rank) * h_in * 2);
    memset(sa + static_cast<size_t>(rank) * h_in, 0, static_cast<size_t>(R - rank) * h_in * 2);
    if (rank == R) {
      memcpy(sbp, B_host, static_cast<size_t>(h_out) * R * 2);
    } else {
      for (int j = 0; j < h_out; ++j) {
        memcpy(sbp + static_cast<size_t>(j) * R, B_host + static_cast<size_t>(j) * rank, rank * 2);
        memset(sbp + static_cast<size_t>(j) * R + rank, 0, (R - rank) * 2);
      }
    }
    CUDA_TRY(cudaMemcpyAsync(p->A_pool + p->a_block * slot, sa, p->a_block * 2, cudaMemcpyHostToDevice, p->side));
    CUDA_TRY(cudaMemcpyAsync(p->B_pool + p->b_block * slot, sbp, p->b_block * 2, cudaMemcpyHostToDevice, p->side));
  }
  CUDA_TRY(cudaMemcpyAsync(p->slots_dev + slot, srow, sizeof(SlotRow), cudaMemcpyHostToDevice, p->side));
  CUDA_TRY(cudaEventRecord(sb.done, p->side));
  sb.in_flight = true;
  CUDA_TRY(cudaEventRecord(p->load_ev, p->side));
  p->load_seq += 1;
  return EDGELORA_OK;
}

int edgelora_pool_load_slot(edgelora_pool_t *p, int32_t slot, int32_t rank, float scale,
                            const uint16_t *A_host, const uint16_t *B_host) {
  if (!p || !A_host || !B_host) return EDGELORA_ERR_INVALID_ARG;
  if (slot < 0 || slot >= p->cfg.n_slots) return EDGELORA_ERR_BAD_SLOT;
  if (rank < 1) return EDGELORA_ERR_INVALID_ARG;
  if (rank > p->cfg.max_rank) return EDGELORA_ERR_RANK_TOO_LARGE;
  return stage_and_copy(p, slot, rank, scale, A_host, B_host);
}

int edgelora_pool_load_slot_pinned(edgelora_pool_t *p, int32_t slot, int32_t rank, float scale,
                                   const uint16_t *A_pinned, const uint16_t *B_pinned) {
  if (!p || !A_pinned || !B_pinned) return EDGELORA_ERR_INVALID_ARG;
  if (slot < 0 || slot >= p->cfg.n_slots) return EDGELORA_ERR_BAD_SLOT;
  if (rank != p->R_pad || p->a_q8) return EDGELORA_ERR_INVALID_ARG;  // already in the block's layout: nothing to pad
  cudaPointerAttributes at{};
  if (cudaPointerGetAttributes(&at, A_pinned) != cudaSuccess || at.type != cudaMemoryTypeHost ||
      cudaPointerGetAttributes(&at, B_pinned) != cudaSuccess || at.type != cudaMemoryTypeHost) {
    cudaGetLastError();
    return EDGELORA_ERR_INVALID_ARG;  // not page-locked: use edgelora_pool_load_slot
  }
  // the slot row still goes through a staging buffer (16 bytes the library owns)
  StagingBuf &sb = p->staging[p->next_staging];
  p->next_staging = (p->next_staging + 1) % kStagingBuffers;
  if (sb.in_flight) {
    CUDA_TRY(cudaEventSynchronize(sb.done));
    sb.in_flight = false;
  }
  SlotRow *srow = reinterpret_cast<SlotRow *>(sb.host + slot_row_offset(p));
  SlotRow &mirror = p->slots_host[slot];
  mirror.rank = rank;
  mirror.scale = scale;
  mirror.generation += 1;
  *srow = mirror;
  if (p->use_recorded) CUDA_TRY(cudaStreamWaitEvent(p->side, p->use_ev, 0));
  CUDA_TRY(cudaMemcpyAsync(p->A_pool + p->a_block * slot, A_pinned, p->a_block * 2, cudaMemcpyHostToDevice, p->side));
  CUDA_TRY(cudaMemcpyAsync(p->B_pool + p->b_block * slot, B_pinned, p->b_block * 2, cudaMemcpyHostToDevice, p->side));
  CUDA_TRY(cudaMemcpyAsync(p->slots_dev + slot, srow, sizeof(SlotRow), cudaMemcpyHostToDevice, p->side));
  CUDA_TRY(cudaEventRecord(sb.done, p->side));
  sb.in_flight = true;
  CUDA_TRY(cudaEventRecord(p->load_ev, p->side));
  p->load_seq += 1;
  return EDGELORA_OK;
}

int edgelora_pool_load_slot_q8(edgelora_pool_t *p, int32_t slot, int32_t rank, float scale, const void *A_q8,
                               const void *B_q8) {
  if (!p || !A_q8 || !B_q8) return EDGELORA_ERR_INVALID_ARG;
  if (slot < 0 || slot >= p->cfg.n_slots) return EDGELORA_ERR_BAD_SLOT;
  if (rank < 1 || (p->cfg.h_in % 32)) return EDGELORA_ERR_INVALID_ARG;
  if (rank > p->cfg.max_rank) return EDGELORA_ERR_RANK_TOO_LARGE;
  const int h_in = p->cfg.h_in, h_out = p->cfg.h_out, R = p->R_pad;
  const size_t a_bytes = static_cast<size_t>(rank) * (h_in / 32) * 34;
  const size_t b_bytes = static_cast<size_t>(h_out) * ((rank + 31) / 32) * 34;
  const size_t b_off = (a_bytes + 15) & ~static_cast<size_t>(15);
  const size_t scratch = static_cast<size_t>(p->cfg.max_rank) * (h_in / 32) * 34 + 16 +
                         static_cast<size_t>(h_out) * ((p->cfg.max_rank + 31) / 32) * 34;
  if (!p->q8_dev) CUDA_TRY(el_malloc(&p->q8_dev, scratch));
  StagingBuf &sb = p->staging[p->next_staging];
  p->next_staging = (p->next_staging + 1) % kStagingBuffers;
  if (sb.in_flight) {
    CUDA_TRY(cudaEventSynchronize(sb.done));
    sb.in_flight = false;
  }
  if (p->a_q8) {
    // the pool keeps A in Q8_0: rows [rank, R_pad) are zero blocks; only B is converted on the device
    const size_t a_pad = p->a_block * 2;
    {  // the pool's layout: the signed bytes of all rows, then the block scales of all rows
      const int nb = h_in / 32;
      const uint8_t *src = static_cast<const uint8_t *>(A_q8);
      uint8_t *qplane = sb.host, *dplane = sb.host + static_cast<size_t>(R) * h_in;
      memset(sb.host, 0, a_pad);
      for (int r = 0; r < rank; ++r)
        for (int b = 0; b < nb; ++b) {
          const uint8_t *blk = src + (static_cast<size_t>(r) * nb + b) * 34;
          memcpy(dplane + (static_cast<size_t>(r) * nb + b) * 2, blk, 2);
          memcpy(qplane + static_cast<size_t>(r) * h_in + b * 32, blk + 2, 32);
        }
    }
    const size_t b_off2 = (a_pad + 15) & ~static_cast<size_t>(15);
    memcpy(sb.host + b_off2, B_q8, b_bytes);
    SlotRow *srow2 = reinterpret_cast<SlotRow *>(sb.host + slot_row_offset(p));
    SlotRow &m2 = p->slots_host[slot];
    m2.rank = rank;
    m2.scale = scale;
    m2.generation += 1;
    *srow2 = m2;
    if (p->use_recorded) CUDA_TRY(cudaStreamWaitEvent(p->side, p->use_ev, 0));
    CUDA_TRY(cudaMemcpyAsync(p->A_pool + p->a_block * slot, sb.host, a_pad, cudaMemcpyHostToDevice, p->side));
    CUDA_TRY(cudaMemcpyAsync(p->q8_dev, sb.host + b_off2, b_bytes, cudaMemcpyHostToDevice, p->side));
    CUDA_TRY(launch_q8_to_block(nullptr, p->q8_dev, nullptr, p->B_pool + p->b_block * slot, rank, R, h_in, h_out,
                                p->sms, p->side));
    CUDA_TRY(cudaMemcpyAsync(p->slots_dev + slot, srow2, sizeof(SlotRow), cudaMemcpyHostToDevice, p->side));
    CUDA_TRY(cudaEventRecord(sb.done, p->side));
    sb.in_flight = true;
    CUDA_TRY(cudaEventRecord(p->load_ev, p->side));
    p->load_seq += 1;
    return EDGELORA_OK;
  }
  // the 8-bit form is smaller than the block the staging buffer was sized for
  memcpy(sb.host, A_q8, a_bytes);
  memcpy(sb.host + b_off, B_q8, b_bytes);
  SlotRow *srow = reinterpret_cast<SlotRow *>(sb.host + slot_row_offset(p));
  SlotRow &mirror = p->slots_host[slot];
  mirror.rank = rank;
  mirror.scale = scale;
  mirror.generation += 1;
  *srow = mirror;
  if (p->use_recorded) CUDA_TRY(cudaStreamWaitEvent(p->side, p->use_ev, 0));
  // (the scratch is reused by every load: the copies and conversions of one pool run in order on
  // its side stream)
  CUDA_TRY(cudaMemcpyAsync(p->q8_dev, sb.host, b_off + b_bytes, cudaMemcpyHostToDevice, p->side));
  CUDA_TRY(launch_q8_to_block(p->q8_dev, p->q8_dev + b_off, p->A_pool + p->a_block * slot,
                              p->B_pool + p->b_block * slot, rank, R, h_in, h_out, p->sms, p->side));
  CUDA_TRY(cudaMemcpyAsync(p->slots_dev + slot, srow, sizeof(SlotRow), cudaMemcpyHostToDevice, p->side));
  CUDA_TRY(cudaEventRecord(sb.done, p->side));
  sb.in_flight = true;
  CUDA_TRY(cudaEventRecord(p->load_ev, p->side));
  p->load_seq += 1;
  return EDGELORA_OK;
}

int edgelora_pool_evict_slot(edgelora_pool_t *p, int32_t slot) {
  if (!p) return EDGELORA_ERR_INVALID_ARG;
  if (slot < 0 || slot >= p->cfg.n_slots) return EDGELORA_ERR_BAD_SLOT;
  return stage_and_copy(p, slot, 0, 0.f, nullptr, nullptr);
}

int edgelora_pool_wait_loads(edgelora_pool_t *p) {
  if (!p) return EDGELORA_ERR_INVALID_ARG;
  CUDA_TRY(cudaStreamSynchronize(p->side));
  for (auto &sb : p->staging) sb.in_flight = false;
  return EDGELORA_OK;
}

int edgelora_pool_plan(edgelora_pool_t *p, edgelora_plan_t **plan_out) {
  if (!p || !plan_out) return EDGELORA_ERR_INVALID_ARG;
  *plan_out = p->plan;
  return EDGELORA_OK;
}

int edgelora_pool_set_option(edgelora_pool_t *p, int32_t option, int32_t value) {
  if (!p) return EDGELORA_ERR_INVALID_ARG;
  switch (option) {
    case EDGELORA_OPT_REGIME:
      if (value < 0 || value > 2) return EDGELORA_ERR_INVALID_ARG;
      p->opt_regime = value;
      return EDGELORA_OK;
    case EDGELORA_OPT_PROFILE:
      p->opt_profile = value ? 1 : 0;
      if (p->opt_profile && p->prof.empty()) {
        p->prof.resize(kProfEvents);
        for (auto &r : p->prof) {
          CUDA_TRY(cudaEventCreate(&r.start));
          CUDA_TRY(cudaEventCreate(&r.stop));
        }
      }
      return EDGELORA_OK;
    case EDGELORA_OPT_PDL:
      if (value < 0 || value > 2) return EDGELORA_ERR_INVALID_ARG;
      p->opt_pdl = value;
      return EDGELORA_OK;
    case EDGELORA_OPT_DECODE_SPLITS:
      if (value < 0 || value > kMaxDecodeSplits) return EDGELORA_ERR_INVALID_ARG;
      p->opt_decode_splits = value;
      return EDGELORA_OK;
    case EDGELORA_OPT_WAIT_CYCLES:
      if (value < 0) return EDGELORA_ERR_INVALID_ARG;
      p->wait_cycles = value == 0 ? ptx::kWaitLimitCycles : static_cast<long long>(value) * 1024;
      return EDGELORA_OK;
    case EDGELORA_OPT_SHRINK_ITEMS:
      if (value < 0) return EDGELORA_ERR_INVALID_ARG;
      p->opt_shrink_items = value;
      return EDGELORA_OK;
    case EDGELORA_OPT_SHRINK_DEPTH:
      if (value != 0 && value != 2 && value != 4) return EDGELORA_ERR_INVALID_ARG;
      p->opt_shrink_depth = value;
      return EDGELORA_OK;
    case EDGELORA_OPT_FUSED_DECODE:
      if (value != 0 && value != 1) return EDGELORA_ERR_INVALID_ARG;
      p->opt_fused_decode = value;
      return EDGELORA_OK;
    case EDGELORA_OPT_GATHER_SPLITS:
      if (value < 0 || value > 8) return EDGELORA_ERR_INVALID_ARG;
      p->opt_gather_splits = value;
      return EDGELORA_OK;
    case EDGELORA_OPT_GATHER_MIN_T:
      if (value < 0 || value > kDecodeMaxT) return EDGELORA_ERR_INVALID_ARG;
      p->opt_gather_min_t = value;
      return EDGELORA_OK;
    default:
      return EDGELORA_ERR_INVALID_ARG;
  }
}

int edgelora_pool_last_launch(edgelora_pool_t *p, int64_t info_out[8]) {
  if (!p || !info_out) return EDGELORA_ERR_INVALID_ARG;
  memcpy(info_out, p->last_info, sizeof p->last_info);
  info_out[6] = p->total_launches;
  return EDGELORA_OK;
}

int edgelora_pool_kernel_times(edgelora_pool_t *p, double ms_out[5], int64_t launches_out[5],
                               int32_t reset) {
  if (!p) return EDGELORA_ERR_INVALID_ARG;
  for (size_t i = 0; i < p->prof_used; ++i) {
    ProfRec &r = p->prof[i];
    CUDA_TRY(cudaEventSynchronize(r.stop));
    float ms = 0.f;
    CUDA_TRY(cudaEventElapsedTime(&ms, r.start, r.stop));
    p->prof_ms[r.kernel] += ms;
    p->prof_n[r.kernel] += 1;
  }
  p->prof_used = 0;
  for (int k = 0; k < 5; ++k) {
    if (ms_out) ms_out[k] = p->prof_ms[k];
    if (launches_out) launches_out[k] = p->prof_n[k];
    if (reset) {
      p->prof_ms[k] = 0;
      p->prof_n[k] = 0;
    }
  }
  return EDGELORA_OK;
}

int edgelora_pool_sync_status(edgelora_pool_t *p, uint32_t *bits_out) {
  if (!p) return EDGELORA_ERR_INVALID_ARG;
  CUDA_TRY(cudaDeviceSynchronize());
  uint32_t a = 0, b = 0;
  CUDA_TRY(cudaMemcpy(&a, p->status_dev, 4, cudaMemcpyDeviceToHost));
  CUDA_TRY(cudaMemcpy(&b, p->plan->pv.status, 4, cudaMemcpyDeviceToHost));
  CUDA_TRY(cudaMemset(p->status_dev, 0, 4));
  CUDA_TRY(cudaMemset(p->plan->pv.status, 0, 8));
  const uint32_t bits = a | b;
  if (bits_out) *bits_out = bits;
  // a wait that ran out can leave arrival counters between their values: nothing is in flight now
  if (bits & EDGELORA_STATUS_TIMEOUT)
    CUDA_TRY(cudaMemset(p->group_counters, 0, sizeof(int32_t) * (kDecodeMaxT * 8 + 32)));
  if (bits & EDGELORA_STATUS_BOUNDS) {  // checked build: which test failed first
    uint32_t site = 0;
    CUDA_TRY(cudaMemcpy(&site, p->status_dev + 1, 4, cudaMemcpyDeviceToHost));
    CUDA_TRY(cudaMemset(p->status_dev + 1, 0, 4));
    snprintf(g_last_error, sizeof g_last_error, "a kernel's index test failed (test %u)", site);
    return EDGELORA_ERR_BOUNDS;
  }
  if (bits & EDGELORA_STATUS_TIMEOUT) return EDGELORA_ERR_TIMEOUT;
  if (edgelora_check_guards() != EDGELORA_OK) return EDGELORA_ERR_BOUNDS;  // always intact in the normal build
  if (bits & EDGELORA_STATUS_BAD_ADAPTER_ID) return EDGELORA_ERR_BAD_ADAPTER_ID;
  if (bits & EDGELORA_STATUS_SLOT_EMPTY) return EDGELORA_ERR_SLOT_EMPTY;
  return EDGELORA_OK;
}

int edgelora_plan_sync_status(edgelora_plan_t *plan, void *stream, uint32_t *bits_out) {
  if (!plan) return EDGELORA_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  CUDA_TRY(cudaStreamSynchronize(s));
  uint32_t bits = 0;
  CUDA_TRY(cudaMemcpy(&bits, plan->pv.status, 4, cudaMemcpyDeviceToHost));
  CUDA_TRY(cudaMemset(plan->pv.status, 0, 4));
  if (bits_out) *bits_out = bits;
  if (bits & EDGELORA_STATUS_BOUNDS) return EDGELORA_ERR_BOUNDS;
  if (bits & EDGELORA_STATUS_TIMEOUT) return EDGELORA_ERR_TIMEOUT;
  if (bits & EDGELORA_STATUS_BAD_ADAPTER_ID) return EDGELORA_ERR_BAD_ADAPTER_ID;
  if (bits & EDGELORA_STATUS_SLOT_EMPTY) return EDGELORA_ERR_SLOT_EMPTY;
  return EDGELORA_OK;
}

int edgelora_pool_selftest_wait(edgelora_pool_t *p, void *stream) {
  if (!p) return EDGELORA_ERR_INVALID_ARG;
  // only with a lowered limit: at the default the kernel would spin for seconds
  if (p->wait_cycles > (1LL << 24)) return EDGELORA_ERR_INVALID_ARG;
  CUDA_TRY(launch_wait_selftest(p->status_dev, p->wait_cycles, static_cast<cudaStream_t>(stream)));
  return EDGELORA_OK;
}

// The layer.  Decode regime (T <= 256): routing + shrink in one kernel, then the base product with
// the expand and the split-K reduction fused in.  Prefill regime: plan, gather shrink for short
// runs, segment shrink for long runs, base product with the expand fused in.
}  // extern "C"

namespace edgelora {
int lora_linear_impl(edgelora_pool *p, edgelora_plan *plan, const int32_t *ids_dev, const void *W_dev,
                     const void *x_dev, int32_t T, void *y_dev, cudaStream_t stream, bool skip_shrink,
                     const NextShrink *next, bool independent) {
  if (!p || !plan || T < 0) return EDGELORA_ERR_INVALID_ARG;
  if (T == 0) return EDGELORA_OK;
  if (!W_dev || !x_dev || !y_dev) return EDGELORA_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(W_dev) | reinterpret_cast<uintptr_t>(x_dev) |
       reinterpret_cast<uintptr_t>(y_dev)) & 15)
    return EDGELORA_ERR_INVALID_ARG;
  if (T > p->cfg.max_tokens || T > plan->max_tokens) return EDGELORA_ERR_TOO_MANY_TOKENS;
  if (plan->n_slots != p->cfg.n_slots) return EDGELORA_ERR_INVALID_ARG;
  if (!ids_dev && plan->last_T != T) return EDGELORA_ERR_INVALID_ARG;
  const int h_in = p->cfg.h_in, h_out = p->cfg.h_out, R = p->R_pad;
  const bool capturing = stream_capturing(stream);
  const bool pdl = p->opt_pdl >= 1 && !p->opt_profile;        // between the kernels of this call
  // first kernel vs earlier stream work: when the pool's option says so, or when the caller (a set
  // of sites) knows that this call does not consume what the call before it produces
  const bool pdl_first = (p->opt_pdl >= 2 || (independent && p->opt_pdl >= 1)) && !p->opt_profile;
  const uint16_t *x = static_cast<const uint16_t *>(x_dev);
  int launches = 0;

  // Order this call behind every load issued so far, once per stream and load (a wait node
  // between two calls of one stream would also keep them from overlapping).  A captured call
  // records no such wait: see the header for what a graph's owner has to do instead.
  if (p->load_seq != 0 && !capturing) {
    auto it = std::find_if(p->load_waited.begin(), p->load_waited.end(),
                           [&](const std::pair<cudaStream_t, uint64_t> &e) { return e.first == stream; });
    if (it == p->load_waited.end()) {
      if (p->load_waited.size() >= 64) p->load_waited.clear();  // streams come and go: start over
      p->load_waited.emplace_back(stream, 0);
      it = p->load_waited.end() - 1;
    }
    if (it->second != p->load_seq) {
      CUDA_TRY(cudaStreamWaitEvent(stream, p->load_ev, 0));
      it->second = p->load_seq;
    }
  }

  int regime = (T <= kDecodeMaxT) ? 1 : 2;
  if (p->opt_regime == 2) regime = 2;
  if (p->opt_regime == 1 && T > kDecodeMaxT) return EDGELORA_ERR_INVALID_ARG;
  const int kb_total = (h_in + kBlockK - 1) / kBlockK;

  GemmParams g{};
  g.T = T;
  g.h_in = h_in;
  g.h_out = h_out;
  g.kb_total = kb_total;
  g.R_pad = R;
  g.max_tokens = p->cfg.max_tokens;
  g.ids_valid = plan->pv.ids_valid;
  g.slots = p->slots_dev;
  g.B_pool = p->B_pool;
  g.zws = p->zws;
  g.zws_out = p->zws;
  g.y = static_cast<uint16_t *>(y_dev);
  g.sgmv_tiles = plan->pv.sgmv_tiles;
  g.counts = plan->pv.counts;
  g.ids = ids_dev ? ids_dev : plan->pv.ids_valid;
  g.n_slots = p->cfg.n_slots;
  g.mt_count = plan->pv.mt_count;
  g.mt_list = plan->pv.mt_list;
  g.status = p->status_dev;
  g.wait_cycles = p->wait_cycles;

  auto smem_for = [](int stages, int BN, int extra = 0) {
    // alignment slack + operand ring + barriers (512) + decode extras (3456, rounded up)
    // (+ the prefill epilogue's staging area, 1024-aligned because every part before it is)
    return static_cast<size_t>(1024 + stages * (kTileM * kBlockK * 2 + BN * kBlockK * 2) + 4096 + extra);
  };
  auto stages_for = [&](int BN, int k_blocks_per_cta, size_t budget) {
    int s = static_cast<int>((budget - 5120) / (kTileM * kBlockK * 2 + BN * kBlockK * 2));
    return std::max(1, std::min({s, kMaxStages, std::max(2, k_blocks_per_cta)}));
  };
  auto pow2_cols = [](int cols) {
    int c = 32;
    while (c < cols) c <<= 1;
    return c;
  };

  // The shrink of a pool as a job of the tile kernel: segment tiles for the long runs of a large
  // batch (tile list from the plan) and gather tiles for every other token.  `decode`: no segment
  // tiles, the K split count is chosen on the device from the number of adapters the batch touches,
  // and whoever completes a tile last adds its splits into the final z plane.
  const bool sgmv = T > kDecodeMaxT;
  struct ShrinkJob {
    GemmParams s;
    CUtensorMap mx, ma, mg;
    int grid = 1;
    size_t smem = 0;
  };
  // Inside a set of sites the shrink tiles ride on another site's base-product launch, where few
  // large items fit into the slack of its last wave better than many small ones; on its own the
  // shrink is split until every SM has an item.
  const bool in_set = skip_shrink || next != nullptr;
  auto zsplits_of = [&](const edgelora_pool *q) {
    if (!sgmv) return 1;
    const int kbt = (q->cfg.h_in + kBlockK - 1) / kBlockK;
    const int tiles_est = std::max(1, T / kTileM);
    // (inside a set: items of about 32 K blocks, so that a wide input does not make them long)
    int z = std::max(1, std::min({in_set ? std::max(2, std::min(8, kbt / 32)) : 8, q->sms / tiles_est, kbt / 4}));
    const int kb_per = (kbt + z - 1) / z;
    return (kbt + kb_per - 1) / kb_per;
  };
  auto shrink_job = [&](edgelora_pool *q, const uint16_t *xq, bool decode, int ring_rows, ShrinkJob *out) -> int {
    const int kbt = (q->cfg.h_in + kBlockK - 1) / kBlockK;
    const int Rq = q->R_pad;
    GemmParams s{};
    s.mode = kModeSgmv;
    s.T = T;
    s.h_in = q->cfg.h_in;
    s.h_out = q->cfg.h_out;
    s.kb_total = kbt;
    s.R_pad = Rq;
    s.BN = Rq;
    s.max_tokens = q->cfg.max_tokens;
    s.zsplits = decode ? 1 : zsplits_of(q);
    s.splits = decode ? q->opt_gather_splits : s.zsplits;  // 0: the kernel picks the gather tiles' split count
    while (s.splits > 1 && (s.splits - 1) * ((kbt + s.splits - 1) / s.splits) >= kbt) --s.splits;  // no empty split
    s.kb_per = (kbt + s.zsplits - 1) / s.zsplits;
    s.gather = 1;
    s.finalize = decode ? 1 : 0;
    // token rows of one gather pass: what the ring's C region holds (given when the job rides on
    // another job's ring), 64 on its own ring (deep pipeline; a tile rarely has more tokens)
    s.gN = ring_rows > 0 ? std::min(256, ring_rows / 16 * 16) : std::min(64, round_up(T, 16));
    s.ring_rows = ring_rows > 0 ? ring_rows : std::max(Rq, s.gN);
    s.acc_cols = s.ring_rows;
    s.stages = stages_for(s.ring_rows, std::max(s.kb_per, 8), kSmemBudget);
    s.n_acc = 2;
    s.tmem_cols = pow2_cols(2 * s.acc_cols);
    // upper bound of its tiles (the true count is on the device): segment tiles x splits + one gather
    // tile per 128 / R_pad adapters x splits
    const int max_gt = (std::min(T, q->cfg.n_slots) * Rq + kTileM - 1) / kTileM;
    s.n_mtiles = (plan->pv.max_sgmv_tiles + max_gt) * std::max(s.zsplits, 1);
    s.ids_valid = plan->pv.ids_valid;
    s.ids = plan->pv.ids_valid;
    s.n_slots = q->cfg.n_slots;
    s.slots = q->slots_dev;
    s.B_pool = q->B_pool;
    s.zws = q->zws;
    s.zws_out = q->zws;
    s.sgmv_tiles = plan->pv.sgmv_tiles;
    s.counts = plan->pv.counts;
    s.mt_count = plan->pv.mt_count;
    s.mt_list = plan->pv.mt_list;
    s.perm_short = plan->pv.perm_short;
    s.gs_short = plan->pv.gs_short;
    s.group_adapter = plan->pv.group_adapter;
    s.tile_counters = q->group_counters;
    s.status = q->status_dev;
    s.wait_cycles = q->wait_cycles;
    out->s = s;
    out->grid = q->sms;
    out->smem = smem_for(s.stages, s.ring_rows);
    int rc2 = get_tmap(q, &out->mx, xq, q->cfg.h_in, T, 0, kTileM);
    if (rc2) return rc2;
    rc2 = get_tmap(q, &out->mg, xq, q->cfg.h_in, T, 0, 1);
    if (rc2) return rc2;
    // the A blocks as one 2D matrix [n_slots * R_pad][h_in]: slot a is rows [a R_pad, (a + 1) R_pad)
    return get_tmap(q, &out->ma, q->A_pool, q->cfg.h_in, static_cast<uint64_t>(Rq) * q->cfg.n_slots, 0, Rq);
  };
  // decode batches above this size take the plan kernel + tensor-core gather tiles; smaller ones
  // the single shrink kernel that derives the routing itself (a launch less)
  const int kGatherMinT = p->opt_gather_min_t;
  // a pool that keeps A in Q8_0 is served by the decode shrink kernel only (it decodes the blocks as
  // it streams them); the tensor-core shrink tiles need bfloat16 operand tiles
  if (p->a_q8 && (regime != 1 || T > kGatherMinT)) return EDGELORA_ERR_INVALID_ARG;

  if (regime == 1) {
    // ---------------------------------------------------------------- decode
    const int32_t *ids_in = ids_dev ? ids_dev : plan->pv.ids_valid;
    plan->last_T = T;
    auto launch_shrink = [&]() -> int {
      if (T > kGatherMinT) {
        if (ids_dev) {
          ProfScope ps(p, 0, stream);
          launch_plan(ids_dev, T, plan->n_slots, plan->pv, pdl_first, stream);
          CUDA_TRY(cudaGetLastError());
          ++launches;
        }
        ShrinkJob sj;
        int rc = shrink_job(p, x, true, 0, &sj);
        if (rc) return rc;
        ProfScope ps(p, 2, stream);
        CUDA_TRY(launch_gemm(sj.mx, sj.ma, sj.mg, sj.s, sj.grid, sj.smem, ids_dev ? pdl : pdl_first, stream));
        ++launches;
      } else
      {
        ProfScope ps(p, 1, stream);
        // When calls overlap (EDGELORA_OPT_PDL = 2) a small batch's shrink runs under the previous
        // call's base product, so its length does not matter but its tail does: one K chunk per
        // item (no pass that adds chunks) and few CTAs (they take SM resources from the base product).
        const bool overlapped = pdl_first && T <= 64;
        // ring depth 2 lets two CTAs share an SM: twice the warps in flight with half the ring each,
        // which suits a kernel bound by the per-warp chain of copy issue, wait and FMAs (measured on
        // the 200-adapter down_proj: 45.8 us against 49.8 us with depth 4)
        const int shrink_depth = T <= 64 ? 2 : (p->opt_shrink_depth == 4 ? 4 : 2);
        const int cta_cap = shrink_depth == 2 && T > 64 ? 2 * p->sms : p->sms;
        // Large batches: few, long items (about 0.6 per warp) beat many short ones, whose ring ramp-up and
        // chunk sums add up: 92 us per step with 2 K chunks on the 1000-adapter down_proj, 96 with 3-4,
        // 100 with 12, 104 with 1.  Small batches: four items per warp.
        const int auto_target = T > 64 ? 5 * cta_cap : 4 * 8 * cta_cap;
        const int target = p->opt_shrink_items > 0 ? p->opt_shrink_items : (overlapped ? 1 : auto_target);
        // at most T token blocks x (R / 8) row groups x K chunks warp items, eight warps per CTA
        const int n_ksteps = (h_in + kShrinkStepElems - 1) / kShrinkStepElems;
        const int max_chunks = target == 1 ? 1 : std::max(1, std::min(kMaxZSplits, n_ksteps / 4));
        const int max_items = std::min(T, p->cfg.n_slots) * (R / 8) * max_chunks;
        const int grid = std::max(1, std::min(cta_cap - 1, (max_items + 7) / 8)) + 1;  // + the publishing CTA
        CUtensorMap ma, mx, md;
        // A rows: bfloat16, or for a pool that keeps A in Q8_0 two planes per slot: the signed bytes
        // [R_pad][h_in] (taken as 16-bit elements: 128 per K step) and the half-precision block scales
        // [R_pad][h_in / 32] (8 per K step); both planes have the slot's byte stride
        int rc;
        if (p->a_q8) {
          const uint64_t slot_bytes = p->a_block * 2;
          rc = get_tmap(p, &ma, p->A_pool, h_in / 2, R, p->cfg.n_slots, 8, kShrinkStepElems / 2, h_in, slot_bytes);
          if (rc) return rc;
          rc = get_tmap(p, &md, reinterpret_cast<const uint8_t *>(p->A_pool) + static_cast<size_t>(R) * h_in, h_in / 32, R,
                        p->cfg.n_slots, 8, kShrinkStepElems / 32, h_in / 16, slot_bytes);
        } else {
          rc = get_tmap(p, &ma, p->A_pool, h_in, R, p->cfg.n_slots, 8, kShrinkStepElems);
          md = ma;
        }
        if (rc) return rc;
        rc = get_tmap(p, &mx, x, h_in, T, 0, 1, kShrinkStepElems);
        if (rc) return rc;
        CUDA_TRY(launch_decode_shrink(ma, md, mx, ids_in, p->slots_dev, plan->pv, p->zws, p->group_counters,
                                      T, h_in, R, p->cfg.n_slots, p->cfg.max_tokens, target, grid,
                                      p->status_dev, pdl_first, p->a_q8, shrink_depth, stream));
        ++launches;
      }
      return 0;
    };
    int N = 32;  // tokens on the UMMA N axis: a power of two so that the cluster's owners get
    while (N < T) N <<= 1;  // equal power-of-two column blocks
    const int row_tiles = (h_out + kTileM - 1) / kTileM;
    const int stage_bytes = kTileM * kBlockK * 2 + N * kBlockK * 2;
    const int ctas_per_sm = (stage_bytes * 4 + 5120 <= static_cast<int>(kSmemBudget / 2)) ? 2 : 1;
    int want = p->opt_decode_splits > 0 ? p->opt_decode_splits
                                        : std::max(1, (p->sms * ctas_per_sm) / row_tiles);
    want = std::min({want, kMaxDecodeSplits, std::max(1, kb_total / 2)});
    int splits = 1;
    while (splits * 2 <= want) splits <<= 1;
    int kb_per = (kb_total + splits - 1) / splits;
    while (splits > 1 && kb_per * (splits - 1) >= kb_total) {  // every split needs a K block
      splits >>= 1;
      kb_per = (kb_total + splits - 1) / splits;
    }
    g.mode = kModeDecode;
    g.BN = N;
    g.splits = splits;
    g.kb_per = kb_per;
    g.n_mtiles = row_tiles;
    g.n_ntiles = 1;
    g.zsplits = 1;   // the decode shrink leaves the summed z in the plane after the partial ones
    g.zws = p->zws + static_cast<size_t>(kMaxZSplits) * p->cfg.max_tokens * R;
    const size_t budget = ctas_per_sm == 2 ? kSmemBudget / 2 : kSmemBudget;
    g.stages = stages_for(N, kb_per + 8, budget);
    // Small batches: the expand moves to the owners of the cluster reduction (at most 64 16-byte
    // loads of B per thread), so the main loop does not depend on the shrink at all.
    g.expand_in_reduce = (splits > 1 && N <= 64 && (N / splits) <= 16 && (N / splits) * (R / 8) <= 64) ? 1 : 0;
    if (g.expand_in_reduce && p->opt_decode_splits == 0) {
      // one CTA per SM leaves room for the shrink kernel's CTAs, so that the two kernels run side
      // by side (measured on 4096 -> 4096, T = 32: 18.4 us per step with 4 splits, 24.4 with 8)
      while (splits > 1 && row_tiles * splits > p->sms) splits >>= 1;
      kb_per = (kb_total + splits - 1) / splits;
      g.splits = splits;
      g.kb_per = kb_per;
      g.expand_in_reduce = (splits > 1 && (N / splits) <= 16 && (N / splits) * (R / 8) <= 64) ? 1 : 0;
      g.stages = stages_for(N, kb_per + 8, budget);
    }
    // the cluster's reduction buffer (N x 128 fp32, plus z of the owner's tokens) overlays the ring
    while (splits > 1 && g.stages * stage_bytes < N * kTileM * 4 + (N / splits) * R * 4 && g.stages < kMaxStages)
      ++g.stages;
    g.n_acc = 1;
    g.ring_rows = N;
    g.acc_cols = N;
    g.tmem_cols = pow2_cols(N);
    CUtensorMap mr, mc, mb;
    int rc = get_tmap(p, &mr, W_dev, h_in, h_out, 0, kTileM);
    if (rc) return rc;
    rc = get_tmap(p, &mc, x, h_in, T, 0, N);
    if (rc) return rc;
    rc = get_tmap(p, &mb, p->B_pool, R, h_out, p->cfg.n_slots, kTileM);
    if (rc) return rc;
    const int grid = row_tiles * splits;
    // Small batches in one launch: the shrink runs on the idle builder warps of the base product's CTAs
    // and on spare CTAs in front of them (SMs the grid leaves empty), and the owners of the cluster
    // reduction wait for its arrival counter.  CTAs of one grid wait for one another here, so every
    // cluster of the launch must be resident at once: checked against the device's occupancy figure.
    bool fused = false;
    if (getenv("EDGELORA_LOG"))
      fprintf(stderr, "edgelora: decode T %d N %d splits %d grid %d expand_in_reduce %d ctas_per_sm %d\n", T, N, splits,
              grid, g.expand_in_reduce, ctas_per_sm);
    // (Calls that may overlap the call before them keep the two launches: a one-launch grid holds every
    // SM until its last CTA is done, so consecutive calls cannot overlap; measured on 4096 -> 4096,
    // T = 32: 17.0 us per step in one launch against 9.7 us in two when the calls are independent, and
    // 16.9 against 19.7 us when each call waits for the one before.)
    if (p->opt_fused_decode && !pdl_first && g.expand_in_reduce && T <= 64 && T <= kGatherMinT && ids_dev &&
        !p->a_q8 && h_in % 8 == 0) {
      FusedDecode f{};
      // room behind the ring for the B_a rows and z of an owner's tokens, when it fits
      // (2: and for the cluster reduction's buffer, which then does not have to wait for the ring)
      size_t stage_extra = static_cast<size_t>(N / splits) * (kTileM * R * 2 + R * 4);
      f.b_stage = smem_for(g.stages, N, static_cast<int>(stage_extra)) <= kSmemBudget ? 1 : 0;
      const size_t with_buf = ((stage_extra + 1023) & ~static_cast<size_t>(1023)) + static_cast<size_t>(N) * kTileM * 4;
      if (f.b_stage && smem_for(g.stages, N, static_cast<int>(with_buf)) <= kSmemBudget) {
        f.b_stage = 2;
        stage_extra = with_buf;
      }
      const size_t smem = smem_for(g.stages, N, f.b_stage ? static_cast<int>(stage_extra) : 0);
      const uint64_t key = (static_cast<uint64_t>(splits) << 32) | static_cast<uint64_t>(smem);
      if (p->fused_key != key) {
        p->fused_key = key;
        p->fused_max_ctas = gemm_fused_max_ctas(splits, smem);
      }
      const int spare = std::max(0, std::min(p->fused_max_ctas - grid, 32) / splits * splits);
      if (spare > 0) {  // every CTA resident at once, and a spare CTA to publish the routing plan
        const int n_teams = 2 * spare + grid;
        const int n_ksteps = (h_in + kShrinkStepElems - 1) / kShrinkStepElems;
        int ks = std::max(1, std::min(kMaxZSplits, n_ksteps / 4));
        while (ks > 1 && T * (R / 8) * ks > 2 * n_teams) ks >>= 1;
        f.n_ctas = spare;
        f.ks = ks;
        f.x_wait = 1;  // x may be the output of the call before this one
        f.A_pool = p->A_pool;
        f.x = x;
        f.z = p->zws;
        f.sync = p->group_counters + kDecodeMaxT * 8 + 8;
        f.pv = plan->pv;
        ProfScope ps(p, 3, stream);
        CUDA_TRY(launch_gemm_fused(mr, mc, g, f, smem, p->opt_pdl != 0, stream));
        ++launches;
        fused = true;
        p->last_info[2] = grid + spare;
        p->last_info[3] = splits;
      }
    }
    if (!fused) {
      rc = launch_shrink();
      if (rc) return rc;
    }
    if (!fused) {
      ProfScope ps(p, 3, stream);
      // Launched under the shrink's tail: a base-product CTA cannot share an SM with the shrink's CTAs
      // (shared memory), but the shrink's CTAs end at different times, and on the SMs that are free
      // early the base K blocks, which need no z, start at once (14336 -> 4096, T = 256: 99 us per
      // step against 104; with the one-CTA-per-SM shrink of four ring stages it was the other way
      // round, 178 against 122 us).
      CUDA_TRY(launch_gemm(mr, mc, mb, g, grid, smem_for(g.stages, N), pdl, stream));
      ++launches;
      p->last_info[2] = grid;
      p->last_info[3] = splits;
    }
  } else {
    // ---------------------------------------------------------------- prefill
    if (ids_dev) {
      ProfScope ps(p, 0, stream);
      plan->last_T = T;
      launch_plan(ids_dev, T, plan->n_slots, plan->pv, pdl_first, stream);
      CUDA_TRY(cudaGetLastError());
      ++launches;
    }
    g.zsplits = zsplits_of(p);
    if (!skip_shrink) {  // this site's shrink on its own, in front of its base product
      ShrinkJob sj;
      int rc = shrink_job(p, x, false, 0, &sj);
      if (rc) return rc;
      ProfScope ps(p, 2, stream);
      CUDA_TRY(launch_gemm(sj.mx, sj.ma, sj.mg, sj.s, sj.grid, sj.smem, ids_dev ? pdl : pdl_first, stream));
      ++launches;
    }
    CUtensorMap mx;
    int rc = get_tmap(p, &mx, x, h_in, T, 0, kTileM);
    if (rc) return rc;
    const int n_mtiles = (T + kTileM - 1) / kTileM;
    const int tiles256 = n_mtiles * ((h_out + 255) / 256);
    // 256-wide tiles unless they would leave three quarters of the SMs without a tile: a K block costs
    // the producer warp about as much for a 128-wide W tile as for a 256-wide one, so narrow tiles
    // only pay through parallelism
    int BN = (tiles256 * 4 >= p->sms || h_out <= 128) ? 256 : 128;
    BN = std::min(BN, round_up(h_out, 32));
    g.mode = kModePrefill;
    g.heavy_first = in_set ? 1 : 0;  // a serving batch: decode tokens first (see heavy_slots in gemm.cu)
    g.BN = BN;
    g.ring_rows = BN;
    g.acc_cols = BN;
    g.splits = 1;
    g.kb_per = kb_total;
    g.n_mtiles = n_mtiles;
    g.n_ntiles = (h_out + BN - 1) / BN;
    g.stages = stages_for(BN, kb_total, kSmemBudget - kYStageBytes);
    g.n_acc = 2;
    g.tmem_cols = pow2_cols(2 * BN);
    g.y_tma = 1;
    CUtensorMap mc, mb, my;
    rc = get_tmap(p, &my, y_dev, h_out, T, 0, 32, kBlockK);  // y in boxes of 32 rows x 64 columns
    if (rc) return rc;
    rc = get_tmap(p, &mc, W_dev, h_in, h_out, 0, BN);
    if (rc) return rc;
    rc = get_tmap(p, &mb, p->B_pool, R, h_out, p->cfg.n_slots, BN);
    if (rc) return rc;
    int grid = std::min(p->sms, g.n_mtiles * g.n_ntiles);
    // The next site of a set (independent of this one): its shrink rides on this site's
    // base-product launch as extra tiles, on this launch's ring.
    ShrinkJob nj;
    bool fuse_next = false;
    if (next && next->pool) {
      edgelora_pool *q = next->pool;
      if (q->cfg.max_tokens < T || q->cfg.n_slots != plan->n_slots) return EDGELORA_ERR_INVALID_ARG;
      if (q->R_pad <= BN) {
        rc = shrink_job(q, next->x, false, BN, &nj);
        if (rc) return rc;
        fuse_next = true;
        grid = std::min(p->sms, g.n_mtiles * g.n_ntiles + nj.s.n_mtiles);
        // CTAs that get one tile fewer (or none) are free for about a tile's time: that many shrink items
        g.fill_rounds = std::max(1, std::min(8, kb_total / std::max(1, nj.s.kb_per)));
      } else {  // cannot share the ring (a tiny site): on its own, before this site's base product
        rc = shrink_job(q, next->x, false, 0, &nj);
        if (rc) return rc;
        ProfScope ps(q, 2, stream);
        CUDA_TRY(launch_gemm(nj.mx, nj.ma, nj.mg, nj.s, nj.grid, nj.smem, pdl, stream));
        ++launches;
      }
    }
    {
      ProfScope ps(p, 3, stream);
      if (fuse_next)
        CUDA_TRY(launch_gemm2(mx, mc, mb, g, nj.mx, nj.ma, nj.mg, nj.s, grid, smem_for(g.stages, BN, kYStageBytes), pdl,
                              stream, &my));
      else
        CUDA_TRY(launch_gemm(mx, mc, mb, g, grid, smem_for(g.stages, BN, kYStageBytes), pdl, stream, &my));
      ++launches;
    }
    p->last_info[2] = grid;
    p->last_info[3] = 1;
  }

  // (inside a set of sites the set records the events once, after its last site: an event between
  // two kernels would keep them from overlapping)
  if (!capturing && !next && !skip_shrink) {
    CUDA_TRY(cudaEventRecord(p->use_ev, stream));
    p->use_recorded = true;
  }
  p->last_info[0] = launches;
  p->last_info[1] = regime;
  p->last_info[4] = g.stages;
  p->last_info[5] = g.BN;
  p->total_launches += launches;
  return EDGELORA_OK;
}
}  // namespace edgelora

extern "C" {

int edgelora_lora_linear(edgelora_pool_t *pool, const void *W_dev, const void *x_dev,
                         const int32_t *adapter_id_dev, int32_t T, void *y_dev, void *stream) {
  if (!pool) return EDGELORA_ERR_INVALID_ARG;
  if (T > 0 && !adapter_id_dev) return EDGELORA_ERR_INVALID_ARG;
  return lora_linear_impl(pool, pool->plan, adapter_id_dev, W_dev, x_dev, T, y_dev,
                          static_cast<cudaStream_t>(stream));
}

int edgelora_lora_linear_planned(edgelora_pool_t *pool, edgelora_plan_t *plan, const void *W_dev,
                                 const void *x_dev, int32_t T, void *y_dev, void *stream) {
  if (!pool || !plan) return EDGELORA_ERR_INVALID_ARG;
  return lora_linear_impl(pool, plan, nullptr, W_dev, x_dev, T, y_dev,
                          static_cast<cudaStream_t>(stream));
}

int edgelora_lora_linear_host(edgelora_pool_t *p, const void *W_dev, const uint16_t *x_host,
                              const int32_t *adapter_id_host, int32_t T, uint16_t *y_host,
                              void *stream) {
  if (!p || T < 0) return EDGELORA_ERR_INVALID_ARG;
  if (T == 0) return EDGELORA_OK;
  if (!x_host || !adapter_id_host || !y_host) return EDGELORA_ERR_INVALID_ARG;
  if (T > p->cfg.max_tokens) return EDGELORA_ERR_TOO_MANY_TOKENS;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t mt = p->cfg.max_tokens;
  if (!p->hx) {  // first use: pinned staging and device mirrors for one batch
    CUDA_TRY(cudaMallocHost(&p->hx, mt * p->cfg.h_in * 2));
    CUDA_TRY(cudaMallocHost(&p->hy, mt * p->cfg.h_out * 2));
    CUDA_TRY(cudaMallocHost(&p->hids, mt * 4));
    CUDA_TRY(el_malloc(&p->dx, mt * p->cfg.h_in * 2));
    CUDA_TRY(el_malloc(&p->dy, mt * p->cfg.h_out * 2));
    CUDA_TRY(el_malloc(&p->dids, mt * 4));
  }
  const size_t xb = static_cast<size_t>(T) * p->cfg.h_in * 2, yb = static_cast<size_t>(T) * p->cfg.h_out * 2;
  memcpy(p->hx, x_host, xb);
  memcpy(p->hids, adapter_id_host, static_cast<size_t>(T) * 4);
  CUDA_TRY(cudaMemcpyAsync(p->dx, p->hx, xb, cudaMemcpyHostToDevice, s));
  CUDA_TRY(cudaMemcpyAsync(p->dids, p->hids, static_cast<size_t>(T) * 4, cudaMemcpyHostToDevice, s));
  int rc = lora_linear_impl(p, p->plan, p->dids, W_dev, p->dx, T, p->dy, s);
  if (rc != EDGELORA_OK) return rc;
  CUDA_TRY(cudaMemcpyAsync(p->hy, p->dy, yb, cudaMemcpyDeviceToHost, s));
  CUDA_TRY(cudaStreamSynchronize(s));
  memcpy(y_host, p->hy, yb);
  return EDGELORA_OK;
}

int edgelora_lora_linear_host_async(edgelora_pool_t *p, const void *W_dev, const uint16_t *x_host,
                                    const int32_t *adapter_id_host, int32_t T, uint16_t *y_host,
                                    void *stream) {
  if (!p || T < 0) return EDGELORA_ERR_INVALID_ARG;
  if (T == 0) return EDGELORA_OK;
  if (!x_host || !adapter_id_host || !y_host) return EDGELORA_ERR_INVALID_ARG;
  if (T > p->cfg.max_tokens) return EDGELORA_ERR_TOO_MANY_TOKENS;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t mt = p->cfg.max_tokens;
  if (!p->h2d_stream) {  // first use
    CUDA_TRY(cudaStreamCreateWithFlags(&p->h2d_stream, cudaStreamNonBlocking));
    CUDA_TRY(cudaStreamCreateWithFlags(&p->d2h_stream, cudaStreamNonBlocking));
    for (int b = 0; b < 2; ++b) {
      CUDA_TRY(el_malloc(&p->pdx[b], mt * p->cfg.h_in * 2));
      CUDA_TRY(el_malloc(&p->pdy[b], mt * p->cfg.h_out * 2));
      CUDA_TRY(el_malloc(&p->pdids[b], mt * 4));
      CUDA_TRY(cudaEventCreateWithFlags(&p->ev_in[b], cudaEventDisableTiming));
      CUDA_TRY(cudaEventCreateWithFlags(&p->ev_done[b], cudaEventDisableTiming));
      CUDA_TRY(cudaEventCreateWithFlags(&p->ev_out[b], cudaEventDisableTiming));
    }
  }
  const int b = static_cast<int>(p->host_calls & 1);
  const bool reused = p->host_calls >= 2;  // the set was used two calls ago
  ++p->host_calls;
  const size_t xb = static_cast<size_t>(T) * p->cfg.h_in * 2, yb = static_cast<size_t>(T) * p->cfg.h_out * 2;
  // inputs: after the layer that last read this set of mirrors
  if (reused) CUDA_TRY(cudaStreamWaitEvent(p->h2d_stream, p->ev_done[b], 0));
  CUDA_TRY(cudaMemcpyAsync(p->pdx[b], x_host, xb, cudaMemcpyHostToDevice, p->h2d_stream));
  CUDA_TRY(cudaMemcpyAsync(p->pdids[b], adapter_id_host, static_cast<size_t>(T) * 4, cudaMemcpyHostToDevice,
                           p->h2d_stream));
  CUDA_TRY(cudaEventRecord(p->ev_in[b], p->h2d_stream));
  // layer: after its inputs, and after the copy-out that last read this set's y
  CUDA_TRY(cudaStreamWaitEvent(s, p->ev_in[b], 0));
  if (reused) CUDA_TRY(cudaStreamWaitEvent(s, p->ev_out[b], 0));
  int rc = lora_linear_impl(p, p->plan, p->pdids[b], W_dev, p->pdx[b], T, p->pdy[b], s);
  if (rc != EDGELORA_OK) return rc;
  CUDA_TRY(cudaEventRecord(p->ev_done[b], s));
  // result
  CUDA_TRY(cudaStreamWaitEvent(p->d2h_stream, p->ev_done[b], 0));
  CUDA_TRY(cudaMemcpyAsync(y_host, p->pdy[b], yb, cudaMemcpyDeviceToHost, p->d2h_stream));
  CUDA_TRY(cudaEventRecord(p->ev_out[b], p->d2h_stream));
  return EDGELORA_OK;
}

int edgelora_pool_host_sync(edgelora_pool_t *p) {
  if (!p) return EDGELORA_ERR_INVALID_ARG;
  if (p->d2h_stream) CUDA_TRY(cudaStreamSynchronize(p->d2h_stream));
  return EDGELORA_OK;
}

}  // extern "C"
