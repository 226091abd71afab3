// A set of linear sites that see the same mixed batch (paper Section 3.4: every LoRA-augmented
// linear layer of the model is evaluated over the same batch of requests; Section 4.3: the mapping
// from adapter ids to samples is worked out once).  The set builds one routing plan per batch and
// runs its sites back to back; because the sites are independent given their inputs, the shrink of
// site i + 1 is issued together with the kernels of site i (its gather part as a light kernel that
// runs beside them, its segment part as extra tiles of site i's base-product launch), so that only
// the first site's shrink stands alone in front of a base product.
#include <cuda_runtime.h>

#include <cstring>
#include <new>
#include <vector>

#include "guard.h"
#include "pool.h"

using namespace edgelora;

struct edgelora_siteset {
  std::vector<edgelora_pool *> pools;
  std::vector<const void *> W;
  std::vector<int32_t> input_of;
  int32_t n_inputs = 0, max_tokens = 0;
  std::vector<int32_t> in_width;          // h_in of every input
  edgelora_plan *plan = nullptr;
  // host-buffer path (allocated on first use)
  std::vector<uint16_t *> dx;             // [n_inputs] device mirrors of the inputs
  int32_t *dids = nullptr;
  std::vector<uint16_t *> dy;             // [n_sites] device results of the sites that are read back
  std::vector<std::pair<int32_t, uint16_t *>> dy_scratch;  // (h_out, buffer) for the others
  cudaStream_t copy_stream = nullptr;     // read-back of results beside the sites that follow
  std::vector<cudaEvent_t> done_ev;       // [n_sites] recorded behind a site whose result is read back
  std::vector<cudaEvent_t> up_ev;         // [n_inputs] an input uploaded on the second stream has arrived
};

namespace {

bool capturing(cudaStream_t s) {
  cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(s, &st) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  return st != cudaStreamCaptureStatusNone;
}

// after: optional, one event per site (or null): recorded on the stream behind that site's launch.
// before: optional, one event per site (or null): the stream waits for it in front of that site's launch.
int run_sites(edgelora_siteset *s, const void *const *x_dev, const int32_t *ids_dev, int32_t T,
              void *const *y_dev, cudaStream_t stream, const std::vector<cudaEvent_t> *after = nullptr,
              const std::vector<cudaEvent_t> *before = nullptr) {
  int rc = edgelora_plan_build(s->plan, ids_dev, T, stream);
  if (rc != EDGELORA_OK) return rc;
  const int n = static_cast<int>(s->pools.size());
  // The shrinks ride along only in the prefill regime (the decode regime has its own two-kernel
  // form) and only when every pool runs in its default configuration.
  bool pipelined = T > kDecodeMaxT;
  for (auto *p : s->pools) pipelined = pipelined && p->opt_regime == 0 && p->opt_pdl >= 1;
  for (int i = 0; i < n; ++i) {
    NextShrink next;
    if (pipelined && i + 1 < n) {
      next.pool = s->pools[i + 1];
      next.x = static_cast<const uint16_t *>(x_dev[s->input_of[i + 1]]);
    }
    if (before && (*before)[i] && cudaStreamWaitEvent(stream, (*before)[i], 0) != cudaSuccess) return EDGELORA_ERR_CUDA;
    // (decode-sized batches: the sites are independent given their inputs and results, so a
    // site's shrink may start under the previous site's base product)
    rc = lora_linear_impl(s->pools[i], s->plan, nullptr, s->W[i], x_dev[s->input_of[i]], T, y_dev[i], stream,
                          pipelined && i > 0, next.pool ? &next : nullptr, !pipelined && i > 0);
    if (rc != EDGELORA_OK) return rc;
    if (after && (*after)[i] && cudaEventRecord((*after)[i], stream) != cudaSuccess) return EDGELORA_ERR_CUDA;
  }
  if (pipelined && !capturing(stream)) {  // slot loads issued later wait for this step
    for (auto *p : s->pools) {
      if (cudaEventRecord(p->use_ev, stream) != cudaSuccess) return EDGELORA_ERR_CUDA;
      p->use_recorded = true;
    }
  }
  return EDGELORA_OK;
}

}  // namespace

extern "C" {

int edgelora_siteset_create(int32_t n_sites, edgelora_pool_t *const *pools, const void *const *W_dev,
                            const int32_t *input_of_site, int32_t n_inputs, int32_t max_tokens,
                            edgelora_siteset_t **set_out) {
  if (n_sites < 1 || !pools || !W_dev || !input_of_site || n_inputs < 1 || !set_out) return EDGELORA_ERR_INVALID_ARG;
  if (max_tokens == 0) max_tokens = 8192;
  if (max_tokens < 0 || max_tokens > kMaxTokensLimit) return EDGELORA_ERR_TOO_MANY_TOKENS;
  edgelora_siteset *s = new (std::nothrow) edgelora_siteset();
  if (!s) return EDGELORA_ERR_INVALID_ARG;
  s->n_inputs = n_inputs;
  s->max_tokens = max_tokens;
  s->in_width.assign(n_inputs, 0);
  for (int i = 0; i < n_sites; ++i) {
    edgelora_pool *p = pools[i];
    const int in = input_of_site[i];
    bool ok = p && W_dev[i] && in >= 0 && in < n_inputs && p->cfg.n_slots == pools[0]->cfg.n_slots &&
              p->cfg.max_tokens >= max_tokens;
    if (ok) {
      if (s->in_width[in] == 0) s->in_width[in] = p->cfg.h_in;
      ok = s->in_width[in] == p->cfg.h_in;  // every site on an input has that input's width
    }
    if (!ok) {
      delete s;
      return EDGELORA_ERR_INVALID_ARG;
    }
    s->pools.push_back(p);
    s->W.push_back(W_dev[i]);
    s->input_of.push_back(in);
  }
  int rc = edgelora_plan_create(max_tokens, pools[0]->cfg.n_slots, &s->plan);
  if (rc != EDGELORA_OK) {
    delete s;
    return rc;
  }
  s->dx.assign(n_inputs, nullptr);
  s->dy.assign(n_sites, nullptr);
  *set_out = s;
  return EDGELORA_OK;
}

int edgelora_siteset_destroy(edgelora_siteset_t *s) {
  if (!s) return EDGELORA_ERR_INVALID_ARG;
  cudaDeviceSynchronize();
  if (s->plan) edgelora_plan_destroy(s->plan);
  for (auto *q : s->dx) if (q) el_free(q);
  for (auto *q : s->dy) if (q) el_free(q);
  for (auto &e : s->dy_scratch) if (e.second) el_free(e.second);
  if (s->dids) el_free(s->dids);
  for (auto e : s->done_ev) if (e) cudaEventDestroy(e);
  for (auto e : s->up_ev) if (e) cudaEventDestroy(e);
  if (s->copy_stream) cudaStreamDestroy(s->copy_stream);
  cudaGetLastError();
  delete s;
  return EDGELORA_OK;
}

int edgelora_siteset_plan(edgelora_siteset_t *s, edgelora_plan_t **plan_out) {
  if (!s || !plan_out) return EDGELORA_ERR_INVALID_ARG;
  *plan_out = s->plan;
  return EDGELORA_OK;
}

int edgelora_siteset_run(edgelora_siteset_t *s, const void *const *x_dev, const int32_t *adapter_id_dev,
                         int32_t T, void *const *y_dev, void *stream) {
  if (!s || T < 0) return EDGELORA_ERR_INVALID_ARG;
  if (T == 0) return EDGELORA_OK;
  if (T > s->max_tokens) return EDGELORA_ERR_TOO_MANY_TOKENS;
  if (!x_dev || !adapter_id_dev || !y_dev) return EDGELORA_ERR_INVALID_ARG;
  for (int i = 0; i < s->n_inputs; ++i)
    if (!x_dev[i] && s->in_width[i]) return EDGELORA_ERR_INVALID_ARG;
  for (size_t i = 0; i < s->pools.size(); ++i)
    if (!y_dev[i]) return EDGELORA_ERR_INVALID_ARG;
  return run_sites(s, x_dev, adapter_id_dev, T, y_dev, static_cast<cudaStream_t>(stream));
}

int edgelora_siteset_run_host(edgelora_siteset_t *s, const uint16_t *const *x_host,
                              const int32_t *adapter_id_host, int32_t T, uint16_t *const *y_host,
                              void *stream) {
  if (!s || T < 0) return EDGELORA_ERR_INVALID_ARG;
  if (T == 0) return EDGELORA_OK;
  if (T > s->max_tokens) return EDGELORA_ERR_TOO_MANY_TOKENS;
  if (!x_host || !adapter_id_host || !y_host) return EDGELORA_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t mt = s->max_tokens;
  const int n = static_cast<int>(s->pools.size());
#define SET_TRY(expr)                                                                  \
  do {                                                                                 \
    cudaError_t _e = (expr);                                                           \
    if (_e != cudaSuccess) {                                                           \
      set_last_cuda_error(_e, #expr);                                                  \
      return EDGELORA_ERR_CUDA;                                                        \
    }                                                                                  \
  } while (0)
  // device mirrors, on first use: the inputs, the ids, one result buffer per site that is read
  // back and one shared buffer per output width for the sites that are not
  for (int i = 0; i < s->n_inputs; ++i) {
    if (!s->in_width[i]) continue;
    if (!x_host[i]) return EDGELORA_ERR_INVALID_ARG;
    if (!s->dx[i]) SET_TRY(el_malloc(&s->dx[i], mt * s->in_width[i] * 2));
  }
  if (!s->dids) SET_TRY(el_malloc(&s->dids, mt * 4));
  std::vector<void *> y_dev(n, nullptr);
  for (int i = 0; i < n; ++i) {
    const int32_t h_out = s->pools[i]->cfg.h_out;
    if (y_host[i]) {
      if (!s->dy[i]) SET_TRY(el_malloc(&s->dy[i], mt * h_out * 2));
      y_dev[i] = s->dy[i];
    } else {
      uint16_t *buf = nullptr;
      for (auto &e : s->dy_scratch)
        if (e.first == h_out) buf = e.second;
      if (!buf) {
        SET_TRY(el_malloc(&buf, mt * h_out * 2));
        s->dy_scratch.emplace_back(h_out, buf);
      }
      y_dev[i] = buf;
    }
  }
  // An input that the first launches do not need is uploaded on the second stream, beside them; the
  // launch in front of its first consumer waits for it (a launch also carries the next site's shrink,
  // hence one launch earlier).
  if (!s->copy_stream) SET_TRY(cudaStreamCreateWithFlags(&s->copy_stream, cudaStreamNonBlocking));
  if (s->up_ev.empty()) s->up_ev.assign(s->n_inputs, nullptr);
  std::vector<cudaEvent_t> before(n, nullptr);
  SET_TRY(cudaMemcpyAsync(s->dids, adapter_id_host, static_cast<size_t>(T) * 4, cudaMemcpyHostToDevice, st));
  for (int i = 0; i < s->n_inputs; ++i) {
    if (!s->in_width[i]) continue;
    int first = n;
    for (int k = 0; k < n; ++k)
      if (s->input_of[k] == i) {
        first = k;
        break;
      }
    const int at = first - 1;  // the launch that may already read it
    const size_t bytes = static_cast<size_t>(T) * s->in_width[i] * 2;
    if (at <= 0 || first >= n || before[at]) {
      SET_TRY(cudaMemcpyAsync(s->dx[i], x_host[i], bytes, cudaMemcpyHostToDevice, st));
    } else {
      if (!s->up_ev[i]) SET_TRY(cudaEventCreateWithFlags(&s->up_ev[i], cudaEventDisableTiming));
      SET_TRY(cudaMemcpyAsync(s->dx[i], x_host[i], bytes, cudaMemcpyHostToDevice, s->copy_stream));
      SET_TRY(cudaEventRecord(s->up_ev[i], s->copy_stream));
      before[at] = s->up_ev[i];
    }
  }
  std::vector<const void *> xd(s->dx.begin(), s->dx.end());
  // A result goes back to the host on a second stream as soon as its site is done, beside the sites
  // that follow (an event behind a launch keeps the next launch from starting under it, which is
  // paid only for the sites that are read back).
  if (s->done_ev.empty()) s->done_ev.assign(n, nullptr);
  for (int i = 0; i < n; ++i)
    if (y_host[i] && !s->done_ev[i]) SET_TRY(cudaEventCreateWithFlags(&s->done_ev[i], cudaEventDisableTiming));
  std::vector<cudaEvent_t> after(n, nullptr);
  for (int i = 0; i < n; ++i)
    if (y_host[i]) after[i] = s->done_ev[i];
  int rc = run_sites(s, xd.data(), s->dids, T, y_dev.data(), st, &after, &before);
  if (rc != EDGELORA_OK) return rc;
  for (int i = 0; i < n; ++i)
    if (y_host[i]) {
      SET_TRY(cudaStreamWaitEvent(s->copy_stream, s->done_ev[i], 0));
      SET_TRY(cudaMemcpyAsync(y_host[i], s->dy[i], static_cast<size_t>(T) * s->pools[i]->cfg.h_out * 2,
                              cudaMemcpyDeviceToHost, s->copy_stream));
    }
  SET_TRY(cudaStreamSynchronize(st));
  SET_TRY(cudaStreamSynchronize(s->copy_stream));
#undef SET_TRY
  return EDGELORA_OK;
}

}  // extern "C"
