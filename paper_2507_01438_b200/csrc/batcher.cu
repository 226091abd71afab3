// Request batcher: the slot state machine of the server manager (paper Section 4: a request that
// arrives takes an idle slot, which passes through adapter selection, prompt processing and
// generation; slots in the prompt or generation state form one batch per step) over the adapter
// memory manager (Section 3.3) with the cache-aware choice of Algorithm 1 (Section 3.2).
//
// Host code only.  The batcher decides, step by step, which tokens form the batch and which pool
// slot (= cache block) each token's adapter lives in; the caller loads the adapters it is told to
// load (edgelora_pool_load_slot), runs the layers over the batch and reports how long the step took.
// Time is the caller's: a measured duration, a model, or a constant.
#include <algorithm>
#include <cstdint>
#include <deque>
#include <new>
#include <vector>

#include "../../include/edgelora.h"

namespace {

enum SlotState : int32_t { kIdle = 0, kSelection = 1, kPrompt = 2, kGeneration = 3 };

struct Req {
  int64_t id = 0;
  double arrival = 0, first_token = -1, finish = -1;
  int32_t in_len = 0, out_len = 0;
  std::vector<int64_t> candidates;
  int64_t adapter = -1;
  int32_t block = -1, hit = -1;
};

struct BSlot {
  int32_t state = kIdle;
  Req req;
  int32_t prompt_done = 0, generated = 0, take = 0;  // take: prompt tokens of the current step
};

}  // namespace

struct edgelora_batcher {
  std::vector<BSlot> slots;
  int32_t max_batch_tokens = 0, top_k = 1;
  edgelora_cache_t *cache = nullptr;
  std::deque<Req> queue;
  std::vector<Req> done;
  double now = 0;
  bool step_open = false;
};

extern "C" {

int edgelora_batcher_create(int32_t n_slots, int32_t max_batch_tokens, int32_t top_k,
                            edgelora_cache_t *cache, edgelora_batcher_t **out) {
  if (!out || !cache || n_slots < 1 || max_batch_tokens < n_slots || top_k < 1) return EDGELORA_ERR_INVALID_ARG;
  edgelora_batcher *b = new (std::nothrow) edgelora_batcher;
  if (!b) return EDGELORA_ERR_INVALID_ARG;
  b->slots.resize(n_slots);
  b->max_batch_tokens = max_batch_tokens;
  b->top_k = top_k;
  b->cache = cache;
  *out = b;
  return EDGELORA_OK;
}

int edgelora_batcher_destroy(edgelora_batcher_t *b) {
  if (!b) return EDGELORA_ERR_INVALID_ARG;
  delete b;
  return EDGELORA_OK;
}

int edgelora_batcher_submit(edgelora_batcher_t *b, int64_t request_id, double arrival, int32_t in_len,
                            int32_t out_len, const int64_t *candidates) {
  if (!b || !candidates || in_len < 1 || out_len < 1) return EDGELORA_ERR_INVALID_ARG;
  if (!b->queue.empty() && arrival < b->queue.back().arrival) return EDGELORA_ERR_INVALID_ARG;
  Req r;
  r.id = request_id;
  r.arrival = arrival;
  r.in_len = in_len;
  r.out_len = out_len;
  r.candidates.assign(candidates, candidates + b->top_k);
  for (int64_t c : r.candidates)
    if (c < 0) return EDGELORA_ERR_INVALID_ARG;
  b->queue.push_back(std::move(r));
  return EDGELORA_OK;
}

int edgelora_batcher_next_batch(edgelora_batcher_t *b, int32_t capacity, int32_t *token_block,
                                int32_t *token_slot, int32_t *n_tokens_out, int32_t *n_decode_out,
                                int64_t *load_key, int32_t *load_block, int32_t *n_loads_out, double *now_out) {
  if (!b || !token_block || !token_slot || !n_tokens_out || !n_decode_out || !load_key || !load_block ||
      !n_loads_out || capacity < b->max_batch_tokens || b->step_open)
    return EDGELORA_ERR_INVALID_ARG;
  int32_t n_loads = 0;
  for (;;) {
    // admission: arrival order, lowest idle slot first
    for (auto &s : b->slots)
      if (s.state == kIdle && !b->queue.empty() && b->queue.front().arrival <= b->now) {
        s.req = std::move(b->queue.front());
        b->queue.pop_front();
        s.state = kSelection;
        s.prompt_done = s.generated = 0;
      }
    // selection (Algorithm 1): the first resident candidate, else the first candidate is loaded
    for (auto &s : b->slots) {
      if (s.state != kSelection) continue;
      int64_t choice = s.req.candidates[0];
      for (int64_t c : s.req.candidates) {
        int32_t blk = -1;
        if (edgelora_cache_lookup(b->cache, c, &blk) == EDGELORA_OK && blk >= 0) {
          choice = c;
          break;
        }
      }
      int32_t blk = -1, hit = 0;
      int64_t evicted = -1;
      const int rc = edgelora_cache_acquire(b->cache, choice, 1, &blk, &hit, &evicted);
      if (rc == EDGELORA_ERR_CACHE_FULL) continue;  // every block is held: try again next step
      if (rc != EDGELORA_OK) return rc;
      s.req.adapter = choice;
      s.req.block = blk;
      s.req.hit = hit;
      s.state = kPrompt;
      if (!hit) {
        load_key[n_loads] = choice;
        load_block[n_loads] = blk;
        ++n_loads;
      }
    }
    bool running = false, selecting = false;
    for (auto &s : b->slots) {
      running = running || s.state == kPrompt || s.state == kGeneration;
      selecting = selecting || s.state == kSelection;
    }
    if (running) break;
    if (selecting) return EDGELORA_ERR_CACHE_FULL;  // nothing runs and nothing can be admitted
    if (b->queue.empty()) {
      *n_tokens_out = *n_decode_out = *n_loads_out = 0;
      if (now_out) *now_out = b->now;
      return 0;  // every submitted request is finished
    }
    b->now = std::max(b->now, b->queue.front().arrival);  // idle: jump to the next arrival
  }
  int32_t n = 0;
  for (size_t i = 0; i < b->slots.size(); ++i)
    if (b->slots[i].state == kGeneration) {
      token_block[n] = b->slots[i].req.block;
      token_slot[n] = static_cast<int32_t>(i);
      ++n;
    }
  const int32_t n_decode = n;
  int32_t budget = b->max_batch_tokens - n_decode;
  for (size_t i = 0; i < b->slots.size(); ++i) {
    BSlot &s = b->slots[i];
    s.take = 0;
    if (s.state != kPrompt || budget <= 0) continue;
    s.take = std::min(budget, s.req.in_len - s.prompt_done);
    for (int32_t k = 0; k < s.take; ++k) {
      token_block[n] = s.req.block;
      token_slot[n] = static_cast<int32_t>(i);
      ++n;
    }
    budget -= s.take;
  }
  b->step_open = true;
  *n_tokens_out = n;
  *n_decode_out = n_decode;
  *n_loads_out = n_loads;
  if (now_out) *now_out = b->now;
  return 1;
}

int edgelora_batcher_complete_step(edgelora_batcher_t *b, double seconds) {
  if (!b || !b->step_open || !(seconds >= 0)) return EDGELORA_ERR_INVALID_ARG;
  b->step_open = false;
  b->now += seconds;
  for (auto &s : b->slots) {
    bool emitted = false;
    if (s.state == kGeneration) {
      s.generated += 1;
      emitted = true;
    } else if (s.state == kPrompt && s.take > 0) {
      s.prompt_done += s.take;
      s.take = 0;
      if (s.prompt_done == s.req.in_len) {
        s.state = kGeneration;
        s.generated = 1;
        s.req.first_token = b->now;
        emitted = true;
      }
    }
    if (emitted && s.generated == s.req.out_len) {
      s.req.finish = b->now;
      edgelora_cache_release(b->cache, s.req.adapter);
      b->done.push_back(std::move(s.req));
      s.state = kIdle;
      s.req = Req();
    }
  }
  return EDGELORA_OK;
}

int edgelora_batcher_finished(const edgelora_batcher_t *b, int32_t capacity, int64_t *request_id,
                              double *arrival, double *first_token, double *finish, int64_t *adapter,
                              int32_t *hit, int32_t *n_out) {
  if (!b || !n_out) return EDGELORA_ERR_INVALID_ARG;
  const int32_t n = static_cast<int32_t>(b->done.size());
  *n_out = n;
  if (capacity < n) return capacity == 0 ? EDGELORA_OK : EDGELORA_ERR_INVALID_ARG;
  for (int32_t i = 0; i < n; ++i) {
    const Req &r = b->done[i];
    if (request_id) request_id[i] = r.id;
    if (arrival) arrival[i] = r.arrival;
    if (first_token) first_token[i] = r.first_token;
    if (finish) finish[i] = r.finish;
    if (adapter) adapter[i] = r.adapter;
    if (hit) hit[i] = r.hit;
  }
  return EDGELORA_OK;
}

}  // extern "C"
