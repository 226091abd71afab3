// Adapter memory manager, host side (paper Section 3.3: a pool of pre-allocated blocks caches the
// resident adapters, a needed adapter that is not resident takes a free block or the block of an
// evicted one; Section 4.2: recency list + membership set + stack of free blocks).
//
// Pure host code: it decides which block (= slot of an adapter pool) a key lives in; the caller
// moves the bytes with edgelora_pool_load_slot, which already runs on a side stream beside the
// layer calls.  Recency is an intrusive doubly linked list over the blocks (O(1) touch and evict),
// membership a hash map from key to block, the free blocks a stack handed out in ascending order.
// The frequency policy scans the unpinned blocks for the fewest uses (ties: least recently used).
#include <cstdint>
#include <new>
#include <unordered_map>
#include <vector>

#include "../../include/edgelora.h"

struct edgelora_cache {
  int32_t n_blocks = 0, policy = 0;
  std::vector<int64_t> key;        // per block; valid while resident
  std::vector<int32_t> prev, next; // recency list over blocks: head = least recently used
  std::vector<int64_t> uses;
  std::vector<int32_t> pins;
  std::vector<uint8_t> resident;
  std::vector<int32_t> free_stack;
  std::unordered_map<int64_t, int32_t> where;
  int32_t head = -1, tail = -1;
  int64_t hits = 0, misses = 0, evictions = 0;

  void unlink(int32_t b) {
    if (prev[b] >= 0) next[prev[b]] = next[b]; else head = next[b];
    if (next[b] >= 0) prev[next[b]] = prev[b]; else tail = prev[b];
    prev[b] = next[b] = -1;
  }
  void push_back(int32_t b) {  // most recently used end
    prev[b] = tail;
    next[b] = -1;
    if (tail >= 0) next[tail] = b; else head = b;
    tail = b;
  }
  int32_t victim() const {
    int32_t best = -1;
    for (int32_t b = head; b >= 0; b = next[b]) {  // least recently used first
      if (pins[b] > 0) continue;
      if (policy == EDGELORA_CACHE_LRU) return b;
      if (best < 0 || uses[b] < uses[best]) best = b;
    }
    return best;
  }
};

extern "C" {

int edgelora_cache_create(int32_t n_blocks, int32_t policy, edgelora_cache_t **out) {
  if (!out || n_blocks < 1 || (policy != EDGELORA_CACHE_LRU && policy != EDGELORA_CACHE_LFU))
    return EDGELORA_ERR_INVALID_ARG;
  edgelora_cache *c = new (std::nothrow) edgelora_cache;
  if (!c) return EDGELORA_ERR_INVALID_ARG;
  c->n_blocks = n_blocks;
  c->policy = policy;
  c->key.assign(n_blocks, -1);
  c->prev.assign(n_blocks, -1);
  c->next.assign(n_blocks, -1);
  c->uses.assign(n_blocks, 0);
  c->pins.assign(n_blocks, 0);
  c->resident.assign(n_blocks, 0);
  for (int32_t b = n_blocks - 1; b >= 0; --b) c->free_stack.push_back(b);  // pop gives 0, 1, 2, ...
  c->where.reserve(static_cast<size_t>(n_blocks) * 2);
  *out = c;
  return EDGELORA_OK;
}

int edgelora_cache_destroy(edgelora_cache_t *c) {
  delete c;
  return EDGELORA_OK;
}

int edgelora_cache_lookup(const edgelora_cache_t *c, int64_t key, int32_t *slot_out) {
  if (!c || !slot_out) return EDGELORA_ERR_INVALID_ARG;
  auto it = c->where.find(key);
  *slot_out = it == c->where.end() ? -1 : it->second;
  return EDGELORA_OK;
}

int edgelora_cache_acquire(edgelora_cache_t *c, int64_t key, int32_t pin, int32_t *slot_out,
                           int32_t *hit_out, int64_t *evicted_key_out) {
  if (!c || !slot_out || key < 0) return EDGELORA_ERR_INVALID_ARG;
  if (evicted_key_out) *evicted_key_out = -1;
  auto it = c->where.find(key);
  if (it != c->where.end()) {
    const int32_t b = it->second;
    ++c->hits;
    c->unlink(b);
    c->push_back(b);
    ++c->uses[b];
    if (pin) ++c->pins[b];
    *slot_out = b;
    if (hit_out) *hit_out = 1;
    return EDGELORA_OK;
  }
  int32_t b;
  if (!c->free_stack.empty()) {
    b = c->free_stack.back();
    c->free_stack.pop_back();
  } else {
    b = c->victim();
    if (b < 0) return EDGELORA_ERR_CACHE_FULL;  // every block is held by a running request
    if (evicted_key_out) *evicted_key_out = c->key[b];
    c->where.erase(c->key[b]);
    c->unlink(b);
    ++c->evictions;
  }
  ++c->misses;
  c->key[b] = key;
  c->resident[b] = 1;
  c->uses[b] = 1;
  c->pins[b] = pin ? 1 : 0;
  c->where.emplace(key, b);
  c->push_back(b);
  *slot_out = b;
  if (hit_out) *hit_out = 0;
  return EDGELORA_OK;
}

// Paper Algorithm 1, second half (Section 3.2): of the k adapters with the highest router scores,
// in descending order of score (equal scores: lower index first), the first resident one is
// used; if none is resident the best-scored one is admitted (and has to be loaded).
int edgelora_cache_select(edgelora_cache_t *c, const float *scores, int32_t n, int32_t k, int32_t pin,
                          int64_t *key_out, int32_t *slot_out, int32_t *hit_out, int64_t *evicted_key_out) {
  if (!c || !scores || n < 1 || k < 1 || !key_out || !slot_out) return EDGELORA_ERR_INVALID_ARG;
  if (k > n) k = n;
  // k passes of selection: k is a handful (the paper's settings use 3), n up to thousands
  std::vector<int32_t> top;
  std::vector<uint8_t> taken(static_cast<size_t>(n), 0);
  top.reserve(k);
  for (int32_t r = 0; r < k; ++r) {
    int32_t best = -1;
    for (int32_t j = 0; j < n; ++j) {
      if (taken[j]) continue;
      if (best < 0 || scores[j] > scores[best]) best = j;
    }
    taken[best] = 1;
    top.push_back(best);
  }
  int64_t chosen = top[0];
  for (int32_t t : top) {
    if (c->where.find(t) != c->where.end()) {
      chosen = t;
      break;
    }
  }
  *key_out = chosen;
  return edgelora_cache_acquire(c, chosen, pin, slot_out, hit_out, evicted_key_out);
}

int edgelora_cache_release(edgelora_cache_t *c, int64_t key) {
  if (!c) return EDGELORA_ERR_INVALID_ARG;
  auto it = c->where.find(key);
  if (it == c->where.end() || c->pins[it->second] <= 0) return EDGELORA_ERR_INVALID_ARG;
  --c->pins[it->second];
  return EDGELORA_OK;
}

int edgelora_cache_prefill(edgelora_cache_t *c, const int64_t *keys, int32_t n, int32_t *blocks_out) {
  if (!c || !keys || n < 0 || n > c->n_blocks) return EDGELORA_ERR_INVALID_ARG;
  if (!c->where.empty()) return EDGELORA_ERR_INVALID_ARG;  // only before serving starts
  for (int32_t i = 0; i < n; ++i) {
    if (keys[i] < 0 || c->where.count(keys[i])) return EDGELORA_ERR_INVALID_ARG;  // distinct keys
    int32_t blk = -1;
    const int rc = edgelora_cache_acquire(c, keys[i], 0, &blk, nullptr, nullptr);
    if (rc != EDGELORA_OK) return rc;
    if (blocks_out) blocks_out[i] = blk;
  }
  c->misses = 0;  // the counters describe the serving phase
  return EDGELORA_OK;
}

int edgelora_cache_stats(const edgelora_cache_t *c, int64_t *hits, int64_t *misses, int64_t *evictions,
                         int32_t *resident) {
  if (!c) return EDGELORA_ERR_INVALID_ARG;
  if (hits) *hits = c->hits;
  if (misses) *misses = c->misses;
  if (evictions) *evictions = c->evictions;
  if (resident) *resident = static_cast<int32_t>(c->where.size());
  return EDGELORA_OK;
}

}  // extern "C"
