"""CPU oracle of the adapter memory manager -- TEST INFRASTRUCTURE, not product code.

Paper Section 3.3: the adapters that do not fit stay outside; a pool of pre-allocated blocks, each
the size of one adapter, caches the resident ones; a needed adapter that is not resident takes a
free block, and when none is free a resident adapter is evicted and its block handed over.
Section 4.2: the resident set is kept as a recency list plus a set for membership, the free blocks
as a stack, and the pool is filled up before serving starts.  Section 3.3 also names a
frequency-based policy; both are written out here.

Everything is plain Python over lists, in the order the text gives; nothing is shared with the
CUDA library.  Readings where the text is silent: free blocks are handed out in ascending index
order; an adapter a running request holds (``pin``) is never the victim; LFU breaks ties by
recency (the least recently used of the least frequently used goes); a key's use count restarts at
one when it comes back after an eviction.
"""
from typing import List, Optional, Tuple

LRU, LFU = 0, 1


class AdapterCache:
    def __init__(self, n_blocks: int, policy: int = LRU):
        assert n_blocks >= 1 and policy in (LRU, LFU)
        self.n_blocks = n_blocks
        self.policy = policy
        self.free: List[int] = list(range(n_blocks - 1, -1, -1))  # a stack: pop() gives 0, 1, 2, ...
        self.order: List[int] = []        # resident keys, least recently used first
        self.slot = {}                    # key -> block
        self.uses = {}                    # key -> uses since it became resident
        self.pins = {}                    # key -> requests holding it
        self.hits = self.misses = self.evictions = 0

    def lookup(self, key: int) -> int:
        return self.slot.get(key, -1)

    def _victim(self) -> Optional[int]:
        candidates = [k for k in self.order if self.pins.get(k, 0) == 0]  # recency order kept
        if not candidates:
            return None
        if self.policy == LRU:
            return candidates[0]
        fewest = min(self.uses[k] for k in candidates)
        return next(k for k in candidates if self.uses[k] == fewest)

    def acquire(self, key: int, pin: bool = False) -> Tuple[int, bool, int]:
        """Returns (block, hit, evicted key or -1).  Raises when every block is pinned."""
        if key in self.slot:
            self.hits += 1
            self.order.remove(key)
            self.order.append(key)
            self.uses[key] += 1
            if pin:
                self.pins[key] = self.pins.get(key, 0) + 1
            return self.slot[key], True, -1
        evicted = -1
        if self.free:
            block = self.free.pop()
        else:
            victim = self._victim()
            if victim is None:
                raise RuntimeError("every block is held by a running request")
            block = self.slot.pop(victim)
            self.order.remove(victim)
            del self.uses[victim]
            self.pins.pop(victim, None)
            self.evictions += 1
            evicted = victim
        self.misses += 1
        self.slot[key] = block
        self.order.append(key)
        self.uses[key] = 1
        if pin:
            self.pins[key] = 1
        return block, False, evicted

    def prefill(self, keys) -> List[int]:
        """Section 4.2: before serving starts the cache is filled with (the caller's choice of)
        adapters; the counters then start at zero."""
        assert not self.slot and len(set(keys)) == len(keys) <= self.n_blocks
        blocks = [self.acquire(int(k))[0] for k in keys]
        self.hits = self.misses = 0
        return blocks

    def release(self, key: int) -> None:
        assert self.pins.get(key, 0) > 0
        self.pins[key] -= 1

    def resident(self) -> int:
        return len(self.slot)


def select_adapter(cache: AdapterCache, scores, k: int, pin: bool = False):
    """Cache-aware adapter selection (paper Algorithm 1, second half; Section 3.2): of the k
    adapters with the highest router scores, taken in descending order of score, the first one
    that is resident is used; if none is, the one with the highest score is loaded.  Scores are
    compared as given (float32); equal scores rank by adapter index.
    Returns (adapter, block, hit, evicted key or -1)."""
    import numpy as np
    s = np.asarray(scores, dtype=np.float32)
    order = sorted(range(len(s)), key=lambda j: (-float(s[j]), j))
    top = order[:max(1, min(k, len(order)))]
    for a in top:
        if cache.lookup(a) >= 0:
            block, hit, evicted = cache.acquire(a, pin)
            return a, block, hit, evicted
    block, hit, evicted = cache.acquire(top[0], pin)
    return top[0], block, hit, evicted
