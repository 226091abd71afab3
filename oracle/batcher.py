"""CPU oracle of the request batcher (slot state machine) -- TEST INFRASTRUCTURE, not product code.

Paper Section 4 ("Slot state machine"): a request that arrives goes to an idle slot and the slot
passes through adapter selection (Algorithm 1), prompt processing and generation; slots in the
prompt or generation state are grouped into one batch per step.  Section 5.1 ("Workload trace"):
requests arrive by a Gamma process, name an adapter by a power law and have uniform input and output
lengths; the number of slots gamma bounds the requests in flight, the others queue; the metrics are
throughput, average request latency, average first-token latency and SLO attainment (first token
within 6 seconds).  Section 3.3 adds the hit rate of the adapter cache.

Everything below is plain Python over lists, one step at a time, in that order.  Time is virtual:
the caller says how long each step took.  Readings where the text is silent:
  - requests are admitted in arrival order, each into the idle slot with the lowest index;
  - the adapter of a request is chosen once, when it is admitted (Algorithm 1 over the request's
    k candidate adapters in their given order: the first resident one, else the first one is
    loaded), and is held in the cache until the request finishes; when every block is held by
    other requests the slot stays in the selection state and tries again in the next step;
  - a step's batch holds one token of every generating slot (slot order) followed by the prompt
    tokens of the slots in the prompt state (slot order), a prompt being cut where the batch's
    token budget ends and continued in the next step;
  - the step that consumes the last prompt token also yields the request's first output token, at
    the end of that step; every later step yields one more token; a request with out_len tokens
    is finished at the end of the step that yields its last one;
  - when nothing is in flight the clock jumps to the next arrival.
"""
from typing import List, Optional

from .cache import AdapterCache

IDLE, SELECTION, PROMPT, GENERATION = 0, 1, 2, 3


class Request:
    def __init__(self, rid, arrival, in_len, out_len, candidates):
        self.rid, self.arrival, self.in_len, self.out_len = rid, float(arrival), int(in_len), int(out_len)
        self.candidates = [int(c) for c in candidates]
        self.adapter = -1      # chosen adapter (key)
        self.block = -1        # its block in the cache = slot of the adapter pool
        self.hit = None        # whether the chosen adapter was resident
        self.first_token = None
        self.finish = None


class Slot:
    def __init__(self):
        self.state = IDLE
        self.req: Optional[Request] = None
        self.prompt_done = 0
        self.generated = 0


class Batcher:
    def __init__(self, n_slots: int, max_batch_tokens: int, cache: AdapterCache):
        assert n_slots >= 1 and max_batch_tokens >= n_slots
        self.slots = [Slot() for _ in range(n_slots)]
        self.max_batch_tokens = max_batch_tokens
        self.cache = cache
        self.queue: List[Request] = []   # submitted, not yet admitted, in arrival order
        self.done: List[Request] = []
        self.now = 0.0
        self._plan = None                # the batch handed out and not yet completed

    def submit(self, rid, arrival, in_len, out_len, candidates):
        assert not self.queue or arrival >= self.queue[-1].arrival, "submit in arrival order"
        assert in_len >= 1 and out_len >= 1 and len(candidates) >= 1
        self.queue.append(Request(rid, arrival, in_len, out_len, candidates))

    def _select(self, slot: Slot) -> Optional[tuple]:
        """Algorithm 1 on the request's ordered candidates.  Returns (key, block) of a load, or None."""
        r = slot.req
        choice = next((a for a in r.candidates if self.cache.lookup(a) >= 0), r.candidates[0])
        try:
            block, hit, _ = self.cache.acquire(choice, pin=True)
        except RuntimeError:
            return None                           # every block is held: stay in selection
        r.adapter, r.block, r.hit = choice, block, hit
        slot.state = PROMPT
        return None if hit else (choice, block)

    def next_batch(self):
        """Forms the next step's batch.  Returns None when every submitted request is finished,
        else a dict: now, token_block (pool slot per token), token_slot (batcher slot per token),
        n_decode, loads [(key, block)] the caller has to perform before the step."""
        assert self._plan is None, "complete_step first"
        while True:
            # admission, in arrival order, lowest idle slot first
            for s in self.slots:
                if s.state == IDLE and self.queue and self.queue[0].arrival <= self.now:
                    s.req = self.queue.pop(0)
                    s.state, s.prompt_done, s.generated = SELECTION, 0, 0
            loads = []
            for s in self.slots:
                if s.state == SELECTION:
                    got = self._select(s)
                    if got:                      # a miss: (key, block) to load
                        loads.append(got)
            if any(s.state in (PROMPT, GENERATION) for s in self.slots):
                break
            if any(s.state == SELECTION for s in self.slots):
                raise RuntimeError("every cache block is held and nothing is running")
            if not self.queue:
                return None
            self.now = max(self.now, self.queue[0].arrival)   # idle: jump to the next arrival
        token_block, token_slot, prompt_take = [], [], {}
        for i, s in enumerate(self.slots):
            if s.state == GENERATION:
                token_block.append(s.req.block)
                token_slot.append(i)
        n_decode = len(token_block)
        budget = self.max_batch_tokens - n_decode
        for i, s in enumerate(self.slots):
            if s.state == PROMPT and budget > 0:
                take = min(budget, s.req.in_len - s.prompt_done)
                prompt_take[i] = take
                token_block += [s.req.block] * take
                token_slot += [i] * take
                budget -= take
        self._plan = (n_decode, prompt_take)
        return {"now": self.now, "token_block": token_block, "token_slot": token_slot,
                "n_decode": n_decode, "loads": loads}

    def complete_step(self, dt: float):
        """The step handed out by next_batch took dt seconds."""
        assert self._plan is not None and dt >= 0
        n_decode, prompt_take = self._plan
        self._plan = None
        self.now += dt
        for i, s in enumerate(self.slots):
            emitted = False
            if s.state == GENERATION:
                s.generated += 1
                emitted = True
            elif s.state == PROMPT and i in prompt_take:
                s.prompt_done += prompt_take[i]
                if s.prompt_done == s.req.in_len:
                    s.state, s.generated = GENERATION, 1
                    s.req.first_token = self.now
                    emitted = True
            if emitted and s.generated == s.req.out_len:
                s.req.finish = self.now
                self.cache.release(s.req.adapter)
                self.done.append(s.req)
                s.state, s.req = IDLE, None

    def run(self, step_time):
        """Drives the machine to the end; step_time(batch) -> seconds.  Returns the finished requests."""
        while True:
            b = self.next_batch()
            if b is None:
                return self.done
            self.complete_step(step_time(b))


def metrics(done: List[Request], slo_seconds: float = 6.0) -> dict:
    """Section 5.1 metrics over finished requests (plus the cache hit rate of Section 3.3)."""
    n = len(done)
    if n == 0:
        return {"requests": 0}
    span = max(r.finish for r in done) - min(r.arrival for r in done)
    return {"requests": n,
            "throughput_req_s": n / span if span > 0 else float("inf"),
            "avg_latency_s": sum(r.finish - r.arrival for r in done) / n,
            "avg_first_token_s": sum(r.first_token - r.arrival for r in done) / n,
            "slo_attainment": sum(1 for r in done if r.first_token - r.arrival <= slo_seconds) / n,
            "hit_rate": sum(1 for r in done if r.hit) / n}
