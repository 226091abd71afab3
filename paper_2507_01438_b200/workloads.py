"""Seeded synthetic inputs for the batch-LoRA linear layer.

This module only draws random numbers and packs them as bfloat16 bit patterns
(numpy uint16); it holds none of the layer's arithmetic, so both the CUDA tests
and the CPU reference checks can take their inputs from it.

Value recipe (all workloads): W, A, B ~ N(0, 0.02), x ~ N(0, 1), drawn in fp32
with numpy ``Generator(PCG64(seed))`` and rounded to nearest-even bf16; every
adapter has scale 2.0.  Adapter popularity for the many-tenant workloads is the
bounded power law of the paper's workload generator (Section 5, "Workload"):
P(i) = i^-s / sum_j j^-s over ranks 1..n, rank i mapped to a slot through a
seeded permutation so that popular adapters are not neighbours in memory.
"""
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

SCALE = 2.0
STD_W = 0.02


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 to bfloat16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) exactly to fp32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(rng: np.random.Generator, shape, std: float) -> np.ndarray:
    a = rng.standard_normal(shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    return f32_to_bf16_bits(a)


def bounded_zipf_ids(rng: np.random.Generator, n_tokens: int, n_adapters: int,
                     s: float) -> np.ndarray:
    """Slot ids drawn from P(i) ~ i^-s over ranks 1..n, rank -> slot by a seeded permutation."""
    w = np.arange(1, n_adapters + 1, dtype=np.float64) ** (-s)
    w /= w.sum()
    rank_to_slot = rng.permutation(n_adapters).astype(np.int32)
    ranks = rng.choice(n_adapters, size=n_tokens, p=w)
    return rank_to_slot[ranks].astype(np.int32)


@dataclass
class Adapter:
    A: np.ndarray      # uint16 [rank, h_in]
    B: np.ndarray      # uint16 [h_out, rank]
    scale: float

    @property
    def rank(self) -> int:
        return int(self.A.shape[0])


@dataclass
class Workload:
    """One linear site plus one mixed batch."""
    name: str
    h_in: int
    h_out: int
    n_slots: int
    max_rank: int
    W: np.ndarray                    # uint16 [h_out, h_in]
    x: np.ndarray                    # uint16 [T, h_in]
    ids: np.ndarray                  # int32 [T]
    adapters: Dict[int, Adapter] = field(default_factory=dict)   # slot -> adapter
    regime: str = "decode"           # "decode" (gather-by-token) or "prefill" (segments)

    @property
    def T(self) -> int:
        return int(self.x.shape[0])

    def distinct_adapters(self) -> List[int]:
        return sorted(set(int(a) for a in self.ids if a >= 0))

    def algorithmic_bytes(self) -> int:
        """W once, each distinct adapter once (true rank), x once, y once."""
        b = 2 * self.h_in * self.h_out + 2 * self.T * (self.h_in + self.h_out)
        for a in self.distinct_adapters():
            b += 2 * self.adapters[a].rank * (self.h_in + self.h_out)
        return b

    def algorithmic_flops(self) -> int:
        f = 2 * self.T * self.h_in * self.h_out
        for a in self.ids:
            if a >= 0:
                f += 2 * self.adapters[int(a)].rank * (self.h_in + self.h_out)
        return f


def _make_adapters(rng, slots, ranks, h_in, h_out) -> Dict[int, Adapter]:
    out = {}
    for a, r in zip(slots, ranks):
        A = normal_bf16(rng, (r, h_in), STD_W)
        B = normal_bf16(rng, (h_out, r), STD_W)
        out[int(a)] = Adapter(A, B, SCALE)
    return out


def tiny(seed: int = 0) -> Workload:
    """256 -> 256, 4 adapters of rank 8, 16 tokens with ids uniform over {-1..3}."""
    rng = np.random.Generator(np.random.PCG64(seed))
    h_in = h_out = 256
    W = normal_bf16(rng, (h_out, h_in), STD_W)
    ad = _make_adapters(rng, range(4), [8] * 4, h_in, h_out)
    x = normal_bf16(rng, (16, h_in), 1.0)
    ids = rng.integers(-1, 4, size=16).astype(np.int32)
    return Workload("tiny", h_in, h_out, 4, 8, W, x, ids, ad, "decode")


def q_proj_decode(seed: int = 1, h: int = 4096, n: int = 32, rank: int = 16) -> Workload:
    """4096 -> 4096, 32 adapters of rank 16, 32 decode tokens each with its own adapter."""
    rng = np.random.Generator(np.random.PCG64(seed))
    W = normal_bf16(rng, (h, h), STD_W)
    ad = _make_adapters(rng, range(n), [rank] * n, h, h)
    x = normal_bf16(rng, (n, h), 1.0)
    ids = rng.permutation(n).astype(np.int32)
    return Workload("q_proj_decode", h, h, n, rank, W, x, ids, ad, "decode")


def gate_up_prefill(seed: int = 2, h_in: int = 4096, h_out: int = 14336, n_req: int = 8,
                    seg_len: int = 512, rank: int = 16) -> Workload:
    """4096 -> 14336, 8 requests x 512 tokens as contiguous segments, one adapter each."""
    rng = np.random.Generator(np.random.PCG64(seed))
    W = normal_bf16(rng, (h_out, h_in), STD_W)
    ad = _make_adapters(rng, range(n_req), [rank] * n_req, h_in, h_out)
    x = normal_bf16(rng, (n_req * seg_len, h_in), 1.0)
    order = rng.permutation(n_req).astype(np.int32)
    ids = np.repeat(order, seg_len).astype(np.int32)
    return Workload("gate_up_prefill", h_in, h_out, n_req, rank, W, x, ids, ad, "prefill")


def down_proj_many_tenant(seed: int = 3, h_in: int = 14336, h_out: int = 4096,
                          n_adapters: int = 1000, rank: int = 64, n_tokens: int = 256,
                          zipf_s: float = 1.1, base_only_frac: float = 0.10,
                          only_used: bool = False) -> Workload:
    """14336 -> 4096, 1000 resident adapters of rank 64, 256 tokens with Zipf(1.1) ids, 10% id -1.

    ``only_used=True`` draws values only for the adapters the batch touches (the
    other slots stay empty); ids and the values of touched adapters are the same
    either way because every adapter has its own sub-seed.
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    W = normal_bf16(rng, (h_out, h_in), STD_W)
    x = normal_bf16(rng, (n_tokens, h_in), 1.0)
    ids = bounded_zipf_ids(rng, n_tokens, n_adapters, zipf_s)
    n_base = int(round(base_only_frac * n_tokens))
    ids[rng.choice(n_tokens, size=n_base, replace=False)] = -1
    used = set(int(a) for a in ids if a >= 0)
    ad = {}
    for a in range(n_adapters):
        if only_used and a not in used:
            continue
        sub = np.random.Generator(np.random.PCG64([seed, 1000 + a]))
        ad.update(_make_adapters(sub, [a], [rank], h_in, h_out))
    return Workload("down_proj_many_tenant", h_in, h_out, n_adapters, rank, W, x, ids, ad, "decode")


# Llama-3.1-8B projection shapes (h_in, h_out) per decoder layer.
LLAMA8B_SITES: List[Tuple[str, int, int]] = [
    ("q", 4096, 4096), ("k", 4096, 1024), ("v", 4096, 1024), ("o", 4096, 4096),
    ("gate", 4096, 14336), ("up", 4096, 14336), ("down", 14336, 4096),
]
LLAMA8B_LAYERS = 32


@dataclass
class FullSetBatch:
    """The mixed batch shared by all 224 sites of the full projection set."""
    ids: np.ndarray                 # int32 [2112]
    ranks: np.ndarray               # int32 [128], rank of each adapter (same at all its sites)
    x4096: np.ndarray               # uint16 [T, 4096]
    x14336: np.ndarray              # uint16 [T, 14336]
    n_slots: int = 128
    max_rank: int = 32


def full_set_batch(seed: int = 4, n_adapters: int = 128, n_decode: int = 64,
                   n_prefill: int = 2, prefill_len: int = 1024, zipf_s: float = 1.1) -> FullSetBatch:
    """64 decode tokens (Zipf ids) first, then 2 prefill segments of 1024 tokens on two further adapters."""
    rng = np.random.Generator(np.random.PCG64(seed))
    ranks = rng.choice(np.array([8, 16, 32], dtype=np.int32), size=n_adapters).astype(np.int32)
    dec = bounded_zipf_ids(rng, n_decode, n_adapters, zipf_s)
    free = [a for a in rng.permutation(n_adapters) if a not in set(dec.tolist())]
    pre = np.array(free[:n_prefill], dtype=np.int32)
    ids = np.concatenate([dec, np.repeat(pre, prefill_len)]).astype(np.int32)
    T = ids.shape[0]
    x4096 = normal_bf16(rng, (T, 4096), 1.0)
    x14336 = normal_bf16(rng, (T, 14336), 1.0)
    return FullSetBatch(ids, ranks, x4096, x14336, n_adapters, 32)


def full_set_site(batch: FullSetBatch, layer: int, site: int, seed: int = 4,
                  only_used: bool = True) -> Workload:
    """One of the 224 independent sites (layer 0..31, site index into LLAMA8B_SITES)."""
    name, h_in, h_out = LLAMA8B_SITES[site]
    rng = np.random.Generator(np.random.PCG64([seed, layer, site]))
    W = normal_bf16(rng, (h_out, h_in), STD_W)
    used = set(int(a) for a in batch.ids if a >= 0)
    ad = {}
    for a in range(batch.n_slots):
        if only_used and a not in used:
            continue
        sub = np.random.Generator(np.random.PCG64([seed, layer, site, a]))
        ad.update(_make_adapters(sub, [a], [int(batch.ranks[a])], h_in, h_out))
    x = batch.x4096 if h_in == 4096 else batch.x14336
    return Workload(f"full_set_L{layer}_{name}", h_in, h_out, batch.n_slots, batch.max_rank,
                    W, x, batch.ids, ad, "prefill")


@dataclass
class Trace:
    """A synthetic request trace (paper Section 5.1, "Workload trace")."""
    arrival: np.ndarray      # float64 [n] seconds, ascending
    in_len: np.ndarray       # int32 [n] prompt tokens
    out_len: np.ndarray      # int32 [n] tokens to generate
    candidates: np.ndarray   # int64 [n, k] the router's k adapters in descending order of confidence


def serving_trace(seed: int = 5, n_adapters: int = 100, alpha: float = 1.0, rate: float = 0.5,
                  cv: float = 1.0, duration: float = 300.0, in_range=(8, 256), out_range=(8, 128),
                  top_k: int = 3) -> Trace:
    """Gamma arrivals (shape 1/cv^2, scale cv^2/rate), adapter by the bounded power law with
    exponent alpha, lengths uniform over the closed ranges.  The first candidate of a request is its
    power-law adapter; the other k-1 are further distinct draws from the same law, standing in for
    the rest of the router's top-k list."""
    rng = np.random.Generator(np.random.PCG64(seed))
    gaps = rng.gamma(shape=1.0 / (cv * cv), scale=(cv * cv) / rate, size=int(duration * rate * 4) + 16)
    t = np.cumsum(gaps)
    t = t[t < duration]
    n = len(t)
    w = np.arange(1, n_adapters + 1, dtype=np.float64) ** (-alpha)
    w /= w.sum()
    rank_to_adapter = rng.permutation(n_adapters)
    k = min(top_k, n_adapters)
    cand = np.zeros((n, k), dtype=np.int64)
    for i in range(n):
        cand[i] = rank_to_adapter[rng.choice(n_adapters, size=k, replace=False, p=w)]
    in_len = rng.integers(in_range[0], in_range[1] + 1, size=n).astype(np.int32)
    out_len = rng.integers(out_range[0], out_range[1] + 1, size=n).astype(np.int32)
    return Trace(t.astype(np.float64), in_len, out_len, cand)


def q8_0_encode(values: np.ndarray) -> np.ndarray:
    """Packs rows of float32 values into Q8_0 blocks (input preparation for adapters that arrive in
    the paper's storage format): per 32 values d = max|v| / 127 as half precision, q = round(v / d).
    Rows are padded with zeros to a multiple of 32.  Returns uint8 [..., n_blocks, 34]."""
    v = np.asarray(values, dtype=np.float32)
    n = v.shape[-1]
    nb = (n + 31) // 32
    pad = np.zeros(v.shape[:-1] + (nb * 32,), dtype=np.float32)
    pad[..., :n] = v
    blk = pad.reshape(v.shape[:-1] + (nb, 32))
    d = (np.abs(blk).max(axis=-1) / np.float32(127.0)).astype(np.float16)
    df = d.astype(np.float32)
    q = np.zeros_like(blk)
    nz = df > 0
    q[nz] = np.rint(blk[nz] / df[nz][..., None])
    q = np.clip(q, -127, 127).astype(np.int8)
    out = np.zeros(v.shape[:-1] + (nb, 34), dtype=np.uint8)
    out[..., 0:2] = np.ascontiguousarray(d.astype("<f2"))[..., None].view(np.uint8)   # little endian
    out[..., 2:] = q.view(np.uint8)
    return out


def q4_0_encode(values: np.ndarray) -> np.ndarray:
    """Packs rows of float32 values into Q4_0 blocks (input preparation for base weights that arrive in
    the paper's storage format): per 32 values the element of largest magnitude m fixes d = m / -8 (half
    precision), codes c = clamp(round(v / d) + 8, 0, 15); byte j = c[j] | c[j + 16] << 4.  The row length
    must be a multiple of 32.  Returns uint8 [..., n_blocks, 18]."""
    v = np.asarray(values, dtype=np.float32)
    n = v.shape[-1]
    assert n % 32 == 0
    blk = v.reshape(v.shape[:-1] + (n // 32, 32))
    idx = np.abs(blk).argmax(axis=-1)
    m = np.take_along_axis(blk, idx[..., None], axis=-1)[..., 0]
    d = (m / np.float32(-8.0)).astype(np.float16)
    df = d.astype(np.float32)
    inv = np.zeros_like(df)
    nz = df != 0
    inv[nz] = np.float32(1.0) / df[nz]
    c = np.clip(np.floor(blk * inv[..., None] + np.float32(8.5)), 0, 15).astype(np.uint8)
    out = np.zeros(v.shape[:-1] + (n // 32, 18), dtype=np.uint8)
    out[..., 0:2] = np.ascontiguousarray(d.astype("<f2"))[..., None].view(np.uint8)
    out[..., 2:] = c[..., :16] | (c[..., 16:] << 4)
    return out
