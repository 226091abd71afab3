"""CPU oracle for Q8_0 adapters -- TEST INFRASTRUCTURE, not product code.

Paper Section 5.1: "All LoRA adapters are quantized using the Q8_0 format".  Q8_0 is the published
ggml block format: 32 consecutive values of a row share one IEEE half-precision scale d and are
stored as signed bytes q, the value being d * q; a block is 34 bytes, d first (little endian).
The layer with such adapters is the layer of Section 3.4 with A and B replaced by their decoded
values; this file decodes in float64 (exactly: d has 11 significant bits, q 7) and evaluates the
low-rank term token by token in float64 on top of the base product of the C oracle.

Section 5.1's model table also stores the base weights in Q8_0 or Q4_0.  Q4_0 is the published ggml
format of 18 bytes per 32 consecutive values: the half-precision scale d, then 16 bytes; byte j holds
value j in its low four bits and value j + 16 in its high four bits, each an unsigned code c with
value d * (c - 8).  `weights_decode` turns a matrix kept in either format into float64 values; the
layer then rounds each to bfloat16 (nearest even), which is the W of Section 3.4.

Readings: A is blocked along h_in (each of its `rank` rows is h_in / 32 blocks); B is blocked
along the rank (each of its h_out rows is ceil(rank / 32) blocks, entries past the rank ignored),
since the format blocks the contiguous dimension of a matrix.
"""
import numpy as np

from . import api

BLOCK, BLOCK_BYTES = 32, 34


def q8_0_decode(blocks: np.ndarray, n_values: int) -> np.ndarray:
    """blocks: uint8 [..., n_blocks, 34] -> float64 [..., n_values] (n_values <= 32 * n_blocks)."""
    blocks = np.asarray(blocks, dtype=np.uint8)
    assert blocks.shape[-1] == BLOCK_BYTES
    lead = blocks.shape[:-2]
    out = np.zeros(lead + (blocks.shape[-2] * BLOCK,), dtype=np.float64)
    flat_b = blocks.reshape(-1, blocks.shape[-2], BLOCK_BYTES)
    flat_o = out.reshape(-1, blocks.shape[-2] * BLOCK)
    for r in range(flat_b.shape[0]):
        for b in range(flat_b.shape[1]):
            blk = flat_b[r, b]
            d = float(np.frombuffer(blk[:2].tobytes(), dtype="<f2")[0])
            for i in range(BLOCK):
                q = int(blk[2 + i]) - 256 if blk[2 + i] >= 128 else int(blk[2 + i])
                flat_o[r, b * BLOCK + i] = d * q
    return out[..., :n_values]


Q4_BLOCK_BYTES = 18


def q4_0_decode(blocks: np.ndarray, n_values: int) -> np.ndarray:
    """blocks: uint8 [..., n_blocks, 18] -> float64 [..., n_values] (n_values <= 32 * n_blocks)."""
    blocks = np.asarray(blocks, dtype=np.uint8)
    assert blocks.shape[-1] == Q4_BLOCK_BYTES
    lead = blocks.shape[:-2]
    out = np.zeros(lead + (blocks.shape[-2] * BLOCK,), dtype=np.float64)
    flat_b = blocks.reshape(-1, blocks.shape[-2], Q4_BLOCK_BYTES)
    flat_o = out.reshape(-1, blocks.shape[-2] * BLOCK)
    for r in range(flat_b.shape[0]):
        for b in range(flat_b.shape[1]):
            blk = flat_b[r, b]
            d = float(np.frombuffer(blk[:2].tobytes(), dtype="<f2")[0])
            for j in range(16):
                byte = int(blk[2 + j])
                flat_o[r, b * BLOCK + j] = d * ((byte & 0x0F) - 8)
                flat_o[r, b * BLOCK + j + 16] = d * ((byte >> 4) - 8)
    return out[..., :n_values]


def weights_decode(fmt: str, blocks: np.ndarray, h_in: int) -> np.ndarray:
    """fmt "q8_0" or "q4_0"; blocks uint8 [h_out, h_in / 32, 34 or 18] -> float64 [h_out, h_in]."""
    assert h_in % BLOCK == 0 and blocks.shape[1] == h_in // BLOCK
    return q8_0_decode(blocks, h_in) if fmt == "q8_0" else q4_0_decode(blocks, h_in)


def lora_linear_q8(W_bits, x_bits, ids, adapters):
    """y[t] = W x[t] + s_a B_a (A_a x[t]) with A_a, B_a given in Q8_0.

    adapters: {slot: (A_q8 uint8 [rank, h_in/32, 34], B_q8 uint8 [h_out, ceil(rank/32), 34], rank, scale)}.
    The base product comes from the C oracle (all ids -1), the low-rank term is added per token."""
    ids = np.asarray(ids, dtype=np.int32)
    T = len(ids)
    h_out, h_in = W_bits.shape
    y = api.lora_linear(W_bits, x_bits, np.full(T, -1, dtype=np.int32), api.AdapterSet(max(adapters) + 1 if adapters else 1))
    x = (np.asarray(x_bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    decoded = {}
    for t in range(T):
        a = int(ids[t])
        if a < 0:
            continue
        if a not in decoded:
            A_q8, B_q8, rank, scale = adapters[a]
            decoded[a] = (q8_0_decode(A_q8, h_in), q8_0_decode(B_q8, rank), float(scale))
        A, Bm, s = decoded[a]
        z = np.array([sum(A[i, k] * x[t, k] for k in range(h_in)) for i in range(A.shape[0])]) \
            if h_in <= 64 else A @ x[t]
        y[t] += s * (Bm @ z)
    return y
