"""CPU oracle of the adapter router's scoring head -- TEST INFRASTRUCTURE, not product code.

Paper Section 3.2: the router is a multi-label classifier over the prompt; its output is one score
s_j in [0, 1] per adapter j.  Section 5.1 describes it as the base model with a classification
head.  The head is written out here as the plain definition, in float64:
s[b][j] = sigmoid(sum_k W_r[j][k] * h[b][k] + bias[j]), h = the prompt's final hidden state.
Inputs are bf16 bit patterns widened exactly.  (Training the router and the backbone pass that
produces h are outside this package.)
"""
import numpy as np


def _widen(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def router_scores(Wr_bits: np.ndarray, bias, h_bits: np.ndarray) -> np.ndarray:
    """Wr [n, hidden] and h [B, hidden] as uint16 bf16 patterns, bias [n] float or None -> [B, n] float64."""
    W = _widen(Wr_bits)
    h = _widen(h_bits)
    v = h @ W.T
    if bias is not None:
        v = v + np.asarray(bias, dtype=np.float64)[None, :]
    out = np.empty_like(v)
    pos = v >= 0
    out[pos] = 1.0 / (1.0 + np.exp(-v[pos]))
    e = np.exp(v[~pos])
    out[~pos] = e / (1.0 + e)
    return out
