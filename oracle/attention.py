"""TEST INFRASTRUCTURE -- plain CPU statement of the attention step of a DiT block; shares
nothing with the CUDA path.

The rollout models of Section 4.1 (FLUX.1, SD3.5, SANA) are diffusion transformers; the method
quantizes their linear layers (Section 3) and leaves scaled-dot-product attention in BF16.  What is
computed here is the textbook definition, per batch element and head:

    O = softmax(Q K^T / sqrt(d)) V        (no mask, no dropout; softmax over the keys)

on BF16 inputs in FP64.  Reading where the paper is silent: the scale is 1/sqrt(d) with d the head
dimension (the convention of the models named above).
"""
from __future__ import annotations

import numpy as np


def attention_head(q: np.ndarray, k: np.ndarray, v: np.ndarray) -> np.ndarray:
    """q [Sq, d], k [Skv, d], v [Skv, d] (FP64 values of BF16 inputs) -> [Sq, d] in FP64."""
    q, k, v = (np.asarray(a, dtype=np.float64) for a in (q, k, v))
    d = q.shape[1]
    s = (q @ k.T) / np.sqrt(np.float64(d))          # a library matmul as one step
    s = s - s.max(axis=1, keepdims=True)            # softmax is invariant to a per-row shift
    p = np.exp(s)
    return (p @ v) / p.sum(axis=1, keepdims=True)


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, rows=None) -> np.ndarray:
    """q [B, Sq, H, d], k and v [B, Skv, H, d] -> [B, Sq, H, d]; `rows`: only these query rows."""
    B, Sq, H, d = q.shape
    idx = np.arange(Sq) if rows is None else np.asarray(rows)
    out = np.empty((B, len(idx), H, d), dtype=np.float64)
    for b in range(B):
        for h in range(H):
            out[b, :, h, :] = attention_head(q[b, idx, h, :], k[b, :, h, :], v[b, :, h, :])
    return out


def attention_joint(first, second):
    """Two token streams that attend jointly (first stream's tokens, then the second's): (q, k, v) each
    [B, S_i, H, d].  The plain definition on the concatenated sequence, split back per stream."""
    q, k, v = (np.concatenate((a, b), axis=1) for a, b in zip(first, second))
    out = attention(q, k, v)
    n = first[0].shape[1]
    return out[:, :n], out[:, n:]


def attention_tolerance(ref: np.ndarray, v: np.ndarray) -> np.ndarray:
    """Bound for a kernel that rounds the probabilities and the output to BF16 and sums in FP32.

    Output rounding: 2^-9 |O|.  Probabilities rounded to BF16 before the product with V: each p_i
    is off by at most 2^-9 p_i, so the numerator moves by at most 2^-9 sum p_i |v_i| <= 2^-9 l
    max|v|, and the row sum l is formed from the unrounded p: 2^-9 max|v| after the division.
    exp2 in hardware (2^-22 relative) and FP32 accumulation of 10^4 terms are far below that.
    Doubled for slack: 2^-8 |O| + 2^-8 max|v| over the head.
    """
    vmax = np.abs(v).max(axis=(1, 3), keepdims=True)   # per batch element and head
    return 2.0 ** -8 * np.abs(ref) + 2.0 ** -8 * vmax
