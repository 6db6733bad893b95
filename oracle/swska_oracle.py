"""fp64 CPU oracle of sliding-window shared-key attention (SW-SKA), the attention half of the
Rodimus+ block.

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU legs may import this
module; the CUDA library and its Python binding never do.

What it computes (Sec. "Shared-Key Attention for Lossless Head Compression": softmax attention,
Eq. "attention_parallel", with ONE key per token shared by all heads, queries and values per head;
combined with a sliding window, each token attends to itself and the W - 1 tokens before it):

    s_ti  = scale * <q^h_t, k_i>                      for  t - W < i <= t   (0 <= i)
    p_ti  = exp(s_ti) / sum_{i'} exp(s_ti')           over the same i'
    o^h_t = sum_i p_ti v^h_i

The definition written out with whole-matrix numpy operations, one (batch, head) at a time: all
scores, the mask, a row-wise softmax with the row maximum subtracted, one matrix product.  No
tiling, no running maxima.  Inputs arrive as float32 (already rounded to the GPU's dtype) and are
promoted to float64.
"""
from __future__ import annotations

import numpy as np


def window_mask(T: int, window: int) -> np.ndarray:
    """M[t, i] = True iff t - window < i <= t."""
    t = np.arange(T)[:, None]
    i = np.arange(T)[None, :]
    return (i <= t) & (i > t - window)


def swska_ref(q, k, v, window: int, scale: float = 1.0) -> np.ndarray:
    """q: [B,H,T,d]; k: [B,T,d] (shared by the H heads); v: [B,H,T,dv].  Returns o [B,H,T,dv]."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    B, H, T, d = q.shape
    assert k.shape == (B, T, d) and v.shape[:3] == (B, H, T) and window >= 1
    o = np.zeros(v.shape, dtype=np.float64)
    if T == 0:
        return o
    mask = window_mask(T, window)
    for b in range(B):
        for h in range(H):
            s = scale * (q[b, h] @ k[b].T)                    # [T, T]
            s = np.where(mask, s, -np.inf)
            s = s - np.max(s, axis=1, keepdims=True)          # the diagonal is always inside
            p = np.exp(s)
            p = p / np.sum(p, axis=1, keepdims=True)
            o[b, h] = p @ v[b, h]
    return o
