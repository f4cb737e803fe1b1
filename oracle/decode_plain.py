"""Plain definition of single-token attention over a compact (compressed, ragged) KV cache: what
a decoding step reads after MixKV has kept `B` rows per head (paper Sec. 3.1: generation continues
on the compressed cache).

TEST INFRASTRUCTURE ONLY, like the rest of this package.  fp64; inputs are bf16 bit patterns
widened exactly.  softmax(q . K^T * scale) V per query head over the rows of its KV head.
"""
from __future__ import annotations

import numpy as np


def _widen(bits: np.ndarray) -> np.ndarray:
    return (np.asarray(bits).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def decode_attention(K_rows, V_rows, row_offsets, q, H: int, G: int, scale: float | None = None):
    """K_rows, V_rows [rows, d] bf16 bits: the compact cache of one layer, rows of (sequence b,
    KV head h) at row_offsets[b*H+h] .. row_offsets[b*H+h+1].  q [batch, H*G, d] bf16 bits: one
    new query token per sequence; query head j reads KV head j // G.  Returns [batch, H*G, d]
    float64.  A head without rows gives zeros."""
    Kf, Vf, qf = _widen(K_rows), _widen(V_rows), _widen(q)
    batch, HG, d = qf.shape
    assert HG == H * G
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    out = np.zeros((batch, HG, d))
    for b in range(batch):
        for h in range(H):
            r0, r1 = int(row_offsets[b * H + h]), int(row_offsets[b * H + h + 1])
            if r1 <= r0:
                continue
            Kh, Vh = Kf[r0:r1], Vf[r0:r1]
            for g in range(G):
                s = (Kh @ qf[b, h * G + g]) * scale
                p = np.exp(s - s.max())
                p /= p.sum()
                out[b, h * G + g] = p @ Vh
    return out
