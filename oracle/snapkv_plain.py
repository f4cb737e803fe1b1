"""A second, independently written importance-only selector (plain SnapKV).

TEST INFRASTRUCTURE ONLY.  It exists to pin the oracle's degenerate case: with the
intrinsic term off and the mix reduced to pure importance, MixKV's selection must be
exactly what a plain observation-window compressor keeps (the paper's Sec. 3.2
"extrinsic importance" used alone; Algorithm 1 with only its attention line).

It deliberately shares nothing with ``mixkv_oracle.c``: it is numpy, it forms the
whole [G*W, L] attention matrix with a library matmul, and it pools with a
convolution instead of a neighbour loop.
"""
from __future__ import annotations

import numpy as np


def _bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def snapkv_scores(Kh_bits: np.ndarray, Qg_bits: np.ndarray, pool_kernel: int) -> np.ndarray:
    """Kh [L, d], Qg [G, W, d] bf16 bits -> pooled window-attention score of the P prefix keys."""
    K = _bf16_to_f64(Kh_bits)
    Q = _bf16_to_f64(Qg_bits)
    G, W, d = Q.shape
    L = K.shape[0]
    P = L - W
    logits = Q.reshape(G * W, d) @ K.T / np.sqrt(d)                  # [G*W, L]
    pos_q = P + np.tile(np.arange(W), G)                             # sequence position of each row
    logits = np.where(np.arange(L)[None, :] <= pos_q[:, None], logits, -np.inf)
    logits -= logits.max(axis=1, keepdims=True)
    w = np.exp(logits)
    w /= w.sum(axis=1, keepdims=True)
    vote = w.reshape(G, W, L).mean(axis=1).sum(axis=0)[:P]           # window mean, group sum
    if pool_kernel > 1:
        vote = np.convolve(vote, np.full(pool_kernel, 1.0 / pool_kernel), mode="same")
    return vote


def snapkv_keep(Kh_bits, Qg_bits, pool_kernel: int, budget: int) -> np.ndarray:
    """Positions kept by plain SnapKV: top-(budget - W) prefix keys by score, then the window."""
    G, W, d = Qg_bits.shape
    L = Kh_bits.shape[0]
    P = L - W
    s = snapkv_scores(Kh_bits, Qg_bits, pool_kernel).astype(np.float32)
    b = min(budget - W, P)
    order = np.lexsort((np.arange(P), -s))                           # score desc, position asc
    keep = np.sort(order[:b])
    return np.concatenate([keep, np.arange(P, L)]).astype(np.int64)
