"""Plain definition of the redundancy analysis maps (paper Sec. 1 / Sec. 3.1 and the heat-map
figures: pairwise cosine similarity of the keys, or values, of one head).

TEST INFRASTRUCTURE ONLY, like the rest of this package: tests compare the CUDA library's
block-mean map against it.  It is the definition written out: normalise every row, take the
full L x L matrix of dot products, average it cell by cell.  fp64 throughout; inputs are bf16
bit patterns widened exactly.
"""
from __future__ import annotations

import numpy as np


def _widen(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def block_cosine_map(X_bits: np.ndarray, block: int):
    """X_bits [H, L, d] uint16 (bf16).  Returns (cells [H, T, T], mean [H]), T = ceil(L / block):
    cells[h, I, J] is the mean of cos(x_i, x_j) over i in block I, j in block J, pairs i == j left
    out (so a diagonal cell averages n (n - 1) pairs; 0 when the block has one row); mean[h] is
    the mean over all ordered pairs i != j of the head: the redundancy of Eq. 4.  A zero row has
    cosine 0 with everything."""
    H, L, _ = X_bits.shape
    T = (L + block - 1) // block
    cells = np.zeros((H, T, T))
    mean = np.zeros(H)
    for h in range(H):
        X = _widen(X_bits[h])
        n = np.sqrt((X * X).sum(axis=1))
        Xn = np.where(n[:, None] > 0, X / np.where(n > 0, n, 1.0)[:, None], 0.0)
        Cm = Xn @ Xn.T
        np.fill_diagonal(Cm, 0.0)
        mean[h] = Cm.sum() / (L * (L - 1)) if L > 1 else 0.0
        for I in range(T):
            r0, r1 = I * block, min(L, (I + 1) * block)
            for J in range(T):
                c0, c1 = J * block, min(L, (J + 1) * block)
                pairs = (r1 - r0) * (c1 - c0) - ((r1 - r0) if I == J else 0)
                cells[h, I, J] = Cm[r0:r1, c0:c1].sum() / pairs if pairs > 0 else 0.0
    return cells, mean
