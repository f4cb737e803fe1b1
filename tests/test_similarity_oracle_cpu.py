"""Pins for the plain block-mean cosine map (the redundancy analysis of the paper's heat-map
figures): closed forms, the relation to Eq. 4, brute force."""
import numpy as np

import oracle
from oracle import similarity_plain
from paper_2510_20707_b200 import synth

RNG = np.random.default_rng(77)


def bf16(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def test_identical_rows_and_orthonormal_rows():
    v = RNG.standard_normal(16)
    X = np.tile(v, (1, 40, 1)) * (1 + np.arange(40))[None, :, None]   # same direction, any length
    cells, mean = similarity_plain.block_cosine_map(bf16(np.round(X * 8) / 8), 16)
    assert cells.shape == (1, 3, 3)
    assert np.allclose(cells, 1.0, atol=2e-2) and np.allclose(mean, 1.0, atol=2e-2)
    E = np.eye(16)[None] * 3.0                                         # orthogonal rows
    cells, mean = similarity_plain.block_cosine_map(bf16(E), 4)
    assert np.array_equal(cells, np.zeros((1, 4, 4))) and mean[0] == 0.0
    P = np.concatenate([np.eye(8), -np.eye(8)])[None]                  # +- pairs
    cells, mean = similarity_plain.block_cosine_map(bf16(P), 8)
    assert np.isclose(mean[0], -1.0 / 15.0)
    assert np.allclose(cells[0, 0, 1], -1.0 / 8.0) and np.allclose(cells[0, 0, 0], 0.0)


def test_mean_is_eq4_and_cells_average_to_it():
    H, L, d, block = 3, 150, 32, 64
    X = RNG.standard_normal((H, L, d)) + RNG.standard_normal((H, 1, d)) * 1.5
    Xb = bf16(X)
    cells, mean = similarity_plain.block_cosine_map(Xb, block)
    T = cells.shape[1]
    n = np.array([min(block, L - I * block) for I in range(T)], dtype=np.float64)
    for h in range(H):
        assert np.allclose(cells[h], cells[h].T, rtol=1e-12)
        w = np.outer(n, n) - np.diag(n)
        assert np.isclose((cells[h] * w).sum() / (L * (L - 1)), mean[h], rtol=1e-12)
        rbar = oracle.key_geometry(Xb[h])[1]                           # Eq. 4, closed form
        assert np.isclose(mean[h], rbar, rtol=1e-9, atol=1e-12)


def test_brute_force_cell_and_zero_rows():
    L, d, block = 20, 8, 6
    X = RNG.standard_normal((1, L, d))
    X[0, 7] = 0.0
    Xb = bf16(X)
    cells, _ = similarity_plain.block_cosine_map(Xb, block)
    Xw = synth.bf16_bits_to_f32(Xb[0]).astype(np.float64)

    def cos(i, j):
        a, b = Xw[i], Xw[j]
        na, nb = np.linalg.norm(a), np.linalg.norm(b)
        return 0.0 if na == 0 or nb == 0 else float(a @ b) / (na * nb)

    I, J = 1, 3                                                        # block 3 is ragged (2 rows)
    acc = [cos(i, j) for i in range(6, 12) for j in range(18, 20)]
    assert np.isclose(cells[0, I, J], np.mean(acc), rtol=1e-12)
    acc = [cos(i, j) for i in range(6, 12) for j in range(6, 12) if i != j]
    assert np.isclose(cells[0, 1, 1], np.mean(acc), rtol=1e-12)
