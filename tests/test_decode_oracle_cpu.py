"""Pins for the plain decode attention over a compact cache."""
import numpy as np

from oracle import decode_plain
from paper_2510_20707_b200 import synth

RNG = np.random.default_rng(5)


def bf16(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def wide(bits):
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


def test_zero_query_averages_values_and_ragged_offsets():
    H, G, d = 2, 3, 16
    offs = np.array([0, 5, 12])           # head 0 keeps 5 rows, head 1 keeps 7
    K, V = bf16(RNG.standard_normal((12, d))), bf16(RNG.standard_normal((12, d)))
    out = decode_plain.decode_attention(K, V, offs, bf16(np.zeros((1, H * G, d))), H, G)
    for j in range(H * G):
        r0, r1 = offs[j // G], offs[j // G + 1]
        assert np.allclose(out[0, j], wide(V[r0:r1]).mean(axis=0), rtol=1e-13)


def test_sharp_query_picks_its_row_and_weights_sum_to_one():
    H, G, d = 1, 2, 8
    K = np.eye(8)[:6] * 40.0
    V = RNG.standard_normal((6, d))
    q = np.zeros((1, 2, d)); q[0, 0, 3] = 40.0; q[0, 1, 5] = 40.0
    out = decode_plain.decode_attention(bf16(K), bf16(V), np.array([0, 6]), bf16(q), H, G, scale=1.0)
    assert np.allclose(out[0, 0], wide(bf16(V))[3], atol=1e-12)
    assert np.allclose(out[0, 1], wide(bf16(V))[5], atol=1e-12)
    ones = decode_plain.decode_attention(bf16(K), bf16(np.ones((6, d))), np.array([0, 6]), bf16(q), H, G)
    assert np.allclose(ones, 1.0, rtol=1e-13)


def test_matches_scalar_loops_and_shift_invariance():
    H, G, d, n = 2, 2, 4, 5
    K, V, q = bf16(RNG.standard_normal((2 * n, d))), bf16(RNG.standard_normal((2 * n, d))), bf16(RNG.standard_normal((1, 4, d)))
    offs = np.array([0, n, 2 * n])
    out = decode_plain.decode_attention(K, V, offs, q, H, G, scale=0.5)
    Kw, Vw, qw = wide(K), wide(V), wide(q)
    for j in range(4):
        h = j // G
        w = [np.exp(0.5 * sum(Kw[h * n + r, c] * qw[0, j, c] for c in range(d))) for r in range(n)]
        ref = [sum(w[r] * Vw[h * n + r, c] for r in range(n)) / sum(w) for c in range(d)]
        assert np.allclose(out[0, j], ref, rtol=1e-12)
    # an empty head gives zeros
    out2 = decode_plain.decode_attention(K, V, np.array([0, 0, n]), q, H, G)
    assert np.array_equal(out2[0, :G], np.zeros((G, d)))
