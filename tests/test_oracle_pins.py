"""Pins for the CPU oracle: closed forms, invariants, brute force and special cases.

None of these retype the oracle's own loops: each compares an oracle function with a
value fixed by the mathematics (a harmonic sum, an orthonormal set, a brute-force
cosine matrix, a library sort / convolution, an independently written selector).
The paper prints no worked numeric example, so there is no printed value to pin to;
the equations cited are Sec. 3.2 (importance, diversity), Eq. 2, Eq. 3-5 and
Algorithm 1.
"""
import numpy as np
import pytest

import oracle
from oracle import snapkv_plain
from paper_2510_20707_b200 import synth

RNG = np.random.default_rng(1234)


def bf16(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def f64(bits):
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


# ------------------------------------------------------------------ bf16 rounding
def test_bf16_round_to_nearest_even_matches_torch():
    torch = pytest.importorskip("torch")
    x = np.concatenate([RNG.standard_normal(5000).astype(np.float32) * 7,
                        np.array([1.00390625, 1.01171875, 0.0, -0.0, 3.0e-39, 65280.0], np.float32)])
    ours = synth.f32_to_bf16_bits(x)
    theirs = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, theirs)
    assert np.array_equal(synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(ours)), ours)


# ------------------------------------------------------------------ window softmax
def test_softmax_rows_sum_to_one_and_mass_is_G():
    G, W, L, d = 3, 5, 41, 16
    K, Q = bf16(RNG.standard_normal((L, d))), bf16(RNG.standard_normal((G, W, d)) * 3)
    s, rows = oracle.window_attention(K, Q)
    assert np.allclose(rows, 1.0, atol=1e-13)
    assert abs(s.sum() - G) < 1e-12          # every row has mass 1, /W per row, W rows, G heads
    assert (s >= 0).all()


def test_zero_queries_give_harmonic_closed_form():
    # Q = 0 => each row is uniform over the P+j+1 keys it may see
    G, W, L, d, k = 7, 32, 200, 8, 7
    P = L - W
    K = bf16(RNG.standard_normal((L, d)))
    s, _ = oracle.window_attention(K, np.zeros((G, W, d), np.uint16))
    const = (G / W) * sum(1.0 / (P + j + 1) for j in range(W))
    assert np.allclose(s[:P], const, rtol=1e-13)
    # window column P+t is seen only by rows j >= t
    for t in (0, 5, W - 1):
        assert np.isclose(s[P + t], (G / W) * sum(1.0 / (P + j + 1) for j in range(t, W)), rtol=1e-13)
    pooled = oracle.pool(s[:P], k, 0)
    assert np.allclose(pooled[3:P - 3], const, rtol=1e-13)
    for e, frac in ((0, 4 / 7), (1, 5 / 7), (2, 6 / 7)):
        assert np.isclose(pooled[e], const * frac, rtol=1e-13)
        assert np.isclose(pooled[P - 1 - e], const * frac, rtol=1e-13)


def test_causal_mask_direction_and_scale():
    # all keys zero except the very last one, which is c*q: only the last window row may
    # see it.  Row j < W-1: uniform over P+j+1 keys.  Row W-1: the last key has logit
    # c*|q|^2/sqrt(d), the other L-1 keys logit 0.
    G, W, L, d = 1, 4, 12, 16
    P = L - W
    q = np.zeros(d, np.float32); q[:4] = [1.0, -2.0, 0.5, 1.5]
    c = 2.0
    K = np.zeros((L, d), np.float32); K[L - 1] = c * q
    Q = np.tile(q, (G, W, 1))
    s, rows = oracle.window_attention(bf16(K), bf16(Q))
    big = np.exp(c * float(q @ q) / np.sqrt(d))
    expect_prefix = (1.0 / W) * (sum(1.0 / (P + j + 1) for j in range(W - 1)) + 1.0 / (L - 1 + big))
    assert np.allclose(s[:P], expect_prefix, rtol=1e-12)
    assert np.isclose(s[L - 1], (1.0 / W) * big / (L - 1 + big), rtol=1e-12)


def test_matched_key_gets_the_vote_and_gqa_grouping():
    # head 1's queries all point at key 7 of head 1; head 0's queries at key 3 of head 0
    H, G, W, L, d = 2, 2, 4, 40, 32
    K = RNG.standard_normal((H, L, d)).astype(np.float32)
    Q = np.empty((1, H * G, W, d), np.float32)
    Q[0, 0:G] = 4 * K[0, 3]
    Q[0, G:2 * G] = 4 * K[1, 7]
    p = oracle.Params(kv_heads=H, gqa_ratio=G, head_dim=d, window=W, pool_kernel=1, budget=8,
                      use_vnorm=0, mix_mode=1)
    out = oracle.scores(bf16(K), None, bf16(Q), p)
    assert out["s_ex"][0].argmax() == 3 and out["s_ex"][1].argmax() == 7


def test_window_attention_matches_independent_numpy_softmax():
    G, W, L, d = 4, 6, 77, 32
    K, Q = bf16(RNG.standard_normal((L, d))), bf16(RNG.standard_normal((G, W, d)) * 2)
    s, _ = oracle.window_attention(K, Q)
    ref = snapkv_plain.snapkv_scores(K, Q, pool_kernel=1)
    assert np.allclose(s[:L - W], ref, rtol=1e-12, atol=1e-15)
    ref7 = snapkv_plain.snapkv_scores(K, Q, pool_kernel=7)
    assert np.allclose(oracle.pool(s[:L - W], 7, 0), ref7, rtol=1e-12, atol=1e-15)


def test_max_pool_brute_force():
    x = RNG.standard_normal(53)
    for k in (1, 3, 7):
        ref = np.array([x[max(0, i - k // 2):i + k // 2 + 1].max() for i in range(x.size)])
        assert np.array_equal(oracle.pool(x, k, 1), ref)
    assert np.array_equal(oracle.pool(x, 1, 0), x)


# ------------------------------------------------------------------ redundancy, Eq. 3-4
def brute_cosine(Kf):
    Kn = Kf / np.linalg.norm(Kf, axis=1, keepdims=True)
    return Kn @ Kn.T


@pytest.mark.parametrize("L,d", [(2, 8), (17, 16), (64, 128)])
def test_rbar_equals_brute_force_off_diagonal_mean(L, d):
    K = bf16(RNG.standard_normal((L, d)) + 0.8)
    R = brute_cosine(f64(K))
    off = (R.sum() - np.trace(R)) / (L * (L - 1))
    s_div, rbar, kbar = oracle.key_geometry(K)
    assert abs(rbar - off) < 1e-12
    # diversity score = minus the mean cosine to every key (itself included)
    assert np.allclose(s_div, -R.mean(axis=1), atol=1e-13)
    # mean of the diversity scores = -|kbar|^2 = -(rbar (L-1) + 1) / L
    assert abs(s_div.mean() + kbar @ kbar) < 1e-13
    assert abs(s_div.mean() + (rbar * (L - 1) + 1) / L) < 1e-13


def test_rbar_special_cases():
    d = 16
    eye = np.eye(d, dtype=np.float32) * 3.0
    assert abs(oracle.key_geometry(bf16(eye))[1]) < 1e-15                    # orthogonal keys
    same = np.tile(RNG.standard_normal(d).astype(np.float32), (9, 1))
    assert abs(oracle.key_geometry(bf16(same))[1] - 1.0) < 1e-12             # identical keys
    v = RNG.standard_normal((5, d)).astype(np.float32)
    pm = np.concatenate([v, -v])                                             # +- pairs sum to zero
    L = pm.shape[0]
    assert abs(oracle.key_geometry(bf16(pm))[1] + 1.0 / (L - 1)) < 1e-12
    K = bf16(RNG.standard_normal((23, d)))
    scale = 2.0 ** RNG.integers(-3, 4, size=23)                              # exact in bf16
    Ks = bf16(f64(K) * scale[:, None])
    a, b = oracle.key_geometry(K), oracle.key_geometry(Ks)
    assert abs(a[1] - b[1]) < 1e-13 and np.allclose(a[0], b[0], atol=1e-13)
    zero = f64(K).copy(); zero[4] = 0.0                                      # a zero key is dropped
    R = brute_cosine(np.delete(zero, 4, axis=0))
    sd, rb, kb = oracle.key_geometry(bf16(zero))
    assert sd[4] == 0.0 and abs(rb - (R.sum() - 23) / (23 * 22)) < 1e-12


# ------------------------------------------------------------------ Eq. 2, Eq. 5
def test_normalisation_invariants_and_mix_limits():
    P, eps = 301, 1e-6
    s_ex = RNG.random(P) * 1e-3
    vn = 8 + RNG.random(P) * 5
    s_div = -RNG.random(P) * 0.7
    o0 = oracle.mix(s_ex, vn, s_div, 0.0, eps=eps)
    o1 = oracle.mix(s_ex, vn, s_div, 1.0, eps=eps)
    om = oracle.mix(s_ex, vn, s_div, 0.3, eps=eps)
    # VNorm normalised to [0,1] and rescaled to the mean of the attention score (Sec. 3.2)
    s_in = o0["s_in_scaled"]
    m = ((vn - vn.min()) / (vn.max() - vn.min() + eps)).mean()
    assert s_in.min() == 0.0 and s_in.argmax() == vn.argmax() and s_in.argmin() == vn.argmin()
    assert np.isclose(s_in.mean(), s_ex.mean() * m / (m + eps), rtol=1e-12)
    assert np.allclose(o0["s_imp"], s_ex + s_in, rtol=1e-15)                 # Eq. 2
    # diversity normalised to [0,1] and rescaled to the mean importance (Sec. 3.3)
    sd = o0["s_div_scaled"]
    md = ((s_div - s_div.min()) / (s_div.max() - s_div.min() + eps)).mean()
    assert sd.min() == 0.0 and sd.argmax() == s_div.argmax()
    assert np.isclose(sd.mean(), o0["s_imp"].mean() * md / (md + eps), rtol=1e-12)
    ratio = sd[sd > 0] / (s_div - s_div.min())[sd > 0]
    assert np.allclose(ratio, ratio[0], rtol=1e-10)                           # affine in s_div
    # limits of Eq. 5 and linearity in r
    assert np.array_equal(o0["s_comp"], o0["s_imp"])
    assert np.array_equal(o1["s_comp"], o1["s_div_scaled"])
    assert np.allclose(om["s_comp"], 0.7 * o0["s_comp"] + 0.3 * o1["s_comp"], rtol=1e-13)
    # ablation modes nest
    assert np.array_equal(oracle.mix(s_ex, vn, s_div, 0.3, mix_mode=1)["s_comp"], o0["s_imp"])
    assert np.array_equal(oracle.mix(s_ex, vn, s_div, 0.3, mix_mode=2)["s_comp"], s_div)
    assert np.allclose(oracle.mix(s_ex, vn, s_div, 0.3, mix_mode=3)["s_comp"],
                       o0["s_imp"] + o0["s_div_scaled"], rtol=1e-15)
    # VNorm off: importance is the attention score alone
    assert np.array_equal(oracle.mix(s_ex, None, s_div, 0.0, use_vnorm=0)["s_imp"], s_ex)


def test_knorm_variant_rewards_small_key_norms():
    # KNorm (Sec. 3.2): the intrinsic term is minus the key norm, normalised like VNorm.  With
    # importance only, the layer score must equal mix(s_ex, -|K_i|, ...) of the same parts, the
    # key of smallest norm gets the largest intrinsic term, and rescaling V changes nothing.
    H, G, W, L, d = 2, 2, 4, 40, 8
    K = RNG.standard_normal((H, L, d)) * (0.5 + RNG.random((H, L, 1)) * 3)
    V = RNG.standard_normal((H, L, d))
    Q = RNG.standard_normal((1, H * G, W, d))
    Kb, Vb, Qb = bf16(K), bf16(V), bf16(Q)
    pk = oracle.Params(kv_heads=H, gqa_ratio=G, head_dim=d, window=W, pool_kernel=1, budget=12,
                       use_vnorm=2, mix_mode=1)
    pn = oracle.Params(kv_heads=H, gqa_ratio=G, head_dim=d, window=W, pool_kernel=1, budget=12,
                       use_vnorm=0, mix_mode=1)
    sk = oracle.scores(Kb, Vb, Qb, pk)
    s0 = oracle.scores(Kb, Vb, Qb, pn)
    P = L - W
    for h in range(H):
        knorm = np.sqrt((f64(Kb[h, :P]) ** 2).sum(axis=1))
        ref = oracle.mix(s0["s_comp"][h].astype(np.float64), -knorm, np.zeros(P), 0.0,
                         mix_mode=1)["s_comp"]
        assert np.allclose(sk["s_comp"][h], ref, rtol=2e-6, atol=0)
        bonus = sk["s_comp"][h].astype(np.float64) - s0["s_comp"][h]
        assert bonus.argmax() == knorm.argmin() and bonus.argmin() == knorm.argmax()
        assert bonus.min() >= 0.0
    again = oracle.scores(Kb, bf16(V * 7.0), Qb, pk)
    assert np.array_equal(again["s_comp"], sk["s_comp"])


def test_selection_invariant_to_rescaling_attention_scores():
    P = 500
    s_ex = RNG.random(P) ** 4
    vn = 8 + RNG.random(P) * 5
    s_div = -RNG.random(P)
    base = oracle.topb(oracle.mix(s_ex, vn, s_div, 0.4, eps=0.0)["s_comp"], 40)
    for c in (0.125, 8.0):       # powers of two keep float rounding identical
        sc = oracle.mix(c * s_ex, vn, s_div, 0.4, eps=0.0)["s_comp"]
        assert np.array_equal(oracle.topb(sc, 40), base)


# ------------------------------------------------------------------ selection, gather
def test_topb_against_library_sort_with_ties():
    s = RNG.integers(0, 12, size=300).astype(np.float32)        # many ties
    for b in (1, 17, 299, 300):
        ref = np.sort(np.lexsort((np.arange(300), -s))[:b])
        got = oracle.topb(s, b)
        assert np.array_equal(got, ref)
        assert (np.diff(got) > 0).all()
    # all equal => lowest positions win
    assert np.array_equal(oracle.topb(np.ones(50, np.float32), 7), np.arange(7))


def _tiny_layer(seq_lens=(37,), H=2, G=2, W=4, seed=3, **kw):
    wl = synth.small_workload(H=H, G=G, W=W, seq_lens=seq_lens, seed=seed, **kw)
    return wl, synth.make_layer(wl, 0)


def test_budget_at_least_L_keeps_everything_bit_exact():
    wl, x = _tiny_layer(seq_lens=(37,))
    for B in (37, 64):
        p = oracle.Params(kv_heads=2, gqa_ratio=2, window=4, pool_kernel=3, budget=B)
        out = oracle.compress_layer(x["K"], x["V"], x["Q"], p)
        assert np.array_equal(out["K_out"].reshape(2, 37, 128), x["K"])
        assert np.array_equal(out["V_out"].reshape(2, 37, 128), x["V"])
        assert np.array_equal(out["counts"], [[33, 33]])


def test_gather_matches_fancy_indexing_and_keeps_window():
    wl, x = _tiny_layer(seq_lens=(50, 41), H=3)
    p = oracle.Params(kv_heads=3, gqa_ratio=2, window=4, pool_kernel=3, budget=12)
    cu = wl.cu_seqlens
    out = oracle.compress_layer(x["K"], x["V"], x["Q"], p, cu=cu)
    ro, io = out["out_row_offsets"], out["idx_offsets"]
    assert ro[-1] == 2 * 3 * 12 and np.array_equal(np.diff(ro), np.full(6, 12))
    for b in range(2):
        L = cu[b + 1] - cu[b]
        for h in range(3):
            bh = b * 3 + h
            idx = out["idx"][io[bh]:io[bh + 1]]
            assert (np.diff(idx) > 0).all() and idx.max() < L - 4 and idx.size == 8
            keep = np.concatenate([idx, np.arange(L - 4, L)]) + cu[b]
            assert np.array_equal(out["K_out"][ro[bh]:ro[bh + 1]], x["K"][h, keep])
            assert np.array_equal(out["V_out"][ro[bh]:ro[bh + 1]], x["V"][h, keep])


def test_ragged_batch_equals_sequences_one_by_one():
    wl, x = _tiny_layer(seq_lens=(33, 58, 40), H=2)
    cu = wl.cu_seqlens
    p = oracle.Params(kv_heads=2, gqa_ratio=2, window=4, pool_kernel=3, budget=10)
    full = oracle.scores(x["K"], x["V"], x["Q"], p, cu=cu)
    for b in range(3):
        sl = slice(cu[b], cu[b + 1])
        one = oracle.scores(x["K"][:, sl], x["V"][:, sl], x["Q"][b:b + 1], p)
        po = cu[b] - 4 * b
        P = cu[b + 1] - cu[b] - 4
        assert np.array_equal(full["s_comp"][:, po:po + P], one["s_comp"])
        assert np.array_equal(full["rbar"][b], one["rbar"][0])


def test_position_permutation_permutes_scores_without_pooling():
    # with pool_kernel = 1 nothing couples neighbouring positions, so permuting the prefix
    # keys/values permutes the scores and maps the selected set
    wl, x = _tiny_layer(seq_lens=(45,), H=1)
    p = oracle.Params(kv_heads=1, gqa_ratio=2, window=4, pool_kernel=1, budget=14)
    perm = np.concatenate([RNG.permutation(41), np.arange(41, 45)])
    a = oracle.compress_layer(x["K"], x["V"], x["Q"], p)
    b = oracle.compress_layer(x["K"][:, perm], x["V"][:, perm], x["Q"], p)
    assert np.allclose(b["s_comp"][0], a["s_comp"][0][perm[:41]], rtol=1e-6)
    assert set(perm[b["idx"]]) == set(a["idx"])


# ------------------------------------------------------------------ degenerate = SnapKV
@pytest.mark.parametrize("variant", ["literal", "calibrated"])
def test_importance_only_equals_plain_snapkv_on_C1(variant):
    wl = synth.CONFIGS["C1"]
    x = synth.make_layer(wl, 0, variant)
    p = oracle.Params(kv_heads=4, gqa_ratio=7, budget=64, use_vnorm=0, mix_mode=1)
    out = oracle.compress_layer(x["K"], x["V"], x["Q"], p)
    io = out["idx_offsets"]
    for h in range(4):
        keep = snapkv_plain.snapkv_keep(x["K"][h], x["Q"][0, h * 7:(h + 1) * 7], 7, 64)
        got = np.concatenate([out["idx"][io[h]:io[h + 1]], np.arange(992, 1024)])
        assert np.array_equal(got, keep)


def test_orthogonal_keys_reduce_mixkv_to_importance():
    # r = 0 exactly (Eq. 4) => Eq. 5 returns s_imp => same selection as importance only
    H, G, W, d = 1, 2, 4, 128
    L = 96
    K = np.zeros((H, L, d), np.float32)
    K[0, np.arange(L), np.arange(L)] = 2.0 ** RNG.integers(-1, 3, size=L)
    V = RNG.standard_normal((H, L, d)).astype(np.float32)
    Q = RNG.standard_normal((1, H * G, W, d)).astype(np.float32) * 3
    kw = dict(kv_heads=H, gqa_ratio=G, window=W, pool_kernel=3, budget=24)
    a = oracle.compress_layer(bf16(K), bf16(V), bf16(Q), oracle.Params(mix_mode=0, **kw))
    b = oracle.compress_layer(bf16(K), bf16(V), bf16(Q), oracle.Params(mix_mode=1, **kw))
    assert np.array_equal(a["s_comp"], b["s_comp"]) and np.array_equal(a["idx"], b["idx"])


def test_identical_keys_pick_lowest_positions():
    # identical keys: r = 1, every diversity score equal => normalised to 0 => all
    # s_comp equal (0) => lowest positions win
    H, G, W, d, L = 1, 1, 4, 128, 40
    K = np.tile(RNG.standard_normal(d).astype(np.float32), (H, L, 1))
    V = RNG.standard_normal((H, L, d)).astype(np.float32)
    Q = RNG.standard_normal((1, G, W, d)).astype(np.float32)
    p = oracle.Params(kv_heads=H, gqa_ratio=G, window=W, pool_kernel=1, budget=10)
    out = oracle.compress_layer(bf16(K), bf16(V), bf16(Q), p)
    s = oracle.scores(bf16(K), bf16(V), bf16(Q), p)
    assert abs(s["rbar"][0, 0] - 1.0) < 1e-6
    # the spread of the diversity scores is rounding noise (<= 1e-15), far below eps, so the
    # normalised diversity and with it every mixed score vanishes
    assert np.abs(out["s_comp"]).max() < 1e-9
    assert out["idx"].size == 6 and (np.diff(out["idx"]) > 0).all()


# ------------------------------------------------------------------ adaptive budgets
def test_adaptive_budgets_invariants_and_brute_force():
    H, W, B = 4, 4, 20
    P = 60
    s = (RNG.random((H, P)) ** 3).astype(np.float32)
    s[2] *= 4                                                    # one head dominates
    p = oracle.Params(kv_heads=H, gqa_ratio=1, window=W, budget=B, budget_mode=1, ada_floor=0.25)
    out = oracle.select(s, p)
    counts = out["counts"][0]
    f = int(np.floor(np.float32(0.25) * (B - W)))
    assert counts.sum() == H * (B - W) and counts.min() >= f and counts[2] == counts.max()
    # brute force: global top-N over the flattened scores, ties to the lower flat position
    N = H * (B - W - f)
    flat = s.reshape(-1)
    top = np.lexsort((np.arange(flat.size), -flat))[:N]
    ref = f + np.bincount(top // P, minlength=H)
    assert np.array_equal(counts, ref)
    io = out["idx_offsets"]
    for h in range(H):
        assert np.array_equal(out["idx"][io[h]:io[h + 1]],
                              np.sort(np.lexsort((np.arange(P), -s[h]))[:counts[h]]))
    # floor = 1 and H = 1 both reduce to fixed budgets
    fixed = oracle.select(s, oracle.Params(kv_heads=H, gqa_ratio=1, window=W, budget=B))
    one = oracle.select(s, oracle.Params(kv_heads=H, gqa_ratio=1, window=W, budget=B,
                                         budget_mode=1, ada_floor=1.0))
    assert np.array_equal(fixed["idx"], one["idx"]) and np.array_equal(fixed["counts"], one["counts"])
    s1 = s[:1].copy()
    a = oracle.select(s1, oracle.Params(kv_heads=1, gqa_ratio=1, window=W, budget=B, budget_mode=1))
    b = oracle.select(s1, oracle.Params(kv_heads=1, gqa_ratio=1, window=W, budget=B))
    assert np.array_equal(a["idx"], b["idx"])
    # a cap that binds: budget larger than the prefix
    big = oracle.select(s, oracle.Params(kv_heads=H, gqa_ratio=1, window=W, budget=P + W + 5,
                                         budget_mode=1))
    assert np.array_equal(big["counts"][0], np.full(H, P))


def test_invalid_arguments_are_rejected():
    wl, x = _tiny_layer(seq_lens=(37,))
    with pytest.raises(ValueError):
        oracle.scores(x["K"], x["V"], x["Q"],
                      oracle.Params(kv_heads=2, gqa_ratio=2, window=4, pool_kernel=4))
    with pytest.raises(ValueError):
        oracle.select(np.zeros((2, 33), np.float32),
                      oracle.Params(kv_heads=2, gqa_ratio=2, window=4, budget=4))
    with pytest.raises(ValueError):
        oracle.scores(x["K"][:, :4], x["V"][:, :4], x["Q"],
                      oracle.Params(kv_heads=2, gqa_ratio=2, window=4, pool_kernel=3))
