"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the
same seeded inputs (tolerances in tests/parity.py)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_20707_b200 import binding, synth
from parity import (check_gather, check_rbar, check_scores, check_selection, params_pair,
                    run_layer_parity, run_layers_parity, to_bits, to_dev)

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("variant", ["literal", "calibrated"])
def test_c1_full_layer(variant):
    run_layer_parity(synth.CONFIGS["C1"], 0, variant)


@pytest.mark.parametrize("H,G,W,L,B,pool", [
    (1, 1, 16, 17, 17, 1),        # a single candidate position
    (2, 2, 8, 33, 12, 3),
    (2, 1, 16, 257, 40, 7),
    (3, 3, 16, 1000, 100, 5),     # several chunks with a ragged tail
    (1, 7, 32, 513, 64, 7),       # one key past a chunk boundary
    (2, 4, 32, 1537, 96, 7),
    (1, 15, 16, 700, 80, 9),      # G*W = 240, the largest supported tile
])
def test_odd_shapes(H, G, W, L, B, pool):
    wl = synth.small_workload(H=H, G=G, W=W, seq_lens=(L,), pool_kernel=pool, budget=B, seed=L)
    run_layer_parity(wl)


def test_ragged_batch_fixed_and_adaptive():
    wl = synth.small_workload(H=4, G=2, W=16, seq_lens=(300, 1025, 47, 640), pool_kernel=7,
                              budget=48, seed=5)
    run_layer_parity(wl)
    run_layer_parity(synth.with_budget(wl, 48, budget_mode=1), variant="calibrated")


@pytest.mark.parametrize("kw", [
    dict(pool_mode=1), dict(use_vnorm=0), dict(use_vnorm=2), dict(use_vnorm=2, mix_mode=1),
    dict(mix_mode=1), dict(mix_mode=2), dict(mix_mode=3),
    dict(use_vnorm=0, mix_mode=1), dict(eps=1e-3), dict(softmax_scale=0.05),
])
def test_modes(kw):
    wl = synth.small_workload(H=2, G=2, W=16, seq_lens=(900,), pool_kernel=7, budget=80, seed=11)
    run_layer_parity(wl, variant="calibrated", **kw)


def test_budget_at_least_L_keeps_everything():
    wl = synth.small_workload(H=2, G=2, W=16, seq_lens=(200,), budget=200, seed=2)
    x = synth.make_layer(wl, 0)
    _, pg = params_pair(wl)
    out = binding.compress_layer(to_dev(x["K"]), to_dev(x["V"]), to_dev(x["Q"]), pg)
    torch.cuda.synchronize()
    assert out["out_row_offsets"].tolist() == [0, 200, 400]
    assert np.array_equal(to_bits(out["K_out"]).reshape(2, 200, 128), x["K"])
    assert np.array_equal(to_bits(out["V_out"]).reshape(2, 200, 128), x["V"])


def test_offline_head_weights():
    wl = synth.small_workload(H=2, G=2, W=16, seq_lens=(500,), budget=60, seed=4)
    x = synth.make_layer(wl, 0, "calibrated")
    po, pg = params_pair(wl)
    rin = np.array([[0.15, 0.85]], np.float32)
    ref = oracle.scores(x["K"], x["V"], x["Q"], po, rbar_in=rin)
    got = binding.scores(to_dev(x["K"]), to_dev(x["V"]), to_dev(x["Q"]), pg,
                         rbar_in=torch.from_numpy(rin).cuda())
    check_scores("s_comp", got["s_comp"].cpu().numpy(), ref["s_comp"], wl.cu_seqlens, 16)
    check_rbar(got["rbar"].cpu().numpy(), ref["rbar"].astype(np.float64))


def test_select_with_ties_is_exact():
    # on caller-supplied scores the selection is integer work: bit-identical to the oracle
    rng = np.random.default_rng(0)
    H, P, W = 3, 5000, 16
    s = rng.integers(0, 50, size=(H, P)).astype(np.float32)
    s[1] = 1.0                                                # a head of all-equal scores
    s[2, ::7] = -0.0
    for mode in (0, 1):
        po = oracle.Params(kv_heads=H, gqa_ratio=1, window=W, budget=W + 333, budget_mode=mode)
        pg = binding.Params(kv_heads=H, gqa_ratio=1, window=W, budget=W + 333, budget_mode=mode)
        ref = oracle.select(s, po)
        got = binding.select(torch.from_numpy(s).cuda(), pg)
        offs = got["idx_offsets"].cpu().numpy()
        assert np.array_equal(got["counts"].cpu().numpy(), ref["counts"].reshape(-1))
        assert np.array_equal(offs, ref["idx_offsets"])
        assert np.array_equal(got["idx"].cpu().numpy()[:offs[-1]], ref["idx"])


def test_identical_keys_head():
    # r = 1: the mix is pure diversity, whose spread is rounding noise; only the things
    # that stay well defined are checked (rbar, the count, valid ascending indices)
    H, G, W, L = 1, 1, 16, 300
    rng = np.random.default_rng(3)
    K = np.tile(rng.standard_normal(128).astype(np.float32), (H, L, 1))
    V = rng.standard_normal((H, L, 128)).astype(np.float32)
    Q = rng.standard_normal((1, G, W, 128)).astype(np.float32)
    pg = binding.Params(kv_heads=H, gqa_ratio=G, window=W, budget=48)
    out = binding.compress_layer(to_dev(synth.f32_to_bf16_bits(K)), to_dev(synth.f32_to_bf16_bits(V)),
                                 to_dev(synth.f32_to_bf16_bits(Q)), pg)
    torch.cuda.synchronize()
    idx = out["idx"].cpu().numpy()[:32]
    assert out["counts"].tolist() == [32] and (np.diff(idx) > 0).all() and idx.max() < L - W


@pytest.mark.parametrize("name,layer", [("C2", 0), ("C2", 27), ("C5", 0)])
def test_full_size_layers(name, layer):
    run_layer_parity(synth.CONFIGS[name], layer, "calibrated")


@pytest.mark.parametrize("name,layer", [("C2", 1), ("C3", 7), ("C4", 2), ("C5", 5)])
def test_full_size_layers_literal_keys(name, layer):
    # the recipe as written (no shared per-head offset): mean key cosine near 0.05 (vision) or 0
    # (text), the other regime of the diversity min-max and of Eq. 5
    run_layer_parity(synth.CONFIGS[name], layer, "literal")


def test_knorm_variant_full_size_and_batched():
    # key-norm intrinsic term (Sec. 3.2 ablation): V is not read for the scores
    run_layer_parity(synth.CONFIGS["C5"], 3, variant="calibrated", use_vnorm=2)
    wl = synth.small_workload(H=2, G=4, W=32, seq_lens=(1500, 700), pool_kernel=7, budget=96,
                              seed=61, centroids=8)
    wl = synth.replace(wl, layers=4)
    run_layers_parity(wl, range(4), use_vnorm=2)


def test_c4_ragged_adaptive_layer():
    run_layer_parity(synth.CONFIGS["C4"], 0, "calibrated")


@pytest.mark.parametrize("name", ["C3", "C3b"])
def test_c3_long_video_layer(name):
    run_layer_parity(synth.CONFIGS[name], 13, "calibrated")


# ---- several layers in one call (mixkv_compress_layers)
def test_layers_batched_small_ragged():
    wl = synth.small_workload(H=3, G=2, W=16, seq_lens=(300, 1025, 47), pool_kernel=7, budget=48,
                              seed=9)
    wl = synth.replace(wl, layers=5)
    run_layers_parity(wl, range(5))
    run_layers_parity(synth.with_budget(wl, 48, budget_mode=1), range(5))
    run_layers_parity(wl, range(3), pad_rows=24, pool_mode=1)


def test_layers_batched_c2():
    run_layers_parity(synth.CONFIGS["C2"], (0, 13, 27, 5))


def test_layers_batched_c4_adaptive():
    run_layers_parity(synth.CONFIGS["C4"], (0, 1))


def test_layers_batched_c3_c5():
    run_layers_parity(synth.CONFIGS["C3"], (3, 20))
    run_layers_parity(synth.CONFIGS["C5"], (0, 31))


def test_bench_launch_configuration_sampled():
    # the call bench.py times: all 28 layers of C3 in one mixkv_compress_layers call; the oracle
    # checks three sampled layers (first, middle, last), the rest by properties that hold at any
    # size: counts, ascending in-range indices, offsets, and the window rows at the end of
    # every (layer, head) block being bit-exact copies
    wl = synth.CONFIGS["C3"]
    NL, H, W, B = wl.layers, wl.kv_heads, wl.window, wl.budget
    L = wl.total_tokens
    po, pg = params_pair(wl)
    K = torch.empty((NL, H, L, 128), dtype=torch.bfloat16, device="cuda")
    V = torch.empty_like(K)
    Q = torch.empty((NL, 1, H * wl.gqa_ratio, W, 128), dtype=torch.bfloat16, device="cuda")
    sampled = {}
    for layer in range(NL):
        x = synth.make_layer(wl, layer, "calibrated")
        K[layer], V[layer], Q[layer] = to_dev(x["K"]), to_dev(x["V"]), to_dev(x["Q"])
        if layer in (0, NL // 2, NL - 1):
            sampled[layer] = x
    out = binding.compress_layers(K, V, Q, pg)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    P = L - W
    counts = out["counts"].cpu().numpy()
    offs = out["idx_offsets"].cpu().numpy()
    ro = out["out_row_offsets"].cpu().numpy()
    idx = out["idx"].cpu().numpy()
    assert (counts == B - W).all()
    assert (offs == np.arange(H + 1) * (B - W)).all() and (ro == np.arange(H + 1) * B).all()
    sel = idx.reshape(NL, H, B - W)
    assert (np.diff(sel, axis=2) > 0).all() and sel.min() >= 0 and sel.max() < P
    Ko = out["K_out"].view(NL, H, B, 128)
    Vo = out["V_out"].view(NL, H, B, 128)
    assert torch.equal(Ko[:, :, B - W:], K[:, :, P:]) and torch.equal(Vo[:, :, B - W:], V[:, :, P:])
    gidx = torch.from_numpy(sel).cuda().long()[..., None].expand(-1, -1, -1, 128)
    assert torch.equal(Ko[:, :, :B - W], torch.gather(K, 2, gidx))
    assert torch.equal(Vo[:, :, :B - W], torch.gather(V, 2, gidx))
    cu = wl.cu_seqlens
    for layer, x in sampled.items():
        ref_s = oracle.scores(x["K"], x["V"], x["Q"], po)
        ref = oracle.select(ref_s["s_comp"], po)
        check_scores(f"s_comp[layer {layer}]", out["s_comp"][layer].cpu().numpy(), ref_s["s_comp"],
                     cu, W)
        check_selection(idx[layer], offs[layer], counts[layer], ref, ref_s["s_comp"], cu, W, H)


def test_bench_launch_configuration_c4_and_c5():
    # the calls bench.py times for the other two multi-layer workloads, at full size.  C4: 28
    # layers x 8 ragged sequences with adaptive budgets = 224 (sequence, layer) pairs, which
    # takes the budget kernel with one CTA per pair and the select + gather tail with one CTA
    # per head; C5: 32 layers x 8 heads = 256 units through the fused tail.  The oracle checks
    # sampled layers, properties that need no oracle check every layer.
    wl = synth.CONFIGS["C4"]
    run_layers_parity(wl, range(wl.layers), check=(0, 14, 27), properties=True)
    wl = synth.CONFIGS["C5"]
    run_layers_parity(wl, range(wl.layers), check=(9, 31), properties=True)


def test_prefix_longer_than_the_tail_cache():
    # 140000 candidates of one head: more than eight CTAs of a cluster keep in shared memory, so
    # the call takes the unfused route and the select + gather tail reads its keys from global
    # memory in every pass
    wl = synth.small_workload(H=1, G=1, W=16, seq_lens=(140016,), pool_kernel=5, budget=272,
                              seed=33, centroids=8)
    run_layer_parity(wl, variant="calibrated")


@pytest.mark.parametrize("H,lens,levels", [
    (8, (16400,) * 19, 3),        # one CTA per sequence, keys not cached, no candidate list
    (8, (16400,) * 19, 1 << 20),  # one CTA per sequence, keys not cached, candidate list
    (8, (60016,), 5),             # cluster of eight, keys not cached, no candidate list
    (8, (60016,), 1 << 20),       # cluster of eight, keys not cached, candidate list
])
def test_adaptive_budgets_on_many_keys_are_exact(H, lens, levels):
    # adaptive budgets on caller-supplied scores are integer work: bit-identical to the oracle.
    # These shapes hold more keys per CTA than its shared memory caches; with few score levels
    # the bin left after the first digit pass is larger than the candidate list.
    W = 16
    rng = np.random.default_rng(levels % 97)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    Ptot = int(cu[-1]) - len(lens) * W
    s = (rng.integers(0, levels, size=(H, Ptot)) / np.float32(levels)).astype(np.float32)
    po = oracle.Params(kv_heads=H, gqa_ratio=1, window=W, budget=W + 200, budget_mode=1)
    pg = binding.Params(kv_heads=H, gqa_ratio=1, window=W, budget=W + 200, budget_mode=1)
    ref = oracle.select(s, po, cu=cu if len(lens) > 1 else None)
    got = binding.select(torch.from_numpy(s).cuda(), pg,
                         cu_seqlens=[int(c) for c in cu] if len(lens) > 1 else None)
    offs = got["idx_offsets"].cpu().numpy()
    assert np.array_equal(got["counts"].cpu().numpy(), ref["counts"].reshape(-1))
    assert np.array_equal(offs, ref["idx_offsets"])
    assert np.array_equal(got["idx"].cpu().numpy()[:offs[-1]], ref["idx"])


@pytest.mark.parametrize("levels", [0, 50, 3000000])
def test_whole_head_ctas_select_exactly(levels):
    # 80 (sequence, head) units of 20000 candidates: one 1024-thread CTA per unit with the keys
    # in shared memory.  Few score levels leave more keys in the bin after two digits than the
    # key list takes (the four-pass search), many levels a few hundred (the list), levels = 0
    # real-valued scores; a head of equal scores and negative zeros ride along.  Integer work:
    # bit-identical to the oracle.
    H, B, W, P = 8, 10, 16, 20000
    rng = np.random.default_rng(levels + 3)
    cu = (np.arange(B + 1) * (P + W)).astype(np.int32)
    if levels:
        s = (rng.integers(0, levels, size=(H, B * P)) / np.float32(levels)).astype(np.float32)
    else:
        s = rng.standard_normal((H, B * P)).astype(np.float32) ** 2
    s[1, :P] = 0.25
    s[2, ::5] = -0.0
    po = oracle.Params(kv_heads=H, gqa_ratio=1, window=W, budget=W + 333)
    pg = binding.Params(kv_heads=H, gqa_ratio=1, window=W, budget=W + 333)
    ref = oracle.select(s, po, cu=cu)
    got = binding.select(torch.from_numpy(s).cuda(), pg, cu_seqlens=[int(c) for c in cu])
    assert int(got["status"].item()) == 0
    offs = got["idx_offsets"].cpu().numpy()
    assert np.array_equal(got["counts"].cpu().numpy(), ref["counts"].reshape(-1))
    assert np.array_equal(offs, ref["idx_offsets"])
    assert np.array_equal(got["idx"].cpu().numpy()[:offs[-1]], ref["idx"])


def test_long_sequence_cluster_tail():
    # 65536 keys per head: the cluster shape of the tail kernel with 16 positions per thread
    wl = synth.small_workload(H=2, G=4, W=32, seq_lens=(65536,), pool_kernel=7, budget=512,
                              seed=31, centroids=32)
    run_layer_parity(wl, variant="calibrated")


def test_many_units_long_prefix_and_widest_query_tile():
    # 80 (layer, head) units of 45000 candidates: too long for one CTA per head, so the call
    # falls back to clusters; G*W = 240 is the widest supported query tile
    wl = synth.small_workload(H=2, G=15, W=16, seq_lens=(45016,), pool_kernel=5, budget=300,
                              seed=32, centroids=16)
    wl = synth.replace(wl, layers=40)
    run_layers_parity(wl, range(40), check=(0, 17, 39))


def test_repeated_calls_are_bit_identical_widest_query_tile():
    # G*W = 240 leaves pass 2 room for three V stages only, which the two pairs of value-norm
    # warps then share in turn (with four, each pair has its own): the same call thirty times
    # over must give the same bits every time, value norms included (they reach s_comp through
    # the intrinsic term).  A warp that read a V stage before its copy had landed would show
    # here.
    wl = synth.small_workload(H=2, G=15, W=16, seq_lens=(45016,), pool_kernel=5, budget=300,
                              seed=33, centroids=16)
    wl = synth.replace(wl, layers=6)
    _, pg = params_pair(wl)
    xs = [synth.make_layer(wl, l, "calibrated") for l in range(6)]
    K, V, Q = (torch.stack([to_dev(x[k]) for x in xs]) for k in ("K", "V", "Q"))
    first = None
    for _ in range(30):
        out = binding.compress_layers(K, V, Q, pg)
        torch.cuda.synchronize()
        assert int(out["status"].item()) == 0
        if first is None:
            first = out
            continue
        for key in ("s_comp", "idx", "idx_offsets", "out_row_offsets"):
            assert torch.equal(first[key], out[key]), key
        assert torch.equal(first["V_out"].view(torch.int16), out["V_out"].view(torch.int16))


def test_workspace_needs_no_clearing():
    # Every word of the workspace that a kernel reads was written earlier in the same call:
    # whatever the workspace holds (all ones, all zeros, random bytes, what an earlier call on
    # another shape left) the results are bit-identical.
    wl = synth.small_workload(H=3, G=4, W=16, seq_lens=(3000, 1500), pool_kernel=5, budget=96,
                              seed=41, centroids=8)
    x = synth.make_layer(wl, 0, "calibrated")
    _, pg = params_pair(wl)
    K, V, Q = to_dev(x["K"]), to_dev(x["V"]), to_dev(x["Q"])
    cu = [int(c) for c in wl.cu_seqlens]
    nbytes = binding.workspace_size(pg, wl.batch, wl.total_tokens, max(wl.seq_lens))
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    gen = torch.Generator(device="cuda").manual_seed(5)
    results = []
    for fill in ("ones", "zeros", "random", "reuse", "other-shape-first"):
        if fill == "ones":
            ws.fill_(255)
        elif fill == "zeros":
            ws.zero_()
        elif fill == "random":
            ws.copy_(torch.randint(0, 256, (nbytes,), dtype=torch.uint8, device="cuda",
                                   generator=gen))
        elif fill == "other-shape-first":
            wl2 = synth.small_workload(H=3, G=4, W=16, seq_lens=(700,), pool_kernel=5, budget=96,
                                       seed=42, centroids=8)
            x2 = synth.make_layer(wl2, 0, "literal")
            o2 = binding.compress_layer(to_dev(x2["K"]), to_dev(x2["V"]), to_dev(x2["Q"]), pg,
                                        workspace=ws)
            assert int(o2["status"].item()) == 0
        out = binding.compress_layer(K, V, Q, pg, cu_seqlens=cu, workspace=ws)
        torch.cuda.synchronize()
        assert int(out["status"].item()) == 0
        results.append(out)
    first = results[0]
    n_rows = int(first["out_row_offsets"][-1].item())
    for out in results[1:]:
        for key in ("s_comp", "idx_offsets", "counts", "out_row_offsets"):
            assert torch.equal(first[key], out[key]), key
        n_idx = int(first["idx_offsets"][-1].item())
        assert torch.equal(first["idx"][:n_idx], out["idx"][:n_idx])
        assert torch.equal(first["K_out"][:n_rows].view(torch.int16), out["K_out"][:n_rows].view(torch.int16))
        assert torch.equal(first["V_out"][:n_rows].view(torch.int16), out["V_out"][:n_rows].view(torch.int16))


def test_graph_capture_and_replay():
    # A call recorded into a CUDA graph meets, at every replay, the workspace as the run before
    # left it; nothing in it is counted or carried over.  Two replays on new K / V / Q (copied
    # into the captured buffers) must each match the oracle.
    wl = synth.small_workload(H=3, G=4, W=16, seq_lens=(2600, 900), pool_kernel=5, budget=80,
                              seed=71, centroids=8)
    po, pg = params_pair(wl)
    cu = wl.cu_seqlens
    cu_list = [int(c) for c in cu]
    xs = [synth.make_layer(wl, layer, "calibrated") for layer in range(3)]
    K, V, Q = (to_dev(xs[0][k]).clone() for k in ("K", "V", "Q"))
    ws = torch.empty(binding.workspace_size(pg, wl.batch, wl.total_tokens, max(wl.seq_lens)),
                     dtype=torch.uint8, device="cuda")
    out = binding.compress_layer(K, V, Q, pg, cu_seqlens=cu_list, workspace=ws)   # outside capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(graph, stream=side):
        binding.compress_layer(K, V, Q, pg, cu_seqlens=cu_list, workspace=ws, out=out)
    H, W = wl.kv_heads, wl.window
    for x in xs[1:]:
        K.copy_(to_dev(x["K"])), V.copy_(to_dev(x["V"])), Q.copy_(to_dev(x["Q"]))
        out["status"].zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert int(out["status"].item()) == 0
        ref_s = oracle.scores(x["K"], x["V"], x["Q"], po, cu=cu)
        ref = oracle.select(ref_s["s_comp"], po, cu=cu)
        check_scores("s_comp", out["s_comp"].cpu().numpy(), ref_s["s_comp"], cu, W)
        offs = out["idx_offsets"].cpu().numpy()
        idx = out["idx"].cpu().numpy()
        check_selection(idx, offs, out["counts"].cpu().numpy(), ref, ref_s["s_comp"], cu, W, H)
        ro = out["out_row_offsets"].cpu().numpy()
        check_gather(x["K"], to_bits(out["K_out"]), ro, idx, offs, cu, W, H)
        check_gather(x["V"], to_bits(out["V_out"]), ro, idx, offs, cu, W, H)


def test_given_head_budgets_ragged():
    # static per-head budgets (rows to keep, window included) chosen outside: below the window,
    # above B, above the number of candidates of the short sequence, and everything between
    wl = synth.small_workload(H=3, G=4, W=16, seq_lens=(900, 150, 2300), pool_kernel=5,
                              budget=200, seed=51, centroids=8)
    wl = synth.replace(wl, layers=3)
    rng = np.random.default_rng(7)
    hb = rng.integers(0, 260, size=(3, wl.batch * wl.kv_heads))
    hb[0, 0], hb[0, 1], hb[1, 4], hb[2, 8] = 5, 16, 1000, 17
    run_layers_parity(wl, range(3), head_budgets=hb)
    # max pooling takes the unfused route (pooled-score sums, mix, then select + gather)
    run_layers_parity(wl, range(3), head_budgets=hb, pool_mode=1)


def test_layer_schedule_budgets():
    # budgets falling linearly with depth (same total as a uniform budget of 96 rows per head)
    n = 6
    sched = binding.layer_budget_schedule(n, 96, 32, 600)
    assert sched == oracle.layer_budget_schedule(n, 96, 32, 600) and sum(sched) == n * 96
    wl = synth.small_workload(H=4, G=7, W=32, seq_lens=(4096,), pool_kernel=7, budget=sched[0],
                              seed=52, centroids=16)
    wl = synth.replace(wl, layers=n)
    hb = np.repeat(np.asarray(sched)[:, None], wl.kv_heads, axis=1)
    out = run_layers_parity(wl, range(n), head_budgets=hb, check=(0, 3, 5))
    kept = out["out_row_offsets"][:, -1].cpu().numpy()
    assert kept.tolist() == [wl.kv_heads * b for b in sched]


def test_bounded_wait_reports_timeout_and_context_survives():
    # a wait that nothing satisfies ends by itself after the limit, the status word says so,
    # and the next call on the same context works
    status, seconds = binding.selftest_bounded_wait()
    assert status == -5 and binding.status_string(status) == "device-side bounded wait expired"
    assert 1.5 < seconds < 4.0
    wl = synth.small_workload(H=2, G=2, W=16, seq_lens=(600,), pool_kernel=5, budget=64, seed=81)
    run_layer_parity(wl, variant="literal")
