"""The seeded input generators: shapes, determinism, and the key statistics the paper
quotes for its workloads (Sec. 1 / Fig. 1-2: mean key cosine 0.2-0.4 for text keys,
0.6-0.8 for vision keys, heads spread from below 0.3 to above 0.9)."""
import numpy as np

import oracle
from paper_2510_20707_b200 import synth


def test_shapes_and_determinism():
    for name in ("C1", "C2"):
        wl = synth.CONFIGS[name]
        a, b = synth.make_layer(wl, 0), synth.make_layer(wl, 0)
        assert a["K"].shape == (wl.kv_heads, wl.total_tokens, 128) and a["K"].dtype == np.uint16
        assert a["V"].shape == a["K"].shape
        assert a["Q"].shape == (wl.batch, wl.kv_heads * wl.gqa_ratio, wl.window, 128)
        assert all(np.array_equal(a[k], b[k]) for k in a)
    c = synth.make_layer(synth.CONFIGS["C2"], 1)
    assert not np.array_equal(c["K"], synth.make_layer(synth.CONFIGS["C2"], 0)["K"])


def test_config_table_matches_the_stated_workloads():
    C = synth.CONFIGS
    assert C["C1"].seq_lens == (1024,) and C["C1"].budget == 64 and C["C1"].vision_tokens == (896,)
    assert C["C2"].layers == 28 and C["C2"].seq_lens == (4096,) and C["C2"].budget == 128
    assert C["C3"].seq_lens == (32768,) and C["C3"].budget == 256 and C["C3b"].budget == 512
    assert C["C3"].frames * C["C3"].frame_tokens + 256 == 32768
    assert C["C4"].batch == 8 and C["C4"].budget_mode == 1
    assert all(2048 <= L <= 8192 for L in C["C4"].seq_lens)
    assert all(0.6 <= v / L <= 0.9 for v, L in zip(C["C4"].vision_tokens, C["C4"].seq_lens))
    assert C["C5"].kv_heads == 8 and C["C5"].gqa_ratio == 4 and C["C5"].layers == 32
    assert C["C4"].cu_seqlens[-1] == C["C4"].total_tokens


def test_calibrated_variants_reach_the_quoted_cosine_bands():
    x = synth.make_layer(synth.CONFIGS["C1"], 0, "calibrated")
    r = [oracle.key_geometry(x["K"][h])[1] for h in range(4)]
    assert r[0] < 0.35 and 0.6 < r[2] < 0.8 and r[3] > 0.85
    lit = synth.make_layer(synth.CONFIGS["C1"], 0, "literal")
    assert all(oracle.key_geometry(lit["K"][h])[1] < 0.1 for h in range(4))
    wl = synth.small_workload(H=8, G=1, W=8, seq_lens=(2048,), kind="text")
    t = synth.make_layer(wl, 0, "calibrated")
    rt = [oracle.key_geometry(t["K"][h])[1] for h in range(8)]
    assert 0.17 < rt[0] < 0.23 and 0.37 < rt[7] < 0.43


def test_shared_offset_leaves_the_window_softmax_almost_unchanged():
    wl = synth.small_workload(H=1, G=2, W=8, seq_lens=(300,), centroids=8)
    a, b = synth.make_layer(wl, 0, "literal"), synth.make_layer(wl, 0, "calibrated")
    sa, _ = oracle.window_attention(a["K"][0], a["Q"][0])
    sb, _ = oracle.window_attention(b["K"][0], b["Q"][0])
    # identical up to the bf16 rounding of the shifted keys
    assert np.corrcoef(sa[:292], sb[:292])[0, 1] > 0.99


def test_c1_oracle_selection_has_not_drifted():
    import os
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "c1_oracle_selection.txt")
    rows = [np.array(l.split(), dtype=np.int64) for l in open(path) if not l.startswith("#")]
    wl = synth.CONFIGS["C1"]
    x = synth.make_layer(wl, 0, "literal")
    p = oracle.Params(kv_heads=4, gqa_ratio=7, budget=64)
    out = oracle.compress_layer(x["K"], x["V"], x["Q"], p)
    io = out["idx_offsets"]
    for h in range(4):
        assert np.array_equal(out["idx"][io[h]:io[h + 1]], rows[h])
