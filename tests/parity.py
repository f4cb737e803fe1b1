"""Comparison rules between the CUDA library and the CPU oracle.

Tolerances (fp32 accumulation from bf16 inputs, as the library computes):
  scores     |gpu - ref| <= 2e-3 * max(|ref_i|, mean_i |ref|) per (sequence, head).  The
             mean term is needed because the min-max normalisations of Sec. 3.2 / 3.3 make
             some scores exactly zero, where a relative error is undefined.
  rbar       |gpu - ref| <= 2e-3 * |ref| + 1e-5
  indices    identical sets, except positions whose oracle score lies within
             2 * 2e-3 * max(|tau|, mean |ref|) of the oracle's threshold score tau (the
             b-th largest): there both answers are correct.
  K/V rows   bit-exact against a gather by the library's own indices.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2510_20707_b200 import binding, synth

REL = 2e-3


def to_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def to_bits(t: torch.Tensor) -> np.ndarray:
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def params_pair(wl: synth.Workload, **kw):
    base = dict(kv_heads=wl.kv_heads, gqa_ratio=wl.gqa_ratio, window=wl.window,
                pool_kernel=wl.pool_kernel, budget=wl.budget, budget_mode=wl.budget_mode,
                ada_floor=wl.ada_floor)
    base.update(kw)
    return oracle.Params(**base), binding.Params(**base)


def seq_slices(wl_cu, W, batch):
    """(prefix offset, P) of every sequence inside the [H, Ptot] score layout."""
    return [(int(wl_cu[b]) - b * W, int(wl_cu[b + 1] - wl_cu[b]) - W) for b in range(batch)]


def check_scores(name, gpu: np.ndarray, ref: np.ndarray, cu, W, rel=REL):
    batch = len(cu) - 1
    for b, (po, P) in enumerate(seq_slices(cu, W, batch)):
        for h in range(ref.shape[0]):
            r = ref[h, po:po + P].astype(np.float64)
            g = gpu[h, po:po + P].astype(np.float64)
            tol = rel * np.maximum(np.abs(r), np.abs(r).mean())
            bad = np.abs(g - r) > tol
            assert not bad.any(), (
                f"{name}: seq {b} head {h}: {bad.sum()} of {P} outside tolerance; worst at "
                f"{np.argmax(np.abs(g - r) / np.maximum(tol, 1e-300))}: gpu {g[np.argmax(np.abs(g - r))]} "
                f"ref {r[np.argmax(np.abs(g - r))]}")


def check_rbar(gpu: np.ndarray, ref: np.ndarray, rel=REL):
    assert np.all(np.abs(gpu.astype(np.float64) - ref) <= rel * np.abs(ref) + 1e-5), (gpu, ref)


def check_selection(gpu_idx, gpu_offsets, gpu_counts, ref, ref_scores, cu, W, H, rel=REL,
                    counts_slack=None):
    """Index sets per (b, h) against the oracle's, allowing swaps only at near-ties."""
    batch = len(cu) - 1
    ro = ref["idx_offsets"]
    for b, (po, P) in enumerate(seq_slices(cu, W, batch)):
        for h in range(H):
            bh = b * H + h
            g = gpu_idx[gpu_offsets[bh]:gpu_offsets[bh + 1]]
            r = ref["idx"][ro[bh]:ro[bh + 1]]
            assert g.size == gpu_counts[bh]
            assert (np.diff(g) > 0).all() and (g.size == 0 or (g.min() >= 0 and g.max() < P))
            if counts_slack is None:
                assert g.size == r.size, f"count mismatch seq {b} head {h}: {g.size} vs {r.size}"
            else:
                assert abs(g.size - r.size) <= counts_slack
            s = ref_scores[h, po:po + P].astype(np.float64)
            if r.size == 0 or r.size == P:
                assert g.size == r.size
                continue
            tau = np.sort(s)[::-1][min(r.size, g.size) - 1]
            band = 2 * rel * max(abs(tau), np.abs(s).mean())
            diff = np.setxor1d(g, r)
            assert np.all(np.abs(s[diff] - tau) <= band), (
                f"seq {b} head {h}: {diff.size} differing indices, "
                f"{np.sum(np.abs(s[diff] - tau) > band)} of them outside the tie band")


def check_gather(Kbits, out_bits, row_offsets, idx, idx_offsets, cu, W, H):
    """Rows of the compact cache are bit-exact copies of the selected rows, then the window."""
    batch = len(cu) - 1
    for b in range(batch):
        L = int(cu[b + 1] - cu[b])
        for h in range(H):
            bh = b * H + h
            sel = idx[idx_offsets[bh]:idx_offsets[bh + 1]]
            keep = np.concatenate([sel, np.arange(L - W, L)]) + int(cu[b])
            got = out_bits[row_offsets[bh]:row_offsets[bh + 1]]
            assert got.shape[0] == keep.size
            assert np.array_equal(got, Kbits[h, keep]), f"gather mismatch seq {b} head {h}"


def run_layer_parity(wl: synth.Workload, layer: int = 0, variant: str = "literal", **kw):
    """Full compress_layer on the GPU against the oracle.  Returns both results."""
    x = synth.make_layer(wl, layer, variant)
    po, pg = params_pair(wl, **kw)
    cu = wl.cu_seqlens
    cu_arg = None if wl.batch == 1 else cu
    ref_s = oracle.scores(x["K"], x["V"], x["Q"], po, cu=cu_arg)
    ref = oracle.select(ref_s["s_comp"], po, cu=cu_arg)
    K, V, Q = to_dev(x["K"]), to_dev(x["V"]), to_dev(x["Q"])
    cu_list = None if wl.batch == 1 else [int(c) for c in cu]
    gs = binding.scores(K, V, Q, pg, cu_seqlens=cu_list)
    out = binding.compress_layer(K, V, Q, pg, cu_seqlens=cu_list)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0 and int(gs["status"].item()) == 0
    H, W = wl.kv_heads, wl.window
    check_rbar(gs["rbar"].cpu().numpy(), ref_s["rbar"].astype(np.float64))
    check_scores("s_ex", gs["s_ex"].cpu().numpy(), ref_s["s_ex"], cu, W)
    check_scores("s_div", gs["s_div"].cpu().numpy(), ref_s["s_div"], cu, W)
    check_scores("s_comp", gs["s_comp"].cpu().numpy(), ref_s["s_comp"], cu, W)
    assert torch.equal(gs["s_comp"], out["s_comp"]), "scores differ between the two entry points"
    offs = out["idx_offsets"].cpu().numpy()
    idx = out["idx"].cpu().numpy()
    counts = out["counts"].cpu().numpy()
    slack = None if po.budget_mode == 0 else 2
    check_selection(idx, offs, counts, ref, ref_s["s_comp"], cu, W, H, counts_slack=slack)
    ro = out["out_row_offsets"].cpu().numpy()
    assert np.array_equal(ro, offs + np.arange(wl.batch * H + 1) * W)
    check_gather(x["K"], to_bits(out["K_out"]), ro, idx, offs, cu, W, H)
    check_gather(x["V"], to_bits(out["V_out"]), ro, idx, offs, cu, W, H)
    return out, ref, ref_s


def check_layer_properties(out, n, K, V, wl, Bp, adaptive):
    """What holds for every layer of a call whatever the scores are (used for the layers the
    oracle does not recompute): counts within their bounds (and summing to the sequence's
    total under adaptive budgets), offsets = prefix sums, indices strictly ascending inside
    the candidates, and every output row a bit-exact copy of the row its index names, the W
    window rows last."""
    H, W, cu = wl.kv_heads, wl.window, wl.cu_seqlens
    counts = out["counts"][n].cpu().numpy()
    offs = out["idx_offsets"][n].cpu().numpy()
    ro = out["out_row_offsets"][n].cpu().numpy()
    idx = out["idx"][n].cpu().numpy()
    assert np.array_equal(offs, np.concatenate([[0], np.cumsum(counts)]))
    assert np.array_equal(ro, offs + np.arange(wl.batch * H + 1) * W)
    rows = []
    for b in range(wl.batch):
        P = int(cu[b + 1] - cu[b]) - W
        c = counts[b * H:(b + 1) * H]
        assert (c >= 0).all() and (c <= P).all()
        if adaptive is True:
            assert c.sum() == min(H * Bp, H * P) or (c == P).any()
        elif adaptive is False:
            assert (c == min(Bp, P)).all()
        for h in range(H):
            g = idx[offs[b * H + h]:offs[b * H + h + 1]]
            assert (np.diff(g) > 0).all() and (g.size == 0 or (g.min() >= 0 and g.max() < P))
            rows.append(torch.from_numpy(
                np.concatenate([g, np.arange(P, P + W)]).astype(np.int64) + int(cu[b])
                + h * int(cu[-1])))
    src = torch.cat(rows).cuda()
    n_rows = int(ro[-1])
    assert src.numel() == n_rows
    for X, Xo in ((K, out["K_out"]), (V, out["V_out"])):
        flat = X[n].reshape(-1, 128).view(torch.int16)      # rows (h, position) of this layer
        assert torch.equal(Xo[n][:n_rows].view(torch.int16), flat[src])


def run_layers_parity(wl: synth.Workload, layers, variant: str = "calibrated", pad_rows: int = 0,
                      check=None, head_budgets=None, properties=False, **kw):
    """mixkv_compress_layers over several layers at once against the oracle, layer by layer
    (only the positions listed in `check`, if given).  pad_rows > 0 leaves a gap between the
    layers of K / V (a strided layer dimension).  head_budgets (array [len(layers), batch*H],
    rows to keep per head, window included) takes the budgeted entry point and the oracle's
    select_given.  properties=True also checks every layer of the call by the properties
    that need no oracle (check_layer_properties)."""
    po, pg = params_pair(wl, **kw)
    cu = wl.cu_seqlens
    cu_arg = None if wl.batch == 1 else cu
    cu_list = None if wl.batch == 1 else [int(c) for c in cu]
    xs = [synth.make_layer(wl, l, variant) for l in layers]
    H, W, NL = wl.kv_heads, wl.window, len(xs)
    Ltot = wl.total_tokens

    def stack(name):
        t = torch.stack([to_dev(x[name]) for x in xs])
        if pad_rows and name != "Q":
            buf = torch.zeros((NL, H * Ltot + pad_rows, 128), dtype=torch.bfloat16, device="cuda")
            buf[:, :H * Ltot] = t.reshape(NL, H * Ltot, 128)
            t = buf[:, :H * Ltot].view(NL, H, Ltot, 128)
        return t

    K, V, Q = stack("K"), stack("V"), stack("Q")
    hb_dev = None
    if head_budgets is not None:
        head_budgets = np.asarray(head_budgets, dtype=np.int32).reshape(NL, wl.batch * H)
        hb_dev = torch.from_numpy(head_budgets).cuda()
    out = binding.compress_layers(K, V, Q, pg, cu_seqlens=cu_list, head_budgets=hb_dev)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    for n, x in enumerate(xs):
        if properties:
            check_layer_properties(out, n, K, V, wl, po.budget - W,
                                   None if head_budgets is not None else po.budget_mode == 1)
        if check is not None and n not in check:
            continue
        ref_s = oracle.scores(x["K"], x["V"], x["Q"], po, cu=cu_arg)
        if head_budgets is None:
            ref = oracle.select(ref_s["s_comp"], po, cu=cu_arg)
        else:
            ref = oracle.select_given(ref_s["s_comp"], head_budgets[n], po, cu=cu)
            assert np.array_equal(out["counts"][n].cpu().numpy().reshape(wl.batch, H),
                                  ref["counts"])
        check_scores(f"s_comp[layer {n}]", out["s_comp"][n].cpu().numpy(), ref_s["s_comp"], cu, W)
        offs = out["idx_offsets"][n].cpu().numpy()
        idx = out["idx"][n].cpu().numpy()
        counts = out["counts"][n].cpu().numpy()
        slack = None if po.budget_mode == 0 else 2
        check_selection(idx, offs, counts, ref, ref_s["s_comp"], cu, W, H, counts_slack=slack)
        ro = out["out_row_offsets"][n].cpu().numpy()
        assert np.array_equal(ro, offs + np.arange(wl.batch * H + 1) * W)
        check_gather(x["K"], to_bits(out["K_out"][n]), ro, idx, offs, cu, W, H)
        check_gather(x["V"], to_bits(out["V_out"][n]), ro, idx, offs, cu, W, H)
    return out
