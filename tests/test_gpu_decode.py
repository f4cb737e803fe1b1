"""GPU parity of mixkv_decode_attention (one query token over the compact cache) against the
plain fp64 definition.  The compact caches fed to the kernel are built by the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from oracle import decode_plain
from paper_2510_20707_b200 import binding, synth
from parity import params_pair

pytestmark = pytest.mark.gpu
RTOL, ATOL = 2e-4, 2e-5   # fp32 accumulation of exact bf16 products, weights carried as two bf16


def bits_to_dev(a):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda().view(torch.bfloat16)


def run(wl, n_layers, **kw):
    po, _ = params_pair(wl, **kw)
    H, G, B = wl.kv_heads, wl.gqa_ratio, po.budget
    cu = wl.cu_seqlens
    rows_cap = wl.batch * H * B
    Kc = np.zeros((n_layers, rows_cap, 128), np.uint16)
    Vc = np.zeros_like(Kc)
    offs = np.zeros((n_layers, wl.batch * H + 1), np.int32)
    rng = np.random.default_rng(wl.seed)
    q = synth.f32_to_bf16_bits(rng.standard_normal((n_layers, wl.batch, H * G, 128)).astype(np.float32))
    refs = []
    for l in range(n_layers):
        x = synth.make_layer(wl, l, "calibrated")
        c = oracle.compress_layer(x["K"], x["V"], x["Q"], po, cu=None if wl.batch == 1 else cu)
        n = c["K_out"].shape[0]
        Kc[l, :n], Vc[l, :n], offs[l] = c["K_out"], c["V_out"], c["out_row_offsets"]
        refs.append(decode_plain.decode_attention(c["K_out"], c["V_out"], c["out_row_offsets"], q[l], H, G))
    most = int(np.diff(offs, axis=1).max())      # adaptive budgets may give a head more than B rows
    out = binding.decode_attention(bits_to_dev(Kc), bits_to_dev(Vc), torch.from_numpy(offs).cuda(),
                                   bits_to_dev(q), H, G, max_rows=most)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    for l in range(n_layers):
        assert np.allclose(got[l], refs[l], rtol=RTOL, atol=ATOL), f"layer {l}"
    return got


def test_fixed_budget_cache_gqa7():
    wl = synth.small_workload(H=4, G=7, W=32, seq_lens=(2048,), pool_kernel=7, budget=128, seed=71,
                              centroids=16)
    run(wl, 3)


def test_ragged_adaptive_cache():
    wl = synth.small_workload(H=3, G=4, W=16, seq_lens=(900, 200, 1500), pool_kernel=5, budget=96,
                              seed=72, centroids=8)
    run(synth.with_budget(wl, 96, budget_mode=1), 2)


@pytest.mark.parametrize("rows,G", [((4096, 1000, 4096, 37), 7), ((20000, 513), 4), ((256, 257), 16)])
def test_long_rows_split_over_a_cluster(rows, G):
    # heads with thousands of rows (a large budget, or a cache that was not compressed): the rows
    # of a head are dealt out 16 at a time over the warps of a cluster, each with a running
    # softmax; two layers, ragged heads (row counts that are no multiple of 16), G on both sides
    # of 8 (the second half of the 16 head slots), a sharp row so that the running reference moves
    H, NL = len(rows), 2
    rng = np.random.default_rng(sum(rows))
    cap = int(sum(rows))
    K = rng.standard_normal((NL, cap, 128)).astype(np.float32)
    V = rng.standard_normal((NL, cap, 128)).astype(np.float32)
    q = rng.standard_normal((NL, 1, H * G, 128)).astype(np.float32)
    K[0, rows[0] - 3] = 6.0 * q[0, 0, 0]          # one key far above the rest, late in head 0
    Kb, Vb, qb = (synth.f32_to_bf16_bits(a) for a in (K, V, q))
    offs = np.tile(np.concatenate([[0], np.cumsum(rows)]).astype(np.int32), (NL, 1))
    out = binding.decode_attention(bits_to_dev(Kb), bits_to_dev(Vb), torch.from_numpy(offs).cuda(),
                                   bits_to_dev(qb), H, G, max_rows=max(rows)).cpu().numpy()
    for l in range(NL):
        ref = decode_plain.decode_attention(Kb[l], Vb[l], offs[l], qb[l], H, G)
        assert np.allclose(out[l], ref, rtol=RTOL, atol=ATOL), f"layer {l}"


@pytest.mark.parametrize("G", [1, 8, 9, 13])
def test_step_edges_and_head_counts(G):
    # heads of 1, 15, 16, 17 and 33 rows (below, at and past one 16-row step) for group sizes at
    # the edges of the 8 + 8 head slots of a tile
    rows, NL = (1, 15, 16, 17, 33), 2
    H = len(rows)
    rng = np.random.default_rng(100 + G)
    cap = int(sum(rows))
    Kb, Vb, qb = (synth.f32_to_bf16_bits(rng.standard_normal(sh).astype(np.float32))
                  for sh in ((NL, cap, 128), (NL, cap, 128), (NL, 1, H * G, 128)))
    offs = np.tile(np.concatenate([[0], np.cumsum(rows)]).astype(np.int32), (NL, 1))
    out = binding.decode_attention(bits_to_dev(Kb), bits_to_dev(Vb), torch.from_numpy(offs).cuda(),
                                   bits_to_dev(qb), H, G, max_rows=max(rows)).cpu().numpy()
    for l in range(NL):
        ref = decode_plain.decode_attention(Kb[l], Vb[l], offs[l], qb[l], H, G)
        assert np.allclose(out[l], ref, rtol=RTOL, atol=ATOL), f"layer {l}"


def test_repeated_calls_are_bit_identical():
    # the steps of a head go to fixed warps and the partial results are merged in a fixed order
    # (warps through shared memory, CTAs through distributed shared memory): twenty calls on the
    # same cache give the same bits
    rows, NL, G = (3000, 517, 2048), 3, 7
    H = len(rows)
    rng = np.random.default_rng(7)
    cap = int(sum(rows))
    Kb, Vb, qb = (synth.f32_to_bf16_bits(rng.standard_normal(sh).astype(np.float32))
                  for sh in ((NL, cap, 128), (NL, cap, 128), (NL, 1, H * G, 128)))
    offs = torch.from_numpy(np.tile(np.concatenate([[0], np.cumsum(rows)]).astype(np.int32), (NL, 1))).cuda()
    K, V, q = bits_to_dev(Kb), bits_to_dev(Vb), bits_to_dev(qb)
    first = binding.decode_attention(K, V, offs, q, H, G, max_rows=max(rows))
    for _ in range(20):
        again = binding.decode_attention(K, V, offs, q, H, G, max_rows=max(rows))
        assert torch.equal(first, again)


def test_empty_head_short_rows_and_bad_arguments():
    H, G = 2, 2
    rng = np.random.default_rng(3)
    K = synth.f32_to_bf16_bits(rng.standard_normal((1, 40, 128)).astype(np.float32))
    V = synth.f32_to_bf16_bits(rng.standard_normal((1, 40, 128)).astype(np.float32))
    q = synth.f32_to_bf16_bits(rng.standard_normal((1, 1, H * G, 128)).astype(np.float32))
    offs = np.array([[0, 0, 33]], np.int32)          # head 0 keeps nothing, head 1 keeps 33 rows
    out = binding.decode_attention(bits_to_dev(K), bits_to_dev(V), torch.from_numpy(offs).cuda(),
                                   bits_to_dev(q), H, G, max_rows=64).cpu().numpy()
    ref = decode_plain.decode_attention(K[0], V[0], offs[0], q[0], H, G)
    assert np.array_equal(out[0, 0, :G], np.zeros((G, 128)))
    assert np.allclose(out[0], ref, rtol=RTOL, atol=ATOL)
    with pytest.raises(binding.MixKVError):
        binding.decode_attention(bits_to_dev(K), bits_to_dev(V), torch.from_numpy(offs).cuda(),
                                 bits_to_dev(q), H, G, max_rows=0)
