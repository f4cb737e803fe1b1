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
RTOL, ATOL = 2e-4, 2e-5   # fp32 dot products of 128 terms, approximate exp2, sums over <= B rows


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
