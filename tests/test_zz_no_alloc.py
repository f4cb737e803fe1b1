"""The no-allocation entry point, mixkv_scores_static, against mixkv_scores.

Some users of the library cannot hand it a workspace: an engine that gave all free HBM to
its own KV pool at start-up, a plug-in inside another program's step loop where cudaMalloc
would stall the device, a binding without an allocator.  For them the library carries a
fixed scratch array of its own.  This file checks, through the C ABI, that scoring with that
built-in scratch gives bit for bit what scoring with a caller workspace gives (the same
kernels run in the same order, only the scratch address differs) and agrees with the CPU
oracle, on two calls in a row (the second on a different, shorter problem, so stale contents
of the shared array from the first call would show), and that a problem too large for the
array is refused with its own status code.  It is collected last on purpose: a run that
stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_20707_b200 import binding, synth
from parity import check_rbar, check_scores, params_pair, to_dev

pytestmark = pytest.mark.gpu


def _both(wl, variant):
    x = synth.make_layer(wl, 0, variant)
    po, pg = params_pair(wl)
    K, V, Q = to_dev(x["K"]), to_dev(x["V"]), to_dev(x["Q"])
    cu = None if wl.batch == 1 else [int(c) for c in wl.cu_seqlens]
    ref = binding.scores(K, V, Q, pg, cu_seqlens=cu)
    torch.cuda.synchronize()
    got = binding.scores_static(K, V, Q, pg, cu_seqlens=cu)
    torch.cuda.synchronize()
    assert int(got["status"].item()) == 0 and int(ref["status"].item()) == 0
    for name in ("s_ex", "s_div", "s_comp", "rbar"):
        assert torch.equal(got[name], ref[name]), name
    want = oracle.scores(x["K"], x["V"], x["Q"], po, cu=None if wl.batch == 1 else wl.cu_seqlens)
    for name in ("s_ex", "s_div", "s_comp"):
        check_scores(name, got[name].cpu().numpy(), want[name], wl.cu_seqlens, wl.window)
    check_rbar(got["rbar"].cpu().numpy(), want["rbar"].astype(np.float64))


def test_static_scratch_matches_workspace_on_two_calls_in_a_row():
    first = synth.small_workload(H=3, G=2, W=16, seq_lens=(1500, 333), pool_kernel=7, budget=64,
                                 seed=21)
    second = synth.small_workload(H=2, G=4, W=32, seq_lens=(777,), pool_kernel=5, budget=96,
                                  seed=22)
    _both(first, "calibrated")
    _both(second, "literal")


def test_too_large_for_the_static_scratch_is_refused():
    # 8 heads x 64k tokens needs far more than the built-in array; nothing may be enqueued
    H, L = 8, 65536
    pg = binding.Params(kv_heads=H, gqa_ratio=4, budget=256)
    K = torch.zeros((H, L, 128), dtype=torch.bfloat16, device="cuda")
    Q = torch.zeros((1, H * 4, 32, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.MixKVError) as e:
        binding.scores_static(K, K, Q, pg)
    assert e.value.status == -6
    assert "scratch" in binding.status_string(-6)
