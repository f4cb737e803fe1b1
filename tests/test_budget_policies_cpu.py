"""Budget policies chosen outside the kernels (layer schedule, per-head budgets): the oracle's
reading pinned by its invariants, and the library's host-side schedule against it."""
import numpy as np
import pytest

import oracle
from paper_2510_20707_b200 import binding


@pytest.mark.parametrize("n,B,W,t", [(28, 256, 32, 500), (32, 512, 32, 999), (5, 100, 32, 0),
                                      (4, 65, 32, 999), (1, 64, 32, 700), (7, 97, 16, 333),
                                      (2, 33, 32, 999)])
def test_layer_schedule_invariants_and_library_agrees(n, B, W, t):
    sched = oracle.layer_budget_schedule(n, B, W, t)
    assert len(sched) == n
    assert sum(sched) == n * B                      # the total number of rows kept is unchanged
    assert all(a >= b for a, b in zip(sched, sched[1:]))   # lower layers never keep fewer
    assert all(v >= W for v in sched)               # the window is always kept
    if t == 0:
        assert sched == [B] * n
    if n > 1 and t > 0 and B - W >= 4 * n:
        assert sched[0] > sched[-1]
        # linear: the middle of the schedule sits at the uniform budget (up to rounding)
        assert abs(sched[n // 2] + sched[(n - 1) // 2] - 2 * B) <= 2
    assert binding.layer_budget_schedule(n, B, W, t) == sched


def test_layer_schedule_closed_form():
    # n = 3, B' = 100, taper 1/2: 150, 100, 50 candidates exactly
    assert oracle.layer_budget_schedule(3, 132, 32, 500) == [182, 132, 82]


def test_schedule_rejects_bad_arguments():
    for args in [(0, 64, 32, 0), (4, 32, 32, 0), (4, 64, 32, 1000), (4, 64, 32, -1)]:
        with pytest.raises(binding.MixKVError):
            binding.layer_budget_schedule(*args)


def test_select_given_reduces_to_fixed_and_clamps():
    rng = np.random.default_rng(3)
    H, W = 3, 8
    cu = [0, 50, 120]
    s = rng.standard_normal((H, 120 - 2 * W)).astype(np.float32)
    p = oracle.Params(kv_heads=H, gqa_ratio=1, window=W, budget=20)
    fixed = oracle.select(s, p, cu=cu)
    same = oracle.select_given(s, np.full((2, H), 20), p, cu=cu)
    for k in ("idx", "counts", "idx_offsets"):
        assert np.array_equal(fixed[k], same[k]), k
    # budgets below the window keep the window only; budgets above B are cut to B
    g = oracle.select_given(s, [[3, 8, 9], [1000, 20, 13]], p, cu=cu)
    assert g["counts"].tolist() == [[0, 0, 1], [12, 12, 5]]
    # brute force for one head
    P1 = 120 - 50 - W
    col0 = 50 - W
    want = np.sort(np.argsort(-s[2, col0:col0 + P1], kind="stable")[:5])
    got = g["idx"][g["idx_offsets"][5]:g["idx_offsets"][6]]
    assert np.array_equal(got, want)
