"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol
the header declares, sizes workspaces and rejects bad arguments before touching CUDA."""
import ctypes as C
import os
import re

import pytest

from paper_2510_20707_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "mixkv.h")).read()
    declared = set(re.findall(r"\b(mixkv_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_status_strings(lib):
    assert binding.status_string(0) == "ok"
    assert "workspace" in binding.status_string(-3)
    assert "unknown" in binding.status_string(-99)


def test_default_params(lib):
    p = binding._CParams()
    lib.mixkv_default_params(C.byref(p), 4, 7, 128)
    assert (p.kv_heads, p.gqa_ratio, p.head_dim, p.window, p.pool_kernel, p.budget) == (4, 7, 128, 32, 7, 128)
    assert p.use_vnorm == 1 and p.mix_mode == 0 and abs(p.eps - 1e-6) < 1e-12


def test_workspace_size_grows_with_tokens():
    p = binding.Params(kv_heads=4, gqa_ratio=7, budget=128)
    a = binding.workspace_size(p, 1, 4096, 4096)
    b = binding.workspace_size(p, 1, 32768, 32768)
    c = binding.workspace_size(p, 8, 40960, 8192)
    assert 0 < a < b < c < 64 << 20


@pytest.mark.parametrize("kw,status", [
    (dict(pool_kernel=4), -1), (dict(budget=32), -1), (dict(budget=8), -1),
    (dict(head_dim=64), -2), (dict(gqa_ratio=8), -2), (dict(window=24, gqa_ratio=1), -2),
    (dict(mix_mode=7), -1), (dict(ada_floor=1.5), -1), (dict(kv_heads=0), -1),
])
def test_bad_params_are_rejected(kw, status):
    base = dict(kv_heads=4, gqa_ratio=7, budget=64)
    base.update(kw)
    with pytest.raises(binding.MixKVError) as e:
        binding.workspace_size(binding.Params(**base), 1, 1024, 1024)
    assert e.value.status == status


def test_entry_points_validate_before_any_cuda_call(lib):
    # null tensors, short sequences, bad offsets, small workspace: all host-side errors
    p = binding.Params(kv_heads=4, gqa_ratio=7, budget=64).c()
    ws = C.create_string_buffer(1 << 20)
    wsp = C.cast(ws, C.c_void_p).value
    wsp = (wsp + 255) // 256 * 256
    one = C.c_void_p(256)  # a non-null, aligned fake pointer; never dereferenced on error paths
    args = lambda L, wbytes, cu=None, batch=1: (one, one, one, cu, batch, L, C.byref(p), wsp, wbytes,
                                                None, one, one, one, None, None, None, None, None, None)
    assert lib.mixkv_compress_layer(*args(32, 1 << 19)) == -1           # L <= W
    assert lib.mixkv_compress_layer(*args(1024, 1024)) == -3            # workspace too small
    cu = (C.c_int32 * 3)(0, 500, 400)
    assert lib.mixkv_compress_layer(*args(0, 1 << 19, cu, 2)) == -1     # offsets not ascending
    assert lib.mixkv_compress_layer(*args(1024, 1 << 19, None, 2)) == -1  # batch > 1 needs offsets
    assert lib.mixkv_scores(None, one, one, None, 1, 1024, C.byref(p), wsp, 1 << 19, one, None,
                            None, None, None, None, None) == -1
    assert lib.mixkv_select(None, None, 1, 1024, C.byref(p), wsp, 1 << 19, one, one, one, None,
                            None) == -1


def test_stage_names_follow_the_route(lib):
    p = binding.Params(kv_heads=4, gqa_ratio=7, budget=256)
    assert binding.stage_names_for(p, 28, 1, 32768) == ["pass1", "pass2", "tail"]
    # one head-layer of 140000 candidates does not fit the tail kernel's shared memory
    assert binding.stage_names_for(p, 1, 1, 140032) == ["pass1", "pass2", "mixpool", "tail"]
    # 112 units of 65504 candidates: too long for one CTA per head, clusters of eight keep them
    assert binding.stage_names_for(p, 28, 1, 65536) == ["pass1", "pass2", "tail"]
    pa = binding.Params(kv_heads=4, gqa_ratio=7, budget=128, budget_mode=1)
    assert binding.stage_names_for(pa, 28, 8, 8192) == ["pass1", "pass2", "mixpool", "budget", "tail"]
    assert binding.stage_names(p) == ["pass1", "pass2", "tail"]


def test_device_check_without_a_device_or_with_one(lib):
    # no GPU here: the query fails and the entry point says so; on a B200 it reports 10.x
    import torch
    rc, major = binding.device_check()
    if torch.cuda.is_available():
        assert (rc, major) == (0, 10)
    else:
        assert rc == -4 and major == 0
