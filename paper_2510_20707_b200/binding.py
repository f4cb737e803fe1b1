"""ctypes binding of the MixKV C ABI (``include/mixkv.h``).

Argument marshalling only: every function hands device pointers of torch tensors to the
library entry point of the same name and returns the tensors it filled.  No arithmetic of
the method happens here, and nothing falls back to PyTorch ops or the CPU: if
``libmixkv.so`` is missing, :func:`load_library` raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Dict, Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libmixkv.so")

EXPORTS = ("mixkv_default_params", "mixkv_workspace_size", "mixkv_scores", "mixkv_select",
           "mixkv_compress_layer", "mixkv_compress_layer_traced", "mixkv_launches_per_layer",
           "mixkv_stage_name", "mixkv_status_string", "mixkv_scores_static",
           "mixkv_workspace_size_layers", "mixkv_compress_layers",
           "mixkv_compress_layers_budgeted", "mixkv_layer_budget_schedule",
           "mixkv_similarity_workspace_size", "mixkv_similarity_map", "mixkv_decode_attention",
           "mixkv_selftest_bounded_wait", "mixkv_launches_for", "mixkv_stage_name_for",
           "mixkv_device_check")


class MixKVError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: {status_string(status)} ({status})")
        self.status = status


class _CParams(C.Structure):
    _fields_ = [("kv_heads", C.c_int32), ("gqa_ratio", C.c_int32), ("head_dim", C.c_int32),
                ("window", C.c_int32), ("pool_kernel", C.c_int32), ("pool_mode", C.c_int32),
                ("use_vnorm", C.c_int32), ("mix_mode", C.c_int32), ("budget_mode", C.c_int32),
                ("budget", C.c_int32), ("ada_floor", C.c_float), ("eps", C.c_float),
                ("softmax_scale", C.c_float)]


@dataclass
class Params:
    """Mirror of ``mixkv_params`` (see include/mixkv.h for the meaning of each field)."""
    kv_heads: int
    gqa_ratio: int
    head_dim: int = 128
    window: int = 32
    pool_kernel: int = 7
    pool_mode: int = 0
    use_vnorm: int = 1
    mix_mode: int = 0
    budget_mode: int = 0
    budget: int = 64
    ada_floor: float = 0.2
    eps: float = 1e-6
    softmax_scale: float = 0.0

    def c(self) -> _CParams:
        return _CParams(self.kv_heads, self.gqa_ratio, self.head_dim, self.window,
                        self.pool_kernel, self.pool_mode, self.use_vnorm, self.mix_mode,
                        self.budget_mode, self.budget, self.ada_floor, self.eps,
                        self.softmax_scale)


_lib: Optional[C.CDLL] = None


def load_library() -> C.CDLL:
    """Loads libmixkv.so from the package directory; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} not found: build it with `python -m paper_2510_20707_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        lib = C.CDLL(LIB_PATH)
        vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
        lib.mixkv_status_string.restype = C.c_char_p
        lib.mixkv_status_string.argtypes = [C.c_int]
        lib.mixkv_default_params.restype = None
        lib.mixkv_default_params.argtypes = [C.POINTER(_CParams), i32, i32, i32]
        lib.mixkv_workspace_size.argtypes = [C.POINTER(_CParams), i32, C.c_int64, i32,
                                             C.POINTER(sz)]
        lib.mixkv_workspace_size_layers.argtypes = [C.POINTER(_CParams), i32, i32, C.c_int64, i32,
                                                    C.POINTER(sz)]
        lib.mixkv_launches_per_layer.argtypes = [C.POINTER(_CParams)]
        lib.mixkv_launches_for.argtypes = [C.POINTER(_CParams), i32, i32, i32]
        lib.mixkv_stage_name_for.argtypes = [C.POINTER(_CParams), i32, i32, i32, i32]
        lib.mixkv_stage_name_for.restype = C.c_char_p
        lib.mixkv_device_check.argtypes = [C.POINTER(i32)]
        lib.mixkv_scores.argtypes = [vp, vp, vp, C.POINTER(i32), i32, i32, C.POINTER(_CParams),
                                     vp, sz, vp, vp, vp, vp, vp, vp, vp]
        lib.mixkv_scores_static.argtypes = [vp, vp, vp, C.POINTER(i32), i32, i32,
                                            C.POINTER(_CParams), vp, vp, vp, vp, vp, vp, vp]
        lib.mixkv_select.argtypes = [vp, C.POINTER(i32), i32, i32, C.POINTER(_CParams), vp, sz,
                                     vp, vp, vp, vp, vp]
        lib.mixkv_compress_layer.argtypes = [vp, vp, vp, C.POINTER(i32), i32, i32,
                                             C.POINTER(_CParams), vp, sz, vp, vp, vp, vp, vp, vp,
                                             vp, vp, vp, vp]
        lib.mixkv_compress_layer_traced.argtypes = lib.mixkv_compress_layer.argtypes + [
            C.POINTER(vp), i32]
        lib.mixkv_compress_layers.argtypes = [vp, vp, vp, i32, C.c_int64, C.c_int64,
                                              C.POINTER(i32), i32, i32, C.POINTER(_CParams), vp,
                                              sz, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp,
                                              C.POINTER(vp), i32]
        lib.mixkv_compress_layers_budgeted.argtypes = [
            vp, vp, vp, i32, C.c_int64, C.c_int64, C.POINTER(i32), i32, i32, C.POINTER(_CParams),
            vp, sz, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.mixkv_layer_budget_schedule.argtypes = [i32, i32, i32, i32, C.POINTER(i32)]
        lib.mixkv_similarity_workspace_size.argtypes = [i32, i32, i32, C.POINTER(sz)]
        lib.mixkv_similarity_map.argtypes = [vp, i32, i32, i32, i32, vp, sz, vp, vp, vp]
        lib.mixkv_decode_attention.argtypes = [vp, vp, vp, C.c_int64, vp, i32, i32, i32, i32, i32,
                                               C.c_float, i32, vp, vp]
        lib.mixkv_selftest_bounded_wait.argtypes = [vp, vp, vp]
        lib.mixkv_stage_name.restype = C.c_char_p
        lib.mixkv_stage_name.argtypes = [C.POINTER(_CParams), i32]
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load_library().mixkv_status_string(int(status)).decode()


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous(), "tensors handed to the library must be contiguous"
    return t.data_ptr()


def _cu_array(cu: Optional[Sequence[int]]):
    if cu is None:
        return None, 1
    arr = (C.c_int32 * len(cu))(*[int(x) for x in cu])
    return arr, len(cu) - 1


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def workspace_size(params: Params, batch: int, total_tokens: int, max_seq_len: int) -> int:
    out = C.c_size_t(0)
    pc = params.c()
    rc = load_library().mixkv_workspace_size(C.byref(pc), batch, total_tokens, max_seq_len,
                                             C.byref(out))
    if rc != 0:
        raise MixKVError(rc, "mixkv_workspace_size")
    return int(out.value)


def workspace_size_layers(params: Params, n_layers: int, batch: int, total_tokens: int,
                          max_seq_len: int) -> int:
    out = C.c_size_t(0)
    pc = params.c()
    rc = load_library().mixkv_workspace_size_layers(C.byref(pc), n_layers, batch, total_tokens,
                                                    max_seq_len, C.byref(out))
    if rc != 0:
        raise MixKVError(rc, "mixkv_workspace_size_layers")
    return int(out.value)


def launches_per_layer(params: Params) -> int:
    pc = params.c()
    return int(load_library().mixkv_launches_per_layer(C.byref(pc)))


def stage_names(params: Params):
    pc = params.c()
    lib = load_library()
    return [lib.mixkv_stage_name(C.byref(pc), i).decode() for i in range(launches_per_layer(params))]


def stage_names_for(params: Params, n_layers: int, batch: int, max_seq_len: int):
    """Names of the kernels a call of this shape enqueues (mixkv_launches_for /
    mixkv_stage_name_for): the route depends on the longest sequence and the number of units."""
    pc = params.c()
    lib = load_library()
    n = int(lib.mixkv_launches_for(C.byref(pc), n_layers, batch, max_seq_len))
    return [lib.mixkv_stage_name_for(C.byref(pc), n_layers, batch, max_seq_len, i).decode()
            for i in range(n)]


def device_check():
    """mixkv_device_check: (status, major compute capability of the current device)."""
    major = C.c_int32(0)
    rc = int(load_library().mixkv_device_check(C.byref(major)))
    return rc, int(major.value)


def _workspace(params, cu, Ltot, device, workspace):
    batch = 1 if cu is None else len(cu) - 1
    max_len = Ltot if cu is None else max(int(cu[b + 1]) - int(cu[b]) for b in range(batch))
    need = workspace_size(params, batch, Ltot, max_len)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=device)
    return workspace, batch


def scores(K: torch.Tensor, V: Optional[torch.Tensor], Q: torch.Tensor, params: Params,
           cu_seqlens: Optional[Sequence[int]] = None, rbar_in: Optional[torch.Tensor] = None,
           workspace: Optional[torch.Tensor] = None, stream=None,
           want_parts: bool = True) -> Dict[str, torch.Tensor]:
    """mixkv_scores: K, V [H, Ltot, 128] bf16, Q [batch, H*G, W, 128] bf16 (device tensors)."""
    H, Ltot, d = K.shape
    workspace, batch = _workspace(params, cu_seqlens, Ltot, K.device, workspace)
    Ptot = Ltot - batch * params.window
    f32 = dict(dtype=torch.float32, device=K.device)
    out = {"s_comp": torch.empty((H, Ptot), **f32)}
    if want_parts:
        out["s_ex"] = torch.empty((H, Ptot), **f32)
        out["s_div"] = torch.empty((H, Ptot), **f32)
        out["rbar"] = torch.empty((batch, H), **f32)
    status = torch.zeros(1, dtype=torch.int32, device=K.device)
    cu, _ = _cu_array(cu_seqlens)
    pc = params.c()
    rc = load_library().mixkv_scores(
        _ptr(K), _ptr(V), _ptr(Q), cu, batch, Ltot, C.byref(pc), _ptr(workspace),
        workspace.numel(), _ptr(out["s_comp"]), _ptr(out.get("s_ex")), _ptr(out.get("s_div")),
        _ptr(out.get("rbar")), _ptr(rbar_in), _ptr(status), _stream(stream))
    if rc != 0:
        raise MixKVError(rc, "mixkv_scores")
    out["status"] = status
    return out


def scores_static(K: torch.Tensor, V: Optional[torch.Tensor], Q: torch.Tensor, params: Params,
                  cu_seqlens: Optional[Sequence[int]] = None,
                  rbar_in: Optional[torch.Tensor] = None, stream=None) -> Dict[str, torch.Tensor]:
    """mixkv_scores_static: the same scores as :func:`scores`, for callers that cannot give
    the library a workspace.  The scratch the kernels need lives inside the library (a fixed
    array, see MIXKV_STATIC_SCRATCH_BYTES in the header), so this function hands over inputs
    and outputs only; the output tensors below are the caller's, as in :func:`scores`.
    Raises MixKVError (status -6) when the problem is too large for the built-in array.
    Calls on one device share that array: do not let two of them overlap on the GPU."""
    H, Ltot, d = K.shape
    batch = 1 if cu_seqlens is None else len(cu_seqlens) - 1
    Ptot = Ltot - batch * params.window
    f32 = dict(dtype=torch.float32, device=K.device)
    out = {"s_comp": torch.empty((H, Ptot), **f32), "s_ex": torch.empty((H, Ptot), **f32),
           "s_div": torch.empty((H, Ptot), **f32), "rbar": torch.empty((batch, H), **f32)}
    status = torch.zeros(1, dtype=torch.int32, device=K.device)
    cu, _ = _cu_array(cu_seqlens)
    pc = params.c()
    rc = load_library().mixkv_scores_static(
        _ptr(K), _ptr(V), _ptr(Q), cu, batch, Ltot, C.byref(pc), _ptr(out["s_comp"]),
        _ptr(out["s_ex"]), _ptr(out["s_div"]), _ptr(out["rbar"]), _ptr(rbar_in), _ptr(status),
        _stream(stream))
    if rc != 0:
        raise MixKVError(rc, "mixkv_scores_static")
    out["status"] = status
    return out


def select(s: torch.Tensor, params: Params, cu_seqlens: Optional[Sequence[int]] = None,
           workspace: Optional[torch.Tensor] = None, stream=None) -> Dict[str, torch.Tensor]:
    """mixkv_select on scores [H, Ptot] fp32 (device tensor)."""
    H, Ptot = s.shape
    batch = 1 if cu_seqlens is None else len(cu_seqlens) - 1
    Ltot = Ptot + batch * params.window
    workspace, batch = _workspace(params, cu_seqlens, Ltot, s.device, workspace)
    i32 = dict(dtype=torch.int32, device=s.device)
    cap = max(batch * H * (params.budget - params.window), 1)
    out = {"idx": torch.empty(cap, **i32), "counts": torch.empty(batch * H, **i32),
           "idx_offsets": torch.empty(batch * H + 1, **i32)}
    status = torch.zeros(1, **i32)
    cu, _ = _cu_array(cu_seqlens)
    pc = params.c()
    rc = load_library().mixkv_select(_ptr(s), cu, batch, Ltot, C.byref(pc), _ptr(workspace),
                                     workspace.numel(), _ptr(out["idx"]), _ptr(out["counts"]),
                                     _ptr(out["idx_offsets"]), _ptr(status), _stream(stream))
    if rc != 0:
        raise MixKVError(rc, "mixkv_select")
    out["status"] = status
    return out


def compress_layer(K: torch.Tensor, V: torch.Tensor, Q: torch.Tensor, params: Params,
                   cu_seqlens: Optional[Sequence[int]] = None,
                   rbar_in: Optional[torch.Tensor] = None,
                   workspace: Optional[torch.Tensor] = None, stream=None,
                   out: Optional[Dict[str, torch.Tensor]] = None,
                   want_aux: bool = True, trace_events=None) -> Dict[str, torch.Tensor]:
    """mixkv_compress_layer.  Returns K_out / V_out [batch*H*B, 128] (rows beyond
    out_row_offsets[-1] are untouched), out_row_offsets and, if want_aux, idx / counts /
    idx_offsets / s_comp.  `out` lets a caller reuse output tensors across calls."""
    H, Ltot, d = K.shape
    workspace, batch = _workspace(params, cu_seqlens, Ltot, K.device, workspace)
    Ptot = Ltot - batch * params.window
    if out is None:
        i32 = dict(dtype=torch.int32, device=K.device)
        rows = batch * H * params.budget
        out = {"K_out": torch.empty((rows, d), dtype=torch.bfloat16, device=K.device),
               "V_out": torch.empty((rows, d), dtype=torch.bfloat16, device=K.device),
               "out_row_offsets": torch.empty(batch * H + 1, **i32),
               "status": torch.zeros(1, **i32)}
        if want_aux:
            cap = max(batch * H * (params.budget - params.window), 1)
            out["idx"] = torch.empty(cap, **i32)
            out["counts"] = torch.empty(batch * H, **i32)
            out["idx_offsets"] = torch.empty(batch * H + 1, **i32)
            out["s_comp"] = torch.empty((H, Ptot), dtype=torch.float32, device=K.device)
    cu, _ = _cu_array(cu_seqlens)
    pc = params.c()
    args = (_ptr(K), _ptr(V), _ptr(Q), cu, batch, Ltot, C.byref(pc), _ptr(workspace),
            workspace.numel(), _ptr(rbar_in), _ptr(out["K_out"]), _ptr(out["V_out"]),
            _ptr(out["out_row_offsets"]), _ptr(out.get("idx")), _ptr(out.get("counts")),
            _ptr(out.get("idx_offsets")), _ptr(out.get("s_comp")), _ptr(out["status"]),
            _stream(stream))
    if trace_events is None:
        rc = load_library().mixkv_compress_layer(*args)
    else:
        # trace_events: a ctypes array of cudaEvent_t handles (see mixkv_compress_layer_traced)
        rc = load_library().mixkv_compress_layer_traced(*args, trace_events, len(trace_events))
    if rc != 0:
        raise MixKVError(rc, "mixkv_compress_layer")
    return out


def compress_layers(K: torch.Tensor, V: torch.Tensor, Q: torch.Tensor, params: Params,
                    cu_seqlens: Optional[Sequence[int]] = None,
                    rbar_in: Optional[torch.Tensor] = None,
                    workspace: Optional[torch.Tensor] = None, stream=None,
                    out: Optional[Dict[str, torch.Tensor]] = None,
                    want_aux: bool = True, trace_events=None,
                    head_budgets: Optional[torch.Tensor] = None) -> Dict[str, torch.Tensor]:
    """mixkv_compress_layers: K, V [n_layers, H, Ltot, 128], Q [n_layers, batch, H*G, W, 128]
    (bf16 device tensors; the layer dimension may be strided, the rest contiguous).  Returns
    K_out / V_out [n_layers, batch*H*B, 128], out_row_offsets [n_layers, batch*H+1] and, if
    want_aux, idx [n_layers, cap] / counts / idx_offsets / s_comp.  With head_budgets (int32
    device tensor [n_layers, batch*H], rows to keep per head, window included) the call goes to
    mixkv_compress_layers_budgeted."""
    NL, H, Ltot, d = K.shape
    batch = 1 if cu_seqlens is None else len(cu_seqlens) - 1
    max_len = Ltot if cu_seqlens is None else max(int(cu_seqlens[b + 1]) - int(cu_seqlens[b])
                                                 for b in range(batch))
    if workspace is None:
        workspace = torch.empty(workspace_size_layers(params, NL, batch, Ltot, max_len),
                                dtype=torch.uint8, device=K.device)
    for t in (K, V, Q):
        assert t[0].is_contiguous(), "each layer must be contiguous"
    assert V.stride(0) == K.stride(0), "K and V must share their layer stride"
    Ptot = Ltot - batch * params.window
    lens = [Ltot] if cu_seqlens is None else [int(cu_seqlens[b + 1]) - int(cu_seqlens[b])
                                              for b in range(batch)]
    cap = max(sum(H * min(params.budget - params.window, L - params.window) for L in lens), 1)
    if out is None:
        i32 = dict(dtype=torch.int32, device=K.device)
        rows = batch * H * params.budget
        out = {"K_out": torch.empty((NL, rows, d), dtype=torch.bfloat16, device=K.device),
               "V_out": torch.empty((NL, rows, d), dtype=torch.bfloat16, device=K.device),
               "out_row_offsets": torch.empty((NL, batch * H + 1), **i32),
               "status": torch.zeros(1, **i32)}
        if want_aux:
            out["idx"] = torch.empty((NL, cap), **i32)
            out["counts"] = torch.empty((NL, batch * H), **i32)
            out["idx_offsets"] = torch.empty((NL, batch * H + 1), **i32)
            out["s_comp"] = torch.empty((NL, H, Ptot), dtype=torch.float32, device=K.device)
    cu, _ = _cu_array(cu_seqlens)
    pc = params.c()
    ev, n_ev = (None, 0) if trace_events is None else (trace_events, len(trace_events))
    if head_budgets is not None:
        assert head_budgets.dtype == torch.int32 and head_budgets.is_contiguous()
        assert tuple(head_budgets.shape) == (NL, batch * H) and trace_events is None
        rc = load_library().mixkv_compress_layers_budgeted(
            K.data_ptr(), V.data_ptr(), Q.data_ptr(), NL, K.stride(0), Q.stride(0), cu, batch,
            Ltot, C.byref(pc), _ptr(workspace), workspace.numel(), _ptr(rbar_in),
            _ptr(head_budgets), _ptr(out["K_out"]), _ptr(out["V_out"]),
            _ptr(out["out_row_offsets"]), _ptr(out.get("idx")), _ptr(out.get("counts")),
            _ptr(out.get("idx_offsets")), _ptr(out.get("s_comp")), _ptr(out["status"]),
            _stream(stream))
        if rc != 0:
            raise MixKVError(rc, "mixkv_compress_layers_budgeted")
        return out
    rc = load_library().mixkv_compress_layers(
        K.data_ptr(), V.data_ptr(), Q.data_ptr(), NL, K.stride(0), Q.stride(0), cu, batch, Ltot,
        C.byref(pc), _ptr(workspace), workspace.numel(), _ptr(rbar_in), _ptr(out["K_out"]),
        _ptr(out["V_out"]), _ptr(out["out_row_offsets"]), _ptr(out.get("idx")),
        _ptr(out.get("counts")), _ptr(out.get("idx_offsets")), _ptr(out.get("s_comp")),
        _ptr(out["status"]), _stream(stream), ev, n_ev)
    if rc != 0:
        raise MixKVError(rc, "mixkv_compress_layers")
    return out


def layer_budget_schedule(n_layers: int, budget: int, window: int, taper_permille: int):
    """mixkv_layer_budget_schedule: rows to keep per head of each layer (host list), falling
    linearly with depth, total n_layers * budget."""
    arr = (C.c_int32 * n_layers)()
    rc = load_library().mixkv_layer_budget_schedule(n_layers, budget, window, taper_permille, arr)
    if rc != 0:
        raise MixKVError(rc, "mixkv_layer_budget_schedule")
    return [int(v) for v in arr]


def similarity_map(X: torch.Tensor, block: int, want_mean: bool = True, stream=None):
    """mixkv_similarity_map: X [heads, L, 128] bf16 device tensor -> (cells [heads, T, T] fp32,
    mean [heads] fp32 or None): block-mean cosine similarity of the rows of every head."""
    heads, L, d = X.shape
    assert X.is_contiguous() and X.dtype == torch.bfloat16
    need = C.c_size_t(0)
    rc = load_library().mixkv_similarity_workspace_size(heads, L, block, C.byref(need))
    if rc != 0:
        raise MixKVError(rc, "mixkv_similarity_workspace_size")
    ws = torch.empty(need.value, dtype=torch.uint8, device=X.device)
    T = (L + block - 1) // block
    cells = torch.empty((heads, T, T), dtype=torch.float32, device=X.device)
    mean = torch.empty(heads, dtype=torch.float32, device=X.device) if want_mean else None
    rc = load_library().mixkv_similarity_map(X.data_ptr(), heads, L, d, block, ws.data_ptr(),
                                             ws.numel(), cells.data_ptr(), _ptr(mean),
                                             _stream(stream))
    if rc != 0:
        raise MixKVError(rc, "mixkv_similarity_map")
    return cells, mean


def decode_attention(K_cache: torch.Tensor, V_cache: torch.Tensor, out_row_offsets: torch.Tensor,
                     q: torch.Tensor, kv_heads: int, gqa_ratio: int, max_rows: int,
                     softmax_scale: float = 0.0, stream=None) -> torch.Tensor:
    """mixkv_decode_attention: K_cache / V_cache [n_layers, rows_cap, 128] bf16 (the compact
    cache), out_row_offsets [n_layers, batch*H+1] int32, q [n_layers, batch, H*G, 128] bf16 ->
    [n_layers, batch, H*G, 128] fp32."""
    NL, rows_cap, d = K_cache.shape
    batch = q.shape[1]
    assert K_cache.is_contiguous() and V_cache.is_contiguous() and q.is_contiguous()
    assert out_row_offsets.dtype == torch.int32 and out_row_offsets.is_contiguous()
    out = torch.empty(q.shape, dtype=torch.float32, device=q.device)
    rc = load_library().mixkv_decode_attention(
        K_cache.data_ptr(), V_cache.data_ptr(), out_row_offsets.data_ptr(), rows_cap, q.data_ptr(),
        NL, batch, kv_heads, gqa_ratio, d, softmax_scale, max_rows, out.data_ptr(), _stream(stream))
    if rc != 0:
        raise MixKVError(rc, "mixkv_decode_attention")
    return out


def selftest_bounded_wait(stream=None):
    """mixkv_selftest_bounded_wait: returns (status, seconds waited) after the kernel has ended."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    rc = load_library().mixkv_selftest_bounded_wait(status.data_ptr(), waited.data_ptr(),
                                                    _stream(stream))
    if rc != 0:
        raise MixKVError(rc, "mixkv_selftest_bounded_wait")
    torch.cuda.synchronize()
    return int(status.item()), int(waited.item()) * 1e-9
