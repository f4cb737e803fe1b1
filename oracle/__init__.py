"""Python face of the plain CPU oracle (``mixkv_oracle.c``).

TEST INFRASTRUCTURE ONLY: the test suite, the smoke check and the benchmark's
cpu_baseline leg load this; the product (the CUDA library and its binding) never
imports it.  The wrapper only marshals numpy arrays into the C functions; all the
arithmetic lives in the C file, written from the paper (Sec. 3.2-3.3, Algorithm 1).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mixkv_oracle.c")
_LIB = os.path.join(_HERE, "libmixkv_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) if the shared object is missing or stale."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Params(C.Structure):
    _fields_ = [("kv_heads", C.c_int32), ("gqa_ratio", C.c_int32), ("head_dim", C.c_int32),
                ("window", C.c_int32), ("pool_kernel", C.c_int32), ("pool_mode", C.c_int32),
                ("use_vnorm", C.c_int32), ("mix_mode", C.c_int32), ("budget_mode", C.c_int32),
                ("budget", C.c_int32), ("ada_floor", C.c_double), ("eps", C.c_double),
                ("softmax_scale", C.c_double)]


@dataclass
class Params:
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

    def c(self) -> _Params:
        # ada_floor and eps are float parameters of the library; the oracle sees the
        # same float-rounded values, widened to double
        return _Params(self.kv_heads, self.gqa_ratio, self.head_dim, self.window,
                       self.pool_kernel, self.pool_mode, self.use_vnorm, self.mix_mode,
                       self.budget_mode, self.budget, float(np.float32(self.ada_floor)),
                       float(np.float32(self.eps)), float(np.float32(self.softmax_scale)))


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.mixkv_oracle_threads.restype = C.c_int
    return _lib


def threads() -> int:
    return int(lib().mixkv_oracle_threads())


def set_threads(n: int) -> None:
    lib().mixkv_oracle_set_threads(C.c_int(n))


def _p(a: Optional[np.ndarray], ctype):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.POINTER(ctype))


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16
    return a


def _cu(cu, L=None):
    if cu is None:
        cu = [0, int(L)]
    return np.ascontiguousarray(np.asarray(cu, dtype=np.int32))


# ------------------------------------------------------------------ step functions
def window_attention(Kh: np.ndarray, Qg: np.ndarray, scale: Optional[float] = None):
    """Kh [L, d] bf16 bits, Qg [G, W, d] bf16 bits -> (s_ex_raw [L], row_sums [G*W]), float64."""
    Kh, Qg = _u16(Kh), _u16(Qg)
    L, d = Kh.shape
    G, W, _ = Qg.shape
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    s = np.empty(L, dtype=np.float64)
    rs = np.empty(G * W, dtype=np.float64)
    lib().mixkv_oracle_window_attention(_p(Kh, C.c_uint16), _p(Qg, C.c_uint16), G, W, L, d,
                                        C.c_double(scale), _p(s, C.c_double), _p(rs, C.c_double))
    return s, rs


def pool(x: np.ndarray, k: int, mode: int = 0) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty_like(x)
    lib().mixkv_oracle_pool(_p(x, C.c_double), x.shape[0], k, mode, _p(out, C.c_double))
    return out


def row_norms(X: np.ndarray) -> np.ndarray:
    X = _u16(X)
    n, d = X.shape
    out = np.empty(n, dtype=np.float64)
    lib().mixkv_oracle_row_norms(_p(X, C.c_uint16), n, d, _p(out, C.c_double))
    return out


def key_geometry(Kh: np.ndarray):
    """Kh [L, d] bf16 bits -> (s_div [L], rbar, kbar [d]), float64."""
    Kh = _u16(Kh)
    L, d = Kh.shape
    s_div = np.empty(L, dtype=np.float64)
    kbar = np.empty(d, dtype=np.float64)
    r = C.c_double(0.0)
    lib().mixkv_oracle_key_geometry(_p(Kh, C.c_uint16), L, d, _p(s_div, C.c_double), C.byref(r),
                                    _p(kbar, C.c_double))
    return s_div, float(r.value), kbar


def mix(s_ex, vnorm, s_div, rbar: float, use_vnorm: int = 1, mix_mode: int = 0,
        eps: float = 1e-6) -> Dict[str, np.ndarray]:
    s_ex = np.ascontiguousarray(s_ex, dtype=np.float64)
    s_div = np.ascontiguousarray(s_div, dtype=np.float64)
    P = s_ex.shape[0]
    vn = None if vnorm is None else np.ascontiguousarray(vnorm, dtype=np.float64)
    out = {k: np.empty(P, dtype=np.float64)
           for k in ("s_comp", "s_imp", "s_div_scaled", "s_in_scaled")}
    lib().mixkv_oracle_mix(_p(s_ex, C.c_double), _p(vn, C.c_double), _p(s_div, C.c_double), P,
                           C.c_double(rbar), use_vnorm, mix_mode, C.c_double(eps),
                           _p(out["s_comp"], C.c_double), _p(out["s_imp"], C.c_double),
                           _p(out["s_div_scaled"], C.c_double), _p(out["s_in_scaled"], C.c_double))
    return out


def topb(s: np.ndarray, b: int) -> np.ndarray:
    s = np.ascontiguousarray(s, dtype=np.float32)
    idx = np.empty(b, dtype=np.int32)
    lib().mixkv_oracle_topb(_p(s, C.c_float), s.shape[0], b, _p(idx, C.c_int32))
    return idx


# ------------------------------------------------------------------ layer functions
def scores(K, V, Q, params: Params, cu=None, rbar_in=None) -> Dict[str, np.ndarray]:
    """All score vectors of one layer.  K, V [H, Ltot, d], Q [batch, H*G, W, d] (bf16 bits)."""
    K, Q = _u16(K), _u16(Q)
    V = None if V is None else _u16(V)
    H, Ltot, d = K.shape
    cu = _cu(cu, Ltot)
    batch = cu.shape[0] - 1
    Ptot = Ltot - batch * params.window
    out = {"s_comp": np.empty((H, Ptot), np.float32), "s_ex": np.empty((H, Ptot), np.float32),
           "s_ex_raw": np.empty((H, Ptot), np.float32), "s_div": np.empty((H, Ptot), np.float32),
           "rbar": np.empty((batch, H), np.float32)}
    rin = None if rbar_in is None else np.ascontiguousarray(rbar_in, dtype=np.float32)
    pc = params.c()
    rc = lib().mixkv_oracle_scores(_p(K, C.c_uint16), _p(V, C.c_uint16), _p(Q, C.c_uint16),
                                   _p(cu, C.c_int32), batch, C.byref(pc),
                                   _p(out["s_comp"], C.c_float), _p(out["s_ex"], C.c_float),
                                   _p(out["s_ex_raw"], C.c_float), _p(out["s_div"], C.c_float),
                                   _p(out["rbar"], C.c_float), _p(rin, C.c_float))
    if rc != 0:
        raise ValueError("oracle: invalid arguments")
    return out


def select(s: np.ndarray, params: Params, cu=None) -> Dict[str, np.ndarray]:
    """Budgets and top-B on given scores [H, Ptot]."""
    s = np.ascontiguousarray(s, dtype=np.float32)
    H, Ptot = s.shape
    if cu is None:
        cu = [0, Ptot + params.window]
    cu = _cu(cu)
    batch = cu.shape[0] - 1
    cap = int(Ptot)  # never more than every candidate
    idx = np.empty(H * cap, dtype=np.int32)
    counts = np.empty(batch * H, dtype=np.int32)
    offs = np.empty(batch * H + 1, dtype=np.int32)
    pc = params.c()
    rc = lib().mixkv_oracle_select(_p(s, C.c_float), _p(cu, C.c_int32), batch, C.byref(pc),
                                   _p(idx, C.c_int32), _p(counts, C.c_int32), _p(offs, C.c_int32))
    if rc != 0:
        raise ValueError("oracle: invalid arguments")
    return {"idx": idx[:offs[-1]].copy(), "counts": counts.reshape(batch, H), "idx_offsets": offs}


def gather(X, idx, idx_offsets, params: Params, cu=None):
    X = _u16(X)
    H, Ltot, d = X.shape
    cu = _cu(cu, Ltot)
    batch = cu.shape[0] - 1
    rows = int(idx_offsets[-1]) + batch * H * params.window
    out = np.empty((rows, d), dtype=np.uint16)
    ro = np.empty(batch * H + 1, dtype=np.int32)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    offs = np.ascontiguousarray(idx_offsets, dtype=np.int32)
    lib().mixkv_oracle_gather(_p(X, C.c_uint16), _p(cu, C.c_int32), batch, H, d, params.window,
                              _p(idx, C.c_int32), _p(offs, C.c_int32), _p(out, C.c_uint16),
                              _p(ro, C.c_int32))
    return out, ro


def compress_layer(K, V, Q, params: Params, cu=None, rbar_in=None) -> Dict[str, np.ndarray]:
    """Score, select and gather one layer."""
    K, V, Q = _u16(K), _u16(V), _u16(Q)
    H, Ltot, d = K.shape
    cu = _cu(cu, Ltot)
    batch = cu.shape[0] - 1
    Ptot = Ltot - batch * params.window
    s_comp = np.empty((H, Ptot), np.float32)
    cap_rows = H * Ltot
    K_out = np.empty((cap_rows, d), np.uint16)
    V_out = np.empty((cap_rows, d), np.uint16)
    ro = np.empty(batch * H + 1, np.int32)
    idx = np.empty(H * Ptot, np.int32)
    counts = np.empty(batch * H, np.int32)
    offs = np.empty(batch * H + 1, np.int32)
    rin = None if rbar_in is None else np.ascontiguousarray(rbar_in, dtype=np.float32)
    pc = params.c()
    rc = lib().mixkv_oracle_compress_layer(
        _p(K, C.c_uint16), _p(V, C.c_uint16), _p(Q, C.c_uint16), _p(cu, C.c_int32), batch,
        C.byref(pc), _p(rin, C.c_float), _p(s_comp, C.c_float), _p(K_out, C.c_uint16),
        _p(V_out, C.c_uint16), _p(ro, C.c_int32), _p(idx, C.c_int32), _p(counts, C.c_int32),
        _p(offs, C.c_int32))
    if rc != 0:
        raise ValueError("oracle: invalid arguments")
    rows = int(ro[-1])
    return {"s_comp": s_comp, "K_out": K_out[:rows].copy(), "V_out": V_out[:rows].copy(),
            "out_row_offsets": ro, "idx": idx[:offs[-1]].copy(),
            "counts": counts.reshape(batch, H), "idx_offsets": offs}


# ------------------------------------------------------------------ budgets chosen outside
# The paper plugs its scores into compressors that only differ in how many rows a layer or a
# head keeps (Sec. 4.1; related work: PyramidKV layer schedules, SparseMM / HeadKV per-head
# shares).  These two functions are plain Python on top of `topb`; the paper prints no formula
# for either policy, so the schedule below is the reading taken here (parity unpinned by the
# paper; pinned by its invariants: total kept, monotone, taper 0 = uniform).
def select_given(s: np.ndarray, head_budgets, params: Params, cu=None) -> Dict[str, np.ndarray]:
    """Top-b on given scores [H, Ptot] with the rows to keep per (sequence, head) given
    (window included): head (b, h) selects min(max(budget - W, 0), B - W, P_b) candidates."""
    s = np.ascontiguousarray(s, dtype=np.float32)
    H, Ptot = s.shape
    W = params.window
    if cu is None:
        cu = [0, Ptot + W]
    cu = _cu(cu)
    batch = cu.shape[0] - 1
    hb = np.asarray(head_budgets, dtype=np.int64).reshape(batch, H)
    counts = np.zeros((batch, H), dtype=np.int32)
    offs = np.zeros(batch * H + 1, dtype=np.int32)
    parts = []
    for b in range(batch):
        P = int(cu[b + 1] - cu[b]) - W
        p0 = int(cu[b]) - b * W
        for h in range(H):
            take = int(min(max(int(hb[b, h]) - W, 0), params.budget - W, P))
            counts[b, h] = take
            parts.append(topb(s[h, p0:p0 + P], take) if take > 0 else np.empty(0, np.int32))
            offs[b * H + h + 1] = offs[b * H + h] + take
    idx = np.concatenate(parts) if parts else np.empty(0, np.int32)
    return {"idx": idx.astype(np.int32), "counts": counts, "idx_offsets": offs}


def layer_budget_schedule(n_layers: int, budget: int, window: int, taper_permille: int):
    """Rows to keep per head of each layer, falling linearly with depth, same total as a
    uniform `budget`: with B' = budget - window and t = taper_permille / 1000, layer l gets
    floor(B' (1 + t (1 - 2 l / (n - 1)))) candidates, the candidates lost to the rounding go
    to the lowest layers one by one, and the window is added back."""
    from fractions import Fraction
    if n_layers == 1:
        return [budget]
    Bp = budget - window
    t = Fraction(taper_permille, 1000)
    cand = [int((Bp * (1 + t * (1 - Fraction(2 * l, n_layers - 1)))) // 1) for l in range(n_layers)]
    short = n_layers * Bp - sum(cand)
    for l in range(short):
        cand[l] += 1
    return [c + window for c in cand]
