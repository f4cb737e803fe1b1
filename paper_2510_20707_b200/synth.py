"""Seeded synthetic inputs for the MixKV prefill-compression workloads.

This module only draws random tensors and rounds them to bf16 bit patterns.  It
holds none of the method's arithmetic (no scores, no softmax, no selection), so
that the CPU oracle and the CUDA path can both be fed the identical bytes it
produces without sharing any code of their own.

Every tensor is returned as a ``numpy.uint16`` array of bf16 bit patterns:
  K, V : [H, Ltot, d]         keys / values of one layer (all sequences concatenated)
  Q    : [batch, H*G, W, d]   the last W (observation-window) queries of each sequence

Workloads follow the key statistics the paper reports (Sec. 1 / Fig. 1-2: mean
pairwise key cosine 0.2-0.4 for text-only LLM keys, 0.6-0.8 for vision keys,
heads spread from below 0.3 to above 0.9; Sec. 3.2: observation window 32;
Tables 1 and 3: budgets 64-1024; Fig. 4: context 32,000).  Two variants exist:

  "literal"     exactly the recipe of the workload description;
  "calibrated"  the same draw plus one shared offset vector per head, whose
                squared norm x_h * d is chosen so that the head's mean pairwise
                cosine lands in the band quoted above (an offset common to all
                keys of a head shifts every logit of a query by the same
                constant, so the window softmax is untouched).
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Tuple

import numpy as np

HEAD_DIM = 128


# --------------------------------------------------------------------------- bf16
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round-to-nearest-even) and return the 16-bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    out = ((u + rounding) >> np.uint32(16)).astype(np.uint16)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to float32 exactly."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# ---------------------------------------------------------------------- workloads
@dataclass(frozen=True)
class Workload:
    name: str
    layers: int
    kv_heads: int          # H
    gqa_ratio: int         # G
    window: int            # W
    pool_kernel: int
    budget: int            # B, rows kept per head including the window
    budget_mode: int       # 0 fixed, 1 adaptive (per sequence total B*H)
    seq_lens: Tuple[int, ...]          # one entry per sequence of the batch
    kind: str              # "image", "video", "batch", "text"
    centroids: int = 0     # per head (per frame for "video")
    vision_tokens: Tuple[int, ...] = ()  # per sequence
    frames: int = 0
    frame_tokens: int = 0
    seed: int = 0
    head_dim: int = HEAD_DIM
    ada_floor: float = 0.2

    @property
    def batch(self) -> int:
        return len(self.seq_lens)

    @property
    def total_tokens(self) -> int:
        return int(sum(self.seq_lens))

    @property
    def cu_seqlens(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.seq_lens)]).astype(np.int32)


def _c4_lengths(seed: int) -> Tuple[Tuple[int, ...], Tuple[int, ...]]:
    rng = np.random.default_rng(np.random.SeedSequence([seed, 4, 999_999]))
    lens = rng.integers(2048, 8193, size=8)
    frac = rng.uniform(0.6, 0.9, size=8)
    vis = np.floor(lens * frac).astype(np.int64)
    return tuple(int(x) for x in lens), tuple(int(x) for x in vis)


def _configs() -> Dict[str, Workload]:
    c4_lens, c4_vis = _c4_lengths(0)
    return {
        # single layer, L=1024: 896 vision keys around 16 centroids/head, 128 text keys
        "C1": Workload("C1", 1, 4, 7, 32, 7, 64, 0, (1024,), "image", centroids=16,
                       vision_tokens=(896,)),
        # Qwen2-VL-7B-shaped prefill, L=4096: 3584 vision keys, 64 centroids/head
        "C2": Workload("C2", 28, 4, 7, 32, 7, 128, 0, (4096,), "image", centroids=64,
                       vision_tokens=(3584,)),
        # long video, L=32768 = 32 frames x 1016 tokens + 256 text tokens
        "C3": Workload("C3", 28, 4, 7, 32, 7, 256, 0, (32768,), "video", centroids=32,
                       frames=32, frame_tokens=1016, vision_tokens=(32 * 1016,)),
        "C3b": Workload("C3b", 28, 4, 7, 32, 7, 512, 0, (32768,), "video", centroids=32,
                        frames=32, frame_tokens=1016, vision_tokens=(32 * 1016,)),
        # batched serving, ragged, adaptive budgets
        "C4": Workload("C4", 28, 4, 7, 32, 7, 128, 1, c4_lens, "batch", centroids=64,
                       vision_tokens=c4_vis),
        # Llama-3-8B-shaped text-only
        "C5": Workload("C5", 32, 8, 4, 32, 7, 256, 0, (16384,), "text"),
    }


CONFIGS: Dict[str, Workload] = _configs()
_CFG_ID = {"C1": 1, "C2": 2, "C3": 3, "C3b": 3, "C4": 4, "C5": 5}

# squared-norm multipliers x_h of the shared per-head offset ("calibrated" variant)
_VISION_X = (0.4, 1.2, 2.4, 10.0)          # mean cosine about 0.26, 0.52, 0.68, 0.90


def _text_x(h: int, H: int) -> float:
    rho = 0.2 + 0.2 * (h / max(H - 1, 1))   # 0.2 .. 0.4 across heads
    return rho / (1.0 - rho)


def _rng(wl: Workload, layer: int, tensor: int, extra: int = 0) -> np.random.Generator:
    cfg = _CFG_ID.get(wl.name, 99)
    return np.random.default_rng(np.random.SeedSequence([wl.seed, cfg, layer, tensor, extra]))


def _normal(rng: np.random.Generator, shape) -> np.ndarray:
    return rng.standard_normal(shape, dtype=np.float32)


def _vision_keys(rng, n_tokens: int, centroids: np.ndarray, noise: float) -> np.ndarray:
    """n_tokens keys, each one of the given centroids plus N(0, noise^2) noise."""
    pick = rng.integers(0, centroids.shape[0], size=n_tokens)
    return centroids[pick] + noise * _normal(rng, (n_tokens, centroids.shape[1]))


def make_keys(wl: Workload, layer: int, variant: str = "literal") -> np.ndarray:
    """float32 keys [H, Ltot, d] before bf16 rounding."""
    H, d = wl.kv_heads, wl.head_dim
    K = np.empty((H, wl.total_tokens, d), dtype=np.float32)
    cu = wl.cu_seqlens
    for h in range(H):
        for b, L in enumerate(wl.seq_lens):
            rng = _rng(wl, layer, 0, h * 1024 + b)
            seg = K[h, cu[b]:cu[b] + L]
            if wl.kind == "text":
                seg[:] = _normal(rng, (L, d))
                x = _text_x(h, H)
            else:
                nv = wl.vision_tokens[b]
                if wl.kind == "video":
                    rho = 0.98
                    c = _normal(rng, (wl.centroids, d))
                    for f in range(wl.frames):
                        if f > 0:
                            c = rho * c + np.float32(np.sqrt(1 - rho * rho)) * _normal(rng, c.shape)
                        lo = f * wl.frame_tokens
                        seg[lo:lo + wl.frame_tokens] = _vision_keys(rng, wl.frame_tokens, c, 0.35)
                else:
                    c = _normal(rng, (wl.centroids, d))
                    seg[:nv] = _vision_keys(rng, nv, c, 0.35)
                seg[nv:] = _normal(rng, (L - nv, d))
                x = _VISION_X[h % len(_VISION_X)]
            if variant == "calibrated":
                m = _normal(rng, (d,))
                m *= np.float32(np.sqrt(x * d) / np.linalg.norm(m))
                seg += m
            elif variant != "literal":
                raise ValueError(f"unknown variant {variant!r}")
    return K


def make_layer(wl: Workload, layer: int, variant: str = "literal") -> Dict[str, np.ndarray]:
    """bf16 bit patterns of one layer's K, V [H, Ltot, d] and Q [batch, H*G, W, d]."""
    H, G, W, d = wl.kv_heads, wl.gqa_ratio, wl.window, wl.head_dim
    K = make_keys(wl, layer, variant)
    V = _normal(_rng(wl, layer, 1), (H, wl.total_tokens, d))
    Q = _normal(_rng(wl, layer, 2), (wl.batch, H * G, W, d))
    return {"K": f32_to_bf16_bits(K), "V": f32_to_bf16_bits(V), "Q": f32_to_bf16_bits(Q)}


def small_workload(name: str = "tiny", *, H: int = 2, G: int = 2, W: int = 4,
                   seq_lens=(37,), pool_kernel: int = 3, budget: int = 12,
                   budget_mode: int = 0, seed: int = 0, kind: str = "image",
                   centroids: int = 4, vision_frac: float = 0.75,
                   ada_floor: float = 0.2) -> Workload:
    """A freely shaped workload for tests (odd lengths, ragged batches, tiny heads)."""
    seq_lens = tuple(int(x) for x in seq_lens)
    vis = tuple(int(L * vision_frac) for L in seq_lens)
    return Workload(name, 1, H, G, W, pool_kernel, budget, budget_mode, seq_lens, kind,
                    centroids=centroids, vision_tokens=vis, seed=seed, ada_floor=ada_floor)


def with_budget(wl: Workload, budget: int, budget_mode: Optional[int] = None) -> Workload:
    return replace(wl, budget=budget,
                   budget_mode=wl.budget_mode if budget_mode is None else budget_mode)
