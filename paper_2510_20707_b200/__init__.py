"""B200-native MixKV prefill KV-cache compression (arxiv 2510.20707).

The product is ``libmixkv.so`` (hand-written sm_100a CUDA behind a C ABI declared in
``include/mixkv.h``); :mod:`paper_2510_20707_b200.binding` is a thin ctypes layer over it
that marshals torch tensors into pointers.  There is no CPU fallback: the binding raises
if the library has not been built.
"""
from .binding import (MixKVError, Params, compress_layer, compress_layers, launches_per_layer,
                      load_library, scores, select, workspace_size, workspace_size_layers)

__all__ = ["MixKVError", "Params", "compress_layer", "compress_layers", "launches_per_layer",
           "load_library", "scores", "select", "workspace_size", "workspace_size_layers"]
