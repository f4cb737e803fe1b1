"""Writes c1_oracle_selection.txt: what the CPU oracle keeps on workload C1 (seed 0).

Calls only the oracle and the seeded input generators; nothing from the CUDA path.
Run from the repository root:  python tests/golden/make_c1_selection.py
"""
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))

import oracle  # noqa: E402
from paper_2510_20707_b200 import synth  # noqa: E402


def main() -> None:
    wl = synth.CONFIGS["C1"]
    x = synth.make_layer(wl, 0, "literal")
    p = oracle.Params(kv_heads=wl.kv_heads, gqa_ratio=wl.gqa_ratio, window=wl.window,
                      pool_kernel=wl.pool_kernel, budget=wl.budget)
    out = oracle.compress_layer(x["K"], x["V"], x["Q"], p)
    io = out["idx_offsets"]
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "c1_oracle_selection.txt")
    with open(path, "w") as f:
        f.write("# oracle selection on C1 (Algorithm 1; H=4, G=7, L=1024, W=32, pool 7, B=64), seed 0\n")
        for h in range(wl.kv_heads):
            f.write(" ".join(str(int(i)) for i in out["idx"][io[h]:io[h + 1]]) + "\n")


if __name__ == "__main__":
    main()
