"""Writes the stored oracle traces under tests/golden/.  Calls only the CPU oracle and the
seeded workload generators; run from the repository root:  python tests/golden/make_golden.py"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import workloads                                   # noqa: E402
from oracle import osscar_oracle as orc            # noqa: E402


def main():
    wl = workloads.config("c1", seed=0)
    X = wl.x_full().float().numpy().astype(np.float64)
    W = wl.weight().numpy().astype(np.float64)
    H, G, const = orc.gram(X, W, wl.damp)
    S0, _ = orc.init_support(H, W, wl.g, wl.k)
    run = orc.Search(H, G, const, wl.g, S0, mode="strict").run(wl.max_swaps)
    S, _, obj, swaps = run.result()
    out = {"workload": "c1 seed 0 (dense 64x64, keep 32, <=50 swaps, strict oracle)",
           "const": const, "init_support": [int(s) for s in S0],
           "swap_trace": [[int(a), int(b)] for a, b in swaps],
           "obj_trace": [float(o) for o in obj], "final_support": [int(s) for s in S],
           "stop_reason": run.stop_reason}
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "c1_seed0_trace.json"), "w") as fh:
        json.dump(out, fh, indent=1)


if __name__ == "__main__":
    main()
