"""Writes tests/golden/seed0_stats.json: statistics of the oracle's result on
the five seeded workloads.  Calls only the input generators and the CPU oracle
(never the CUDA library).  Run from the repository root:

    python tests/golden/make_seed0_stats.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2609_36800_b200 import synth  # noqa: E402


def main():
    out = {}
    for wl in synth.WORKLOADS:
        X, W, bits, alpha = synth.make_inputs(wl)
        Y = oracle.gemm(X, W, bits, alpha)
        out[wl.name] = {
            "B": wl.B, "m": wl.m, "K": wl.K, "N": wl.N, "seed": wl.seed,
            "x000_bits": int(X[0, 0, 0]), "w00_bits": int(W[0, 0]),
            "bits_first": int(bits[0, 0, 0]), "bits_last": int(bits[-1, -1, -1]),
            "alpha_first": float(alpha[0]), "alpha_last": float(alpha[-1]),
            "y_first": float(Y[0, 0, 0]), "y_last": float(Y[-1, -1, -1]),
            "y_mid": float(Y[wl.B // 2, wl.m // 2, wl.N // 2]),
            "y_absmax": float(np.abs(Y).max()), "y_fro": float(np.linalg.norm(Y)),
            "y_sum": float(Y.sum()), "count_abs_ge_4": int((np.abs(Y) >= 4).sum()),
            "count_abs_ge_8": int((np.abs(Y) >= 8).sum()),
        }
        print(wl.name, out[wl.name], flush=True)
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "seed0_stats.json"), "w") as f:
        json.dump(out, f, indent=1, sort_keys=True)


if __name__ == "__main__":
    main()
