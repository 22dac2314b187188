"""Writes the per-head thresholds of the 720P Wan-14B-shaped workload (config 4).

The configuration asks for a global retained-block budget of 15 % "with tau_h chosen per head to
meet it" -- a stand-in for the output of the paper's offline budgeted calibration, which needs the
real model.  This script finds, for every head of the step-0 synthetic tensors, the tau_h at which
the oracle's top-p selection keeps 15 % of that head's block pairs (bisection), using ONLY the CPU
oracle (oracle/heart_oracle.py) and the seeded input generator.  Its output is pasted into
paper_2605_14513_b200/inputs.py (_TAU_WAN14B_720P).

    python tests/golden/calibrate_tau_wan14b_720p.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import heart_oracle as oracle  # noqa: E402
from paper_2605_14513_b200 import inputs  # noqa: E402

BUDGET = 0.15


def main():
    wl = inputs.workload("wan14b-720p")
    N, D, b, nb = wl.N, wl.D, wl.block, wl.n_blocks
    scale = 1.0 / np.sqrt(D)
    taus = []
    for h in range(wl.H):
        E = inputs.positional(wl.grid, D, h, "cpu") * float(wl.pos_scale[h])
        Q = (inputs.normal(wl.seed, 0, 0, h * N * D, N * D, "cpu").view(N, D) + E).to(inputs.torch.bfloat16)[None]
        K = (inputs.normal(wl.seed, 1, 0, h * N * D, N * D, "cpu").view(N, D) + E).to(inputs.torch.bfloat16)[None]
        Qp = oracle.block_pool(inputs.bits(Q), b)[0]
        Kp = oracle.block_pool(inputs.bits(K), b)[0]
        P = np.stack([oracle.block_probs(Qp[I], Kp, scale) for I in range(nb)])

        def density(tau):
            return sum(oracle.top_p(P[I], tau)[1] for I in range(nb)) / float(nb * nb)

        lo, hi = 0.5, 0.9999
        for _ in range(14):
            mid = 0.5 * (lo + hi)
            if density(mid) < BUDGET:
                lo = mid
            else:
                hi = mid
        tau = round(0.5 * (lo + hi), 4)
        taus.append(tau)
        print(f"head {h:2d}: tau = {tau:.4f}  density = {density(tau):.4f}", flush=True)
    print("_TAU_WAN14B_720P = np.array([" + ", ".join(f"{t:.4f}" for t in taus) + "])")


if __name__ == "__main__":
    main()
