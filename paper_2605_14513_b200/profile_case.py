"""A few layer-steps of one benchmark workload and nothing else: the command to put under a profiler.

    python -m paper_2605_14513_b200.profile_case --workload wan1.3b-480p [--heads 6] [--steps 3]
                                                 [--estimator pooled|antidiag]

--heads H runs the first H heads of the workload only (same tokens, block size and per-head
parameters): every head is independent, so DRAM traffic and kernel time scale with H, and a capture
that would hold tens of GB at full size stays small.  Prints one line with the per-step time.
"""
import argparse
import dataclasses
import sys

import torch

from . import heart, inputs


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="wan1.3b-480p")
    ap.add_argument("--heads", type=int, default=0)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--estimator", default="pooled", choices=["pooled", "antidiag"])
    a = ap.parse_args(argv)
    wl = inputs.workload(a.workload)
    if a.heads and a.heads < wl.H:
        h = a.heads
        wl = dataclasses.replace(wl, H=h, tau=wl.tau[:h], delta=wl.delta[:h], eps=wl.eps[:h], pos_scale=wl.pos_scale[:h])
    flags = heart.ESTIMATOR_ANTIDIAG if a.estimator == "antidiag" else 0
    cfg = heart.make_config(wl.B, wl.H, wl.N, wl.block, flags=flags)
    st, ws = heart.State(cfg), heart.new_workspace(cfg)
    delta = torch.tensor(wl.delta, dtype=torch.float64, device="cuda")
    tau = torch.tensor(wl.tau, dtype=torch.float64, device="cuda")
    seq = inputs.Sequence(wl, "cuda")
    O = None
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(a.steps + 1)]
    for t in range(a.steps):
        Q, K, V = seq.bf16()
        if O is None:
            O = torch.empty_like(Q)
        ev[t].record()
        heart.heart_step(cfg, Q, K, V, delta, tau, st, O, ws)
        if t + 1 < a.steps:
            seq.advance()
    ev[a.steps].record()
    torch.cuda.synchronize()
    assert heart.heart_get_status(ws) == 0
    dens = float(st.kv_cnt.double().mean()) / wl.n_blocks
    print(f"{wl.name} H={wl.H} estimator={a.estimator}: {a.steps} steps, last step "
          f"{ev[a.steps - 1].elapsed_time(ev[a.steps]):.3f} ms (input generation of the next step not included), "
          f"density {dens:.3f}")
    return 0


if __name__ == "__main__":
    sys.exit(main())
