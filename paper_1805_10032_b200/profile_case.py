"""Runs a few Zeno steps of one benchmark configuration, optionally shrunk, for a profiler to capture.

    python -m paper_1805_10032_b200.profile_case --config 5 --d 4194304 --steps 3
    python -m paper_1805_10032_b200.profile_case --config 4 --steps 2

The least-squares configuration holds 21.7 GB at full size, too much for a multi-pass capture; --d gives it a
smaller parameter count (every operand is still far larger than the L2).  Prints the kernels of one step.
"""
from __future__ import annotations

import argparse

import torch

from . import synthetic as syn
from . import zeno


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, required=True, choices=[1, 2, 3, 4, 5, 6])
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--d", type=int, default=0, help="configuration 5 only: parameter count")
    ap.add_argument("--n-r", type=int, default=0)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device")
    ov = {}
    if args.d and args.config == 5:
        ov["d"] = args.d
    if args.n_r:
        ov["n_r"] = args.n_r
    w = syn.make_config(args.config, device="cuda", **ov)
    out = torch.empty(w.d, dtype=torch.float32, device="cuda")
    with zeno.from_workload(w) as z:
        for _ in range(args.steps):
            z.step(w.x, w.V, w.features, w.targets, w.gamma, w.rho, w.b, out=out)
        torch.cuda.synchronize()
        z.check_device_status()
        z.profile(True)
        z.step(w.x, w.V, w.features, w.targets, w.gamma, w.rho, w.b, out=out)
        torch.cuda.synchronize()
        print("kernels of a step:", ", ".join(f"{n} {ms * 1e3:.1f} us" for n, ms in z.profile_read(0)))


if __name__ == "__main__":
    main()
