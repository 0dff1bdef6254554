"""Timing sweeps of the Zeno step over the hyperparameters the paper varies (Experiments, "Hyperparameter
Sensitivity": the Zeno batch size n_r, and rho and b in its appendix; the remark after Corollary 2 on n_r).

    python -m paper_1805_10032_b200.sweep --config 2 --n-r 1 4 32 128 [--steps 100]
    python -m paper_1805_10032_b200.sweep --config 2 --b 0 4 8 16 19
    python -m paper_1805_10032_b200.sweep --config 3 --baselines     (Zeno_b, Median and Krum_b on the same V)

Prints one markdown table row per setting: microseconds per step (steps enqueued back to back, CUDA events
around the loop) and the kernels that served it with their share of the profiled time -- which shows where
the step moves from one kernel family to another as n_r grows.  Timing only: the arithmetic is checked by
the parity tests.
"""
from __future__ import annotations

import argparse

import torch

from . import synthetic as syn
from . import zeno


def time_setting(index, steps, **ov):
    w = syn.make_config(index, device="cuda", **ov)
    out = torch.empty(w.d, dtype=torch.float32, device="cuda")
    with zeno.from_workload(w) as z:
        def step():
            z.step(w.x, w.V, w.features, w.targets, w.gamma, w.rho, w.b, out=out)
        for _ in range(5):
            step()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            step()
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) / steps * 1e3
        z.profile(True)
        n = min(steps, 48)
        for _ in range(n):
            step()
        acc = {}
        for back in range(n):
            for j, (name, ms) in enumerate(z.profile_read(back)):
                acc.setdefault(f"{j}:{name}", []).append(ms * 1e3)
        z.profile(False)
        z.check_device_status()
    kernels = ", ".join(f"{k.split(':')[1]} {sum(v) / len(v):.1f}" for k, v in acc.items())
    return us, kernels


def time_baselines(index, steps):
    """The three aggregation rules on the same candidates: Zeno_b (the whole step), the marginal Median and
    Krum_b, microseconds per call, and the bytes each must at least read (V once) against the time."""
    w = syn.make_config(index, device="cuda")
    out = torch.empty(w.d, dtype=torch.float32, device="cuda")
    rows = []
    with zeno.from_workload(w) as z:
        calls = [("Zeno_b (score, rank, trimmed mean)", lambda: z.step(w.x, w.V, w.features, w.targets, w.gamma, w.rho, w.b, out=out)),
                 ("Median", lambda: z.median(w.V, out=out))]
        if w.m <= 128 and w.m - w.b - 2 >= 1:
            calls.append((f"Krum_b (b = {w.b})", lambda: z.krum(w.V, w.b)))
        for name, fn in calls:
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(steps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            rows.append((name, e0.elapsed_time(e1) / steps * 1e3))
    v_bytes = w.m * w.d * w.V.element_size()
    return rows, v_bytes


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=2, choices=[1, 2, 3, 4, 5, 6])
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--n-r", type=int, nargs="*", default=[])
    ap.add_argument("--b", type=int, nargs="*", default=[])
    ap.add_argument("--rho", type=float, nargs="*", default=[])
    ap.add_argument("--baselines", action="store_true",
                    help="time Zeno_b, Median and Krum_b on the configuration's candidates instead of sweeping")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("the sweep needs a CUDA device")
    if args.baselines:
        rows, v_bytes = time_baselines(args.config, args.steps)
        print(f"| config {args.config}: rule | us / call | V read once at this time (GB/s) |")
        print("|---|---|---|")
        for name, us in rows:
            print(f"| {name} | {us:.1f} | {v_bytes / us / 1e3:.0f} |")
        return
    print(f"| config {args.config} with | us / step | kernels (us each, profiled pass) |")
    print("|---|---|---|")
    for key, values in (("n_r", args.n_r), ("b", args.b), ("rho", args.rho)):
        for v in values:
            us, kernels = time_setting(args.config, args.steps, **{key: v})
            print(f"| {key} = {v} | {us:.1f} | {kernels} |", flush=True)


if __name__ == "__main__":
    main()
