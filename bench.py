#!/usr/bin/env python
"""Benchmark of the Zeno aggregation step (scores -> ranking -> trimmed mean).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]

One step = one zeno_step call: f_r(x), the m candidate losses f_r(x - gamma v_i) with the
squared norms, the top-(m-b) ranking and the trimmed mean, on one batch of synthetic input.
Prints ONE JSON line: steps/s with the inputs resident in HBM (`value`), the same through the
host-memory entry point with the copies inside the timed region (`e2e`), the dominant kernel's
achieved bandwidth against the measured HBM peak (`roofline`), and the float64 CPU oracle timed
on the host cores (`cpu_baseline`).

--gpus N (under torchrun, one rank per GPU): the step does not shard without a collective this
library does not have, so the ranks run independent replicas of the workload; `value` is the sum.
--impl reference: times the CPU oracle as it stands (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "zeno_steps_per_sec"
UNIT = "steps/s"
L2_BYTES = 126 * 1024 * 1024
FALLBACK_HBM_GBS = 6650.0


# ----------------------------------------------------------------------------- helpers

def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as fh:
            d = json.load(fh)
        return float(d["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) from one ncu capture of
# the kernel on the named configuration (summaries under profiles/), valid only while the kernel's
# sources are unchanged.  Configuration 5 is too large to capture: its figure is the d = 2^22 case
# scaled by the parameters processed (reads x 16, the slab writes as they are).
_CSRC = "paper_1805_10032_b200/csrc/"
NCU_TRAFFIC = {
    ("0:stream_tf32x3", 2): {"bytes": 136.90e6, "sources": ["zeno_stream_tc.cu", "zeno_tc.cuh"],
                             "sha256_16": "3fefb930ccc7aac0"},
    ("2:layer_tc_head", 2): {"bytes": 25.34e6, "sources": ["zeno_layer_tc.cu", "zeno_tc.cuh"],
                             "sha256_16": "21d9b6d50ed88f88"},
    ("1:layer_tc", 3): {"bytes": 656.8e6, "sources": ["zeno_layer_tc.cu", "zeno_tc.cuh"],
                        "sha256_16": "21d9b6d50ed88f88"},
    ("1:layer_tc", 4): {"bytes": 1421.5e6, "sources": ["zeno_layer_tc.cu", "zeno_tc.cuh"],
                        "sha256_16": "21d9b6d50ed88f88"},
    ("2:layer_tc", 4): {"bytes": 1485.8e6, "sources": ["zeno_layer_tc.cu", "zeno_tc.cuh"],
                        "sha256_16": "21d9b6d50ed88f88"},
    ("0:lsq_tc", 5): {"bytes": 16 * 1359.08e6 + 3.8e6, "sources": ["zeno_lsq_tc.cu", "zeno_tc.cuh"],
                      "sha256_16": "7e611b2739f3b4f4"},
}


def measured_traffic(kernel_key, config):
    """kernel_key: position in the step and name, as in the per-kernel list ("0:stream_tf32x3")."""
    import hashlib
    ent = NCU_TRAFFIC.get((kernel_key, config))
    if not ent:
        return None
    try:
        digest = hashlib.sha256()
        for name in ent["sources"]:
            with open(os.path.join(ROOT, _CSRC + name), "rb") as fh:
                digest.update(fh.read())
        if digest.hexdigest()[:16] != ent["sha256_16"]:
            return None          # the kernel changed since the counters were taken
    except OSError:
        return None
    return ent["bytes"]


def algorithmic_bytes(w):
    """Bytes the step itself must move (padding excluded): the score pass reads V, x and the batch
    once; the aggregate pass reads the m-b selected rows once more and writes d floats."""
    s = 2 if w.dtype == "bf16" else 4
    feats = w.n_r * w.dims[0] * 4 + w.n_r * 4
    score = w.m * w.d * s + w.d * s + feats
    agg = (w.m - w.b) * w.d * s + w.d * 4
    return score, agg


def layer_bytes(w, layer):
    """Algorithmic bytes of one layer launch: that layer's slice of V (m rows) and of x, plus its
    input activations ((m+1) n_r in floats, or the shared features for layer 0) and outputs."""
    s = 2 if w.dtype == "bf16" else 4
    i, o = w.dims[layer], w.dims[layer + 1]
    params = o * i + (o if w.has_bias else 0)
    acts_in = w.n_r * i * 4 * (1 if layer == 0 else w.m + 1)
    acts_out = (w.m + 1) * w.n_r * o * 4
    return (w.m + 1) * params * s + acts_in + acts_out


class ClockSampler:
    """SM clock and throttle reasons read through NVML (read-only) by a background thread every
    few milliseconds while the timed regions run."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap"}

    def __init__(self, gpu_index, period_s=0.005):
        self.gpu, self.period = gpu_index, period_s
        self.samples, self.reason_bits, self.max_mhz = [], 0, None
        self._stop = None
        self._thread = None

    def start(self):
        import threading
        try:
            import pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            index = self.gpu
            if visible:
                ids = [v.strip() for v in visible.split(",") if v.strip()]
                if self.gpu < len(ids) and ids[self.gpu].isdigit():
                    index = int(ids[self.gpu])
            handle = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM))
        except Exception:
            return
        self._stop = threading.Event()

        def run():
            while not self._stop.is_set():
                try:
                    self.samples.append(float(pynvml.nvmlDeviceGetClockInfo(handle, pynvml.NVML_CLOCK_SM)))
                    self.reason_bits |= int(pynvml.nvmlDeviceGetCurrentClocksEventReasons(handle))
                except Exception:
                    pass
                self._stop.wait(self.period)

        self._thread = threading.Thread(target=run, daemon=True)
        self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join(timeout=2)
        out = {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": len(self.samples)}
        if self.samples:
            out["sm_mhz"] = statistics.median(self.samples)
        out["reasons"] = sorted(name for bit, name in self.REASONS.items() if self.reason_bits & bit)
        return out


def whole_job_rate(ms_local, units_per_rank, world, dist=None, device="cpu"):
    """Whole-job throughput from per-rank device times: the job takes as long as its slowest rank
    (MAX over ranks), and every rank contributed units_per_rank units.  Returns (units/s, ms)."""
    ms = float(ms_local)
    if dist is not None and world > 1:
        import torch
        t = torch.tensor([ms], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    return world * units_per_rank / (ms * 1e-3), ms


def kind_code(w):
    return 1 if w.kind == "lsq" else 0


def oracle_step_seconds(w, m_sample=None):
    """One oracle step on (a candidate subset of) the workload; returns (seconds, candidates)."""
    import numpy as np
    from oracle import zeno_oracle
    from paper_1805_10032_b200 import synthetic as syn
    m = w.m if m_sample is None else min(m_sample, w.m)
    b = min(w.b, m - 1)
    V = syn.to_numpy_params(w.V[:m])
    x = syn.to_numpy_params(w.x)
    f = w.features.cpu().numpy()
    t = w.targets.cpu().numpy()
    dt = 1 if w.dtype == "bf16" else 0
    t0 = time.perf_counter()
    zeno_oracle.step(kind_code(w), dt, w.dims, w.has_bias, x, V, w.ldv, m, f, t,
                     float(np.float32(w.gamma)), float(np.float32(w.rho)), b)
    return time.perf_counter() - t0, m


# ----------------------------------------------------------------------------- reference arm

def run_reference(args, rank, world):
    if rank != 0:
        return 0
    from oracle import zeno_oracle
    from paper_1805_10032_b200 import synthetic as syn
    zeno_oracle.build()
    w = syn.make_config(args.config)
    cores = zeno_oracle.num_threads()
    # bound the whole run to a few minutes: time one full step, then shrink the candidate sample
    t_full, _ = oracle_step_seconds(w)
    total_steps = args.steps + args.warmup
    budget = 150.0
    m_sample = w.m
    if t_full * total_steps > budget:
        m_sample = max(1, int((budget / total_steps) / t_full * (w.m + 1)) - 1)
    scale = (w.m + 1) / (m_sample + 1)     # the oracle's work is linear in the models evaluated
    for _ in range(args.warmup):
        oracle_step_seconds(w, m_sample)
    times = [oracle_step_seconds(w, m_sample)[0] * scale for _ in range(args.steps)]
    per_step = sum(times) / len(times)
    value = 1.0 / per_step
    sample = (f"all {w.m} candidates" if m_sample == w.m else
              f"first {m_sample} of {w.m} candidates per step, time scaled by (m+1)/(m_s+1)")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(w, args.config),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def workload_config(w, index):
    return {"workload": f"config{index}: {w.kind} dims={list(w.dims)} dtype={w.dtype} m={w.m} "
                        f"b={w.b} n_r={w.n_r} gamma={w.gamma} rho={w.rho} d={w.d} ldv={w.ldv}",
            "m": w.m, "b": w.b, "n_r": w.n_r, "d": w.d}


# ----------------------------------------------------------------------------- our arm

def run_ours(args, rank, world, local_rank):
    import torch
    from paper_1805_10032_b200 import build as zbuild
    from paper_1805_10032_b200 import synthetic as syn
    from paper_1805_10032_b200 import zeno

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the Zeno step has no CPU path")
    zbuild.build()
    dev = local_rank
    torch.cuda.set_device(dev)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", dev))

    # inputs: enough distinct sets that the rotation exceeds 4x the L2 capacity
    gen_device = "cuda" if args.config >= 3 else "cpu"      # the large workloads are generated on the device
    shrink = {"d": args.lsq_d} if (args.config == 5 and args.lsq_d > 0) else {}
    w0 = syn.make_config(args.config, device=gen_device, **shrink)
    score_b, agg_b = algorithmic_bytes(w0)
    set_bytes = w0.V.numel() * w0.V.element_size() + w0.features.numel() * 4
    n_sets = max(1, min(8, -(-4 * L2_BYTES // set_bytes)))
    sets = [w0] + [syn.make_config(args.config, seed=syn.BASE_SEED + args.config + 1000 * (i + 1),
                                   device=gen_device, **shrink) for i in range(n_sets - 1)]
    dsets = [(s.x.cuda(), s.V.cuda(), s.features.cuda(), s.targets.cuda()) for s in sets]
    z = zeno.from_workload(w0, device=dev)
    out = torch.empty(w0.d, dtype=torch.float32, device="cuda")
    scores = torch.empty(w0.m, dtype=torch.float32, device="cuda")
    idx = torch.empty(w0.m - w0.b, dtype=torch.int32, device="cuda")

    def step(i):
        x, V, f, t = dsets[i % n_sets]
        z.step(x, V, f, t, w0.gamma, w0.rho, w0.b, out=out, scores=scores, idx=idx)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    launches_per_step = 0
    step(0)
    launches_per_step = z.last_launch_count

    # ---- timed region 1: K steps, inputs resident in HBM
    sampler = ClockSampler(dev)
    sampler.start()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        step(i)
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    z.check_device_status()      # a kernel that gave up on a bounded wait voids the timing

    # ---- timed region 2: the same K steps with an event around every kernel; the steps are
    # enqueued in batches and read afterwards, so the GPU never waits for the host between events
    z.profile(True)
    per_kernel = {}
    order = []
    done = 0
    while done < args.steps:
        batch = min(48, args.steps - done)
        for i in range(batch):
            step(done + i)
        for back in range(batch - 1, -1, -1):
            for j, (name, ms) in enumerate(z.profile_read(back)):
                key = f"{j}:{name}"
                if key not in per_kernel:
                    per_kernel[key] = []
                    order.append(key)
                per_kernel[key].append(ms)
        done += batch
    z.profile(False)
    z.check_device_status()
    clocks = sampler.stop()

    value, ms_total = whole_job_rate(ms_total, args.steps, world, dist, "cuda")
    ms_per_step = ms_total / args.steps

    # ---- launch floor: as many of the library's smallest kernel (the one-block ranking of m scores)
    # back to back as a step has launches -- what the step would cost if its kernels did no work
    lib = zeno.load_library()
    floor_calls = 200
    def floor_pass():
        for _ in range(floor_calls * launches_per_step):
            lib.zeno_select(z._h, scores.data_ptr(), w0.m, w0.b, idx.data_ptr(), None)
    floor_pass()
    barrier()
    e0.record()
    floor_pass()
    e1.record()
    barrier()
    launch_floor_us = e0.elapsed_time(e1) * 1e3 / floor_calls

    # ---- end to end through the host-memory entry point (copies inside the timed region)
    hx, hV = sets[0].x.cpu().pin_memory(), sets[0].V.cpu().pin_memory()
    hf, ht = sets[0].features.cpu().pin_memory(), sets[0].targets.cpu().pin_memory()
    hout = torch.empty(w0.d, dtype=torch.float32).pin_memory()
    e2e_steps = max(3, min(args.steps, 20 if args.config <= 3 else 3))
    for _ in range(2):
        z.step_host(hx, hV, hf, ht, w0.gamma, w0.rho, w0.b, hout)
    barrier()
    t0 = time.perf_counter()
    e0.record()
    for _ in range(e2e_steps):
        z.step_host(hx, hV, hf, ht, w0.gamma, w0.rho, w0.b, hout)
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    e2e_value, e2e_ms = whole_job_rate(e2e_ms, e2e_steps, world, dist, "cuda")
    h2d = (hx.numel() * hx.element_size() + hV.numel() * hV.element_size() + hf.numel() * 4
           + ht.numel() * 4)
    d2h = hout.numel() * 4

    if rank != 0:
        return 0

    # ---- roofline of the dominant kernel
    peak, peak_kind = measured_peaks()
    kern = []
    for key in order:
        v = per_kernel[key]
        kern.append({"kernel": key, "avg_us": 1e3 * sum(v) / len(v)})
    total_us = sum(k["avg_us"] for k in kern) or 1.0
    for k in kern:
        k["share"] = k["avg_us"] / total_us
    top = max(kern, key=lambda k: k["avg_us"])
    top_name = top["kernel"].split(":")[1]
    # which dense layer a kernel of the list evaluates (the split-K combine belongs to none)
    layer_of, layer = {}, 0
    for k in kern:
        name = k["kernel"].split(":")[1]
        if name in ("stream_tf32x3", "layer_tc", "mlp_layer", "mlp_layer_mma", "mlp_head_loss_tail"):
            layer_of[k["kernel"]] = [layer]
            layer += 1
        elif name == "layer_tc_head":           # a hidden layer with the small last layer folded in
            layer_of[k["kernel"]] = [layer, layer + 1]
            layer += 2
    if top["kernel"] in layer_of:
        top_bytes = sum(layer_bytes(w0, l) for l in layer_of[top["kernel"]])
    elif top_name in ("lsq_stream", "lsq_tc"):
        top_bytes = score_b
    elif top_name == "aggregate":
        top_bytes = agg_b
    else:
        top_bytes = 0
    achieved = top_bytes / (top["avg_us"] * 1e-6) / 1e9
    step_bytes = score_b + agg_b
    roofline = {
        "bound": "hbm", "kernel": top["kernel"], "achieved": achieved, "peak": peak,
        "unit": "GB/s", "frac": achieved / peak, "traffic": None if shrink else measured_traffic(top["kernel"], args.config),
        "peak_source": peak_kind,
        "bytes_per_launch": top_bytes, "avg_us": top["avg_us"],
        "timed": "second pass over the same K steps, enqueued back to back with a CUDA event around every kernel",
        "launch_floor_us": launch_floor_us,
        "step": {"algorithmic_bytes": step_bytes,
                 "achieved_GBs": step_bytes / (ms_per_step * 1e-3) / 1e9,
                 "frac_of_hbm_peak": step_bytes / (ms_per_step * 1e-3) / 1e9 / peak,
                 "roofline_us": step_bytes / (peak * 1e9) * 1e6},
        "kernels": kern,
    }

    # ---- CPU baseline: the oracle on a bounded sample of the same workload
    from oracle import zeno_oracle
    zeno_oracle.build()
    t_full, _ = oracle_step_seconds(w0, None if args.config in (1, 2, 3) else 3)
    m_s = w0.m if args.config in (1, 2, 3) else 3
    reps = max(1, min(5, int(12.0 / max(t_full, 1e-3))))
    ts = [oracle_step_seconds(w0, m_s)[0] for _ in range(reps)]
    t_step = (sum(ts) / len(ts)) * (w0.m + 1) / (m_s + 1)
    cpu = {"value": 1.0 / t_step, "unit": UNIT, "cores": zeno_oracle.num_threads(), "kind": "oracle",
           "sample": (f"{reps} full steps" if m_s == w0.m else
                      f"{reps} steps over the first {m_s} of {w0.m} candidates, scaled by (m+1)/(m_s+1)")}

    cfg = workload_config(w0, args.config)
    cfg["l2_policy"] = (f"inputs rotate over {n_sets} distinct sets ({n_sets * set_bytes / 1e6:.0f} MB"
                        f" > 4x L2)" if n_sets > 1 else "one input set, larger than 4x L2")
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16/f32" if w0.dtype == "bf16" else "f32",
        "data": "synthetic", "config": cfg, "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps},
        "gpu_launches": launches_per_step * args.steps, "launches_per_step": launches_per_step,
        "roofline": roofline, "cpu_baseline": cpu,
    }
    print(json.dumps(line))
    z.close()
    if dist is not None:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", type=int, default=2, help="benchmark configuration 1..5 (default 2)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--lsq-d", type=int, default=0,
                    help="configuration 5 only: a smaller parameter count, for profiler captures of the "
                         "least-squares kernels on a case that holds a few GB (not a benchmark line)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        return run_reference(args, rank, world)
    return run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    sys.exit(main())
