#!/usr/bin/env python
"""Benchmark of the Zeno aggregation step (scores -> ranking -> trimmed mean).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]

One step = one zeno_step call: f_r(x), the m candidate losses f_r(x - gamma v_i) with the
squared norms, the top-(m-b) ranking and the trimmed mean, on one batch of synthetic input.

Without --config the run covers all five benchmark configurations: the headline numbers (`value`,
`ms_per_step`, `roofline`, `e2e`, `cpu_baseline`) are those of the largest single-GPU one,
configuration 5, timed over exactly K steps; `per_config` holds one record for each of
configurations 1-5 (its own step count, per-step percentiles, the dominant kernel's roofline, the
step-level fraction of the roofline, the launch floor, the clocks seen).  With --config C only that
configuration is timed (the form the profiler commands under profiles/ use).

Prints ONE JSON line: steps/s with the inputs resident in HBM (`value`), the same through the
host-memory entry point with the copies inside the timed region (`e2e`), the dominant kernel's
achieved bandwidth against the measured HBM peak (`roofline`), and the float64 CPU oracle timed
on the host cores (`cpu_baseline`).

--gpus N (under torchrun, one rank per GPU): the ranks run independent replicas of the workload
(no collective on the data path); `value` is the sum over ranks, timed as the slowest rank.
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
FALLBACK_BF16_TFLOPS = 1400.0          # sustained figure of the fallback measurement
NOMINAL_HBM_GBS = 8000.0               # the peak the target is stated against ("~8 TB/s")
TF32_OVER_BF16 = 1.1 / 2.25            # nominal dense tensor peaks: tf32 over bf16
HEADLINE_CONFIG = 5
# timed steps per configuration when the command line gives none
DEFAULT_STEPS = {1: 200, 2: 200, 3: 200, 4: 50, 5: 20}


# ----------------------------------------------------------------------------- helpers

def measured_peaks():
    """(HBM GB/s, sustained bf16 TFLOP/s, "measured" | "fallback")."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as fh:
            d = json.load(fh)
        return float(d["hbm_gbs"]), float(d.get("bf16_tflops_sustained", FALLBACK_BF16_TFLOPS)), "measured"
    return FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS, "fallback"


# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) from one ncu capture of
# the kernel on the named configuration (summaries under profiles/), valid only while the kernel's
# sources are unchanged.  Configuration 5 is too large to capture: its figure is the d = 2^22 case
# scaled by the parameters processed (reads x 16, the slab writes as they are).
_CSRC = "paper_1805_10032_b200/csrc/"
NCU_TRAFFIC = {
    ("0:lsq_tc", 5): {"bytes": 2.1751e+10, "sources": ["zeno_lsq_tc.cu", "zeno_tc.cuh"], "sha256_16": "1f142f64bf1a0db1"},
    ("1:layer_tc", 4): {"bytes": 1.4225e+09, "sources": ["zeno_layer_tc.cu", "zeno_tc.cuh"], "sha256_16": "f0b30a6b2bae6de9"},
    ("2:layer_tc", 4): {"bytes": 1.4892e+09, "sources": ["zeno_layer_tc.cu", "zeno_tc.cuh"], "sha256_16": "f0b30a6b2bae6de9"},
    ("3:layer_tc", 4): {"bytes": 3.6208e+08, "sources": ["zeno_layer_tc.cu", "zeno_tc.cuh"], "sha256_16": "f0b30a6b2bae6de9"},
    ("5:aggregate", 4): {"bytes": 1.6506e+09, "sources": ["zeno_aggregate.cu"], "sha256_16": "d4ebd34a19b63638"},
    ("1:layer_tc", 3): {"bytes": 6.5876e+08, "sources": ["zeno_layer_tc.cu", "zeno_tc.cuh"], "sha256_16": "f0b30a6b2bae6de9"},
    ("3:layer_tc", 3): {"bytes": 1.3774e+08, "sources": ["zeno_layer_tc.cu", "zeno_tc.cuh"], "sha256_16": "f0b30a6b2bae6de9"},
    ("0:stream_tf32x3", 2): {"bytes": 1.3695e+08, "sources": ["zeno_stream_tc.cu", "zeno_tc.cuh"], "sha256_16": "bfb9d41675540c43"},
    ("2:layer_tc_head", 2): {"bytes": 2.5343e+07, "sources": ["zeno_layer_tc.cu", "zeno_tc.cuh"], "sha256_16": "f0b30a6b2bae6de9"},
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


def algorithmic_flops(w):
    """2 n_r (#weights) (m + 1): one multiply-add per weight, sample and model."""
    if w.kind == "lsq":
        weights = w.d
    else:
        weights = sum(w.dims[l] * w.dims[l + 1] for l in range(len(w.dims) - 1))
    return 2.0 * w.n_r * weights * (w.m + 1)


def tensor_time_us(w, bf16_tflops):
    """Time of the step's contraction at the tensor peak of the type it runs in: bfloat16 models
    at the measured bf16 rate; binary32 models as three tf32 products per multiply-add (both
    operands split in two terms, the smallest product dropped) at bf16 x the nominal tf32/bf16
    ratio."""
    if w.dtype == "bf16":
        return algorithmic_flops(w) / (bf16_tflops * 1e12) * 1e6
    return 3.0 * algorithmic_flops(w) / (bf16_tflops * TF32_OVER_BF16 * 1e12) * 1e6


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


def percentile(sorted_vals, q):
    if not sorted_vals:
        return None
    pos = q * (len(sorted_vals) - 1)
    lo = int(pos)
    hi = min(lo + 1, len(sorted_vals) - 1)
    return sorted_vals[lo] + (sorted_vals[hi] - sorted_vals[lo]) * (pos - lo)


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


def input_sets(index):
    """How many distinct input sets the timed loop rotates over, and the bytes of one set."""
    from paper_1805_10032_b200 import synthetic as syn
    c = syn.describe_config(index)
    s = 2 if c["dtype"] == "bf16" else 4
    set_bytes = c["m"] * c["ldv"] * s + c["n_r"] * c["dims"][0] * 4
    return max(1, min(8, -(-4 * L2_BYTES // set_bytes))), set_bytes


def workload_config(index):
    """The `config` object of the JSON line: the same for both arms, built from the recipe alone."""
    from paper_1805_10032_b200 import synthetic as syn
    c = syn.describe_config(index)
    n_sets, set_bytes = input_sets(index)
    if n_sets == 1:
        l2 = "one input set, larger than 4x L2"
    elif n_sets * set_bytes > 4 * L2_BYTES:
        l2 = f"inputs rotate over {n_sets} distinct sets ({n_sets * set_bytes / 1e6:.0f} MB > 4x L2)"
    else:
        l2 = (f"inputs rotate over {n_sets} distinct sets ({n_sets * set_bytes / 1e6:.0f} MB); L2-resident: this "
              "configuration is bound by launch latency, not by bytes")
    return {"workload": f"config{index}: {c['kind']} dims={list(c['dims'])} dtype={c['dtype']} m={c['m']} "
                        f"b={c['b']} n_r={c['n_r']} gamma={c['gamma']} rho={c['rho']} d={c['d']} ldv={c['ldv']}",
            "m": c["m"], "b": c["b"], "n_r": c["n_r"], "d": c["d"], "l2_policy": l2}


def reference_workload(index, m_sample):
    """The configuration, or for the two largest ones a cut of m_sample honest candidates drawn by
    the same recipe: the host need not hold 17 GB of candidates to time a sample of them."""
    from paper_1805_10032_b200 import synthetic as syn
    if index == 5 and m_sample < 64:
        return syn.make_config(5, m=m_sample, b=min(24, m_sample - 1), n_noise=0)
    if index == 4 and m_sample < 32:
        return syn.make_config(4, m=m_sample, b=min(12, m_sample - 1), faults=[])
    return syn.make_config(index)


# ----------------------------------------------------------------------------- reference arm

# float64 oracle on the host cores: rough seconds per evaluated model (candidate or x itself) on a
# 16-core box, used only to pick a sample size before anything is generated
_ORACLE_MODEL_SECONDS = {1: 1e-5, 2: 0.008, 3: 0.016, 4: 2.5, 5: 0.9}


def run_reference(args, rank, world):
    if rank != 0:
        return 0
    from oracle import zeno_oracle
    zeno_oracle.build()
    index = args.config or HEADLINE_CONFIG
    steps = args.steps if args.steps else DEFAULT_STEPS[index]
    total_steps = steps + args.warmup
    budget = 150.0                       # seconds of oracle time for the whole run
    full_m = {1: 20, 2: 20, 3: 100, 4: 32, 5: 64}[index]
    per_model = _ORACLE_MODEL_SECONDS[index]
    m_sample = full_m
    if per_model * (full_m + 1) * total_steps > budget:
        m_sample = max(1, int(budget / total_steps / per_model) - 1)
        m_sample = min(m_sample, full_m)
    w = reference_workload(index, m_sample)
    cores = zeno_oracle.num_threads()
    scale = (full_m + 1) / (m_sample + 1)     # the oracle's work is linear in the models evaluated
    for _ in range(args.warmup):
        oracle_step_seconds(w, m_sample)
    times = [oracle_step_seconds(w, m_sample)[0] * scale for _ in range(steps)]
    per_step = sum(times) / len(times)
    value = 1.0 / per_step
    sample = (f"all {full_m} candidates" if m_sample == full_m else
              f"first {m_sample} of {full_m} candidates per step, time scaled by (m+1)/(m_s+1)")
    cfg = workload_config(index)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": cfg,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ----------------------------------------------------------------------------- our arm

class Runner:
    """State shared by the per-configuration measurements of one process."""

    def __init__(self, rank, world, local_rank):
        import torch
        self.torch = torch
        self.rank, self.world, self.dev = rank, world, local_rank
        self.dist = None
        torch.cuda.set_device(self.dev)
        if world > 1:
            import torch.distributed as dist
            dist.init_process_group("nccl", device_id=torch.device("cuda", self.dev))
            self.dist = dist
        self.hbm_peak, self.bf16_peak, self.peak_kind = measured_peaks()

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()


def bench_config(R, index, steps, warmup, headline):
    """Times one configuration.  Returns (record, extras): the per-configuration record and, for
    the headline configuration, what the top-level JSON keys need."""
    torch = R.torch
    from paper_1805_10032_b200 import synthetic as syn
    from paper_1805_10032_b200 import zeno

    # inputs: enough distinct sets that the rotation exceeds 4x the L2 capacity (at most 8 sets:
    # configuration 1 stays L2-resident whatever is done, it is bound by launch latency)
    gen_device = "cuda" if index >= 3 else "cpu"      # the large workloads are generated on the device
    w0 = syn.make_config(index, device=gen_device)
    score_b, agg_b = algorithmic_bytes(w0)
    n_sets, set_bytes = input_sets(index)
    sets = [w0] + [syn.make_config(index, seed=syn.BASE_SEED + index + 1000 * (i + 1), device=gen_device)
                   for i in range(n_sets - 1)]
    dsets = [(s.x.cuda(), s.V.cuda(), s.features.cuda(), s.targets.cuda()) for s in sets]
    z = zeno.from_workload(w0, device=R.dev)
    out = torch.empty(w0.d, dtype=torch.float32, device="cuda")
    scores = torch.empty(w0.m, dtype=torch.float32, device="cuda")
    idx = torch.empty(w0.m - w0.b, dtype=torch.int32, device="cuda")

    def step(i):
        x, V, f, t = dsets[i % n_sets]
        z.step(x, V, f, t, w0.gamma, w0.rho, w0.b, out=out, scores=scores, idx=idx)

    for i in range(warmup):
        step(i)
    step(0)
    launches_per_step = z.last_launch_count

    # ---- timed region 1: K steps, inputs resident in HBM
    sampler = ClockSampler(R.dev)
    sampler.start()
    R.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        step(i)
    e1.record()
    R.barrier()
    ms_total = e0.elapsed_time(e1)
    z.check_device_status()      # a kernel that gave up on a bounded wait voids the timing

    # ---- per-step times for the percentiles: the same K steps with an event between steps
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    marks[0].record()
    for i in range(steps):
        step(i)
        marks[i + 1].record()
    torch.cuda.synchronize()
    per_step_us = sorted(marks[i].elapsed_time(marks[i + 1]) * 1e3 for i in range(steps))

    # ---- timed region 2: the same K steps with an event around every kernel; the steps are
    # enqueued in batches and read afterwards, so the GPU never waits for the host between events
    z.profile(True)
    per_kernel = {}
    order = []
    done = 0
    while done < steps:
        batch = min(48, steps - done)
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

    value, ms_total = whole_job_rate(ms_total, steps, R.world, R.dist, "cuda")
    ms_per_step = ms_total / steps

    # ---- launch floor: as many of the library's smallest kernel (the one-block ranking of m scores)
    # back to back as a step has launches -- what the step would cost if its kernels did no work
    lib = zeno.load_library()
    floor_calls = 200

    def floor_pass():
        for _ in range(floor_calls * launches_per_step):
            lib.zeno_select(z._h, scores.data_ptr(), w0.m, w0.b, idx.data_ptr(), None)
    floor_pass()
    R.barrier()
    e0.record()
    floor_pass()
    e1.record()
    R.barrier()
    launch_floor_us = e0.elapsed_time(e1) * 1e3 / floor_calls

    extras = {}
    if headline:
        # ---- end to end through the host-memory entry point (copies inside the timed region)
        hx, hV = sets[0].x.cpu().pin_memory(), sets[0].V.cpu().pin_memory()
        hf, ht = sets[0].features.cpu().pin_memory(), sets[0].targets.cpu().pin_memory()
        hout = torch.empty(w0.d, dtype=torch.float32).pin_memory()
        e2e_steps = max(3, min(steps, 20 if index <= 3 else 3))
        for _ in range(2):
            z.step_host(hx, hV, hf, ht, w0.gamma, w0.rho, w0.b, hout)
        R.barrier()
        e0.record()
        for _ in range(e2e_steps):
            z.step_host(hx, hV, hf, ht, w0.gamma, w0.rho, w0.b, hout)
        e1.record()
        R.barrier()
        e2e_value, _ = whole_job_rate(e0.elapsed_time(e1), e2e_steps, R.world, R.dist, "cuda")
        h2d = (hx.numel() * hx.element_size() + hV.numel() * hV.element_size() + hf.numel() * 4
               + ht.numel() * 4)
        extras["e2e"] = {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d,
                         "d2h_bytes_per_step": hout.numel() * 4, "steps": e2e_steps}
        del hx, hV, hf, ht, hout

    # ---- roofline of the dominant kernel and of the whole step
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
    hbm_us = step_bytes / (R.hbm_peak * 1e9) * 1e6
    tensor_us = tensor_time_us(w0, R.bf16_peak)
    roofline_us = max(hbm_us, tensor_us)
    roofline = {
        "bound": "hbm" if hbm_us >= tensor_us else "tensor", "kernel": top["kernel"], "achieved": achieved,
        "peak": R.hbm_peak, "unit": "GB/s", "frac": achieved / R.hbm_peak,
        "frac_of_nominal_peak": achieved / NOMINAL_HBM_GBS,
        "traffic": measured_traffic(top["kernel"], index), "peak_source": R.peak_kind,
        "bytes_per_launch": top_bytes, "avg_us": top["avg_us"],
        "timed": "second pass over the same K steps, enqueued back to back with a CUDA event around every kernel",
        "launch_floor_us": launch_floor_us,
        # the step against its roofline = the slower of its bytes at the HBM peak and its flops at the tensor peak
        "step": {"algorithmic_bytes": step_bytes, "algorithmic_flops": algorithmic_flops(w0),
                 "hbm_us": hbm_us, "tensor_us": tensor_us, "roofline_us": roofline_us,
                 "achieved_GBs": step_bytes / (ms_per_step * 1e-3) / 1e9,
                 "frac_of_measured_peak": roofline_us / (ms_per_step * 1e3),
                 "frac_of_nominal_peak": max(step_bytes / (NOMINAL_HBM_GBS * 1e9) * 1e6, tensor_us) / (ms_per_step * 1e3),
                 "target": "0.70 of the roofline, judged against the measured peak"},
        "kernels": kern,
    }
    cfg = workload_config(index)
    record = {"config": index, "workload": cfg["workload"], "steps": steps, "warmup": warmup,
              "value": value, "ms_per_step": ms_per_step,
              "p10_us": percentile(per_step_us, 0.10), "p50_us": percentile(per_step_us, 0.50),
              "p90_us": percentile(per_step_us, 0.90),
              "launches_per_step": launches_per_step, "launch_floor_us": launch_floor_us,
              "step_over_launch_floor": ms_per_step * 1e3 / launch_floor_us if launch_floor_us else None,
              "step_frac_of_roofline": roofline["step"]["frac_of_measured_peak"],
              "l2_policy": cfg["l2_policy"], "clocks": clocks, "roofline": roofline}
    extras.update(cfg=cfg, roofline=roofline, clocks=clocks, value=value, ms_per_step=ms_per_step,
                  launches_per_step=launches_per_step, dtype="bf16/f32" if w0.dtype == "bf16" else "f32")

    if headline and R.rank == 0 and R.world == 1:
        # ---- CPU baseline: the oracle on a bounded sample of the same workload
        from oracle import zeno_oracle
        zeno_oracle.build()
        m_s = w0.m if index in (1, 2, 3) else 3
        t_full, _ = oracle_step_seconds(w0, m_s)
        reps = max(1, min(5, int(12.0 / max(t_full, 1e-3))))
        ts = [oracle_step_seconds(w0, m_s)[0] for _ in range(reps)]
        t_step = (sum(ts) / len(ts)) * (w0.m + 1) / (m_s + 1)
        extras["cpu_baseline"] = {
            "value": 1.0 / t_step, "unit": UNIT, "cores": zeno_oracle.num_threads(), "kind": "oracle",
            "sample": (f"{reps} full steps" if m_s == w0.m else
                       f"{reps} steps over the first {m_s} of {w0.m} candidates, scaled by (m+1)/(m_s+1)")}

    z.close()
    del dsets, sets, w0, out, scores, idx
    torch.cuda.empty_cache()
    return record, extras


def run_ours(args, rank, world, local_rank):
    import torch
    from paper_1805_10032_b200 import build as zbuild

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the Zeno step has no CPU path")
    zbuild.build()
    R = Runner(rank, world, local_rank)
    headline = args.config or HEADLINE_CONFIG
    todo = [args.config] if args.config else [1, 2, 3, 4, 5]
    records, head = [], None
    for index in todo:
        is_head = index == headline
        steps = args.steps if (args.steps and (is_head or args.config)) else max(args.steps or 0, DEFAULT_STEPS[index])
        record, extras = bench_config(R, index, steps, args.warmup, is_head)
        records.append(record)
        if is_head:
            head = (record, extras)
    R.close()
    if rank != 0:
        return 0
    record, ex = head
    line = {
        "metric": METRIC, "value": ex["value"], "unit": UNIT, "n_gpus": world, "steps": record["steps"],
        "warmup": args.warmup, "ms_per_step": ex["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": ex["dtype"],
        "data": "synthetic", "config": ex["cfg"], "clocks": ex["clocks"],
        "e2e": ex.get("e2e"),
        "gpu_launches": ex["launches_per_step"] * record["steps"], "launches_per_step": ex["launches_per_step"],
        "roofline": ex["roofline"], "cpu_baseline": ex.get("cpu_baseline"),
    }
    if not args.config:
        line["per_config"] = records
    else:
        line["percentiles_us"] = {"p10": record["p10_us"], "p50": record["p50_us"], "p90": record["p90_us"]}
    print(json.dumps(line))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0,
                    help="timed steps of the headline configuration (default: 200 for configurations 1-3, "
                         "50 for 4, 20 for 5); the other configurations of a full run take at least their defaults")
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", type=int, default=0, choices=[0, 1, 2, 3, 4, 5],
                    help="time only this benchmark configuration (default: all five, configuration 5 as the headline)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
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
