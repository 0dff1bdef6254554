"""Seeded synthetic inputs for the Zeno aggregation step.

This module builds the *inputs* of the step -- the current parameters x, the
matrix V of m candidate gradients (honest rows plus faulty rows of the kinds
the paper's experiments use: sign-flipped copies, large Gaussian noise, an
omniscient-style scaled negative mean), and the server's small batch -- and
nothing else.  It contains none of the aggregation rule's arithmetic (no score,
no ranking, no trimmed mean) and imports neither the CUDA binding nor the CPU
oracle; both are handed the very same buffers it returns.

The honest gradient g is what a worker would send (Algorithm 1, worker side):
the gradient of the model's mean loss on a separate seeded batch of
``worker_batch`` samples, obtained here with torch autograd.

Workloads 1-5 follow the five benchmark configurations; each recipe takes
overrides so that tests can shrink it while keeping its structure.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional, Sequence

import torch

BASE_SEED = 20260101


@dataclass
class Workload:
    name: str
    kind: str                 # "mlp" (softmax cross-entropy ReLU MLP), "lsq" (least squares) or "cnn"
    dtype: str                # storage type of x and V: "f32" or "bf16"
    dims: tuple               # mlp: layer widths (in, hidden..., classes); lsq: (d, 1);
                              # cnn: (S, C_0, C_1, .., C_Lc, classes): image side, planes per layer, classes
    has_bias: bool
    m: int
    b: int
    n_r: int
    gamma: float
    rho: float
    d: int
    ldv: int
    x: torch.Tensor           # [d]
    V: torch.Tensor           # [m, ldv]; columns >= d are padding (NaN for f32/bf16)
    features: torch.Tensor    # [n_r, dims[0]] float32 (cnn: [n_r, C_0, S, S])
    targets: torch.Tensor     # int32 labels [n_r] (mlp) or float32 y [n_r] (lsq)
    honest: torch.Tensor = field(default=None)  # bool [m], which rows are honest (metadata only)
    seed: int = 0


def param_count(kind: str, dims: Sequence[int], has_bias: bool = True) -> int:
    if kind == "lsq":
        return int(dims[0])
    if kind == "cnn":
        side, chans, classes = dims[0], dims[1:-1], dims[-1]
        lc = len(chans) - 1
        conv = sum(chans[l] * chans[l - 1] * 9 + (chans[l] if has_bias else 0) for l in range(1, lc + 1))
        side //= 2 ** (lc // 2)
        return int(conv + classes * chans[-1] * side * side + (classes if has_bias else 0))
    return int(sum(dims[l + 1] * dims[l] + (dims[l + 1] if has_bias else 0)
                   for l in range(len(dims) - 1)))


def round_up(n: int, q: int) -> int:
    return (n + q - 1) // q * q


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _randn(shape, gen, device, std=1.0):
    return torch.randn(shape, generator=gen, device=device, dtype=torch.float32) * std


def _split_params(flat: torch.Tensor, dims, has_bias):
    """Views of the flat parameter vector: per layer W [out x in] row-major, then b [out]."""
    out = []
    off = 0
    for l in range(len(dims) - 1):
        i, o = dims[l], dims[l + 1]
        W = flat[off:off + o * i].view(o, i)
        off += o * i
        bvec = None
        if has_bias:
            bvec = flat[off:off + o]
            off += o
        out.append((W, bvec))
    return out


def he_init(dims, has_bias, gen, device) -> torch.Tensor:
    """He-initialised weights N(0, 2/fan_in), zero biases, in the flat layout."""
    parts = []
    for l in range(len(dims) - 1):
        i, o = dims[l], dims[l + 1]
        parts.append(_randn((o * i,), gen, device, (2.0 / i) ** 0.5))
        if has_bias:
            parts.append(torch.zeros(o, device=device))
    return torch.cat(parts)


def mlp_gradient(x_flat: torch.Tensor, dims, has_bias, feats, labels) -> torch.Tensor:
    """A worker's gradient of the mean softmax cross-entropy (torch autograd, float32)."""
    p = x_flat.detach().clone().float().requires_grad_(True)
    h = feats
    layers = _split_params(p, dims, has_bias)
    for l, (W, bvec) in enumerate(layers):
        h = torch.nn.functional.linear(h, W, bvec)
        if l + 1 < len(layers):
            h = torch.relu(h)
    loss = torch.nn.functional.cross_entropy(h, labels.long())
    (g,) = torch.autograd.grad(loss, p)
    return g.detach()


def _store(t: torch.Tensor, dtype: str) -> torch.Tensor:
    return t.to(torch.bfloat16) if dtype == "bf16" else t.float()


def _alloc_V(m, d, ldv, dtype, device):
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    V = torch.empty((m, ldv), dtype=tdt, device=device)
    if ldv > d:
        V[:, d:] = float("nan")   # padding must never be read as data
    return V


def _shuffle_rows(m, gen_cpu):
    return torch.randperm(m, generator=gen_cpu)


def make_mlp_workload(name, seed, dims, dtype, m, b, n_r, gamma, rho, honest_std, faults,
                      x_init="he", worker_batch=100, ldv: Optional[int] = None,
                      device="cpu", has_bias=True) -> Workload:
    """faults: list of (count, kind) with kind in
         "signflip"  : -4 * g (all copies identical, as in the paper's bit-flip experiment)
         "noise200"  : i.i.d. N(0, 200^2)
         "omniscient": -1e3 * mean(honest rows)
    """
    dims = tuple(int(v) for v in dims)
    d = param_count("mlp", dims, has_bias)
    ldv = round_up(d, 32) if ldv is None else int(ldv)
    gen = _gen(seed, device)
    gen_cpu = _gen(seed + 7919, "cpu")
    classes = dims[-1]

    if x_init == "he":
        x32 = he_init(dims, has_bias, gen, device)
    else:  # "normal0.1": N(0, variance 0.01)
        x32 = _randn((d,), gen, device, 0.1)
    x = _store(x32, dtype)

    feats = _randn((n_r, dims[0]), gen, device)
    labels = torch.randint(0, classes, (n_r,), generator=gen, device=device, dtype=torch.int32)
    wfeats = _randn((worker_batch, dims[0]), gen, device)
    wlabels = torch.randint(0, classes, (worker_batch,), generator=gen, device=device,
                            dtype=torch.int32)
    g = mlp_gradient(x.float(), dims, has_bias, wfeats, wlabels)

    n_faulty = sum(c for c, _ in faults)
    n_honest = m - n_faulty
    assert n_honest >= 1
    perm = _shuffle_rows(m, gen_cpu)
    V = _alloc_V(m, d, ldv, dtype, device)
    honest = torch.zeros(m, dtype=torch.bool)
    honest_sum = torch.zeros(d, device=device, dtype=torch.float32)
    slot = 0
    for _ in range(n_honest):
        row = _store(g + _randn((d,), gen, device, honest_std), dtype)
        V[perm[slot], :d] = row
        honest[perm[slot]] = True
        honest_sum += row.float()
        slot += 1
    for count, kind in faults:
        if kind == "signflip":
            row = _store(-4.0 * g, dtype)
        elif kind == "omniscient":
            row = _store(-1e3 * (honest_sum / n_honest), dtype)
        for _ in range(count):
            if kind == "noise200":
                row = _store(_randn((d,), gen, device, 200.0), dtype)
            V[perm[slot], :d] = row
            slot += 1
    return Workload(name=name, kind="mlp", dtype=dtype, dims=dims, has_bias=has_bias, m=m, b=b,
                    n_r=n_r, gamma=gamma, rho=rho, d=d, ldv=ldv, x=x, V=V, features=feats,
                    targets=labels, honest=honest, seed=seed)


def _cnn_split(flat, dims, has_bias):
    """Views of the flat parameter vector: [(W[C_l, C_{l-1}, 3, 3], b or None)] and the dense (W, b)."""
    side, chans, classes = dims[0], dims[1:-1], dims[-1]
    lc = len(chans) - 1
    off, conv = 0, []
    for l in range(1, lc + 1):
        n = chans[l] * chans[l - 1] * 9
        W = flat[off:off + n].view(chans[l], chans[l - 1], 3, 3)
        off += n
        bvec = None
        if has_bias:
            bvec = flat[off:off + chans[l]]
            off += chans[l]
        conv.append((W, bvec))
    side //= 2 ** (lc // 2)
    n = classes * chans[-1] * side * side
    W = flat[off:off + n].view(classes, chans[-1] * side * side)
    off += n
    bvec = flat[off:off + classes] if has_bias else None
    return conv, (W, bvec)


def cnn_he_init(dims, has_bias, gen, device) -> torch.Tensor:
    """He-initialised weights N(0, 2/fan_in), zero biases, in the flat layout."""
    side, chans, classes = dims[0], dims[1:-1], dims[-1]
    lc = len(chans) - 1
    parts = []
    for l in range(1, lc + 1):
        parts.append(_randn((chans[l] * chans[l - 1] * 9,), gen, device, (2.0 / (chans[l - 1] * 9)) ** 0.5))
        if has_bias:
            parts.append(torch.zeros(chans[l], device=device))
    side //= 2 ** (lc // 2)
    flat = chans[-1] * side * side
    parts.append(_randn((classes * flat,), gen, device, (2.0 / flat) ** 0.5))
    if has_bias:
        parts.append(torch.zeros(classes, device=device))
    return torch.cat(parts)


def cnn_gradient(x_flat, dims, has_bias, feats, labels) -> torch.Tensor:
    """A worker's gradient of the network's mean cross-entropy (torch autograd, float32): input data for the
    candidates, like mlp_gradient."""
    p = x_flat.detach().clone().float().requires_grad_(True)
    conv, (W, bvec) = _cnn_split(p, dims, has_bias)
    h = feats
    for l, (Wc, bc) in enumerate(conv, start=1):
        h = torch.relu(torch.nn.functional.conv2d(h, Wc, bc, padding=1))
        if l % 2 == 0:
            h = torch.nn.functional.max_pool2d(h, 2)
    z = torch.nn.functional.linear(h.flatten(1), W, bvec)
    loss = torch.nn.functional.cross_entropy(z, labels.long())
    (g,) = torch.autograd.grad(loss, p)
    return g.detach()


def make_cnn_workload(name, seed, dims, dtype, m, b, n_r, gamma, rho, honest_std, faults, worker_batch=32,
                      ldv: Optional[int] = None, device="cpu", has_bias=True) -> Workload:
    """The convolutional model: images N(0, 1), uniform labels, He-initialised x, honest rows = a worker's
    gradient + N(0, honest_std^2), faults as in make_mlp_workload."""
    dims = tuple(int(v) for v in dims)
    d = param_count("cnn", dims, has_bias)
    ldv = round_up(d, 32) if ldv is None else int(ldv)
    gen = _gen(seed, device)
    gen_cpu = _gen(seed + 7919, "cpu")
    side, c0, classes = dims[0], dims[1], dims[-1]
    x = _store(cnn_he_init(dims, has_bias, gen, device), dtype)
    feats = _randn((n_r, c0, side, side), gen, device)
    labels = torch.randint(0, classes, (n_r,), generator=gen, device=device, dtype=torch.int32)
    wfeats = _randn((worker_batch, c0, side, side), gen, device)
    wlabels = torch.randint(0, classes, (worker_batch,), generator=gen, device=device, dtype=torch.int32)
    g = cnn_gradient(x.float(), dims, has_bias, wfeats, wlabels)
    n_faulty = sum(c for c, _ in faults)
    n_honest = m - n_faulty
    assert n_honest >= 1
    perm = _shuffle_rows(m, gen_cpu)
    V = _alloc_V(m, d, ldv, dtype, device)
    honest = torch.zeros(m, dtype=torch.bool)
    honest_sum = torch.zeros(d, device=device, dtype=torch.float32)
    slot = 0
    for _ in range(n_honest):
        row = _store(g + _randn((d,), gen, device, honest_std), dtype)
        V[perm[slot], :d] = row
        honest[perm[slot]] = True
        honest_sum += row.float()
        slot += 1
    for count, kind in faults:
        if kind == "signflip":
            row = _store(-4.0 * g, dtype)
        elif kind == "omniscient":
            row = _store(-1e3 * (honest_sum / n_honest), dtype)
        for _ in range(count):
            if kind == "noise200":
                row = _store(_randn((d,), gen, device, 200.0), dtype)
            V[perm[slot], :d] = row
            slot += 1
    return Workload(name=name, kind="cnn", dtype=dtype, dims=dims, has_bias=has_bias, m=m, b=b, n_r=n_r,
                    gamma=gamma, rho=rho, d=d, ldv=ldv, x=x, V=V, features=feats, targets=labels,
                    honest=honest, seed=seed)


def make_lsq_workload(name, seed, d, m, b, n_r, gamma, rho, honest_std, n_noise, noise_std,
                      ldv: Optional[int] = None, device="cpu") -> Workload:
    """f(x) = ||A x - y||^2 / (2 n_r); A entries N(0, variance 1/d), y ~ N(0,1), x ~ N(0,1);
    honest rows = grad f(x) + N(0, honest_std^2); faulty rows = N(0, noise_std^2)."""
    d = int(d)
    ldv = round_up(d, 32) if ldv is None else int(ldv)
    gen = _gen(seed, device)
    gen_cpu = _gen(seed + 7919, "cpu")
    x = _randn((d,), gen, device)
    A = torch.empty((n_r, d), dtype=torch.float32, device=device)
    for j in range(n_r):
        A[j] = _randn((d,), gen, device, d ** -0.5)
    y = _randn((n_r,), gen, device)
    g = (A.t() @ (A @ x - y)) / n_r          # grad f(x) = A^T (A x - y) / n_r
    perm = _shuffle_rows(m, gen_cpu)
    V = _alloc_V(m, d, ldv, "f32", device)
    honest = torch.zeros(m, dtype=torch.bool)
    for s in range(m):
        if s < m - n_noise:
            V[perm[s], :d] = g + _randn((d,), gen, device, honest_std)
            honest[perm[s]] = True
        else:
            V[perm[s], :d] = _randn((d,), gen, device, noise_std)
    return Workload(name=name, kind="lsq", dtype="f32", dims=(d, 1), has_bias=False, m=m, b=b,
                    n_r=n_r, gamma=gamma, rho=rho, d=d, ldv=ldv, x=x, V=V, features=A,
                    targets=y, honest=honest, seed=seed)


# The five benchmark configurations (1-based): recipe parameters only, no tensors.
CONFIGS = {
    1: dict(dims=(784, 10), dtype="f32", m=20, b=8, n_r=4, gamma=0.1, rho=5e-4,
            honest_std=0.1, faults=[(8, "signflip")], x_init="normal0.1"),
    2: dict(dims=(3072, 512, 512, 10), dtype="f32", m=20, b=8, n_r=32, gamma=0.1, rho=5e-4,
            honest_std=0.1, faults=[(8, "noise200")]),
    3: dict(dims=(3072, 512, 512, 10), dtype="f32", m=100, b=40, n_r=64, gamma=0.05,
            rho=1e-3, honest_std=0.1, faults=[(20, "signflip"), (20, "omniscient")]),
    4: dict(dims=(4096, 4096, 4096, 1000), dtype="bf16", m=32, b=12, n_r=128, gamma=0.1,
            rho=5e-4, honest_std=0.05, faults=[(12, "signflip")]),
    5: dict(d=1 << 26, m=64, b=24, n_r=16, gamma=0.01, rho=1e-4, honest_std=0.01,
            n_noise=24, noise_std=100.0),
    # the shape of the paper's own experiment: a CNN of four convolutional layers and a dense one on
    # 32 x 32 x 3 images, 20 workers, 8 of them faulty, n_r = 4 (the network's widths are this project's)
    6: dict(dims=(32, 3, 32, 32, 64, 64, 10), dtype="f32", m=20, b=8, n_r=4, gamma=0.1, rho=5e-4,
            honest_std=0.02, faults=[(8, "signflip")]),
}


def describe_config(index: int) -> dict:
    """Shape of a benchmark configuration without generating it: kind, dims, dtype, m, b, n_r,
    gamma, rho, d, ldv (the default row pitch)."""
    p = CONFIGS[index]
    if index == 5:
        kind, dims, dtype = "lsq", (p["d"], 1), "f32"
    elif index == 6:
        kind, dims, dtype = "cnn", tuple(p["dims"]), p["dtype"]
    else:
        kind, dims, dtype = "mlp", tuple(p["dims"]), p["dtype"]
    d = param_count(kind, dims)
    return dict(kind=kind, dims=dims, dtype=dtype, m=p["m"], b=p["b"], n_r=p["n_r"], gamma=p["gamma"],
                rho=p["rho"], d=d, ldv=round_up(d, 32))


def make_config(index: int, device="cpu", **ov) -> Workload:
    """The five benchmark configurations (1-based).  Keyword overrides shrink a
    configuration for tests (e.g. dims=(96, 40, 24, 10), m=9, b=3, n_r=5)."""
    seed = ov.pop("seed", BASE_SEED + index)
    if index not in CONFIGS:
        raise ValueError("config index must be 1..6")
    p = dict(CONFIGS[index])
    p.update(ov)
    if index == 5:
        return make_lsq_workload("config5", seed, device=device, **p)
    if index == 6:
        return make_cnn_workload("config6", seed, device=device, **p)
    return make_mlp_workload(f"config{index}", seed, device=device, **p)


# ---- host views for a CPU consumer ------------------------------------------------

def to_numpy_params(t: torch.Tensor):
    """float32 tensors as float32 arrays; bfloat16 tensors as uint16 bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view("uint16")
    return t.numpy()
