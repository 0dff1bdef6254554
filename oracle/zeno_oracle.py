"""ctypes front end of the float64 CPU oracle (oracle/zeno_oracle.c).

TEST INFRASTRUCTURE.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this module; the CUDA library and its Python
binding never do.  It holds no arithmetic of its own: every number comes from
the C file, which states Definition 2 (score) and Definition 3 (aggregation)
of the Zeno paper in plain double precision.

Arrays are numpy: float32 parameters as float32 arrays, bfloat16 parameters
as uint16 arrays holding the raw bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "zeno_oracle.c")
_LIB = os.path.join(_HERE, "libzeno_oracle.so")

LOSS_SOFTMAX_MLP = 0
LOSS_LEAST_SQUARES = 1
LOSS_SOFTMAX_CNN = 2      # dims = [S, C_0, C_1, .., C_Lc, classes]: Lc convolutional layers and a dense one
F32 = 0
BF16 = 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP over candidates)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fopenmp", "-fno-fast-math", "-shared", "-fPIC",
             "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        i32, i64, dbl, vp = ctypes.c_int, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        lib.zo_param_count.restype = i64
        lib.zo_param_count.argtypes = [i32, i32, vp, i32]
        lib.zo_round_to_bf16.restype = dbl
        lib.zo_round_to_bf16.argtypes = [ctypes.c_float]
        lib.zo_candidate_params.restype = None
        lib.zo_candidate_params.argtypes = [vp, vp, i64, i32, dbl, vp]
        lib.zo_loss.restype = dbl
        lib.zo_loss.argtypes = [i32, i32, vp, i32, vp, vp, vp, i32]
        lib.zo_score.restype = i32
        lib.zo_score.argtypes = [i32, i32, i32, vp, i32, vp, vp, i64, i32, vp, vp, i32,
                                 dbl, dbl, vp, vp, vp]
        lib.zo_select.restype = i32
        lib.zo_select.argtypes = [vp, i32, i32, vp]
        lib.zo_aggregate.restype = i32
        lib.zo_aggregate.argtypes = [i32, vp, i64, i64, i32, vp, i32, vp]
        lib.zo_update.restype = None
        lib.zo_update.argtypes = [vp, vp, i64, i32, dbl, vp]
        lib.zo_step.restype = i32
        lib.zo_step.argtypes = [i32, i32, i32, vp, i32, vp, vp, i64, i32, vp, vp, i32,
                                dbl, dbl, i32, vp, vp, vp]
        lib.zo_worker_gradient.restype = i32
        lib.zo_worker_gradient.argtypes = [i32, i32, vp, i32, vp, i32, vp, vp, i32, i32, vp]
        lib.zo_inject_faults.restype = i32
        lib.zo_inject_faults.argtypes = [vp, i64, i32, vp, i32, i32, dbl]
        lib.zo_median.restype = i32
        lib.zo_median.argtypes = [i32, vp, i64, i64, i32, vp]
        lib.zo_krum.restype = i32
        lib.zo_krum.argtypes = [i32, vp, i64, i64, i32, i32, vp, vp, vp]
        lib.zo_cnn_logits.restype = i32
        lib.zo_cnn_logits.argtypes = [i32, vp, i32, vp, vp, vp]
        lib.zo_eval_count.restype = ctypes.c_longlong
        lib.zo_reset_eval_count.restype = None
        lib.zo_num_threads.restype = i32
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _dims(dims):
    return np.ascontiguousarray(np.asarray(dims, dtype=np.int64))


def _n_layers(kind, dm):
    """Layers a dims list describes: its widths minus one, or (convolutional network) minus two,
    since that list starts with the image side."""
    return len(dm) - 2 if kind == LOSS_SOFTMAX_CNN else len(dm) - 1


def _params(a, dtype):
    want = np.uint16 if dtype == BF16 else np.float32
    a = np.ascontiguousarray(a)
    if a.dtype != want:
        raise TypeError(f"parameter array must be {want.__name__}, got {a.dtype}")
    return a


def _targets(kind, t):
    want = np.float32 if kind == LOSS_LEAST_SQUARES else np.int32
    t = np.ascontiguousarray(t)
    if t.dtype != want:
        raise TypeError(f"targets must be {want.__name__}, got {t.dtype}")
    return t


def _features(f):
    f = np.ascontiguousarray(f)
    if f.dtype != np.float32:
        raise TypeError("features must be float32")
    return f


def _check(rc, what):
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


def num_threads() -> int:
    return int(_load().zo_num_threads())


def eval_count() -> int:
    return int(_load().zo_eval_count())


def reset_eval_count() -> None:
    _load().zo_reset_eval_count()


def param_count(kind, dims, has_bias=True) -> int:
    dm = _dims(dims)
    return int(_load().zo_param_count(kind, _n_layers(kind, dm), _ptr(dm), int(has_bias)))


def round_to_bf16(f: float) -> float:
    return float(_load().zo_round_to_bf16(ctypes.c_float(f)))


def candidate_params(x, v, dtype, gamma):
    """w = x - gamma * v as float64 (v=None: w = x)."""
    x = _params(x, dtype)
    d = x.shape[0]
    if v is not None:
        v = _params(v, dtype)
    w = np.empty(d, dtype=np.float64)
    _load().zo_candidate_params(_ptr(x), _ptr(v), d, dtype, float(gamma), _ptr(w))
    return w


def loss(kind, dims, has_bias, w, features, targets):
    """f_r(w) for a float64 parameter vector w."""
    dm = _dims(dims)
    w = np.ascontiguousarray(w, dtype=np.float64)
    features = _features(features)
    targets = _targets(kind, targets)
    n_r = targets.shape[0]
    return float(_load().zo_loss(kind, _n_layers(kind, dm), _ptr(dm), int(has_bias), _ptr(w),
                                 _ptr(features), _ptr(targets), n_r))


def cnn_logits(dims, has_bias, w, feat):
    """The convolutional network's logits for one sample (float64 [classes])."""
    dm = _dims(dims)
    w = np.ascontiguousarray(w, dtype=np.float64)
    feat = _features(feat)
    out = np.empty(int(dm[-1]), dtype=np.float64)
    _check(_load().zo_cnn_logits(len(dm) - 2, _ptr(dm), int(has_bias), _ptr(w), _ptr(feat), _ptr(out)),
           "zo_cnn_logits")
    return out


def score(kind, dtype, dims, has_bias, x, V, ldv, m, features, targets, gamma, rho):
    """Returns (scores[m], losses[m+1], norms[m]) as float64."""
    dm = _dims(dims)
    x = _params(x, dtype)
    V = _params(V, dtype)
    features = _features(features)
    targets = _targets(kind, targets)
    n_r = targets.shape[0]
    s = np.empty(m, dtype=np.float64)
    f = np.empty(m + 1, dtype=np.float64)
    n = np.empty(m, dtype=np.float64)
    rc = _load().zo_score(kind, dtype, _n_layers(kind, dm), _ptr(dm), int(has_bias), _ptr(x), _ptr(V),
                          int(ldv), int(m), _ptr(features), _ptr(targets), n_r,
                          float(gamma), float(rho), _ptr(s), _ptr(f), _ptr(n))
    _check(rc, "zo_score")
    return s, f, n


def select(scores, b):
    s = np.ascontiguousarray(scores, dtype=np.float64)
    m = s.shape[0]
    if not (0 <= b < m):
        raise ValueError("need m > b >= 0")
    idx = np.empty(m - b, dtype=np.int32)
    _check(_load().zo_select(_ptr(s), m, int(b), _ptr(idx)), "zo_select")
    return idx


def aggregate(dtype, V, ldv, d, m, idx):
    V = _params(V, dtype)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    out = np.empty(d, dtype=np.float64)
    _check(_load().zo_aggregate(dtype, _ptr(V), int(ldv), int(d), int(m), _ptr(idx),
                                idx.shape[0], _ptr(out)), "zo_aggregate")
    return out


def worker_gradient(kind, dtype, dims, has_bias, x, features, targets, flip=False):
    """Algorithm 1, a worker's line: the gradient of the mean loss over its own samples at x (float64 [d]);
    softmax regression (a one-layer model) and least squares.  flip: the label-flipping failure."""
    dm = _dims(dims)
    x = _params(x, dtype)
    features = _features(features)
    targets = _targets(kind, targets)
    d = param_count(kind, dims, has_bias)
    g = np.empty(d, dtype=np.float64)
    _check(_load().zo_worker_gradient(kind, len(dm) - 1, _ptr(dm), int(has_bias), _ptr(x), dtype, _ptr(features),
                                      _ptr(targets), targets.shape[0], int(bool(flip)), _ptr(g)),
           "zo_worker_gradient")
    return g


def inject_faults(V, faulty, mode, eps=0.0):
    """The experiments' failures on a float64 candidate matrix [m, d] (returns a modified copy):
    mode 0 bit-flipping with copy-overwrite, mode 1 scaling by eps."""
    V = np.array(V, dtype=np.float64, order="C", copy=True)
    faulty = np.ascontiguousarray(faulty, dtype=np.int32)
    _check(_load().zo_inject_faults(_ptr(V), V.shape[1], V.shape[0], _ptr(faulty), faulty.shape[0], int(mode),
                                    float(eps)), "zo_inject_faults")
    return V


def median(dtype, V, ldv, d, m):
    """Marginal median of the m candidates (the paper's Median baseline): float64 [d]."""
    V = _params(V, dtype)
    out = np.empty(d, dtype=np.float64)
    _check(_load().zo_median(dtype, _ptr(V), int(ldv), int(d), int(m), _ptr(out)), "zo_median")
    return out


def krum(dtype, V, ldv, d, m, b):
    """Krum_b (the paper's Krum baseline): returns (k, sums[m], dist[m, m])."""
    V = _params(V, dtype)
    k = np.zeros(1, dtype=np.int32)
    sums = np.empty(m, dtype=np.float64)
    dist = np.empty((m, m), dtype=np.float64)
    _check(_load().zo_krum(dtype, _ptr(V), int(ldv), int(d), int(m), int(b), _ptr(k), _ptr(sums),
                           _ptr(dist)), "zo_krum")
    return int(k[0]), sums, dist


def update(dtype, x, vbar, gamma):
    """Algorithm 1's server update: x - gamma * vbar, element by element (float64; a bfloat16
    parameter vector is rounded back to bfloat16)."""
    x = _params(x, dtype)
    vbar = np.ascontiguousarray(vbar, dtype=np.float64)
    xnew = np.empty(vbar.shape[0], dtype=np.float64)
    _load().zo_update(_ptr(x), _ptr(vbar), vbar.shape[0], dtype, float(gamma), _ptr(xnew))
    return xnew


def step(kind, dtype, dims, has_bias, x, V, ldv, m, features, targets, gamma, rho, b):
    """Zeno_b: returns (out[d], scores[m], idx[m-b])."""
    dm = _dims(dims)
    x = _params(x, dtype)
    V = _params(V, dtype)
    features = _features(features)
    targets = _targets(kind, targets)
    n_r = targets.shape[0]
    d = param_count(kind, dims, has_bias)
    out = np.empty(d, dtype=np.float64)
    s = np.empty(m, dtype=np.float64)
    idx = np.empty(m - b, dtype=np.int32)
    rc = _load().zo_step(kind, dtype, _n_layers(kind, dm), _ptr(dm), int(has_bias), _ptr(x), _ptr(V),
                         int(ldv), int(m), _ptr(features), _ptr(targets), n_r,
                         float(gamma), float(rho), int(b), _ptr(out), _ptr(s), _ptr(idx))
    _check(rc, "zo_step")
    return out, s, idx
