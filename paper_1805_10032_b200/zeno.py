"""ctypes binding of libzeno.so -- argument marshalling only.

Every step of the Zeno aggregation rule (scores, ranking, trimmed mean) runs in
the CUDA kernels behind the C ABI declared in include/zeno.h; this module turns
torch tensors into device pointers and status codes into exceptions.  There is
no CPU fallback: if the shared library is missing or a call fails, it raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libzeno.so")

MAX_LAYERS = 8
MAX_CANDIDATES = 1024

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(6)
LOSS_SOFTMAX_MLP, LOSS_LEAST_SQUARES, LOSS_SOFTMAX_CNN = 0, 1, 2
FAULT_BIT_FLIP, FAULT_SCALE = 0, 1
F32, BF16 = 0, 1

EXPORTS = (
    "zeno_param_count", "zeno_create", "zeno_destroy", "zeno_score", "zeno_select",
    "zeno_aggregate", "zeno_worker_gradients", "zeno_inject_faults", "zeno_score_partial", "zeno_score_from_sums", "zeno_median", "zeno_krum", "zeno_step", "zeno_step_update", "zeno_run", "zeno_step_host", "zeno_device_status", "zeno_score_lsq_static",
    "zeno_debug_set_wait_limit",
    "zeno_profile", "zeno_profile_read",
    "zeno_last_launch_count",
    "zeno_last_cuda_error", "zeno_last_wait_code", "zeno_status_string",
)


class ModelDesc(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("param_dtype", ctypes.c_int32),
                ("n_layers", ctypes.c_int32), ("has_bias", ctypes.c_int32),
                ("dims", ctypes.c_int64 * (MAX_LAYERS + 1))]


class Batch(ctypes.Structure):
    _fields_ = [("features", ctypes.c_void_p), ("targets", ctypes.c_void_p),
                ("n_r", ctypes.c_int32)]


class ZenoError(RuntimeError):
    def __init__(self, status: int, what: str, detail: str = ""):
        self.status = status
        super().__init__(f"{what}: status {status} ({status_string(status)}){detail}")


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads libzeno.so; raises if it has not been built (python -m paper_1805_10032_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} is missing: build it with `python -m paper_1805_10032_b200.build` "
            "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float
    lib.zeno_param_count.restype = i64
    lib.zeno_param_count.argtypes = [ctypes.POINTER(ModelDesc)]
    lib.zeno_create.restype = i32
    lib.zeno_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(ModelDesc), i32, i32, i32]
    lib.zeno_destroy.restype = i32
    lib.zeno_destroy.argtypes = [vp]
    lib.zeno_score.restype = i32
    lib.zeno_score.argtypes = [vp, vp, vp, i64, i32, ctypes.POINTER(Batch), f32, f32, vp, vp, vp, vp]
    lib.zeno_select.restype = i32
    lib.zeno_select.argtypes = [vp, vp, i32, i32, vp, vp]
    lib.zeno_aggregate.restype = i32
    lib.zeno_aggregate.argtypes = [vp, vp, i64, i32, vp, i32, vp, vp]
    lib.zeno_worker_gradients.restype = i32
    lib.zeno_worker_gradients.argtypes = [vp, vp, vp, vp, i32, i32, vp, vp, i64, vp]
    lib.zeno_inject_faults.restype = i32
    lib.zeno_inject_faults.argtypes = [vp, vp, i64, i32, vp, i32, i32, f32, vp]
    lib.zeno_score_partial.restype = i32
    lib.zeno_score_partial.argtypes = [vp, vp, vp, i64, i32, vp, i32, vp, vp]
    lib.zeno_score_from_sums.restype = i32
    lib.zeno_score_from_sums.argtypes = [vp, vp, vp, i32, i32, f32, f32, vp, vp, vp, vp]
    lib.zeno_median.restype = i32
    lib.zeno_median.argtypes = [vp, vp, i64, i32, vp, vp]
    lib.zeno_krum.restype = i32
    lib.zeno_krum.argtypes = [vp, vp, i64, i32, i32, vp, vp, vp, vp]
    lib.zeno_step.restype = i32
    lib.zeno_step.argtypes = [vp, vp, vp, i64, i32, ctypes.POINTER(Batch), f32, f32, i32, vp, vp, vp, vp]
    lib.zeno_run.restype = i32
    lib.zeno_run.argtypes = [vp, vp, vp, i64, i64, i32, vp, vp, i32, i32, f32, f32, i32, vp, vp, vp]
    lib.zeno_step_update.restype = i32
    lib.zeno_step_update.argtypes = [vp, vp, vp, i64, i32, ctypes.POINTER(Batch), f32, f32, i32, vp, vp, vp, vp]
    lib.zeno_step_host.restype = i32
    lib.zeno_step_host.argtypes = [vp, vp, vp, i64, i32, vp, vp, i32, f32, f32, i32, vp, vp, vp, vp]
    lib.zeno_score_lsq_static.restype = i32
    lib.zeno_score_lsq_static.argtypes = [i32, vp, vp, i64, i64, i32, vp, vp, i32, f32, f32, vp, vp, vp, vp]
    lib.zeno_device_status.restype = i32
    lib.zeno_device_status.argtypes = [vp, vp]
    lib.zeno_debug_set_wait_limit.restype = i32
    lib.zeno_debug_set_wait_limit.argtypes = [vp, ctypes.c_uint32]
    lib.zeno_profile.restype = i32
    lib.zeno_profile.argtypes = [vp, i32]
    lib.zeno_profile_read.restype = i32
    lib.zeno_profile_read.argtypes = [vp, i32, ctypes.POINTER(f32), ctypes.POINTER(ctypes.c_char_p), i32]
    lib.zeno_last_launch_count.restype = i32
    lib.zeno_last_launch_count.argtypes = [vp]
    lib.zeno_last_cuda_error.restype = i32
    lib.zeno_last_cuda_error.argtypes = [vp]
    lib.zeno_last_wait_code.restype = i32
    lib.zeno_last_wait_code.argtypes = [vp]
    lib.zeno_status_string.restype = ctypes.c_char_p
    lib.zeno_status_string.argtypes = [i32]
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().zeno_status_string(int(status)).decode()


def make_desc(kind: int, param_dtype: int, dims: Sequence[int], has_bias: bool = True) -> ModelDesc:
    if len(dims) > MAX_LAYERS + 1:
        raise ValueError("too many layers")
    d = ModelDesc()
    d.kind = kind
    d.param_dtype = param_dtype
    # a convolutional network's list starts with the image side: [S, C_0, C_1, .., C_Lc, classes]
    d.n_layers = len(dims) - 2 if kind == LOSS_SOFTMAX_CNN else len(dims) - 1
    d.has_bias = int(has_bias)
    for i, v in enumerate(dims):
        d.dims[i] = int(v)
    return d


def param_count(desc: ModelDesc) -> int:
    return int(load_library().zeno_param_count(ctypes.byref(desc)))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


class Zeno:
    """A handle for one model shape on one device (zeno_create / zeno_destroy).

    All tensors are CUDA tensors on the handle's device; outputs are allocated by the
    caller side of this binding with torch (device memory is torch's job here)."""

    def __init__(self, kind: int, param_dtype: int, dims: Sequence[int], has_bias: bool = True,
                 m_max: int = 128, n_r_max: int = 128, device: int = 0):
        self._lib = load_library()
        self.desc = make_desc(kind, param_dtype, dims, has_bias)
        self.kind, self.param_dtype = kind, param_dtype
        self.dims = tuple(int(v) for v in dims)
        self.device = int(device)
        self.m_max, self.n_r_max = int(m_max), int(n_r_max)
        self._h = ctypes.c_void_p()
        st = self._lib.zeno_create(ctypes.byref(self._h), ctypes.byref(self.desc), self.m_max,
                                   self.n_r_max, self.device)
        if st != OK:
            self._h = ctypes.c_void_p()
            raise ZenoError(st, "zeno_create")
        self.d = param_count(self.desc)

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self._lib.zeno_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # -- helpers ------------------------------------------------------------------------
    def _check(self, st: int, what: str):
        if st != OK:
            detail = ""
            if st == ERR_CUDA:
                detail = f" [cudaError {self._lib.zeno_last_cuda_error(self._h)}]"
            if st == ERR_TIMEOUT:
                detail = f" [wait code {self._lib.zeno_last_wait_code(self._h):#x}]"
            raise ZenoError(st, what, detail)

    def _batch(self, features: torch.Tensor, targets: torch.Tensor) -> Batch:
        b = Batch()
        b.features = features.data_ptr()
        b.targets = targets.data_ptr()
        b.n_r = int(targets.shape[0])
        return b

    def _dev(self):
        return torch.device("cuda", self.device)

    @property
    def last_launch_count(self) -> int:
        return int(self._lib.zeno_last_launch_count(self._h))

    def check_device_status(self, stream=None):
        """Synchronises and raises if a kernel gave up on a bounded device-side wait."""
        self._check(self._lib.zeno_device_status(self._h, _stream_ptr(stream)), "zeno_device_status")

    def debug_set_wait_limit(self, polls: int):
        """Test hook: polls a bounded device-side wait may take before it gives up (see zeno.h)."""
        self._check(self._lib.zeno_debug_set_wait_limit(self._h, int(polls)), "zeno_debug_set_wait_limit")

    @property
    def last_wait_code(self) -> int:
        return int(self._lib.zeno_last_wait_code(self._h))

    def profile(self, enable: bool = True):
        self._check(self._lib.zeno_profile(self._h, int(enable)), "zeno_profile")

    def profile_read(self, back: int = 0):
        """[(kernel name, milliseconds)] of the call made `back` calls ago, in launch order."""
        cap = 32
        ms = (ctypes.c_float * cap)()
        names = (ctypes.c_char_p * cap)()
        n = self._lib.zeno_profile_read(self._h, int(back), ms, names, cap)
        if n < 0:
            raise ZenoError(ERR_CUDA, "zeno_profile_read")
        return [(names[i].decode(), float(ms[i])) for i in range(n)]

    # -- the four calls -------------------------------------------------------------------
    def score(self, x, V, features, targets, gamma, rho, m=None, ldv=None, want_losses=True,
              want_norms=True, stream=None):
        """Returns (scores[m], losses[m+1] or None, norms[m] or None) as CUDA float32 tensors."""
        m = V.shape[0] if m is None else m
        ldv = V.stride(0) if ldv is None else ldv
        scores = torch.empty(m, dtype=torch.float32, device=self._dev())
        losses = torch.empty(m + 1, dtype=torch.float32, device=self._dev()) if want_losses else None
        norms = torch.empty(m, dtype=torch.float32, device=self._dev()) if want_norms else None
        b = self._batch(features, targets)
        st = self._lib.zeno_score(self._h, _ptr(x), _ptr(V), int(ldv), int(m), ctypes.byref(b),
                                  float(gamma), float(rho), _ptr(scores), _ptr(losses), _ptr(norms),
                                  _stream_ptr(stream))
        self._check(st, "zeno_score")
        return scores, losses, norms

    def select(self, scores, b, m=None, stream=None):
        """Returns idx[m-b] (int32, rank order)."""
        m = scores.shape[0] if m is None else m
        idx = torch.empty(max(m - b, 0), dtype=torch.int32, device=self._dev())
        st = self._lib.zeno_select(self._h, _ptr(scores), int(m), int(b), _ptr(idx),
                                   _stream_ptr(stream))
        self._check(st, "zeno_select")
        return idx

    def aggregate(self, V, idx, m=None, ldv=None, k=None, out=None, stream=None):
        """Returns out[d] float32 = mean of the rows idx of V."""
        m = V.shape[0] if m is None else m
        ldv = V.stride(0) if ldv is None else ldv
        k = idx.shape[0] if k is None else k
        if out is None:
            out = torch.empty(self.d, dtype=torch.float32, device=self._dev())
        st = self._lib.zeno_aggregate(self._h, _ptr(V), int(ldv), int(m), _ptr(idx), int(k),
                                      _ptr(out), _stream_ptr(stream))
        self._check(st, "zeno_aggregate")
        return out

    def worker_gradients(self, x, features, targets, V, label_flip=None, stream=None):
        """Algorithm 1's worker lines: row i of V <- the gradient at x of worker i's mean loss over its own batch
        (features [m, n, in], targets [m, n]); label_flip: int32 [m] device tensor or None."""
        m, n = features.shape[0], features.shape[1]
        st = self._lib.zeno_worker_gradients(self._h, _ptr(x), _ptr(features), _ptr(targets), int(n), int(m),
                                             _ptr(label_flip), _ptr(V), int(V.stride(0)), _stream_ptr(stream))
        self._check(st, "zeno_worker_gradients")
        return V

    def inject_faults(self, V, faulty, mode, eps=0.0, stream=None):
        """The experiments' failures on the rows `faulty` (int32 device tensor) of V, in place."""
        st = self._lib.zeno_inject_faults(self._h, _ptr(V), int(V.stride(0)), int(V.shape[0]), _ptr(faulty),
                                          int(faulty.shape[0]), int(mode), float(eps), _stream_ptr(stream))
        self._check(st, "zeno_inject_faults")
        return V

    def score_partial(self, x, V, features, m=None, ldv=None, sums=None, stream=None):
        """This handle's column slice of the least-squares score sums: float64 [(m+1), (n_r+1)]."""
        m = V.shape[0] if m is None else m
        ldv = V.stride(0) if ldv is None else ldv
        n_r = features.shape[0]
        if sums is None:
            sums = torch.empty((m + 1, n_r + 1), dtype=torch.float64, device=self._dev())
        st = self._lib.zeno_score_partial(self._h, _ptr(x), _ptr(V), int(ldv), int(m), _ptr(features), int(n_r),
                                          _ptr(sums), _stream_ptr(stream))
        self._check(st, "zeno_score_partial")
        return sums

    def score_from_sums(self, sums, targets, gamma, rho, stream=None):
        """Definition 2's scores from the sums of all slices: returns (scores[m], losses[m+1], norms[m])."""
        m, n_r = sums.shape[0] - 1, sums.shape[1] - 1
        scores = torch.empty(m, dtype=torch.float32, device=self._dev())
        losses = torch.empty(m + 1, dtype=torch.float32, device=self._dev())
        norms = torch.empty(m, dtype=torch.float32, device=self._dev())
        st = self._lib.zeno_score_from_sums(self._h, _ptr(sums), _ptr(targets), int(m), int(n_r), float(gamma),
                                            float(rho), _ptr(scores), _ptr(losses), _ptr(norms), _stream_ptr(stream))
        self._check(st, "zeno_score_from_sums")
        return scores, losses, norms

    def median(self, V, m=None, ldv=None, out=None, stream=None):
        """The marginal median of the candidates (the paper's Median baseline): out[d] float32."""
        m = V.shape[0] if m is None else m
        ldv = V.stride(0) if ldv is None else ldv
        if out is None:
            out = torch.empty(self.d, dtype=torch.float32, device=self._dev())
        self._check(self._lib.zeno_median(self._h, _ptr(V), int(ldv), int(m), _ptr(out), _stream_ptr(stream)),
                    "zeno_median")
        return out

    def krum(self, V, b, m=None, ldv=None, want_out=True, stream=None):
        """Krum_b (the paper's Krum baseline): returns (out[d] or None, k int32[1], sums[m])."""
        m = V.shape[0] if m is None else m
        ldv = V.stride(0) if ldv is None else ldv
        out = torch.empty(self.d, dtype=torch.float32, device=self._dev()) if want_out else None
        k = torch.empty(1, dtype=torch.int32, device=self._dev())
        sums = torch.empty(m, dtype=torch.float32, device=self._dev())
        self._check(self._lib.zeno_krum(self._h, _ptr(V), int(ldv), int(m), int(b), _ptr(out), _ptr(k), _ptr(sums),
                                        _stream_ptr(stream)), "zeno_krum")
        return out, k, sums

    def step(self, x, V, features, targets, gamma, rho, b, m=None, ldv=None, out=None,
             scores=None, idx=None, want_scores=True, want_idx=True, stream=None):
        """Zeno_b: returns (out[d], scores[m] or None, idx[m-b] or None)."""
        m = V.shape[0] if m is None else m
        ldv = V.stride(0) if ldv is None else ldv
        if out is None:
            out = torch.empty(self.d, dtype=torch.float32, device=self._dev())
        if scores is None and want_scores:
            scores = torch.empty(m, dtype=torch.float32, device=self._dev())
        if idx is None and want_idx:
            idx = torch.empty(max(m - b, 0), dtype=torch.int32, device=self._dev())
        bt = self._batch(features, targets)
        st = self._lib.zeno_step(self._h, _ptr(x), _ptr(V), int(ldv), int(m), ctypes.byref(bt),
                                 float(gamma), float(rho), int(b), _ptr(out), _ptr(scores), _ptr(idx),
                                 _stream_ptr(stream))
        self._check(st, "zeno_step")
        return out, scores, idx

    def step_update(self, x, V, features, targets, gamma, rho, b, m=None, ldv=None, out=None,
                    scores=None, idx=None, want_out=True, want_scores=True, want_idx=True, stream=None):
        """Zeno_b followed by the server update x <- x - gamma * average, in place and in the pass that
        forms the average.  Returns (out[d] or None, scores[m] or None, idx[m-b] or None)."""
        m = V.shape[0] if m is None else m
        ldv = V.stride(0) if ldv is None else ldv
        if out is None and want_out:
            out = torch.empty(self.d, dtype=torch.float32, device=self._dev())
        if scores is None and want_scores:
            scores = torch.empty(m, dtype=torch.float32, device=self._dev())
        if idx is None and want_idx:
            idx = torch.empty(max(m - b, 0), dtype=torch.int32, device=self._dev())
        bt = self._batch(features, targets)
        st = self._lib.zeno_step_update(self._h, _ptr(x), _ptr(V), int(ldv), int(m), ctypes.byref(bt),
                                        float(gamma), float(rho), int(b), _ptr(out), _ptr(scores),
                                        _ptr(idx), _stream_ptr(stream))
        self._check(st, "zeno_step_update")
        return out, scores, idx

    def run(self, x, V, features, targets, gamma, rho, b, scores=None, idx=None, stream=None):
        """Algorithm 1's server loop: V [steps, m, ldv], features [steps, n_r, in], targets [steps, n_r];
        x is updated in place.  Returns (scores [steps, m], idx [steps, m - b])."""
        steps, m = V.shape[0], V.shape[1]
        ldv, stride = V.stride(1), V.stride(0)
        n_r = features.shape[1]
        assert features.is_contiguous() and targets.is_contiguous()
        if scores is None:
            scores = torch.empty((steps, m), dtype=torch.float32, device=self._dev())
        if idx is None:
            idx = torch.empty((steps, max(m - b, 0)), dtype=torch.int32, device=self._dev())
        st = self._lib.zeno_run(self._h, _ptr(x), _ptr(V), int(ldv), int(stride), int(m), _ptr(features),
                                _ptr(targets), int(n_r), int(steps), float(gamma), float(rho), int(b),
                                _ptr(scores), _ptr(idx), _stream_ptr(stream))
        self._check(st, "zeno_run")
        return scores, idx

    def step_host(self, x, V, features, targets, gamma, rho, b, out, scores=None, idx=None,
                  m=None, ldv=None, stream=None):
        """Host-memory variant: all tensors are CPU tensors (pinned for asynchronous copies);
        `out` (float32 [d]) is filled on return."""
        m = V.shape[0] if m is None else m
        ldv = V.stride(0) if ldv is None else ldv
        st = self._lib.zeno_step_host(self._h, _ptr(x), _ptr(V), int(ldv), int(m), _ptr(features),
                                      _ptr(targets), int(targets.shape[0]), float(gamma), float(rho),
                                      int(b), _ptr(out), _ptr(scores), _ptr(idx), _stream_ptr(stream))
        self._check(st, "zeno_step_host")
        return out


STATIC_MAX_M, STATIC_MAX_N_R = 64, 32


def score_lsq_static(x, V, A, y, gamma, rho, scores, losses=None, norms=None, m=None, ldv=None,
                     device=0, stream=None):
    """zeno_score_lsq_static: least-squares scores with no allocation anywhere -- the caller passes
    every buffer (CUDA tensors: x [d], V [m, ldv], A [n_r, d], y [n_r], scores [m] float32; losses
    [m+1] and norms [m] optional).  For callers that may not call the CUDA allocator; m <= 64 and
    n_r <= 32.  Calls whose kernels could overlap on the GPU must be ordered by the caller."""
    lib = load_library()
    m = V.shape[0] if m is None else m
    ldv = V.stride(0) if ldv is None else ldv
    st = lib.zeno_score_lsq_static(int(device), _ptr(x), _ptr(V), int(ldv), int(x.shape[0]), int(m),
                                   _ptr(A), _ptr(y), int(y.shape[0]), float(gamma), float(rho),
                                   _ptr(scores), _ptr(losses), _ptr(norms), _stream_ptr(stream))
    if st != OK:
        raise ZenoError(st, "zeno_score_lsq_static")
    return scores


def from_workload(w, m_max=None, n_r_max=None, device=0) -> "Zeno":
    """A handle shaped for a synthetic.Workload."""
    kind = {"lsq": LOSS_LEAST_SQUARES, "cnn": LOSS_SOFTMAX_CNN}.get(w.kind, LOSS_SOFTMAX_MLP)
    dt = BF16 if w.dtype == "bf16" else F32
    return Zeno(kind, dt, w.dims, w.has_bias, m_max or w.m, n_r_max or w.n_r, device)
