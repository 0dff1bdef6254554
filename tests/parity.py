"""Shared helpers of the GPU-vs-oracle parity tests (test infrastructure).

Tolerances (from the statement of the task this library serves):
  scores      |s_gpu - s_orc| <= 1e-4 |s_orc|; a candidate whose three terms nearly cancel may meet
              1e-4 (|f_0| + |f_i| + rho n_i) instead, and its condition number is then printed
  selection   identical index sets wherever the oracle's gap between the (m-b)-th and
              (m-b+1)-th score exceeds 1e-3 relative; otherwise the GPU's set must be a valid
              top-(m-b) set up to the score tolerance
  aggregate   relative l2 error <= 1e-5 (against the oracle's mean over the GPU's set when the
              cut falls inside a near-tie)
"""
import numpy as np
import torch

from paper_1805_10032_b200 import synthetic as syn
from paper_1805_10032_b200 import zeno

SCORE_RTOL = 1e-4
GAP_RTOL = 1e-3
AGG_RTOL = 1e-5

KIND = {"mlp": 0, "lsq": 1, "cnn": 2}
DTYPE = {"f32": 0, "bf16": 1}


def oracle_inputs(w):
    """numpy views of a Workload for the oracle."""
    return dict(kind=KIND[w.kind], dtype=DTYPE[w.dtype], dims=w.dims, has_bias=w.has_bias,
                x=syn.to_numpy_params(w.x), V=syn.to_numpy_params(w.V), ldv=w.ldv, m=w.m,
                features=w.features.cpu().numpy(), targets=w.targets.cpu().numpy(),
                gamma=float(np.float32(w.gamma)), rho=float(np.float32(w.rho)))


def oracle_score(oracle, w):
    o = oracle_inputs(w)
    return oracle.score(o["kind"], o["dtype"], o["dims"], o["has_bias"], o["x"], o["V"], o["ldv"],
                        o["m"], o["features"], o["targets"], o["gamma"], o["rho"])


def to_device(w, device="cuda"):
    return (w.x.to(device), w.V.to(device), w.features.to(device), w.targets.to(device))


def assert_scores_close(s_gpu, s_orc, losses_orc=None, norms_orc=None, rho=None, rtol=SCORE_RTOL):
    """Headline criterion: |s_gpu - s_orc| <= rtol |s_orc| for every candidate.

    Definition 2's score is a difference of three terms, so a candidate whose terms nearly cancel
    (an honest update with a small rho: |s| far below f_0) cannot meet a bound relative to |s| from
    binary32 terms.  When the oracle's losses and norms are passed, such a candidate may instead
    meet the conditioning-aware bound rtol (|f_0| + |f_i| + rho n_i); the helper then prints that
    candidate's condition number (|f_0| + |f_i| + rho n_i) / |s_i| and returns the list of
    (index, condition number) pairs that needed it.  Without them only the headline bound counts."""
    s_gpu = np.asarray(s_gpu, dtype=np.float64)
    s_orc = np.asarray(s_orc, dtype=np.float64)
    finite = np.isfinite(s_orc)
    # non-finite oracle scores: the GPU's must be non-finite too
    assert not np.isfinite(s_gpu[~finite]).any(), "GPU score finite where the oracle's is not"
    err = np.abs(s_gpu - s_orc)
    bound = rtol * np.abs(s_orc)
    relaxed = []
    for i in np.flatnonzero(finite):
        if err[i] <= bound[i]:
            continue
        if losses_orc is not None and norms_orc is not None and rho is not None:
            terms = abs(losses_orc[0]) + abs(losses_orc[1 + i]) + rho * norms_orc[i]
            if np.isfinite(terms) and err[i] <= rtol * terms:
                cond = terms / abs(s_orc[i]) if s_orc[i] != 0 else np.inf
                relaxed.append((int(i), float(cond)))
                print(f"score {i}: rel err {err[i] / abs(s_orc[i]):.3e} misses {rtol:g} |s| but meets "
                      f"{rtol:g} (|f0|+|f_i|+rho n_i); condition number {cond:.3e}")
                continue
        raise AssertionError(
            f"score {i}: gpu {s_gpu[i]!r} oracle {s_orc[i]!r} rel err "
            f"{err[i] / max(abs(s_orc[i]), 1e-300):.3e} > {rtol:g}")
    return relaxed


def assert_selection_valid(idx_gpu, s_orc, b, rtol_gap=GAP_RTOL, rtol_score=SCORE_RTOL, oracle=None):
    m = len(s_orc)
    keep = m - b
    idx_gpu = np.asarray(idx_gpu)
    assert idx_gpu.shape == (keep,)
    assert len(set(idx_gpu.tolist())) == keep and idx_gpu.min() >= 0 and idx_gpu.max() < m
    key = np.where(np.isnan(s_orc), -np.inf, s_orc)
    order = np.argsort(-key, kind="stable")
    if b == 0:
        assert sorted(idx_gpu.tolist()) == list(range(m))
        return True
    lo, hi = key[order[keep]], key[order[keep - 1]]      # first rejected, last kept
    gap = hi - lo
    scale = max(abs(hi), abs(lo))
    if np.isfinite(scale) and gap > rtol_gap * scale or (np.isinf(lo) and np.isfinite(hi)):
        assert sorted(idx_gpu.tolist()) == sorted(order[:keep].tolist()), "selected sets differ"
        return True
    # near-tie at the cut: every selected score >= every rejected score - tolerance
    rejected = np.setdiff1d(np.arange(m), idx_gpu)
    tol = 2 * rtol_score * scale if np.isfinite(scale) else 0.0
    assert key[idx_gpu].min() >= key[rejected].max() - tol, "selection is not a valid top set"
    return False


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return np.linalg.norm(a - b) / den if den > 0 else np.linalg.norm(a - b)


def run_step_parity(oracle, w, check_parts=True):
    """Whole-step parity of the CUDA path against the oracle on one workload.  Returns a dict of
    the measured errors."""
    o = oracle_inputs(w)
    s_orc, f_orc, n_orc = oracle_score(oracle, w)
    x, V, feats, tgt = to_device(w)
    with zeno.from_workload(w) as z:
        out, scores, idx = z.step(x, V, feats, tgt, w.gamma, w.rho, w.b)
        launches = z.last_launch_count
        s2, losses, norms = z.score(x, V, feats, tgt, w.gamma, w.rho)
        idx2 = z.select(scores, w.b)
        out2 = z.aggregate(V, idx)
        torch.cuda.synchronize()
    s_gpu = scores.cpu().numpy()
    assert np.array_equal(s_gpu, s2.cpu().numpy(), equal_nan=True), "step and score disagree"
    assert torch.equal(idx, idx2), "step and select disagree"
    assert torch.equal(out, out2), "step and aggregate disagree"
    relaxed = assert_scores_close(s_gpu, s_orc, f_orc, n_orc, o["rho"])
    assert np.allclose(norms.cpu().numpy(), n_orc, rtol=1e-5)
    assert np.allclose(losses.cpu().numpy(), f_orc, rtol=1e-4, atol=1e-6)
    # the ranking itself is integer work: bit-exact against the oracle on the GPU's own scores
    idx_ref = oracle.select(s_gpu.astype(np.float64), w.b)
    assert np.array_equal(idx.cpu().numpy(), idx_ref), "ranking differs on identical scores"
    exact_set = assert_selection_valid(idx.cpu().numpy(), s_orc, w.b)
    agg_ref = oracle.aggregate(o["dtype"], o["V"], w.ldv, w.d, w.m, idx.cpu().numpy())
    err = rel_l2(out.cpu().numpy(), agg_ref)
    assert err <= AGG_RTOL, f"aggregate rel l2 {err:.3e}"
    assert np.isfinite(out.cpu().numpy()).all() or not np.isfinite(agg_ref).all()
    return dict(score_err=float(np.nanmax(np.abs(s_gpu - s_orc) / np.abs(s_orc))), agg_err=float(err),
                exact_set=exact_set, launches=launches, relaxed=relaxed)
