"""Pins for the oracle's baseline aggregation rules (Experiments, "Baselines": Median and Krum),
against what the paper and the mathematics fix -- never against the CUDA path.

  Median : hand values for odd and even m; numpy's median (a library routine) on random data;
           invariance under permutation of the candidates; a minority of arbitrarily large rows
           cannot move a coordinate outside the range of the majority; NaN counts as +infinity
  Krum   : the paper's one-dimensional toy example (tests/golden/krum_toy_example.txt); the sums of
           Definition "Krum" rebuilt from numpy's pairwise distances and partial sorts, and the
           argmin by brute force; m - b - 2 neighbours (b chosen so that one neighbour is left);
           translation invariance; the selected vector is one of the inputs
"""
import os

import numpy as np
import pytest

F32, BF16 = 0, 1
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


# ---------------------------------------------------------------- Median

def test_median_hand_values_odd_and_even(oracle):
    V = np.array([[1, 10], [3, -2], [2, 7]], dtype=np.float32)             # m = 3
    assert oracle.median(F32, V, 2, 2, 3).tolist() == [2.0, 7.0]
    V = np.array([[1, 10], [3, -2], [2, 7], [8, 0]], dtype=np.float32)     # m = 4: mean of the two middle values
    assert oracle.median(F32, V, 2, 2, 4).tolist() == [2.5, 3.5]
    assert oracle.median(F32, V[:1], 2, 2, 1).tolist() == [1.0, 10.0]      # m = 1: the value itself


@pytest.mark.parametrize("m", [2, 5, 20, 33, 100])
def test_median_matches_numpy_and_ignores_row_order(oracle, m):
    r = _rng(m)
    d, ldv = 57, 61
    V = np.full((m, ldv), np.nan, dtype=np.float32)
    V[:, :d] = r.standard_normal((m, d)).astype(np.float32)
    got = oracle.median(F32, V, ldv, d, m)
    assert np.array_equal(got, np.median(V[:, :d].astype(np.float64), axis=0))
    perm = r.permutation(m)
    assert np.array_equal(oracle.median(F32, V[perm].copy(), ldv, d, m), got)


def test_median_bf16_rows_are_promoted_exactly(oracle):
    import torch
    r = _rng(3)
    t = torch.from_numpy(r.standard_normal((7, 16)).astype(np.float32)).to(torch.bfloat16)
    bits = t.view(torch.int16).numpy().view("uint16")
    got = oracle.median(BF16, bits, 16, 16, 7)
    assert np.array_equal(got, np.median(t.float().double().numpy(), axis=0))


def test_median_stays_inside_the_majority_range(oracle):
    r = _rng(9)
    honest = r.standard_normal((11, 40)).astype(np.float32)
    faulty = np.full((8, 40), 1e30, dtype=np.float32)
    faulty[::2] = -1e30
    V = np.concatenate([honest, faulty])
    med = oracle.median(F32, V, 40, 40, 19)
    assert np.all(med >= honest.min(axis=0)) and np.all(med <= honest.max(axis=0))


def test_median_counts_nan_as_plus_infinity(oracle):
    V = np.array([[1.0], [np.nan], [2.0], [3.0], [np.nan]], dtype=np.float32)
    assert oracle.median(F32, V, 1, 1, 5).tolist() == [3.0]                 # sorted: 1 2 3 inf inf
    V = np.array([[1.0], [np.nan], [np.nan]], dtype=np.float32)
    assert oracle.median(F32, V, 1, 1, 3).tolist() == [np.inf]


# ---------------------------------------------------------------- Krum

def test_krum_toy_example_of_the_paper(oracle):
    vals = {}
    with open(os.path.join(GOLDEN, "krum_toy_example.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            key, *rest = line.split()
            vals[key] = [float(v) for v in rest]
    values = np.array(vals["values"], dtype=np.float32).reshape(-1, 1)
    k, sums, dist = oracle.krum(F32, values, 1, 1, len(values), int(vals["b"][0]))
    assert values[k, 0] == vals["krum"][0]
    # by hand: -1 has the other -1 (0) and 0.2 (1.44) as its two neighbours
    assert sums[k] == pytest.approx(1.44, rel=1e-6)
    assert min(sums[2:]) == pytest.approx(1.48, rel=1e-6)


def _krum_by_definition(V, b):
    """Definition "Krum" with numpy's routines: pairwise squared distances, the m - b - 2 smallest
    to the other candidates, brute-force argmin."""
    m = V.shape[0]
    Vd = V.astype(np.float64)
    D = ((Vd[:, None, :] - Vd[None, :, :]) ** 2).sum(axis=2)
    sums = np.empty(m)
    for i in range(m):
        others = np.delete(D[i], i)
        sums[i] = np.sort(others)[:m - b - 2].sum()
    return int(np.argmin(sums)), sums, D


@pytest.mark.parametrize("m,b", [(4, 1), (6, 2), (9, 3), (20, 8), (20, 17), (33, 0)])
def test_krum_matches_the_definition_rebuilt_with_numpy(oracle, m, b):
    r = _rng(100 * m + b)
    d, ldv = 23, 25
    V = np.full((m, ldv), np.nan, dtype=np.float32)
    V[:, :d] = r.standard_normal((m, d)).astype(np.float32)
    V[m // 2, :d] = V[0, :d]                                   # a duplicated candidate: distance exactly zero
    k, sums, dist = oracle.krum(F32, V, ldv, d, m, b)
    k_ref, sums_ref, D_ref = _krum_by_definition(V[:, :d], b)
    assert np.allclose(dist, D_ref, rtol=1e-12, atol=0)
    assert dist[0, m // 2] == 0.0 and np.all(np.diag(dist) == 0.0)
    assert np.allclose(sums, sums_ref, rtol=1e-12)
    assert k == k_ref


def test_krum_is_translation_invariant_and_returns_an_input(oracle):
    r = _rng(5)
    V = r.standard_normal((12, 30)).astype(np.float32)
    k, sums, _ = oracle.krum(F32, V, 30, 30, 12, 4)
    shift = np.float32(0.5)                                     # exactly representable shifts keep the differences
    k2, sums2, _ = oracle.krum(F32, (V.astype(np.float64) + 0.5).astype(np.float32), 30, 30, 12, 4)
    assert k2 == k
    assert np.allclose(sums2, sums, rtol=1e-5)
    assert 0 <= k < 12


def test_krum_needs_a_neighbour(oracle):
    V = np.zeros((5, 3), dtype=np.float32)
    with pytest.raises(Exception):
        oracle.krum(F32, V, 3, 3, 5, 3)                        # m - b - 2 = 0
    k, _, _ = oracle.krum(F32, V, 3, 3, 5, 2)                  # one neighbour: fine, ties go to the lowest index
    assert k == 0


# ---------------------------------------------------------------- the workers' side: gradients and failures
# (Algorithm 1, worker lines; Experiments: label-flipping and bit-flipping failures; the failure model's
# scaled gradient)

MLP, LSQ = 0, 1


def _fd_gradient(oracle, kind, dims, x, feats, tgts, h=1e-6):
    """Central differences of the (already pinned) loss f_r, coordinate by coordinate, in float64."""
    g = np.empty(x.shape[0])
    for k in range(x.shape[0]):
        e = np.zeros_like(x)
        e[k] = h
        g[k] = (oracle.loss(kind, dims, True, x + e, feats, tgts) - oracle.loss(kind, dims, True, x - e, feats, tgts)) / (2 * h)
    return g


def test_worker_gradient_softmax_regression_matches_finite_differences_of_the_loss(oracle):
    r = _rng(21)
    dims = (6, 4)
    d = 6 * 4 + 4
    x = r.standard_normal(d).astype(np.float32)
    feats = r.standard_normal((5, 6)).astype(np.float32)
    labels = r.integers(0, 4, 5).astype(np.int32)
    g = oracle.worker_gradient(MLP, F32, dims, True, x, feats, labels)
    fd = _fd_gradient(oracle, MLP, dims, x.astype(np.float64), feats, labels)
    assert np.allclose(g, fd, rtol=1e-6, atol=1e-8)
    # the label-flipping failure is the gradient on the labels classes - 1 - label
    gf = oracle.worker_gradient(MLP, F32, dims, True, x, feats, labels, flip=True)
    assert np.allclose(gf, oracle.worker_gradient(MLP, F32, dims, True, x, feats, (3 - labels).astype(np.int32)))
    assert not np.allclose(gf, g)
    # a gradient of a softmax model: the bias entries sum to zero (probabilities and one-hot both sum to one)
    assert abs(g[24:].sum()) < 1e-12


def test_worker_gradient_least_squares_is_the_normal_equations_residual(oracle):
    r = _rng(22)
    d, n = 9, 4
    x = r.standard_normal(d).astype(np.float32)
    A = r.standard_normal((n, d)).astype(np.float32)
    y = r.standard_normal(n).astype(np.float32)
    g = oracle.worker_gradient(LSQ, F32, (d, 1), False, x, A, y)
    Ad = A.astype(np.float64)
    assert np.allclose(g, Ad.T @ (Ad @ x.astype(np.float64) - y) / n, rtol=1e-12)
    fd = _fd_gradient(oracle, LSQ, (d, 1), x.astype(np.float64), A, y)
    assert np.allclose(g, fd, rtol=1e-6, atol=1e-8)


def test_inject_faults_bit_flip_copies_one_negated_gradient_and_scaling_multiplies(oracle):
    V = np.arange(20, dtype=np.float64).reshape(5, 4) + 1
    out = oracle.inject_faults(V, [3, 1, 4], 0)
    assert np.array_equal(out[3], -V[3]) and np.array_equal(out[1], -V[3]) and np.array_equal(out[4], -V[3])
    assert np.array_equal(out[[0, 2]], V[[0, 2]])
    out = oracle.inject_faults(V, [0, 2], 1, eps=-4.0)
    assert np.array_equal(out[[0, 2]], -4.0 * V[[0, 2]]) and np.array_equal(out[[1, 3, 4]], V[[1, 3, 4]])
    assert np.array_equal(oracle.inject_faults(V, [], 0), V)
    with pytest.raises(Exception):
        oracle.inject_faults(V, [5], 0)
