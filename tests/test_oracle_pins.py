"""Pins for the float64 oracle: it is checked here against what the paper and the
mathematics fix, never against itself or the CUDA path.

  storage / rounding : bfloat16 round-to-nearest-even vs torch's conversion
  f_r (MLP)          : all-zero parameters give ln(#classes); a hand-worked 2-2-2 network in
                       closed form; torch float64 forward (library routine) on random nets;
                       finite differences vs the textbook softmax-regression gradient
  f_r (least squares): f(x) - f(x - g v) = g <grad f, v> - (g^2/2) v^T H v  (Assumption 2 holds
                       with equality for a quadratic); the L / mu sandwich of Assumption 2
  norm term          : ||(3,4)||^2 = 25; Score differences in rho; gamma = 0
  Score              : Score(0, x) = 0 exactly (Definition 2)
  ranking            : brute-force subset enumeration; Lemma 1 (order statistics of a subset);
                       permutation invariance; duplicated candidates; NaN = minus infinity
  trimmed average    : b = 0 is the plain Mean; b = m - 1 returns one row; Jensen step of the
                       convergence proof (Eq. "str_cvx" with mu = 0) for convex losses
  cost model         : (m + 1) n_r sample evaluations, 84 for the paper's m = 20, n_r = 4
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from paper_1805_10032_b200 import synthetic as syn

MLP, LSQ = 0, 1
F32, BF16 = 0, 1
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


def _random_mlp_problem(seed, dims=(7, 5, 4, 3), m=6, n_r=3, ldv=None, scale=1.0):
    r = _rng(seed)
    d = syn.param_count("mlp", dims, True)
    ldv = d if ldv is None else ldv
    x = (r.standard_normal(d) * 0.5).astype(np.float32)
    V = np.full((m, ldv), np.nan, dtype=np.float32)
    V[:, :d] = (r.standard_normal((m, d)) * scale).astype(np.float32)
    feats = r.standard_normal((n_r, dims[0])).astype(np.float32)
    labels = r.integers(0, dims[-1], n_r).astype(np.int32)
    return d, ldv, x, V, feats, labels


def _torch_mlp_loss(w, dims, feats, labels):
    """Independent float64 forward with torch library ops."""
    p = torch.from_numpy(np.asarray(w, dtype=np.float64))
    h = torch.from_numpy(feats).double()
    off = 0
    L = len(dims) - 1
    for l in range(L):
        i, o = dims[l], dims[l + 1]
        W = p[off:off + o * i].view(o, i); off += o * i
        b = p[off:off + o]; off += o
        h = torch.nn.functional.linear(h, W, b)
        if l + 1 < L:
            h = torch.relu(h)
    return float(torch.nn.functional.cross_entropy(h, torch.from_numpy(labels).long()))


# ---------------------------------------------------------------- storage / rounding

def test_bf16_rounding_matches_library_conversion(oracle):
    r = _rng(1)
    vals = np.concatenate([
        r.standard_normal(4000).astype(np.float32),
        (r.standard_normal(2000) * 1e-30).astype(np.float32),
        (r.standard_normal(2000) * 1e30).astype(np.float32),
        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, -1.00390625, 3.3895314e38, 3.4e38,
                  -3.4e38, 1e-40, 9.2e-41, 2.3e-41, 4.6e-41, 1.1754944e-38, np.inf, -np.inf],
                 dtype=np.float32),
        # every tie between neighbouring bfloat16 values around a few binades
        (np.arange(0, 512, dtype=np.float32) * 2.0 ** -8 + 1.0).astype(np.float32),
        (np.arange(0, 512, dtype=np.float32) * 2.0 ** -140).astype(np.float32),
    ])
    want = torch.from_numpy(vals).to(torch.bfloat16).double().numpy()
    got = np.array([oracle.round_to_bf16(float(v)) for v in vals])
    assert np.array_equal(got, want)
    assert math.isnan(oracle.round_to_bf16(float("nan")))


def test_bf16_storage_is_promoted_exactly(oracle):
    t = (torch.randn(257, generator=torch.Generator().manual_seed(3)) * 3).to(torch.bfloat16)
    w = oracle.candidate_params(syn.to_numpy_params(t), None, BF16, 0.0)
    assert np.array_equal(w, t.double().numpy())


def test_bf16_candidate_is_rounded_difference(oracle):
    g = torch.Generator().manual_seed(4)
    x = torch.randn(1000, generator=g).to(torch.bfloat16)
    v = (torch.randn(1000, generator=g) * 2).to(torch.bfloat16)
    gamma = float(np.float32(0.1))
    w = oracle.candidate_params(syn.to_numpy_params(x), syn.to_numpy_params(v), BF16, gamma)
    # library route: exact float64 difference -> float32 -> bfloat16
    want = (x.double() - gamma * v.double()).float().to(torch.bfloat16).double().numpy()
    assert np.array_equal(w, want)


def test_f32_candidate_is_exact_float64_difference(oracle):
    r = _rng(5)
    x = r.standard_normal(500).astype(np.float32)
    v = r.standard_normal(500).astype(np.float32)
    gamma = float(np.float32(0.05))
    w = oracle.candidate_params(x, v, F32, gamma)
    assert np.array_equal(w, x.astype(np.float64) - gamma * v.astype(np.float64))


def test_param_count_matches_layer_sizes(oracle):
    assert oracle.param_count(MLP, (784, 10)) == 7850
    assert oracle.param_count(MLP, (3072, 512, 512, 10)) == 1841162
    assert oracle.param_count(MLP, (4096, 4096, 4096, 1000)) == 37659624
    assert oracle.param_count(LSQ, (1 << 26, 1), False) == 1 << 26
    assert oracle.param_count(MLP, (3, 2), False) == 6


# ---------------------------------------------------------------- f_r, multi-layer perceptron

@pytest.mark.parametrize("dims", [(784, 10), (12, 8, 5), (9, 6, 6, 1000)])
def test_zero_parameters_give_log_num_classes(oracle, dims):
    d = syn.param_count("mlp", dims, True)
    r = _rng(6)
    feats = r.standard_normal((5, dims[0])).astype(np.float32)
    labels = r.integers(0, dims[-1], 5).astype(np.int32)
    f = oracle.loss(MLP, dims, True, np.zeros(d), feats, labels)
    assert f == pytest.approx(math.log(dims[-1]), rel=1e-14)


def test_hand_worked_two_layer_network(oracle):
    # W1 = I, b1 = (0,-1); W2 = [[1,-1],[0,2]], b2 = (0.5, 0)
    w = np.array([1, 0, 0, 1, 0, -1, 1, -1, 0, 2, 0.5, 0], dtype=np.float64)
    feats = np.array([[2, 3], [-1, 0.5]], dtype=np.float32)
    labels = np.array([0, 1], dtype=np.int32)
    # sample 0: h = relu(2, 2) -> z = (0.5, 4), label 0: loss = log(e^.5 + e^4) - .5
    l0 = 3.5 + math.log1p(math.exp(-3.5))
    # sample 1: pre-activations (-1, -0.5) are both clipped by the ReLU -> z = (0.5, 0),
    #           label 1: loss = log(e^.5 + 1)
    l1 = math.log(math.exp(0.5) + 1.0)
    f = oracle.loss(MLP, (2, 2, 2), True, w, feats, labels)
    assert f == pytest.approx((l0 + l1) / 2, rel=1e-14)
    # each sample alone (mean over n_r = 1)
    assert oracle.loss(MLP, (2, 2, 2), True, w, feats[:1], labels[:1]) == pytest.approx(l0, rel=1e-14)
    assert oracle.loss(MLP, (2, 2, 2), True, w, feats[1:], labels[1:]) == pytest.approx(l1, rel=1e-14)
    # weight layout: swapping the roles of W2's rows must change the answer
    w_t = w.copy(); w_t[6:10] = [1, 0, -1, 2]   # W2 transposed
    assert abs(oracle.loss(MLP, (2, 2, 2), True, w_t, feats, labels) - f) > 1e-3


@pytest.mark.parametrize("dims", [(11, 4), (7, 5, 3), (13, 9, 6, 4), (5, 8, 8, 8, 3)])
def test_mlp_loss_matches_torch_float64_forward(oracle, dims):
    r = _rng(hash(dims) % 1000)
    d = syn.param_count("mlp", dims, True)
    w = r.standard_normal(d)
    feats = r.standard_normal((6, dims[0])).astype(np.float32)
    labels = r.integers(0, dims[-1], 6).astype(np.int32)
    assert oracle.loss(MLP, dims, True, w, feats, labels) == pytest.approx(
        _torch_mlp_loss(w, dims, feats, labels), rel=1e-12)


def test_logsumexp_is_stable_for_huge_logits(oracle):
    # one layer, weights 1e4: logits of size 1e5; the loss is the gap to the largest logit
    w = np.array([1e4, 0, 0, -1e4, 0, 0], dtype=np.float64)   # W = diag(1e4, -1e4), b = 0
    feats = np.array([[10.0, 10.0]], dtype=np.float32)
    assert oracle.loss(MLP, (2, 2), True, w, feats, np.array([1], np.int32)) == pytest.approx(2e5)
    assert oracle.loss(MLP, (2, 2), True, w, feats, np.array([0], np.int32)) == pytest.approx(0.0, abs=1e-12)


def test_score_first_order_term_is_the_textbook_softmax_gradient(oracle):
    # softmax regression: grad f_r = (1/n_r) sum_j (p_j - e_{y_j}) x_j^T ; db = mean(p - e_y)
    dims = (9, 4)
    r = _rng(8)
    d = syn.param_count("mlp", dims, True)
    x = (r.standard_normal(d) * 0.3).astype(np.float32)
    v = r.standard_normal((1, d)).astype(np.float32)
    feats = r.standard_normal((5, 9)).astype(np.float32)
    labels = r.integers(0, 4, 5).astype(np.int32)
    W = x[:36].astype(np.float64).reshape(4, 9); bvec = x[36:].astype(np.float64)
    z = feats.astype(np.float64) @ W.T + bvec
    p = np.exp(z - z.max(1, keepdims=True)); p /= p.sum(1, keepdims=True)
    p[np.arange(5), labels] -= 1.0
    grad = np.concatenate([(p.T @ feats.astype(np.float64)).ravel() / 5, p.mean(0)])
    gdotv = float(grad @ v[0].astype(np.float64))
    gamma = 1e-6
    s, f, n = oracle.score(MLP, F32, dims, True, x, v, d, 1, feats, labels, gamma, 0.0)
    # s = f(x) - f(x - gamma v) = gamma <grad, v> + O(gamma^2)
    assert s[0] / gamma == pytest.approx(gdotv, rel=1e-4)


# ---------------------------------------------------------------- f_r, least squares

def _lsq_problem(seed, d=40, n_r=6, m=5):
    r = _rng(seed)
    A = (r.standard_normal((n_r, d)) / math.sqrt(d)).astype(np.float32)
    y = r.standard_normal(n_r).astype(np.float32)
    x = r.standard_normal(d).astype(np.float32)
    V = r.standard_normal((m, d)).astype(np.float32)
    return A, y, x, V


def test_quadratic_loss_difference_closed_form(oracle):
    A, y, x, V = _lsq_problem(9)
    n_r, d = A.shape
    gamma, rho = float(np.float32(0.3)), float(np.float32(0.01))
    s, f, n = oracle.score(LSQ, F32, (d, 1), False, x, V, d, V.shape[0], A, y, gamma, rho)
    A64, y64, x64, V64 = (a.astype(np.float64) for a in (A, y, x, V))
    grad = A64.T @ (A64 @ x64 - y64) / n_r
    H = A64.T @ A64 / n_r
    for i in range(V.shape[0]):
        diff = gamma * grad @ V64[i] - 0.5 * gamma ** 2 * V64[i] @ H @ V64[i]
        assert f[0] - f[1 + i] == pytest.approx(diff, rel=1e-10)
        assert s[i] == pytest.approx(diff - rho * V64[i] @ V64[i], rel=1e-10)
    assert f[0] == pytest.approx(np.sum((A64 @ x64 - y64) ** 2) / (2 * n_r), rel=1e-13)


def test_assumption2_sandwich_for_least_squares(oracle):
    A, y, x, V = _lsq_problem(10, d=12, n_r=20)
    n_r, d = A.shape
    A64 = A.astype(np.float64)
    ev = np.linalg.eigvalsh(A64.T @ A64 / n_r)
    mu, L = ev[0], ev[-1]
    grad = A64.T @ (A64 @ x.astype(np.float64) - y.astype(np.float64)) / n_r
    gamma = 0.2
    s, f, n = oracle.score(LSQ, F32, (d, 1), False, x, V, d, V.shape[0], A, y, gamma, 0.0)
    for i in range(V.shape[0]):
        u = V[i].astype(np.float64)
        lo = gamma * grad @ u - 0.5 * L * gamma ** 2 * u @ u
        hi = gamma * grad @ u - 0.5 * mu * gamma ** 2 * u @ u
        assert lo - 1e-12 <= s[i] <= hi + 1e-12


# ---------------------------------------------------------------- norm term, Score

def test_norm_of_3_4_is_25(oracle):
    x = np.zeros(2, np.float32)
    V = np.array([[3, 4]], np.float32)
    A = np.zeros((1, 2), np.float32); y = np.zeros(1, np.float32)
    s, f, n = oracle.score(LSQ, F32, (2, 1), False, x, V, 2, 1, A, y, 0.5, 0.125)
    assert n[0] == 25.0 and f[0] == 0.0 and s[0] == -25.0 * 0.125


def test_norm_includes_biases_and_skips_padding(oracle):
    dims = (3, 2)
    d = 8
    V = np.full((2, 11), np.nan, np.float32)
    V[:, :d] = np.arange(16, dtype=np.float32).reshape(2, 8)
    x = np.zeros(d, np.float32)
    feats = np.ones((1, 3), np.float32); labels = np.zeros(1, np.int32)
    s, f, n = oracle.score(MLP, F32, dims, True, x, V, 11, 2, feats, labels, 0.0, 1.0)
    assert n.tolist() == [float(sum(k * k for k in range(8))), float(sum(k * k for k in range(8, 16)))]
    assert np.all(np.isfinite(s))


def test_score_of_zero_update_is_exactly_zero(oracle):
    d, ldv, x, V, feats, labels = _random_mlp_problem(11)
    V[2, :d] = 0.0
    s, f, n = oracle.score(MLP, F32, (7, 5, 4, 3), True, x, V, ldv, 6, feats, labels, 0.1, 5e-4)
    assert s[2] == 0.0 and f[3] == f[0] and n[2] == 0.0


def test_score_difference_in_rho_is_the_norm(oracle):
    d, ldv, x, V, feats, labels = _random_mlp_problem(12, ldv=91)
    a = oracle.score(MLP, F32, (7, 5, 4, 3), True, x, V, ldv, 6, feats, labels, 0.1, 0.25)
    c = oracle.score(MLP, F32, (7, 5, 4, 3), True, x, V, ldv, 6, feats, labels, 0.1, 0.75)
    nrm = (V[:, :d].astype(np.float64) ** 2).sum(1)
    assert np.allclose(a[0] - c[0], 0.5 * nrm, rtol=1e-12)
    assert np.allclose(a[2], nrm, rtol=1e-14)


def test_gamma_zero_keeps_the_smallest_norms(oracle):
    d, ldv, x, V, feats, labels = _random_mlp_problem(13, m=7)
    V[:, :d] *= np.arange(1, 8, dtype=np.float32)[::-1, None]      # norms decrease with the index
    out, s, idx = oracle.step(MLP, F32, (7, 5, 4, 3), True, x, V, ldv, 7, feats, labels, 0.0, 1.0, 3)
    nrm = (V[:, :d].astype(np.float64) ** 2).sum(1)
    assert np.allclose(s, -nrm, rtol=1e-14)
    assert sorted(idx.tolist()) == sorted(np.argsort(nrm)[:4].tolist())
    assert np.allclose(out, V[np.argsort(nrm)[:4], :d].astype(np.float64).mean(0), rtol=1e-13)


# ---------------------------------------------------------------- ranking

def test_selection_is_the_best_subset_by_brute_force(oracle):
    r = _rng(14)
    for m in range(1, 10):
        s = r.standard_normal(m)
        for b in range(0, m):
            idx = oracle.select(s, b)
            best = max(itertools.combinations(range(m), m - b), key=lambda c: sum(s[list(c)]))
            assert sorted(idx.tolist()) == sorted(best)
            assert all(s[idx[i]] >= s[idx[i + 1]] for i in range(len(idx) - 1))


def test_lemma1_order_statistics_of_any_subset(oracle):
    r = _rng(15)
    s = r.standard_normal(12)
    order = oracle.select(s, 0)
    ranked = s[order]
    for size in (1, 3, 7, 12):
        for _ in range(20):
            C = r.choice(12, size, replace=False)
            sub = np.sort(s[C])[::-1]
            assert np.all(ranked[:size] >= sub)


def test_ties_go_to_the_lower_index_and_nan_is_worst(oracle):
    s = np.array([1.0, 2.0, 2.0, np.nan, -np.inf, 2.0, 0.5, np.nan])
    assert oracle.select(s, 0).tolist() == [1, 2, 5, 0, 6, 3, 4, 7]
    assert oracle.select(s, 5).tolist() == [1, 2, 5]
    assert oracle.select(np.array([np.inf, 3.0, np.inf]), 1).tolist() == [0, 2]


def test_select_rejects_bad_b(oracle):
    with pytest.raises(ValueError):
        oracle.select(np.zeros(4), 4)
    with pytest.raises(ValueError):
        oracle.select(np.zeros(4), -1)


def test_step_is_invariant_under_permutation_of_candidates(oracle):
    dims = (7, 5, 4, 3)
    d, ldv, x, V, feats, labels = _random_mlp_problem(16, m=8)
    out, s, idx = oracle.step(MLP, F32, dims, True, x, V, ldv, 8, feats, labels, 0.1, 5e-4, 3)
    perm = _rng(17).permutation(8)
    out_p, s_p, idx_p = oracle.step(MLP, F32, dims, True, x, V[perm], ldv, 8, feats, labels, 0.1, 5e-4, 3)
    assert np.array_equal(s_p, s[perm])
    assert sorted(perm[idx_p].tolist()) == sorted(idx.tolist())
    assert np.allclose(out_p, out, rtol=1e-13, atol=1e-15)


def test_duplicated_candidates_score_equal_and_average_the_same(oracle):
    dims = (7, 5, 4, 3)
    d, ldv, x, V, feats, labels = _random_mlp_problem(18, m=6)
    V[4] = V[1]
    V[5] = V[1]
    out, s, idx = oracle.step(MLP, F32, dims, True, x, V, ldv, 6, feats, labels, 0.1, 5e-4, 2)
    assert s[4] == s[1] == s[5]
    # replacing a selected duplicate by another one leaves the average unchanged
    alt = [4 if i == 1 else i for i in idx.tolist()]
    assert np.allclose(oracle.aggregate(F32, V, ldv, d, 6, np.array(alt, np.int32)),
                       oracle.aggregate(F32, V, ldv, d, 6, idx), rtol=1e-14)


# ---------------------------------------------------------------- trimmed average

def test_b_zero_is_the_plain_mean(oracle):
    dims = (7, 5, 4, 3)
    d, ldv, x, V, feats, labels = _random_mlp_problem(19, m=6, ldv=80)
    out, s, idx = oracle.step(MLP, F32, dims, True, x, V, ldv, 6, feats, labels, 0.1, 5e-4, 0)
    assert sorted(idx.tolist()) == list(range(6))
    assert np.allclose(out, V[:, :d].astype(np.float64).mean(0), rtol=1e-13, atol=1e-16)


def test_b_m_minus_1_returns_the_best_row(oracle):
    dims = (7, 5, 4, 3)
    d, ldv, x, V, feats, labels = _random_mlp_problem(20, m=6)
    out, s, idx = oracle.step(MLP, F32, dims, True, x, V, ldv, 6, feats, labels, 0.1, 5e-4, 5)
    assert idx.tolist() == [int(np.argmax(s))]
    assert np.array_equal(out, V[idx[0], :d].astype(np.float64))


def test_aggregate_bf16_rows_with_library_mean(oracle):
    t = (torch.randn(5, 40, generator=torch.Generator().manual_seed(21)) * 3).to(torch.bfloat16)
    idx = np.array([4, 0, 2], np.int32)
    out = oracle.aggregate(BF16, syn.to_numpy_params(t), 40, 37, 5, idx)
    assert np.allclose(out, t.double().numpy()[[4, 0, 2], :37].mean(0), rtol=1e-14)


# ---------------------------------------------------------------- Algorithm 1's server update

def test_update_hand_values_and_gamma_zero(oracle):
    """x - gamma * vbar on numbers worked by hand; gamma = 0 leaves x as it is."""
    x = np.array([1.0, 2.0, -3.0], np.float32)
    vbar = np.array([0.5, -4.0, 8.0])
    assert np.allclose(oracle.update(F32, x, vbar, 0.1), [0.95, 2.4, -3.8], rtol=1e-15)
    assert np.array_equal(oracle.update(F32, x, vbar, 0.0), x.astype(np.float64))
    xb = torch.tensor([1.5, -0.3125, 96.0]).to(torch.bfloat16)
    assert np.array_equal(oracle.update(BF16, syn.to_numpy_params(xb), vbar, 0.0), xb.double().numpy())


def test_update_of_bf16_parameters_rounds_to_nearest_even(oracle):
    """1 - 2^-9 lies halfway between the bfloat16 neighbours 255/256 and 1: the tie goes to 1 (even);
    1 - 3 * 2^-10 is nearer to 255/256; library route for random values."""
    one = syn.to_numpy_params(torch.tensor([1.0, 1.0]).to(torch.bfloat16))
    got = oracle.update(BF16, one, np.array([2.0 ** -9, 3 * 2.0 ** -10]), 1.0)
    assert got.tolist() == [1.0, 255.0 / 256.0]
    g = torch.Generator().manual_seed(31)
    x = torch.randn(2000, generator=g).to(torch.bfloat16)
    vbar = torch.randn(2000, generator=g, dtype=torch.float64) * 3
    gamma = float(np.float32(0.05))
    want = (x.double() - gamma * vbar).float().to(torch.bfloat16).double().numpy()
    assert np.array_equal(oracle.update(BF16, syn.to_numpy_params(x), vbar.numpy(), gamma), want)


def test_update_after_step_is_x_minus_gamma_times_mean_of_kept_rows(oracle):
    dims = (7, 5, 4, 3)
    d, ldv, x, V, feats, labels = _random_mlp_problem(23, m=6)
    out, s, idx = oracle.step(MLP, F32, dims, True, x, V, ldv, 6, feats, labels, 0.1, 5e-4, 2)
    kept = np.argsort(-s, kind="stable")[:4]
    want = x.astype(np.float64) - 0.1 * V[kept, :d].astype(np.float64).mean(0)
    assert np.allclose(oracle.update(F32, x, out, 0.1), want, rtol=1e-13, atol=1e-16)


def test_aggregate_rejects_out_of_range_index(oracle):
    V = np.zeros((3, 4), np.float32)
    with pytest.raises(RuntimeError):
        oracle.aggregate(F32, V, 4, 4, 3, np.array([0, 3], np.int32))


@pytest.mark.parametrize("kind", ["softmax", "lsq"])
def test_jensen_step_for_convex_losses(oracle, kind):
    # convex f_r (mu = 0): f_r(x - gamma * mean of selected) <= mean of f_r(x - gamma v_(i))
    if kind == "softmax":
        dims = (9, 4); K = MLP; bias = True
        d, ldv, x, V, feats, tgt = _random_mlp_problem(22, dims=dims, m=8)
    else:
        A, y, x, V = _lsq_problem(23, m=8)
        dims = (A.shape[1], 1); K = LSQ; bias = False; d = ldv = A.shape[1]; feats, tgt = A, y
    gamma = 0.1
    out, s, idx = oracle.step(K, F32, dims, bias, x, V, ldv, 8, feats, tgt, gamma, 5e-4, 3)
    _, f, _ = oracle.score(K, F32, dims, bias, x, V, ldv, 8, feats, tgt, gamma, 5e-4)
    f_at_mean = oracle.loss(K, dims, bias, x.astype(np.float64) - gamma * out, feats, tgt)
    assert f_at_mean <= np.mean(f[1 + idx]) + 1e-12


# ---------------------------------------------------------------- cost model

def test_cost_model_84_sample_evaluations(oracle):
    vals = {}
    with open(os.path.join(GOLDEN, "cost_model.txt")) as fh:
        for line in fh:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                vals[k] = int(v)
    m, n_r = vals["m"], vals["n_r"]
    w = syn.make_config(1, dims=(20, 10))
    assert (w.m, w.n_r) == (m, n_r)
    oracle.reset_eval_count()
    oracle.step(MLP, F32, w.dims, True, w.x.numpy(), w.V.numpy(), w.ldv, w.m, w.features.numpy(),
                w.targets.numpy(), w.gamma, w.rho, w.b)
    assert oracle.eval_count() == vals["sample_evaluations"] == (m + 1) * n_r
