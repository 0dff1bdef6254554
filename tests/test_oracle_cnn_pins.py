"""Pins for the oracle's convolutional loss (the paper's experiments train a CNN of four convolutional
layers and one dense layer; the network's exact definition is this project's own and is stated at the
top of oracle/zeno_oracle.c) -- against the mathematics and library routines, never against the CUDA path.

  parameter count : the closed form, layer by layer
  one tap         : a kernel with a single 1 moves the image by that tap (orientation of dy / dx, and
                    that the sum is a cross-correlation, not a convolution with a flipped kernel)
  zero padding    : an all-ones kernel on an all-ones image counts 4 / 6 / 9 pixels at corners, edges, inside
  whole network   : the logits rebuilt with scipy.signal.correlate2d, numpy's max over 2 x 2 windows and a
                    matrix product; the loss with scipy's logsumexp
  identity kernels: the convolutional layers then only pass the (non-negative) image on, and the loss equals
                    the pinned softmax-regression loss (kind 0) on the pooled image
  bias, ReLU, NaN : a negative bias switches a plane off; a NaN pixel makes the loss NaN
"""
import numpy as np
import pytest
from scipy.signal import correlate2d
from scipy.special import logsumexp

MLP, CNN = 0, 2


def _rng(seed):
    return np.random.default_rng(seed)


def _layout(dims, has_bias=True):
    """Offsets of the layers' weights and biases in the flat parameter vector."""
    S, chans, classes = dims[0], dims[1:-1], dims[-1]
    lc = len(chans) - 1
    off, conv = 0, []
    for l in range(1, lc + 1):
        nw = chans[l] * chans[l - 1] * 9
        conv.append((off, off + nw if has_bias else None))
        off += nw + (chans[l] if has_bias else 0)
    side = S // (2 ** (lc // 2))
    flat = chans[-1] * side * side
    dense = (off, off + classes * flat if has_bias else None)
    off += classes * flat + (classes if has_bias else 0)
    return conv, dense, flat, side, off


def _reference_logits(dims, has_bias, w, feat):
    """The same network from library routines."""
    S, chans, classes = dims[0], dims[1:-1], dims[-1]
    conv, dense, flat, side, _ = _layout(dims, has_bias)
    h = np.asarray(feat, dtype=np.float64).reshape(chans[0], S, S)
    for l, (ow, ob) in enumerate(conv, start=1):
        cin, cout = chans[l - 1], chans[l]
        W = w[ow:ow + cout * cin * 9].reshape(cout, cin, 3, 3)
        out = np.zeros((cout,) + h.shape[1:])
        for co in range(cout):
            for ci in range(cin):
                out[co] += correlate2d(h[ci], W[co, ci], mode="same", boundary="fill", fillvalue=0.0)
            if has_bias:
                out[co] += w[ob + co]
        h = np.maximum(out, 0.0)
        if l % 2 == 0:
            c, s, _ = h.shape
            h = h.reshape(c, s // 2, 2, s // 2, 2).max(axis=(2, 4))
    ow, ob = dense
    z = w[ow:ow + classes * flat].reshape(classes, flat) @ h.reshape(-1)
    if has_bias:
        z = z + w[ob:ob + classes]
    return z


def test_parameter_count_is_the_layer_sum(oracle):
    dims = [32, 3, 32, 32, 64, 64, 10]
    want = (3 * 32 * 9 + 32) + (32 * 32 * 9 + 32) + (32 * 64 * 9 + 64) + (64 * 64 * 9 + 64) + (10 * 64 * 8 * 8 + 10)
    assert oracle.param_count(CNN, dims, True) == want == _layout(dims)[4]
    assert oracle.param_count(CNN, dims, False) == want - (32 + 32 + 64 + 64 + 10)
    assert oracle.param_count(CNN, [8, 1, 2, 2, 3], True) == (2 * 9 + 2) + (4 * 9 + 2) + (3 * 2 * 16 + 3)
    # an odd number of convolutional layers, or a side the poolings do not divide, is no network
    assert oracle.param_count(CNN, [8, 1, 2, 3], True) == 0
    assert oracle.param_count(CNN, [6, 1, 2, 2, 2, 2, 3], True) == 0


def _readout_net(S):
    """One plane, two convolutional layers, then a dense layer that reads the pooled plane out:
    logits = the (S/2)^2 pooled values."""
    half = S // 2
    dims = [S, 1, 1, 1, half * half]
    conv, dense, flat, side, d = _layout(dims, True)
    w = np.zeros(d)
    w[dense[0]:dense[0] + flat * flat] = np.eye(flat).reshape(-1)
    return dims, conv, w


@pytest.mark.parametrize("tap", [(0, 0), (0, 1), (0, 2), (1, 0), (1, 2), (2, 0), (2, 1), (2, 2)])
def test_a_single_tap_moves_the_image(oracle, tap):
    S = 8
    dims, conv, w = _readout_net(S)
    dy, dx = tap
    w[conv[0][0] + dy * 3 + dx] = 1.0          # layer 1: out[y][x] = in[y + dy - 1][x + dx - 1]
    w[conv[1][0] + 4] = 1.0                    # layer 2: the centre tap, the identity
    img = _rng(7).random((S, S)).astype(np.float32) + 0.5      # positive: ReLU leaves it alone
    padded = np.zeros((S + 2, S + 2))
    padded[1:-1, 1:-1] = img
    moved = padded[dy:dy + S, dx:dx + S]
    want = moved.reshape(S // 2, 2, S // 2, 2).max(axis=(1, 3)).reshape(-1)
    got = oracle.cnn_logits(dims, True, w, img)
    assert np.array_equal(got, want)


def test_zero_padding_counts_the_pixels_inside(oracle):
    S = 4
    dims = [S, 1, 1, 1, 4]
    conv, dense, flat, side, d = _layout(dims, True)
    w = np.zeros(d)
    w[conv[0][0]:conv[0][0] + 9] = 1.0         # layer 1 sums the 3 x 3 window
    w[conv[1][0] + 4] = 1.0
    w[dense[0]:dense[0] + 16] = np.eye(4).reshape(-1)
    got = oracle.cnn_logits(dims, True, w, np.ones((S, S), dtype=np.float32))
    # window sums: corners 4, edges 6, inside 9; every 2 x 2 pooling window of a 4 x 4 plane holds one inside pixel
    assert got.tolist() == [9.0, 9.0, 9.0, 9.0]
    w[conv[1][0] + 4] = -1.0                   # layer 2 negates: ReLU leaves zeros
    assert oracle.cnn_logits(dims, True, w, np.ones((S, S), dtype=np.float32)).tolist() == [0.0] * 4
    # without pooling inside pixels in the way: read the corner through a one-tap second layer
    w[conv[1][0] + 4] = 0.0
    w[conv[1][0] + 0] = 1.0                    # out[y][x] = h[y - 1][x - 1]: window (0, 0) sees h[0][0] = 4 at most
    got = oracle.cnn_logits(dims, True, w, np.ones((S, S), dtype=np.float32))
    assert got[0] == 4.0 and got[1] == 6.0 and got[2] == 6.0 and got[3] == 9.0


@pytest.mark.parametrize("dims,has_bias,seed", [
    ([8, 3, 4, 5, 7], True, 1),
    ([8, 2, 3, 3, 4, 5, 6], True, 2),
    ([12, 1, 2, 3, 3], False, 3),
    ([16, 3, 6, 6, 8, 8, 10], True, 4),
])
def test_logits_and_loss_from_library_routines(oracle, dims, has_bias, seed):
    r = _rng(seed)
    d = oracle.param_count(CNN, dims, has_bias)
    assert d == _layout(dims, has_bias)[4]
    w = r.standard_normal(d) * 0.3
    n_r = 5
    feats = r.standard_normal((n_r, dims[1], dims[0], dims[0])).astype(np.float32)
    labels = r.integers(0, dims[-1], n_r).astype(np.int32)
    losses = []
    for j in range(n_r):
        z = _reference_logits(dims, has_bias, w, feats[j])
        got = oracle.cnn_logits(dims, has_bias, w, feats[j])
        assert np.allclose(got, z, rtol=1e-12, atol=1e-12)
        losses.append(logsumexp(z) - z[labels[j]])
    got = oracle.loss(CNN, dims, has_bias, w, feats, labels)
    assert got == pytest.approx(np.mean(losses), rel=1e-12)


def test_identity_kernels_reduce_to_softmax_regression(oracle):
    S, C, classes = 8, 3, 5
    dims = [S, C, C, C, C, C, classes]
    conv, dense, flat, side, d = _layout(dims, True)
    r = _rng(11)
    w = np.zeros(d)
    for l, (ow, _) in enumerate(conv):
        W = np.zeros((C, C, 3, 3))
        for c in range(C):
            W[c, c, 1, 1] = 1.0
        w[ow:ow + C * C * 9] = W.reshape(-1)
    w[dense[0]:] = r.standard_normal(d - dense[0])
    n_r = 6
    feats = r.random((n_r, C, S, S)).astype(np.float32)           # non-negative: ReLU is the identity
    labels = r.integers(0, classes, n_r).astype(np.int32)
    pooled = feats.astype(np.float64)
    for _ in range(2):
        n, c, s, _ = pooled.shape
        pooled = pooled.reshape(n, c, s // 2, 2, s // 2, 2).max(axis=(3, 5))
    pooled32 = pooled.reshape(n_r, -1).astype(np.float32)         # maxima of float32 values are float32 values
    assert np.array_equal(pooled32.astype(np.float64), pooled.reshape(n_r, -1))
    want = oracle.loss(MLP, [flat, classes], True, w[dense[0]:], pooled32, labels)
    got = oracle.loss(CNN, dims, True, w, feats, labels)
    assert got == pytest.approx(want, rel=1e-13)


def test_bias_relu_and_nan(oracle):
    S = 4
    dims = [S, 1, 1, 1, 4]
    conv, dense, flat, side, d = _layout(dims, True)
    w = np.zeros(d)
    w[conv[0][0] + 4] = 1.0
    w[conv[1][0] + 4] = 1.0
    w[dense[0]:dense[0] + 16] = np.eye(4).reshape(-1)
    img = np.arange(16, dtype=np.float32).reshape(S, S)
    assert oracle.cnn_logits(dims, True, w, img).tolist() == [5.0, 7.0, 13.0, 15.0]
    w[conv[0][1]] = -6.0                       # layer 1's bias: values up to 6 are switched off
    assert oracle.cnn_logits(dims, True, w, img).tolist() == [0.0, 1.0, 7.0, 9.0]
    w[conv[0][1]] = 0.0
    img[0, 0] = np.nan                         # a NaN pixel reaches every logit: the dense layer's zero weights
    got = oracle.cnn_logits(dims, True, w, img)  # multiply it too (0 x NaN = NaN), as IEEE arithmetic has it
    assert np.isnan(got).all()
    assert np.isnan(oracle.loss(CNN, dims, True, w, img[None, None], np.zeros(1, dtype=np.int32)))


def test_score_uses_the_cnn_loss_per_candidate(oracle):
    dims = [8, 2, 3, 3, 4]
    r = _rng(21)
    d = oracle.param_count(CNN, dims, True)
    m, n_r, gamma, rho = 4, 3, 0.05, 0.01
    x = (r.standard_normal(d) * 0.3).astype(np.float32)
    V = (r.standard_normal((m, d + 3)) * 0.5).astype(np.float32)
    feats = r.standard_normal((n_r, 2, 8, 8)).astype(np.float32)
    labels = r.integers(0, 4, n_r).astype(np.int32)
    s, f, n = oracle.score(CNN, 0, dims, True, x, V, d + 3, m, feats, labels, gamma, rho)
    f0 = oracle.loss(CNN, dims, True, x.astype(np.float64), feats, labels)
    assert f[0] == f0
    for i in range(m):
        wi = x.astype(np.float64) - gamma * V[i, :d].astype(np.float64)
        fi = oracle.loss(CNN, dims, True, wi, feats, labels)
        ni = float(np.sum(V[i, :d].astype(np.float64) ** 2))
        assert f[1 + i] == pytest.approx(fi, rel=1e-14)
        assert n[i] == pytest.approx(ni, rel=1e-14)
        assert s[i] == pytest.approx(f0 - fi - rho * ni, rel=1e-12, abs=1e-15)
