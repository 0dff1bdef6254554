"""The workers' side of Algorithm 1 on the device (gradients of the workers' own batches, the experiments'
failures) against the float64 oracle, and a whole synchronous iteration chained on one stream --
workers' gradients -> failures -> Zeno_b -> update -- against the same chain on the host."""
import numpy as np
import pytest
import torch

from paper_1805_10032_b200 import zeno

import parity as P

pytestmark = pytest.mark.gpu

MLP, LSQ, F32 = 0, 1, 0


@pytest.fixture(scope="module", autouse=True)
def _library():
    from paper_1805_10032_b200 import build as zbuild
    zbuild.build()
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    zeno.load_library()


def _softmax_problem(seed, m=20, n_w=100, dims=(784, 10), n_r=4):
    g = torch.Generator().manual_seed(seed)
    d = dims[0] * dims[1] + dims[1]
    x = torch.randn(d, generator=g) * 0.1
    feats = torch.randn(m, n_w, dims[0], generator=g)
    labels = torch.randint(0, dims[1], (m, n_w), generator=g, dtype=torch.int32)
    sf = torch.randn(n_r, dims[0], generator=g)
    sl = torch.randint(0, dims[1], (n_r,), generator=g, dtype=torch.int32)
    return x, feats, labels, sf, sl, d


def test_softmax_regression_worker_gradients_and_label_flipping(oracle):
    dims = (784, 10)
    x, feats, labels, _, _, d = _softmax_problem(1)
    m = feats.shape[0]
    flip = torch.zeros(m, dtype=torch.int32)
    flip[[2, 5, 11]] = 1
    ldv = d + 6
    V = torch.full((m, ldv), float("nan"), device="cuda")
    with zeno.Zeno(MLP, F32, dims, m_max=m, n_r_max=4) as z:
        z.worker_gradients(x.cuda(), feats.cuda(), labels.cuda(), V, label_flip=flip.cuda())
        torch.cuda.synchronize()
    Vh = V.cpu()
    assert torch.isnan(Vh[:, d:]).all()                                  # the padding is not touched
    for i in range(m):
        want = oracle.worker_gradient(MLP, F32, dims, True, x.numpy(), feats[i].numpy(), labels[i].numpy(),
                                      flip=bool(flip[i]))
        assert P.rel_l2(Vh[i, :d].numpy(), want) <= 2e-6, i


def test_least_squares_worker_gradients(oracle):
    g = torch.Generator().manual_seed(3)
    d, m, n_w = 5003, 6, 9
    x = torch.randn(d, generator=g)
    A = torch.randn(m, n_w, d, generator=g) * d ** -0.5
    y = torch.randn(m, n_w, generator=g)
    V = torch.empty((m, d + 1), device="cuda")
    with zeno.Zeno(LSQ, F32, (d, 1), m_max=m, n_r_max=16) as z:
        z.worker_gradients(x.cuda(), A.cuda(), y.cuda(), V)
        torch.cuda.synchronize()
    for i in range(m):
        want = oracle.worker_gradient(LSQ, F32, (d, 1), False, x.numpy(), A[i].numpy(), y[i].numpy())
        assert P.rel_l2(V[i, :d].cpu().numpy(), want) <= 5e-6, i


@pytest.mark.parametrize("mode,eps", [(zeno.FAULT_BIT_FLIP, 0.0), (zeno.FAULT_SCALE, -4.0)])
def test_failures_match_the_oracle_exactly(oracle, mode, eps):
    g = torch.Generator().manual_seed(7)
    m, d = 9, 1031
    Vh = torch.randn(m, d + 3, generator=g)
    faulty = torch.tensor([6, 1, 8, 3], dtype=torch.int32)
    V = Vh.cuda()
    with zeno.Zeno(LSQ, F32, (d, 1), m_max=m, n_r_max=4) as z:
        z.inject_faults(V, faulty.cuda(), mode, eps)
        torch.cuda.synchronize()
    want = oracle.inject_faults(Vh[:, :d].double().numpy(), faulty.numpy(), mode, eps)
    assert np.array_equal(V[:, :d].cpu().double().numpy(), want)         # negation, copies and a power-of-two scale: exact
    assert torch.equal(V[:, d:].cpu(), Vh[:, d:])


def test_unsupported_models_are_refused():
    with zeno.Zeno(MLP, F32, (20, 8, 4), m_max=4, n_r_max=4) as z:        # a hidden layer: needs back-propagation
        x = torch.zeros(z.d, device="cuda")
        V = torch.zeros((4, z.d), device="cuda")
        with pytest.raises(zeno.ZenoError) as e:
            z.worker_gradients(x, torch.zeros(4, 5, 20, device="cuda"), torch.zeros(4, 5, dtype=torch.int32, device="cuda"), V)
        assert e.value.status == zeno.ERR_UNSUPPORTED


@pytest.mark.parametrize("failure", ["none", "label_flip", "bit_flip"])
def test_whole_synchronous_iterations_on_the_device(oracle, failure):
    """T iterations of Algorithm 1 with m = 20 workers of which q = 12 are faulty (more than half, the case the
    paper is about), every step enqueued on one stream; the host repeats the chain with the oracle."""
    dims, m, n_w, n_r, T, b, q = (784, 10), 20, 100, 4, 3, 12, 12
    gamma, rho = 0.1, 5e-4
    x0, _, _, _, _, d = _softmax_problem(100)
    batches = [_softmax_problem(200 + t, m=m, n_w=n_w, n_r=n_r) for t in range(T)]
    faulty = torch.arange(q, dtype=torch.int32) if failure != "none" else torch.zeros(0, dtype=torch.int32)
    flip = torch.zeros(m, dtype=torch.int32)
    if failure == "label_flip":
        flip[faulty.long()] = 1
    ldv = d + 2
    x = x0.cuda().clone()
    V = torch.zeros((m, ldv), device="cuda")
    all_scores, all_idx = [], []
    with zeno.Zeno(MLP, F32, dims, m_max=m, n_r_max=n_r) as z:
        dev = [(f.cuda(), l.cuda(), sf.cuda(), sl.cuda()) for _, f, l, sf, sl, _ in batches]
        fl, fa = flip.cuda(), faulty.cuda()
        for t in range(T):                       # nothing below waits for the device
            f, l, sf, sl = dev[t]
            z.worker_gradients(x, f, l, V, label_flip=fl)
            if failure == "bit_flip":
                z.inject_faults(V, fa, zeno.FAULT_BIT_FLIP)
            _, s, i = z.step_update(x, V, sf, sl, gamma, rho, b, want_out=False)
            all_scores.append(s)
            all_idx.append(i)
        torch.cuda.synchronize()
        z.check_device_status()
    # the same chain on the host
    x_orc = x0.numpy().copy()
    g32, r32 = float(np.float32(gamma)), float(np.float32(rho))
    for t in range(T):
        _, f, l, sf, sl, _ = batches[t]
        Vd = np.stack([oracle.worker_gradient(MLP, F32, dims, True, x_orc, f[i].numpy(), l[i].numpy(), flip=bool(flip[i]))
                       for i in range(m)])
        if failure == "bit_flip":
            Vd = oracle.inject_faults(Vd, faulty.numpy(), 0)
        V32 = Vd.astype(np.float32)               # the candidates are stored in binary32
        s_orc, f_orc, n_orc = oracle.score(MLP, F32, dims, True, x_orc, V32, d, m, sf.numpy(), sl.numpy(), g32, r32)
        P.assert_scores_close(all_scores[t].cpu().numpy(), s_orc, f_orc, n_orc, r32, rtol=2e-4)
        idx = all_idx[t].cpu().numpy()
        P.assert_selection_valid(idx, s_orc, b, rtol_score=2e-4)
        # (which rows survive is the oracle's business: with synthetic random labels a faulty gradient need not
        # look worse than an honest one, so nothing is asserted about who gets trimmed)
        vbar = oracle.aggregate(F32, V32, d, d, m, idx)
        x_orc = oracle.update(F32, x_orc, vbar, g32).astype(np.float32)
    assert P.rel_l2(x.cpu().numpy(), x_orc) <= 1e-5
