"""Full-size workloads (configurations 3, 4, 5) in the launch configuration bench.py times.

Every candidate's score and the whole mean are compared with the oracle; for the two largest
workloads the oracle works through the candidates a few rows at a time (each candidate's score
depends on no other candidate) and through the mean a block of columns at a time, so that the host
never holds more than a few GB.  The ranking is integer work and is checked bit-exactly on the GPU's
own scores.  Inputs are generated on the device with the seeded recipes and copied to the host for
the oracle: both sides see the same buffers."""
import numpy as np
import pytest
import torch

from paper_1805_10032_b200 import synthetic as syn
from paper_1805_10032_b200 import zeno

import parity as P

pytestmark = [pytest.mark.gpu, pytest.mark.slow]


@pytest.fixture(scope="module", autouse=True)
def _library():
    from paper_1805_10032_b200 import build as zbuild
    zbuild.build()
    assert torch.cuda.is_available()
    zeno.load_library()


def _chunked_oracle_scores(oracle, w, chunk):
    """Oracle scores of every candidate, a few rows at a time (each candidate's score depends on no
    other candidate; f_r(x) is recomputed per chunk and must come out the same)."""
    o_kind, o_dt = P.KIND[w.kind], P.DTYPE[w.dtype]
    x = syn.to_numpy_params(w.x)
    feats, tgt = w.features.cpu().numpy(), w.targets.cpu().numpy()
    gamma, rho = float(np.float32(w.gamma)), float(np.float32(w.rho))
    s_all, f_all, n_all = np.empty(w.m), np.empty(w.m + 1), np.empty(w.m)
    for r0 in range(0, w.m, chunk):
        r1 = min(w.m, r0 + chunk)
        Vs = syn.to_numpy_params(w.V[r0:r1])
        s, f, n = oracle.score(o_kind, o_dt, w.dims, w.has_bias, x, Vs, w.ldv, r1 - r0, feats, tgt, gamma, rho)
        if r0 > 0:
            assert f[0] == f_all[0]
        s_all[r0:r1], n_all[r0:r1] = s, n
        f_all[0] = f[0]
        f_all[1 + r0:1 + r1] = f[1:]
    return s_all, f_all, n_all


def _whole_mean_check(oracle, w, idx, out, block):
    """The oracle's mean over every column, a block of columns at a time."""
    dt = P.DTYPE[w.dtype]
    num, den = 0.0, 0.0
    for c0 in range(0, w.d, block):
        c1 = min(w.d, c0 + block)
        Vb = syn.to_numpy_params(w.V[:, c0:c1].contiguous())
        ref = oracle.aggregate(dt, Vb, c1 - c0, c1 - c0, w.m, idx)
        got = out[c0:c1].cpu().numpy().astype(np.float64)
        num += float(np.sum((got - ref) ** 2))
        den += float(np.sum(ref ** 2))
        assert P.rel_l2(got, ref) <= P.AGG_RTOL, (c0, c1)
    assert (num / den) ** 0.5 <= P.AGG_RTOL


def test_config3_full(oracle):
    w = syn.make_config(3, device="cuda")
    assert (w.m, w.b, w.n_r, w.d) == (100, 40, 64, 1841162)
    with zeno.from_workload(w) as z:
        out, scores, idx = z.step(w.x, w.V, w.features, w.targets, w.gamma, w.rho, w.b)
        torch.cuda.synchronize()
        z.check_device_status()
    s_orc, f_orc, n_orc = P.oracle_score(oracle, w)
    s_gpu = scores.cpu().numpy()
    P.assert_scores_close(s_gpu, s_orc)
    assert np.array_equal(idx.cpu().numpy(), oracle.select(s_gpu.astype(np.float64), w.b))
    P.assert_selection_valid(idx.cpu().numpy(), s_orc, w.b)
    ref = oracle.aggregate(0, syn.to_numpy_params(w.V), w.ldv, w.d, w.m, idx.cpu().numpy())
    assert P.rel_l2(out.cpu().numpy(), ref) <= P.AGG_RTOL


def test_config4_full(oracle):
    w = syn.make_config(4, device="cuda")
    assert (w.m, w.b, w.n_r, w.d) == (32, 12, 128, 37659624) and w.V.dtype == torch.bfloat16
    with zeno.from_workload(w) as z:
        out, scores, idx = z.step(w.x, w.V, w.features, w.targets, w.gamma, w.rho, w.b)
        s2, losses, norms = z.score(w.x, w.V, w.features, w.targets, w.gamma, w.rho)
        torch.cuda.synchronize()
    s_gpu = scores.cpu().numpy()
    faulty = torch.nonzero(~w.honest).flatten().tolist()
    s_orc, f_orc, n_orc = _chunked_oracle_scores(oracle, w, 16)      # all 32 candidates
    P.assert_scores_close(s_gpu, s_orc, f_orc, n_orc, float(np.float32(w.rho)))
    assert np.allclose(norms.cpu().numpy(), n_orc, rtol=1e-5)
    assert np.allclose(losses.cpu().numpy(), f_orc, rtol=1e-4)
    assert np.array_equal(idx.cpu().numpy(), oracle.select(s_gpu.astype(np.float64), w.b))
    P.assert_selection_valid(idx.cpu().numpy(), s_orc, w.b)
    _whole_mean_check(oracle, w, idx.cpu().numpy(), out, 1 << 22)
    # identical sign-flip rows score bit-identically
    assert len({s_gpu[i] for i in faulty}) == 1


def test_config5_full(oracle):
    w = syn.make_config(5, device="cuda")
    assert (w.m, w.b, w.n_r, w.d) == (64, 24, 16, 1 << 26)
    with zeno.from_workload(w) as z:
        out, scores, idx = z.step(w.x, w.V, w.features, w.targets, w.gamma, w.rho, w.b)
        torch.cuda.synchronize()
    s_gpu = scores.cpu().numpy()
    faulty = torch.nonzero(~w.honest).flatten().tolist()
    s_orc, f_orc, n_orc = _chunked_oracle_scores(oracle, w, 8)       # all 64 candidates, 2 GB of rows at a time
    P.assert_scores_close(s_gpu, s_orc, f_orc, n_orc, float(np.float32(w.rho)))
    assert np.array_equal(idx.cpu().numpy(), oracle.select(s_gpu.astype(np.float64), w.b))
    P.assert_selection_valid(idx.cpu().numpy(), s_orc, w.b)
    # every noise row must have been trimmed here: its norm term alone is -6.7e7
    assert not set(idx.cpu().tolist()) & set(faulty)
    _whole_mean_check(oracle, w, idx.cpu().numpy(), out, 1 << 22)
