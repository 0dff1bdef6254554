"""Full-size workloads (configurations 3, 4, 5) in the launch configuration bench.py times.

The oracle cannot evaluate every candidate of the two largest workloads in seconds, so there it
scores a sample of candidates one by one (each candidate's score depends on no other candidate)
and averages sampled column blocks; the ranking is integer work and is checked bit-exactly on the
GPU's own scores.  Inputs are generated on the device with the seeded recipes and copied to the
host for the oracle: both sides see the same buffers."""
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


def _sampled_score_check(oracle, w, rows):
    """Oracle scores of the candidates `rows` only (plus f_r(x)), as a sub-problem with m' rows."""
    o_kind, o_dt = P.KIND[w.kind], P.DTYPE[w.dtype]
    Vs = syn.to_numpy_params(w.V[rows])
    s, f, n = oracle.score(o_kind, o_dt, w.dims, w.has_bias, syn.to_numpy_params(w.x), Vs, w.ldv, len(rows),
                           w.features.cpu().numpy(), w.targets.cpu().numpy(),
                           float(np.float32(w.gamma)), float(np.float32(w.rho)))
    return s, f, n


def _column_block_check(oracle, w, idx, out, blocks):
    dt = P.DTYPE[w.dtype]
    for c0, c1 in blocks:
        Vb = syn.to_numpy_params(w.V[:, c0:c1].contiguous())
        ref = oracle.aggregate(dt, Vb, c1 - c0, c1 - c0, w.m, idx)
        got = out[c0:c1].cpu().numpy()
        assert P.rel_l2(got, ref) <= P.AGG_RTOL, (c0, c1)


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


def test_config4_full_sampled(oracle):
    w = syn.make_config(4, device="cuda")
    assert (w.m, w.b, w.n_r, w.d) == (32, 12, 128, 37659624) and w.V.dtype == torch.bfloat16
    with zeno.from_workload(w) as z:
        out, scores, idx = z.step(w.x, w.V, w.features, w.targets, w.gamma, w.rho, w.b)
        s2, losses, norms = z.score(w.x, w.V, w.features, w.targets, w.gamma, w.rho)
        torch.cuda.synchronize()
    s_gpu = scores.cpu().numpy()
    honest = torch.nonzero(w.honest).flatten().tolist()
    faulty = torch.nonzero(~w.honest).flatten().tolist()
    rows = [honest[0], faulty[0], honest[-1]]
    s_orc, f_orc, n_orc = _sampled_score_check(oracle, w, rows)
    P.assert_scores_close(s_gpu[rows], s_orc)
    assert np.allclose(norms.cpu().numpy()[rows], n_orc, rtol=1e-5)
    assert abs(losses[0].item() - f_orc[0]) <= 1e-4 * abs(f_orc[0])
    assert np.array_equal(idx.cpu().numpy(), oracle.select(s_gpu.astype(np.float64), w.b))
    _column_block_check(oracle, w, idx.cpu().numpy(), out,
                        [(0, 4096), (16777216 - 1000, 16777216 + 5000), (w.d - 3000, w.d)])
    # identical sign-flip rows score bit-identically
    assert len({s_gpu[i] for i in faulty}) == 1


def test_config5_full_sampled(oracle):
    w = syn.make_config(5, device="cuda")
    assert (w.m, w.b, w.n_r, w.d) == (64, 24, 16, 1 << 26)
    with zeno.from_workload(w) as z:
        out, scores, idx = z.step(w.x, w.V, w.features, w.targets, w.gamma, w.rho, w.b)
        torch.cuda.synchronize()
    s_gpu = scores.cpu().numpy()
    honest = torch.nonzero(w.honest).flatten().tolist()
    faulty = torch.nonzero(~w.honest).flatten().tolist()
    rows = [honest[0], faulty[0], honest[-1]]
    s_orc, f_orc, n_orc = _sampled_score_check(oracle, w, rows)
    P.assert_scores_close(s_gpu[rows], s_orc)
    assert np.array_equal(idx.cpu().numpy(), oracle.select(s_gpu.astype(np.float64), w.b))
    # every noise row must have been trimmed here: its norm term alone is -6.7e7
    assert not set(idx.cpu().tolist()) & set(faulty)
    _column_block_check(oracle, w, idx.cpu().numpy(), out, [(0, 8192), ((1 << 25) - 4096, (1 << 25) + 4096),
                                                             (w.d - 8192, w.d)])
