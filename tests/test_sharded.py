"""The column-sliced Zeno step (least squares) for several GPUs.

CPU part (two gloo ranks): the host logic -- the slicing, the layout of the exchanged sums, the all-reduce and
the order of the calls -- with a stand-in for the four library calls that does what they are documented to do
in numpy, checked against the float64 oracle on the unsliced problem.  GPU part (marked gpu): the real
library with one rank, against the plain step and the oracle.
"""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_column_slices_cover_the_columns_exactly():
    from paper_1805_10032_b200 import sharded
    for d, world in [(1 << 26, 8), (70001, 2), (70001, 3), (31, 4), (0, 2), (4096, 1), (100, 7)]:
        sl = sharded.column_slices(d, world)
        assert len(sl) == world and sl[0][0] == 0 and sl[-1][1] == d
        for (a0, a1), (b0, b1) in zip(sl, sl[1:]):
            assert a1 == b0 and a0 <= a1
        assert all(lo % 32 == 0 for lo, hi in sl if hi > lo)
        sizes = [hi - lo for lo, hi in sl]
        assert all(s == sizes[0] or s < sizes[0] for s in sizes) and sizes[0] - d / world < 32 + 1


class _NumpyStandIn:
    """What the four library calls are documented to compute, in float64 numpy (test scaffolding)."""

    def __init__(self, d):
        self.d = d

    def score_partial(self, x, V, A):
        m, n_r = V.shape[0], A.shape[0]
        s = torch.zeros((m + 1, n_r + 1), dtype=torch.float64)
        Ad, xd, Vd = A.double(), x.double(), V[:, :self.d].double()
        s[0, :n_r] = Ad @ xd
        s[1:, :n_r] = Vd @ Ad.t()
        s[1:, n_r] = (Vd * Vd).sum(dim=1)
        return s

    def score_from_sums(self, sums, y, gamma, rho):
        n_r = sums.shape[1] - 1
        r0 = sums[0, :n_r] - y.double()
        f0 = (r0 ** 2).sum() / (2 * n_r)
        fi = ((r0[None, :] - float(np.float32(gamma)) * sums[1:, :n_r]) ** 2).sum(dim=1) / (2 * n_r)
        scores = f0 - fi - float(np.float32(rho)) * sums[1:, n_r]
        return scores, torch.cat([f0[None], fi]), sums[1:, n_r]

    def select(self, scores, b):
        key = torch.where(torch.isnan(scores), torch.full_like(scores, -float("inf")), scores)
        order = sorted(range(len(key)), key=lambda i: (-key[i].item(), i))
        return torch.tensor(order[:len(key) - b], dtype=torch.int32)

    def aggregate(self, V, idx):
        return V[idx.long(), :self.d].double().mean(dim=0)


def _rank(rank, world, port, q):
    sys.path.insert(0, ROOT)
    from paper_1805_10032_b200 import sharded
    from paper_1805_10032_b200 import synthetic as syn
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = syn.make_config(5, d=6000 + 17, m=13, b=5, n_r=16, n_noise=5)       # every rank generates the same inputs
    lo, hi = sharded.column_slices(w.d, world)[rank]
    x_s, V_s, A_s = w.x[lo:hi], w.V[:, lo:hi].contiguous(), w.features[:, lo:hi].contiguous()
    out_s, scores, idx = sharded.sharded_step(_NumpyStandIn(hi - lo), x_s, V_s, A_s, w.targets, w.gamma, w.rho, w.b)
    q.put((rank, lo, hi, out_s.numpy(), scores.numpy(), idx.numpy()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_on_cpu_agree_with_the_oracle_on_the_unsliced_problem(oracle):
    from paper_1805_10032_b200 import synthetic as syn
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() + 7) % 2000
    procs = [ctx.Process(target=_rank, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=180) for _ in procs), key=lambda t: t[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w = syn.make_config(5, d=6000 + 17, m=13, b=5, n_r=16, n_noise=5)
    out_orc, s_orc, idx_orc = oracle.step(1, 0, w.dims, w.has_bias, w.x.numpy(), w.V.numpy(), w.ldv, w.m,
                                          w.features.numpy(), w.targets.numpy(), float(np.float32(w.gamma)),
                                          float(np.float32(w.rho)), w.b)
    (r0, lo0, hi0, out0, s0, i0), (r1, lo1, hi1, out1, s1, i1) = res
    assert (lo0, hi1) == (0, w.d) and hi0 == lo1
    assert np.array_equal(s0, s1) and np.array_equal(i0, i1)         # every rank holds the same scores and ranking
    assert np.allclose(s0, s_orc, rtol=1e-9)
    assert np.array_equal(i0, idx_orc)
    assert np.allclose(np.concatenate([out0, out1]), out_orc, rtol=1e-12, atol=0)


@pytest.mark.gpu
def test_one_rank_on_the_gpu_matches_the_plain_step_and_the_oracle(oracle):
    from paper_1805_10032_b200 import build as zbuild
    from paper_1805_10032_b200 import sharded
    from paper_1805_10032_b200 import synthetic as syn
    from paper_1805_10032_b200 import zeno
    import parity as P
    zbuild.build()
    for ov in (dict(d=70000, m=13, b=5, n_r=16, n_noise=5), dict(d=4099, m=5, b=2, n_r=3, n_noise=2, ldv=4101)):
        w = syn.make_config(5, **ov)
        x, V, A, y = P.to_device(w)
        with zeno.from_workload(w) as z:
            out_s, scores, idx = sharded.sharded_step(z, x, V, A, y, w.gamma, w.rho, w.b)
            out, s_plain, i_plain = z.step(x, V, A, y, w.gamma, w.rho, w.b)
            torch.cuda.synchronize()
        s_orc, f_orc, n_orc = P.oracle_score(oracle, w)
        P.assert_scores_close(scores.cpu().numpy(), s_orc, f_orc, n_orc, float(np.float32(w.rho)))
        assert torch.equal(idx, i_plain) and torch.equal(out_s, out)
        # the sums are kept in double up to the scores here, in single there: equal to a few ulps of the terms
        assert np.allclose(scores.cpu().numpy(), s_plain.cpu().numpy(), rtol=1e-5, atol=1e-6)


@pytest.mark.gpu
def test_two_slices_on_one_gpu_add_up(oracle):
    """The exchange done by hand: two handles for the two column slices on one device, their sums added."""
    from paper_1805_10032_b200 import sharded
    from paper_1805_10032_b200 import synthetic as syn
    from paper_1805_10032_b200 import zeno
    import parity as P
    w = syn.make_config(5, d=70000 + 48, m=13, b=5, n_r=16, n_noise=5)
    (lo0, hi0), (lo1, hi1) = sharded.column_slices(w.d, 2)
    x, V, A, y = P.to_device(w)
    parts, outs = [], []
    handles = [zeno.Zeno(1, 0, (hi - lo, 1), m_max=w.m, n_r_max=w.n_r) for lo, hi in ((lo0, hi0), (lo1, hi1))]
    try:
        slices = [(x[lo:hi].contiguous(), V[:, lo:hi].contiguous(), A[:, lo:hi].contiguous())
                  for lo, hi in ((lo0, hi0), (lo1, hi1))]
        for z, (xs, Vs, As) in zip(handles, slices):
            parts.append(z.score_partial(xs, Vs, As))
        total = parts[0] + parts[1]
        scores, losses, norms = handles[0].score_from_sums(total, y, w.gamma, w.rho)
        idx = handles[0].select(scores, w.b)
        for z, (xs, Vs, As) in zip(handles, slices):
            outs.append(z.aggregate(Vs, idx))
        torch.cuda.synchronize()
    finally:
        for z in handles:
            z.close()
    s_orc, f_orc, n_orc = P.oracle_score(oracle, w)
    P.assert_scores_close(scores.cpu().numpy(), s_orc, f_orc, n_orc, float(np.float32(w.rho)))
    assert np.allclose(norms.cpu().numpy(), n_orc, rtol=1e-5)
    P.assert_selection_valid(idx.cpu().numpy(), s_orc, w.b)
    ref = oracle.aggregate(0, w.V.numpy(), w.ldv, w.d, w.m, idx.cpu().numpy())
    assert P.rel_l2(torch.cat(outs).cpu().numpy(), ref) <= P.AGG_RTOL
