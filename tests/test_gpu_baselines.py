"""GPU parity of the baseline aggregation rules (Experiments, "Baselines": marginal Median, Krum_b) against
the float64 oracle, through the C ABI, on the same seeded candidate matrices the Zeno tests use."""
import numpy as np
import pytest
import torch

from paper_1805_10032_b200 import synthetic as syn
from paper_1805_10032_b200 import zeno

import parity as P

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _library():
    from paper_1805_10032_b200 import build as zbuild
    zbuild.build()
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    zeno.load_library()


CASES = {
    "cfg1": (1, dict()),                                                       # m = 20: one lane a column
    "cfg2_small_odd_m": (2, dict(dims=(300, 72, 40, 10), n_r=9, m=7, b=2, faults=[(2, "noise200")])),
    "cfg3_m37": (3, dict(dims=(260, 44, 36, 10), m=37, b=15, n_r=7, faults=[(7, "signflip"), (8, "omniscient")])),  # two lanes a column
    "cfg3_m100": (3, dict(dims=(132, 40, 10), m=100, b=40, n_r=5, faults=[(20, "signflip"), (20, "omniscient")])),  # four lanes a column
    "cfg4_bf16": (4, dict(dims=(264, 136, 72, 50), m=9, b=3, n_r=19, faults=[(3, "signflip")])),
    "cfg5_small": (5, dict(d=70001, m=13, b=5, n_r=16, n_noise=5, ldv=70003)),   # unaligned rows
}


# every compiled variant of the sorting network (columns of 8 .. 32 slots in one lane, then 2 .. 32 lanes a
# column) at, below and above its limits, in both storage types; d leaves a ragged last group of columns
MEDIAN_M = [1, 2, 3, 4, 7, 8, 9, 12, 13, 16, 17, 20, 21, 24, 25, 28, 29, 31, 32, 33, 63, 64, 65, 127, 128, 129, 255,
            256, 257, 500, 512, 513, 1000, 1024]


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_median_every_network(oracle, dtype):
    for m in MEDIAN_M:
        if dtype == "fp32":
            w = syn.make_config(5, d=301, m=m, b=0, n_r=4, n_noise=0, ldv=307, seed=1000 + m)
            dt = 0
        else:
            w = syn.make_config(4, dims=(10, 13, 10), m=m, b=0, n_r=4, faults=[], seed=1000 + m)
            dt = 1
        if m >= 5:                                  # ties and special values in some columns
            w.V[1, 0] = w.V[0, 0]
            w.V[m - 1, 1] = float("inf")
            w.V[m // 2, 2] = float("-inf")
            w.V[2, 3] = float("nan")
        want = oracle.median(dt, syn.to_numpy_params(w.V), w.ldv, w.d, w.m)
        with zeno.from_workload(w) as z:
            got = z.median(w.V.cuda()).cpu().numpy().astype(np.float64)
        fin = np.isfinite(want)
        assert np.array_equal(got[~fin], want[~fin]), m
        if m % 2 == 1:
            assert np.array_equal(got, want), (m, np.flatnonzero(got != want)[:5])     # a selection, exactly
        else:                                       # the mean of two stored values formed in binary32: one rounding
            assert np.all(np.abs(got[fin] - want[fin]) <= 1.2e-7 * np.maximum(np.abs(want[fin]), 1e-30) + 1e-45), m


@pytest.mark.parametrize("name", sorted(CASES))
def test_median_matches_oracle(oracle, name):
    index, ov = CASES[name]
    w = syn.make_config(index, **ov)
    dt = P.DTYPE[w.dtype]
    want = oracle.median(dt, syn.to_numpy_params(w.V), w.ldv, w.d, w.m)
    with zeno.from_workload(w) as z:
        got = z.median(w.V.cuda()).cpu().numpy().astype(np.float64)
    if w.m % 2 == 1:
        assert np.array_equal(got, want)            # a selection: the value of one input entry, exactly
    else:
        # the mean of two stored values, formed in binary32: one rounding
        assert np.all(np.abs(got - want) <= 1.2e-7 * np.maximum(np.abs(want), 1e-30) + 1e-45)
    assert P.rel_l2(got, want) <= 1e-6


def test_median_special_values(oracle):
    w = syn.make_config(1, dims=(64, 12), m=5, b=1, faults=[(1, "signflip")])
    w.V[0, 3] = float("nan")
    w.V[1, 3] = float("nan")
    w.V[2, 3] = float("nan")                        # three of five are NaN: the median is +inf
    w.V[4, 7] = float("inf")
    w.V[3, 9] = -float("inf")
    want = oracle.median(0, syn.to_numpy_params(w.V), w.ldv, w.d, w.m)
    with zeno.from_workload(w) as z:
        got = z.median(w.V.cuda()).cpu().numpy().astype(np.float64)
    assert np.array_equal(got, want) and got[3] == np.inf


@pytest.mark.parametrize("name", sorted(CASES))
def test_krum_matches_oracle(oracle, name):
    index, ov = CASES[name]
    w = syn.make_config(index, **ov)
    dt = P.DTYPE[w.dtype]
    b = min(w.b, w.m - 3)
    k_orc, sums_orc, _ = oracle.krum(dt, syn.to_numpy_params(w.V), w.ldv, w.d, w.m, b)
    with zeno.from_workload(w) as z:
        out, k, sums = z.krum(w.V.cuda(), b)
        torch.cuda.synchronize()
    sums = sums.cpu().numpy().astype(np.float64)
    k = int(k.item())
    assert np.allclose(sums, sums_orc, rtol=2e-5, atol=0)
    # the arg min decides an integer: identical wherever the oracle's best two sums are clearly apart,
    # otherwise any candidate whose sum is the minimum up to the tolerance (identical rows tie exactly)
    order = np.argsort(sums_orc, kind="stable")
    if sums_orc[order[1]] - sums_orc[order[0]] > 1e-4 * abs(sums_orc[order[0]]):
        assert k == k_orc
    else:
        assert sums_orc[k] <= sums_orc[order[0]] * (1 + 1e-4)
    assert k == int(np.argmin(sums))                # on its own sums the choice is exact, lowest index first
    assert torch.equal(out.cpu(), w.V[k, :w.d].float())


def test_krum_toy_example_on_the_gpu():
    # Discussion, the one-dimensional toy example: Krum_2({-1, -1, 0.2, 0.4, 1.6, 1.8}) = -1
    V = torch.tensor([[-1.0], [-1.0], [0.2], [0.4], [1.6], [1.8]])
    with zeno.Zeno(1, 0, (1, 1), m_max=6, n_r_max=1) as z:
        out, k, sums = z.krum(V.cuda(), 2)
    assert out.item() == -1.0 and k.item() == 0
    assert sums[0].item() == pytest.approx(1.44, rel=1e-6)


def test_krum_argument_errors_and_limits():
    w = syn.make_config(1, dims=(64, 12), m=6, b=2, faults=[(2, "signflip")])
    V = w.V.cuda()
    with zeno.from_workload(w) as z:
        with pytest.raises(zeno.ZenoError) as e:
            z.krum(V, 4)                            # m - b - 2 = 0 neighbours
        assert e.value.status == zeno.ERR_INVALID_ARG
        with pytest.raises(zeno.ZenoError) as e:
            z.krum(V, -1)
        assert e.value.status == zeno.ERR_INVALID_ARG
    w2 = syn.make_config(1, dims=(16, 4), m=130, b=8, faults=[(8, "signflip")])
    with zeno.from_workload(w2) as z:
        with pytest.raises(zeno.ZenoError) as e:
            z.krum(w2.V.cuda(), 8)
        assert e.value.status == zeno.ERR_UNSUPPORTED
        assert torch.isfinite(z.median(w2.V.cuda())).all()      # the median has no such limit
