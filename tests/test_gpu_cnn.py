"""GPU parity of the convolutional loss (ZENO_LOSS_SOFTMAX_CNN: the model family of the paper's own
experiment, a CNN of four convolutional layers and a dense one) against the float64 oracle, through the
C ABI: whole steps (score, ranking, trimmed mean), the pieces, shapes that leave ragged blocks (planes that
do not fill a block, channel counts that are no multiples of the block's sixteen planes or of the eight
staged at a time, a last group of samples that is not full), both storage types."""
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
    # the experiment's shape at a size the oracle finishes in seconds
    "paper_shape_small": dict(dims=(32, 3, 32, 32, 64, 64, 10), m=6, b=2, n_r=3, faults=[(2, "signflip")]),
    "two_layers": dict(dims=(8, 2, 5, 7, 4), m=7, b=3, n_r=5, faults=[(3, "noise200")]),
    "odd_channels_16x16": dict(dims=(16, 3, 9, 17, 20, 33, 10), m=5, b=2, n_r=6, faults=[(2, "signflip")]),
    "side_12_six_layers": dict(dims=(24, 1, 4, 4, 6, 6, 8, 8, 5), m=4, b=1, n_r=9, faults=[(1, "omniscient")]),
    "many_samples": dict(dims=(8, 3, 8, 8, 12, 12, 10), m=9, b=3, n_r=37, faults=[(3, "signflip")]),
    "no_bias": dict(dims=(16, 3, 8, 8, 10), m=5, b=1, n_r=4, faults=[(1, "signflip")], has_bias=False),
    "bf16": dict(dims=(16, 3, 16, 16, 24, 24, 10), m=6, b=2, n_r=5, faults=[(2, "signflip")], dtype="bf16"),
    "wide_head": dict(dims=(8, 3, 8, 8, 40), m=5, b=2, n_r=4, faults=[(2, "signflip")]),     # 40 classes: separate loss kernel
}


@pytest.mark.parametrize("name", sorted(CASES))
def test_step_matches_oracle(oracle, name):
    w = syn.make_config(6, **CASES[name])
    r = P.run_step_parity(oracle, w)
    assert r["agg_err"] <= P.AGG_RTOL


def test_kernels_of_the_step():
    w = syn.make_config(6, dims=(16, 3, 8, 8, 12, 12, 10), m=5, b=2, n_r=4, faults=[(2, "signflip")])
    x, V, f, t = P.to_device(w)
    with zeno.from_workload(w) as z:
        z.profile(True)
        z.step(x, V, f, t, w.gamma, w.rho, w.b)
        names = [n for n, _ in z.profile_read(0)]
        z.profile(False)
    assert names == ["cnn_conv3x3"] * 4 + ["mlp_head_loss_tail", "aggregate"], names


def test_description_errors():
    ok = (16, 3, 8, 8, 10)
    for dims in [(16, 3, 8, 10),              # an odd number of convolutional layers
                 (34, 3, 8, 8, 10),           # planes larger than 32 x 32
                 (6, 3, 8, 8, 8, 8, 10),      # 6 -> 3: odd before the second pooling
                 (15, 3, 8, 8, 10)]:          # an odd side
        with pytest.raises(zeno.ZenoError) as e:
            zeno.Zeno(zeno.LOSS_SOFTMAX_CNN, zeno.F32, dims, True, 4, 4)
        assert e.value.status == zeno.ERR_INVALID_ARG, dims
    z = zeno.Zeno(zeno.LOSS_SOFTMAX_CNN, zeno.F32, ok, True, 4, 4)
    assert z.d == syn.param_count("cnn", ok)
    z.close()


def test_nan_pixel_and_nan_candidate(oracle):
    w = syn.make_config(6, dims=(8, 2, 4, 4, 5), m=5, b=2, n_r=3, faults=[(2, "signflip")])
    w.V[1, 7] = float("nan")                         # a candidate with a NaN entry ranks last
    s_orc, f_orc, n_orc = P.oracle_score(oracle, w)
    x, V, f, t = P.to_device(w)
    with zeno.from_workload(w) as z:
        out, scores, idx = z.step(x, V, f, t, w.gamma, w.rho, w.b)
    s = scores.cpu().numpy()
    assert np.isnan(s[1]) and np.isnan(s_orc[1])
    assert 1 not in idx.cpu().tolist()
    ok = ~np.isnan(s_orc)
    assert np.allclose(s[ok], s_orc[ok], rtol=1e-3, atol=1e-6)


def test_host_buffers(oracle):
    """zeno_step_host with the convolutional model: the batch is [n_r][C_0][S][S] values per step."""
    w = syn.make_config(6, dims=(8, 3, 8, 8, 10), m=5, b=2, n_r=3, faults=[(2, "signflip")])
    out = torch.empty(w.d, dtype=torch.float32).pin_memory()
    scores = torch.empty(w.m, dtype=torch.float32).pin_memory()
    idx = torch.empty(w.m - w.b, dtype=torch.int32).pin_memory()
    with zeno.from_workload(w) as z:
        z.step_host(w.x.pin_memory(), w.V.pin_memory(), w.features.contiguous().pin_memory(), w.targets.pin_memory(),
                    w.gamma, w.rho, w.b, out, scores=scores, idx=idx)
        x, V, f, t = P.to_device(w)
        out_d, scores_d, idx_d = z.step(x, V, f, t, w.gamma, w.rho, w.b)
    assert torch.equal(out, out_d.cpu()) and torch.equal(scores, scores_d.cpu()) and torch.equal(idx, idx_d.cpu())
