"""GPU parity of zeno_step_update (Zeno_b followed by Algorithm 1's server update x <- x - gamma v)
against the float64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from paper_1805_10032_b200 import synthetic as syn
from paper_1805_10032_b200 import zeno

import parity as P

pytestmark = pytest.mark.gpu

UPDATE_RTOL = 1e-6      # binary32 x: one fused multiply-add on a mean that is within 1e-5 of the oracle's


@pytest.fixture(scope="module", autouse=True)
def _library():
    from paper_1805_10032_b200 import build as zbuild
    zbuild.build()
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    zeno.load_library()


CASES = {
    "cfg1": (1, dict()),
    "cfg2_mid_layers": (2, dict(dims=(520, 200, 136, 10), n_r=21, m=6, b=2, faults=[(2, "noise200")])),
    "cfg2_unaligned": (2, dict(dims=(301, 37, 10), n_r=9, m=7, b=3, faults=[(3, "noise200")])),
    "cfg4_small": (4, dict(dims=(264, 136, 72, 50), m=9, b=3, n_r=19, faults=[(3, "signflip")])),
    "cfg5_small": (5, dict(d=70000, m=13, b=5, n_r=16, n_noise=5)),
}


@pytest.mark.parametrize("name", sorted(CASES))
def test_step_update_matches_oracle(oracle, name):
    index, ov = CASES[name]
    w = syn.make_config(index, **ov)
    o = P.oracle_inputs(w)
    x, V, feats, tgt = P.to_device(w)
    x_new = x.clone()
    with zeno.from_workload(w) as z:
        out_ref, scores_ref, idx_ref = z.step(x, V, feats, tgt, w.gamma, w.rho, w.b)
        out, scores, idx = z.step_update(x_new, V, feats, tgt, w.gamma, w.rho, w.b)
        # the average is optional: the update alone must give the same parameters
        x_only = x.clone()
        none_out, _, _ = z.step_update(x_only, V, feats, tgt, w.gamma, w.rho, w.b, want_out=False)
        torch.cuda.synchronize()
    assert none_out is None
    # everything but x is what zeno_step gives, bit for bit
    assert torch.equal(out, out_ref) and torch.equal(idx, idx_ref)
    assert np.array_equal(scores.cpu().numpy(), scores_ref.cpu().numpy(), equal_nan=True)
    assert torch.equal(x_only, x_new)
    # x against the oracle's update of the oracle's average over the GPU's (already validated) set
    vbar = oracle.aggregate(o["dtype"], o["V"], w.ldv, w.d, w.m, idx.cpu().numpy())
    want = oracle.update(o["dtype"], o["x"], vbar, float(np.float32(w.gamma)))
    got = x_new.double().cpu().numpy() if w.dtype == "f32" else x_new.float().double().cpu().numpy()
    if w.dtype == "f32":
        assert P.rel_l2(got, want) <= UPDATE_RTOL
        # element by element: the step gamma * vbar is small against x, so an absolute bound in units of x
        assert np.max(np.abs(got - want)) <= 4e-7 * max(1.0, np.max(np.abs(want)))
    else:
        # a bfloat16 parameter: the same bfloat16 number, except where the binary32 mean falls on the
        # other side of a rounding boundary -- then the neighbouring one
        diff = np.abs(got - want)
        ulp = np.maximum(np.abs(want), 2.0 ** -126) * 2.0 ** -7
        assert np.all(diff <= ulp), "more than one bfloat16 spacing away"
        assert np.mean(diff == 0) >= 0.999
    assert not torch.equal(x_new, x), "the update changed nothing"


def test_step_update_rejects_missing_x():
    w = syn.make_config(1)
    x, V, feats, tgt = P.to_device(w)
    with zeno.from_workload(w) as z:
        lib = zeno.load_library()
        import ctypes
        bt = z._batch(feats, tgt)
        st = lib.zeno_step_update(z._h, None, V.data_ptr(), w.ldv, w.m, ctypes.byref(bt), 0.1, 5e-4, w.b,
                                  None, None, None, None)
        assert st == zeno.ERR_INVALID_ARG
