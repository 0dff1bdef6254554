"""zeno_run, Algorithm 1's server loop on the device, against the oracle's step and update chained on
the host: T iterations, each with its own candidates and its own batch, x carried from one to the next."""
import numpy as np
import pytest
import torch

from paper_1805_10032_b200 import synthetic as syn
from paper_1805_10032_b200 import zeno

import parity as P

pytestmark = pytest.mark.gpu

T = 3


@pytest.fixture(scope="module", autouse=True)
def _library():
    from paper_1805_10032_b200 import build as zbuild
    zbuild.build()
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    zeno.load_library()


CASES = {
    "cfg1": (1, dict()),
    "cfg2_mid_layers": (2, dict(dims=(520, 200, 136, 10), n_r=21, m=6, b=2, faults=[(2, "noise200")])),
    "cfg4_small": (4, dict(dims=(264, 136, 72, 50), m=9, b=3, n_r=19, faults=[(3, "signflip")])),
    "cfg5_small": (5, dict(d=70000, m=13, b=5, n_r=16, n_noise=5)),
    "cfg6_cnn_small": (6, dict(dims=(8, 3, 8, 8, 12, 12, 10), m=7, b=2, n_r=5, faults=[(2, "signflip")])),
}


@pytest.mark.parametrize("name", sorted(CASES))
def test_server_loop_matches_the_chained_oracle(oracle, name):
    index, ov = CASES[name]
    ws = [syn.make_config(index, seed=syn.BASE_SEED + 31 * t + index, **ov) for t in range(T)]
    w = ws[0]
    V = torch.stack([s.V for s in ws]).cuda()
    feats = torch.stack([s.features for s in ws]).cuda()
    tgts = torch.stack([s.targets for s in ws]).cuda()
    x = w.x.cuda().clone()
    with zeno.from_workload(w) as z:
        scores, idx = z.run(x, V, feats, tgts, w.gamma, w.rho, w.b)
        launches = z.last_launch_count
        # the same loop, one call per iteration
        x2 = w.x.cuda().clone()
        for t in range(T):
            _, s2, i2 = z.step_update(x2, V[t], feats[t], tgts[t], w.gamma, w.rho, w.b, want_out=False)
            assert torch.equal(s2, scores[t]) and torch.equal(i2, idx[t])
        torch.cuda.synchronize()
        z.check_device_status()
    assert torch.equal(x, x2)
    assert launches >= 2 * T

    # the oracle's chain: the stored parameter vector is rounded to its storage type between iterations
    kind, dt = P.KIND[w.kind], P.DTYPE[w.dtype]
    gamma, rho = float(np.float32(w.gamma)), float(np.float32(w.rho))
    x_orc = syn.to_numpy_params(w.x)
    for t in range(T):
        Vt = syn.to_numpy_params(ws[t].V)
        f, tg = ws[t].features.numpy(), ws[t].targets.numpy()
        s_orc, f_orc, n_orc = oracle.score(kind, dt, w.dims, w.has_bias, x_orc, Vt, w.ldv, w.m, f, tg, gamma, rho)
        P.assert_scores_close(scores[t].cpu().numpy(), s_orc, f_orc, n_orc, rho)
        got_idx = idx[t].cpu().numpy()
        P.assert_selection_valid(got_idx, s_orc, w.b)
        vbar = oracle.aggregate(dt, Vt, w.ldv, w.d, w.m, got_idx)
        x_new = oracle.update(dt, x_orc, vbar, gamma)
        if w.dtype == "bf16":
            x_orc = syn.to_numpy_params(torch.from_numpy(x_new).to(torch.bfloat16))    # exact: already bfloat16 values
        else:
            x_orc = x_new.astype(np.float32)
    got = x.float().double().cpu().numpy()
    want = (torch.from_numpy(x_orc.view("int16")).view(torch.bfloat16).float().double().numpy()
            if w.dtype == "bf16" else x_orc.astype(np.float64))
    if w.dtype == "f32":
        assert P.rel_l2(got, want) <= T * 1e-6
    else:
        # a bfloat16 parameter may land on the neighbouring number at a rounding boundary, once per iteration
        ulp = np.maximum(np.abs(want), 2.0 ** -126) * 2.0 ** -7
        assert np.all(np.abs(got - want) <= T * ulp)
        assert np.mean(got == want) >= 0.99
    assert not torch.equal(x.cpu(), w.x)


def test_run_argument_errors():
    w = syn.make_config(1)
    x, V, f, t = P.to_device(w)
    V3 = torch.stack([V, V]).contiguous()
    f3, t3 = torch.stack([f, f]).contiguous(), torch.stack([t, t]).contiguous()
    with zeno.from_workload(w) as z:
        lib = zeno.load_library()
        st = lib.zeno_run(z._h, x.data_ptr(), V3.data_ptr(), w.ldv, w.m * w.ldv - 1, w.m, f3.data_ptr(),
                          t3.data_ptr(), w.n_r, 2, 0.1, 5e-4, w.b, None, None, None)
        assert st == zeno.ERR_INVALID_ARG                      # iterations would overlap
        st = lib.zeno_run(z._h, x.data_ptr(), V3.data_ptr(), w.ldv, w.m * w.ldv, w.m, f3.data_ptr(),
                          t3.data_ptr(), w.n_r, 0, 0.1, 5e-4, w.b, None, None, None)
        assert st == zeno.ERR_INVALID_ARG                      # no iterations
        scores, idx = z.run(x.clone(), V3, f3, t3, w.gamma, w.rho, w.b)
        assert scores.shape == (2, w.m) and idx.shape == (2, w.m - w.b)
