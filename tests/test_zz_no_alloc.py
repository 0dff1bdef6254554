"""zeno_score_lsq_static: the least-squares scores for callers that are not allowed to allocate.

Some users of the library sit in places where cudaMalloc is off limits when a score is needed:
a serving loop that must not touch the CUDA allocator after start-up (an allocation synchronises
the device and stalls every other stream), or a process whose framework has already taken all of
the device memory into its own pool.  The handle-based calls allocate a workspace in zeno_create;
this entry point instead keeps its scratch in a fixed array inside the library, takes every buffer
from the caller, and must give the same numbers as zeno_score.

This file is named so that pytest collects it last.  The entry point is checked on two calls in
a row (the scratch array keeps the previous call's contents, and the second call uses different
data and a different shape), against the handle-based path, through the C ABI.
"""
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
    assert torch.cuda.is_available(), "this test needs a CUDA device"
    zeno.load_library()


def _reference(w):
    x, V, A, y = P.to_device(w)
    with zeno.from_workload(w) as z:
        s, losses, norms = z.score(x, V, A, y, w.gamma, w.rho)
        torch.cuda.synchronize()
    return s.cpu().numpy(), losses.cpu().numpy(), norms.cpu().numpy()


def _static(w, with_optional, check_memory=False):
    x, V, A, y = P.to_device(w)
    # every buffer comes from the caller; the call itself allocates nothing
    scores = torch.full((w.m,), float("nan"), dtype=torch.float32, device="cuda")
    losses = torch.full((w.m + 1,), float("nan"), dtype=torch.float32, device="cuda") if with_optional else None
    norms = torch.full((w.m,), float("nan"), dtype=torch.float32, device="cuda") if with_optional else None
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    zeno.score_lsq_static(x, V, A, y, w.gamma, w.rho, scores, losses, norms, ldv=w.ldv)
    torch.cuda.synchronize()
    if check_memory:
        # not the first call in this process: the device's free memory is what it was before the call
        assert torch.cuda.mem_get_info()[0] == free_before
    return (scores.cpu().numpy(), None if losses is None else losses.cpu().numpy(),
            None if norms is None else norms.cpu().numpy())


def test_two_calls_in_a_row_match_the_handle_based_scores(oracle):
    first = syn.make_config(5, d=70000, m=13, b=5, n_r=16, n_noise=5)
    second = syn.make_config(5, d=33333 * 4, m=40, b=12, n_r=5, n_noise=12, seed=77)
    for call, (w, with_optional) in enumerate(((first, True), (second, False))):
        want_s, want_f, want_n = _reference(w)
        got_s, got_f, got_n = _static(w, with_optional, check_memory=call > 0)
        assert np.all(np.abs(got_s - want_s) <= P.SCORE_RTOL * np.abs(want_s))
        if with_optional:
            assert np.allclose(got_f, want_f, rtol=1e-5, atol=1e-7)
            assert np.allclose(got_n, want_n, rtol=1e-5)
        # and both agree with the float64 oracle
        s_orc, _, _ = P.oracle_score(oracle, w)
        P.assert_scores_close(got_s, s_orc)


@pytest.mark.parametrize("shape", [
    dict(d=4099, m=5, b=2, n_r=3, n_noise=2, ldv=4101),          # rows that are not 16-byte aligned: scalar loads
    dict(d=50000, m=64, b=20, n_r=24, n_noise=20),               # 17..32 samples, every candidate slot in use
    dict(d=20004, m=7, b=2, n_r=32, n_noise=2, gamma=0.1),       # the largest sample count the scratch holds
])
def test_other_kernel_instantiations(oracle, shape):
    w = syn.make_config(5, **shape)
    _static(w, False)                                            # whatever ran before, this is not the first call
    got_s, got_f, got_n = _static(w, True, check_memory=True)
    s_orc, f_orc, n_orc = P.oracle_score(oracle, w)
    P.assert_scores_close(got_s, s_orc, f_orc, n_orc, float(np.float32(w.rho)))
    assert np.allclose(got_n, n_orc, rtol=1e-5)


def test_sizes_beyond_the_fixed_scratch_are_refused():
    w = syn.make_config(5, d=4096, m=zeno.STATIC_MAX_M + 1, b=3, n_r=4, n_noise=3)
    x, V, A, y = P.to_device(w)
    scores = torch.empty(w.m, dtype=torch.float32, device="cuda")
    with pytest.raises(zeno.ZenoError) as e:
        zeno.score_lsq_static(x, V, A, y, w.gamma, w.rho, scores)
    assert e.value.status == zeno.ERR_WORKSPACE
    w2 = syn.make_config(5, d=4096, m=4, b=1, n_r=zeno.STATIC_MAX_N_R + 1, n_noise=1)
    x, V, A, y = P.to_device(w2)
    with pytest.raises(zeno.ZenoError) as e:
        zeno.score_lsq_static(x, V, A, y, w2.gamma, w2.rho, torch.empty(4, dtype=torch.float32, device="cuda"))
    assert e.value.status == zeno.ERR_WORKSPACE
