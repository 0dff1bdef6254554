"""The give-up path of the bounded device-side waits.

Every wait a tensor-core kernel makes on one of its barriers polls a limited number of times.  The
limit is a launch argument; with zeno_debug_set_wait_limit(handle, 0) the first wait that is not
satisfied at its first probe gives up at once.  Nothing goes wrong on the device: the block raises
its abort flag, every role leaves its loop, the teardown waits (with the full limit) for the copies
and MMAs in flight, frees the tensor memory, and writes the status word the host reads.  The tests
check the whole chain: status code, a wait code that names a real barrier, a process that keeps
working, and a fresh handle that gives the right answer again.
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
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    zeno.load_library()


CASES = {
    # kernel id (bits 24-27 of the wait code), workload
    "first_layer_stream": (1, 2, dict(dims=(520, 200, 136, 10), n_r=21, m=6, b=2, faults=[(2, "noise200")])),
    "layer": (2, 4, dict(dims=(264, 136, 72, 50), m=9, b=3, n_r=19, faults=[(3, "signflip")])),
    "least_squares": (3, 5, dict(d=70000, m=13, b=5, n_r=16, n_noise=5)),
}


@pytest.mark.parametrize("name", sorted(CASES))
def test_a_wait_that_runs_out_is_reported_and_leaves_the_context_usable(oracle, name):
    kernel_id, index, ov = CASES[name]
    w = syn.make_config(index, **ov)
    x, V, f, t = P.to_device(w)
    z = zeno.from_workload(w)
    try:
        z.debug_set_wait_limit(0)
        z.step(x, V, f, t, w.gamma, w.rho, w.b)
        with pytest.raises(zeno.ZenoError) as e:
            z.check_device_status()
        assert e.value.status == zeno.ERR_TIMEOUT
        code = z.last_wait_code
        assert (code >> 24) & 0xf in (1, 2, 3)          # a tensor-core kernel of this step
        if name != "first_layer_stream":                # (that step also runs a layer kernel after the stream)
            assert (code >> 24) & 0xf == kernel_id
        assert 0 <= ((code >> 1) & 0xffff) < 64         # an index into that kernel's barrier array
        # the condition is sticky for the handle
        with pytest.raises(zeno.ZenoError):
            z.check_device_status()
    finally:
        z.close()
    # the process and the device are fine: a fresh handle computes the right step
    torch.cuda.synchronize()
    res = P.run_step_parity(oracle, w)
    assert res["launches"] >= 2


def test_default_limit_is_restored_by_a_new_handle():
    w = syn.make_config(5, d=70000, m=13, b=5, n_r=16, n_noise=5)
    x, V, f, t = P.to_device(w)
    with zeno.from_workload(w) as z:
        z.step(x, V, f, t, w.gamma, w.rho, w.b)
        z.check_device_status()                          # no wait gave up
        assert z.last_wait_code == 0
