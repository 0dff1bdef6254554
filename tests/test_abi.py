"""The C-ABI library: it loads without a GPU, exports every symbol include/zeno.h declares, and
its host-side argument checks answer with status codes (no compute call is made here)."""
import ctypes
import os
import re

import pytest

from paper_1805_10032_b200 import build as zbuild
from paper_1805_10032_b200 import zeno

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    zbuild.build()
    return zeno.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "zeno.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(zeno_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert set(names) == set(zeno.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_status_strings(lib):
    seen = {zeno.status_string(s) for s in range(6)}
    assert len(seen) == 6 and "ok" in seen
    assert zeno.status_string(99) == "unknown status"


def test_param_count_on_host(lib):
    assert zeno.param_count(zeno.make_desc(0, 0, (784, 10))) == 7850
    assert zeno.param_count(zeno.make_desc(0, 0, (3072, 512, 512, 10))) == 1841162
    assert zeno.param_count(zeno.make_desc(0, 1, (4096, 4096, 4096, 1000))) == 37659624
    assert zeno.param_count(zeno.make_desc(1, 0, (1 << 26, 1), False)) == 1 << 26
    assert zeno.param_count(zeno.make_desc(0, 0, (5, 3), False)) == 15
    assert zeno.param_count(zeno.make_desc(0, 0, (5, 0))) == 0          # invalid layer width
    assert zeno.param_count(zeno.make_desc(7, 0, (5, 3))) == 0          # unknown loss


def test_create_rejects_bad_arguments_before_touching_cuda(lib):
    h = ctypes.c_void_p()
    good = zeno.make_desc(0, 0, (8, 4))
    cases = [
        (None, 4, 4, zeno.ERR_INVALID_ARG),
        (zeno.make_desc(5, 0, (8, 4)), 4, 4, zeno.ERR_UNSUPPORTED),
        (zeno.make_desc(0, 3, (8, 4)), 4, 4, zeno.ERR_UNSUPPORTED),
        (zeno.make_desc(1, 1, (8, 1), False), 4, 4, zeno.ERR_UNSUPPORTED),   # bf16 least squares
        (zeno.make_desc(0, 0, (8, -1)), 4, 4, zeno.ERR_INVALID_ARG),
        (good, 0, 4, zeno.ERR_INVALID_ARG),
        (good, zeno.MAX_CANDIDATES + 1, 4, zeno.ERR_INVALID_ARG),
        (good, 4, 0, zeno.ERR_INVALID_ARG),
    ]
    for desc, m_max, n_r_max, want in cases:
        st = lib.zeno_create(ctypes.byref(h), ctypes.byref(desc) if desc is not None else None,
                             m_max, n_r_max, 0)
        assert st == want and not h.value
    assert lib.zeno_create(None, ctypes.byref(good), 4, 4, 0) == zeno.ERR_INVALID_ARG


def test_null_handle_calls_return_invalid_arg(lib):
    assert lib.zeno_destroy(None) == zeno.ERR_INVALID_ARG
    assert lib.zeno_select(None, None, 4, 1, None, None) == zeno.ERR_INVALID_ARG
    assert lib.zeno_aggregate(None, None, 4, 4, None, 1, None, None) == zeno.ERR_INVALID_ARG
    assert lib.zeno_last_launch_count(None) == 0


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(zeno, "_lib", None)
    monkeypatch.setattr(zeno, "LIB_PATH", str(tmp_path / "libzeno.so"))
    with pytest.raises(FileNotFoundError):
        zeno.load_library()
