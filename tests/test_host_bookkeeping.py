"""Host-side logic of the library checked without a GPU: the per-device "attribute already set" table that the
kernels' launchers keep (cudaFuncSetAttribute acts on the current device only), compiled into a small host
program from the library's own header, and the convolutional model's parameter count through the C ABI."""
import os
import shutil
import subprocess
import textwrap

import pytest

from paper_1805_10032_b200 import build as zbuild
from paper_1805_10032_b200 import synthetic as syn
from paper_1805_10032_b200 import zeno

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

PROGRAM = textwrap.dedent("""
    #include <cstdio>
    #include "zeno_internal.h"
    int main() {
        zeno::PerDeviceOnce a, b;
        int bad = 0;
        for (int dev = 0; dev < zeno::kMaxDevices; ++dev) bad += !a.need(dev);        // nothing set yet
        a.mark(3);
        bad += a.need(3);                                                              // device 3 is done ...
        bad += !a.need(0) + !a.need(2) + !a.need(4) + !a.need(zeno::kMaxDevices - 1);  // ... and only device 3
        bad += !b.need(3);                                                             // one table per kernel
        a.mark(-1);
        a.mark(zeno::kMaxDevices);                                                     // out of the table: ignored,
        bad += !a.need(-1) + !a.need(zeno::kMaxDevices) + !a.need(1 << 20);            // and always set again
        bad += !a.need(0);
        a.mark(0);
        a.mark(zeno::kMaxDevices - 1);
        bad += a.need(0) + a.need(zeno::kMaxDevices - 1) + a.need(3);
        std::printf("%d\\n", bad);
        return bad;
    }
""")


def test_per_device_attribute_table(tmp_path):
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        pytest.skip("no nvcc")
    src = tmp_path / "once.cu"
    src.write_text(PROGRAM)
    exe = tmp_path / "once"
    subprocess.run([nvcc, "-std=c++17", "-I", os.path.join(ROOT, "paper_1805_10032_b200", "csrc"),
                    "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0 and out.stdout.strip() == "0", out.stdout + out.stderr


def test_cnn_param_count_through_the_abi():
    zbuild.build()
    zeno.load_library()
    for dims in [(32, 3, 32, 32, 64, 64, 10), (8, 2, 5, 7, 4), (24, 1, 4, 4, 6, 6, 8, 8, 5)]:
        desc = zeno.make_desc(zeno.LOSS_SOFTMAX_CNN, zeno.F32, dims, True)
        assert zeno.param_count(desc) == syn.param_count("cnn", dims)
        desc = zeno.make_desc(zeno.LOSS_SOFTMAX_CNN, zeno.F32, dims, False)
        assert zeno.param_count(desc) == syn.param_count("cnn", dims, False)
    for dims in [(16, 3, 8, 10), (34, 3, 8, 8, 10), (6, 3, 8, 8, 8, 8, 10), (15, 3, 8, 8, 10)]:
        assert zeno.param_count(zeno.make_desc(zeno.LOSS_SOFTMAX_CNN, zeno.F32, dims, True)) == 0
