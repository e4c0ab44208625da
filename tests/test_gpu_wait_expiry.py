"""A bounded device-side wait that runs out: the kernel must return (no trap, no hang), the host must read the code,
and a later launch must wait normally although the report has not been read yet.

The kernel is a test-only build around the library's own wait routine (tests/native/wait_probe.cu; it is not part of
liblte.so): its barrier is never armed, so the wait gives up after a few thousand polls.  Nothing faults."""
import ctypes
import os
import subprocess

import pytest

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
SRC = os.path.join(HERE, "native", "wait_probe.cu")
LIB = os.path.join(HERE, "native", "libwait_probe.so")
CSRC = os.path.join(ROOT, "paper_2510_20787_b200", "csrc")


def _build():
    deps = [SRC, os.path.join(CSRC, "tc_common.cuh"), os.path.join(CSRC, "common.cuh")]
    if os.path.exists(LIB) and all(os.path.getmtime(LIB) >= os.path.getmtime(d) for d in deps):
        return LIB
    tmp = LIB + ".tmp.%d" % os.getpid()
    subprocess.check_call([os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc"), "-gencode", "arch=compute_100a,code=sm_100a",
                           "-O2", "-std=c++17", "-shared", "-Xcompiler", "-fPIC", "-I", CSRC, "-I", os.path.join(ROOT, "include"),
                           "-o", tmp, SRC, "-lcudart"])
    os.replace(tmp, LIB)
    return LIB


def test_a_wait_that_runs_out_is_reported_and_does_not_poison_the_next_launch():
    lib = ctypes.CDLL(_build())
    out = (ctypes.c_longlong * 3)()
    assert lib.wait_probe_status() == 0
    # nothing arrives: the first wait gives up (code 77); the launch's second wait then stops early on the abort mark
    assert lib.wait_probe_run(0, out) == 0, "the kernel must return normally"
    assert out[2] == 1
    first, second = out[0], out[1]
    assert second < first, (first, second)                       # about 1024 polls against 4096
    # the report is still unread; a new launch whose barrier is armed waits normally and records nothing new
    assert lib.wait_probe_run(1, out) == 0
    assert out[2] == 1 and out[0] < first
    # another lost wait in a new launch, report still unread: it must run to its own limit again (not be cut short at
    # 1024 polls by the mark of the earlier launch)
    assert lib.wait_probe_run(0, out) == 0
    assert out[0] > 2 * out[1], (out[0], out[1])
    assert lib.wait_probe_status() == 77                          # the code of a wait that gave up; reading clears it
    assert lib.wait_probe_status() == 0
