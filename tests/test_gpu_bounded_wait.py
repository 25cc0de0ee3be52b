"""The bounded mbarrier wait of the tensor-core kernels gives up instead of hanging.

Every wait in the loss kernels is `mbar_wait` from csrc/nat_tc.cuh: it polls, and after its
time limit (or once another role of the block has raised the abort flag) it returns false,
upon which the kernel winds down and reports NAT_DEV_TIMEOUT.  In a healthy run no wait
ever runs out, so this test builds a one-block probe from that same header in which a wait
cannot succeed -- an mbarrier nobody arrives at, nothing in flight -- and checks that the
kernel returns by itself with the flag raised.  Nothing here faults or hangs the GPU.
"""
import ctypes
import os
import shutil
import subprocess

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_wait_on_a_barrier_nobody_signals_returns_with_the_abort_flag(tmp_path):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    if not (os.path.exists(nvcc) or shutil.which(nvcc)):
        pytest.skip("nvcc is not available to build the probe")
    so = tmp_path / "bounded_wait_probe.so"
    cmd = [nvcc, "-std=c++17", "-O2", "-gencode", "arch=compute_100a,code=sm_100a", "-Xcompiler",
           "-fPIC", "-shared", "-I", os.path.join(ROOT, "paper_2603_06619_b200", "csrc"),
           "-o", str(so), os.path.join(ROOT, "tests", "probes", "bounded_wait_probe.cu")]
    r = subprocess.run(cmd, capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    lib = ctypes.CDLL(str(so))
    out = (ctypes.c_uint32 * 6)()
    assert lib.bounded_wait_probe(out) == 0
    gave_up, waited_us, saw_flag, waited2_us, signalled_ok, flag = list(out)
    assert gave_up == 0                       # the 2 ms wait ran out ...
    assert 1900 <= waited_us < 200000         # ... after its limit, not before and not much later
    assert saw_flag == 0 and waited2_us < 1000000   # the 2 s wait left early on the flag
    assert signalled_ok == 1                  # a barrier that is signalled completes
    assert flag == 1                          # and the block's abort flag is raised
