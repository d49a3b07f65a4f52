"""Host-side pieces of the library that need no GPU: the per-device bookkeeping behind the kernels' one-time
set-up (compiled with the host compiler and run), and the argument checks of the newer entry points."""
import ctypes
import os
import subprocess
import tempfile

import pytest

import __graft_entry__ as entry
from paper_2604_08133_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_one_time_kernel_setup_is_kept_per_device():
    src = os.path.join(ROOT, "tests", "cpp", "device_once_test.cpp")
    inc = os.path.join(ROOT, "paper_2604_08133_b200", "csrc")
    with tempfile.TemporaryDirectory() as tmp:
        exe = os.path.join(tmp, "device_once_test")
        subprocess.run(["g++", "-std=c++17", "-O1", "-I", inc, src, "-o", exe], check=True)
        r = subprocess.run([exe], capture_output=True, text=True)
    assert r.returncode == 0 and r.stdout.strip().endswith("ok"), r.stdout + r.stderr


def test_no_kernel_source_keeps_a_process_wide_setup_flag():
    """The launchers remember their set-up per device (PerDeviceOnce), never in a single process-wide flag."""
    csrc = os.path.join(ROOT, "paper_2604_08133_b200", "csrc")
    for name in os.listdir(csrc):
        with open(os.path.join(csrc, name)) as f:
            text = f.read()
        assert "static bool attr_done" not in text and "static bool cattr_done" not in text, name
        if "cudaFuncAttributeMaxDynamicSharedMemorySize" in text:
            assert name == "common.cuh", name


@pytest.fixture(scope="module")
def lib():
    entry.build()
    return B.lib()


def test_routed_layer_call_checks_its_arguments_on_the_host(lib):
    s = B.make_shape(64, 256, 8, 512, 0, 2, 1)
    fake, odd = ctypes.c_void_p(4096), ctypes.c_void_p(4098)
    args = lambda x=fake, n=fake, bmax=100, hint=0, wsb=1 << 30: (
        ctypes.byref(s), x, fake, fake, n, bmax, hint, fake, fake, None, None, None, fake, fake, fake, wsb, None)
    assert lib.moe_layer_forward_routed(*args(bmax=129)) == B.MOE_ERR_BUDGET       # above K_orig*T
    assert lib.moe_layer_forward_routed(*args(bmax=-1)) == B.MOE_ERR_BUDGET
    assert lib.moe_layer_forward_routed(*args(hint=-5)) == B.MOE_ERR_BUDGET
    assert lib.moe_layer_forward_routed(*args(x=odd)) == B.MOE_ERR_ARG
    assert lib.moe_layer_forward_routed(*args(n=odd)) == B.MOE_ERR_ARG             # n_sel not on a 4-byte boundary
    assert lib.moe_layer_forward_routed(*args(wsb=64)) == B.MOE_ERR_WORKSPACE


def test_wait_selftest_and_grouped_ffn_check_their_arguments_on_the_host(lib):
    s = B.make_shape(64, 256, 8, 512, 0, 2, 1)
    fake = ctypes.c_void_p(4096)
    f = lib.moe_selftest_wait_timeout
    assert f(ctypes.byref(s), fake, 64, fake, fake, 10, fake, fake, 1 << 30, None) == B.MOE_ERR_ARG        # limit too small
    assert f(ctypes.byref(s), fake, 64, fake, fake, 1 << 40, fake, fake, 1 << 30, None) == B.MOE_ERR_ARG   # and too large
    assert f(ctypes.byref(s), fake, 0, fake, fake, 1 << 20, fake, fake, 1 << 30, None) == B.MOE_ERR_BUDGET
    assert f(ctypes.byref(s), fake, 64, fake, fake, 1 << 20, fake, fake, 64, None) == B.MOE_ERR_WORKSPACE
    g = lib.moe_grouped_ffn
    assert g(ctypes.byref(s), None, None, fake, 64, fake, fake, fake, fake, fake, 1 << 30, None) == B.MOE_ERR_ARG
    assert g(ctypes.byref(s), fake, None, fake, 129, fake, fake, fake, fake, fake, 1 << 30, None) == B.MOE_ERR_BUDGET
    assert g(ctypes.byref(s), fake, fake, fake, 64, fake, fake, fake, fake, fake, 64, None) == B.MOE_ERR_WORKSPACE
