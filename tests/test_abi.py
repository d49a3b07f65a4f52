"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares;
host-side argument checks answer before anything would be launched."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2604_08133_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    entry.build()
    return B.lib()


def _declared():
    with open(os.path.join(ROOT, "include", "allocmoe.h")) as f:
        src = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    return sorted(set(re.findall(r"\b(moe_[a-z_0-9]+|alloc_t_select|alloc_l_solve)\s*\(", src)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert {"moe_gate", "alloc_t_select", "moe_permute", "moe_grouped_ffn", "moe_combine",
            "moe_layer_forward"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(B.EXPORTS)


def test_status_strings(lib):
    seen = {B.status_string(i) for i in range(7)}
    assert len(seen) == 7 and "ok" in seen


def test_workspace_bytes_is_host_only_and_monotone(lib):
    s = B.make_shape(4096, 2048, 64, 1408, 2, 6, 1)
    a = B.moe_workspace_bytes(s, 2 * 4096)
    b = B.moe_workspace_bytes(s, 6 * 4096)
    assert 0 < a < b
    # x_perm + h + y_perm dominate: budget * (2H + I) * 2 bytes
    assert b >= 6 * 4096 * (2 * 2048 + 1408) * 2
    assert B.moe_workspace_bytes(s, 6 * 4096 + 1) == 0            # beyond K_orig*T
    for bad in (B.make_shape(64, 100, 64, 1408, 0, 6, 1), B.make_shape(64, 2048, 62, 1408, 0, 6, 1),
                B.make_shape(64, 2048, 64, 1408, 0, 6, 7), B.make_shape(0, 2048, 64, 1408, 0, 6, 1),
                B.make_shape(64, 2048, 8, 1408, 0, 9, 1)):
        assert B.moe_workspace_bytes(bad, 64) == 0


def test_host_checks_answer_without_a_device(lib):
    s = B.make_shape(64, 256, 8, 512, 0, 2, 1)
    fake = ctypes.c_void_p(4096)          # aligned, never dereferenced: the checks come first
    odd = ctypes.c_void_p(4100)
    r = lib.moe_layer_forward(ctypes.byref(s), fake, fake, None, fake, fake, None, None, 63, None, fake, fake, fake,
                              1 << 30, None)
    assert r == B.MOE_ERR_BUDGET
    r = lib.moe_layer_forward(ctypes.byref(s), odd, fake, None, fake, fake, None, None, 64, None, fake, fake, fake,
                              1 << 30, None)
    assert r == B.MOE_ERR_ARG
    r = lib.moe_layer_forward(ctypes.byref(s), fake, fake, None, fake, fake, None, None, 64, None, fake, fake, fake,
                              16, None)
    assert r == B.MOE_ERR_WORKSPACE
    r = lib.alloc_t_select(ctypes.byref(s), fake, 200, fake, fake, None, 0, None)
    assert r == B.MOE_ERR_BUDGET
    r = lib.moe_gate(ctypes.byref(s), None, fake, None, None, fake, fake, None)
    assert r == B.MOE_ERR_ARG
