"""The C-ABI library builds for sm_100a, loads, and exports every symbol include/bwla.h declares.

No compute runs here: without a GPU the compute entry points must refuse (BWLA_ERR_UNSUPPORTED) or reject
bad arguments before touching CUDA.
"""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2605_00422_b200 import build
    return C.CDLL(build.build())


def _declared():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(bwla_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert {"bwla_pack_signs", "bwla_rotate_quant_act", "bwla_w1ax_linear"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ but not exported"


def test_binding_lists_the_same_names(lib):
    from paper_2605_00422_b200 import bwla
    assert sorted(bwla.EXPORTS) == _declared()
    for n in bwla.EXPORTS:
        assert callable(getattr(bwla, n))


def test_host_side_logic_without_a_gpu(lib):
    lib.bwla_workspace_bytes.restype = C.c_size_t
    lib.bwla_workspace_bytes.argtypes = [C.c_int64, C.c_int64, C.c_int64, C.c_int, C.c_int]
    lib.bwla_status_string.restype = C.c_char_p
    a = lib.bwla_workspace_bytes(16, 1024, 1024, 16, 6)
    b = lib.bwla_workspace_bytes(32, 1024, 1024, 16, 6)
    assert a > 0 and a % 256 == 0 and b > a
    assert lib.bwla_workspace_bytes(16, 1000, 1024, 16, 6) == 0        # K % 32 != 0
    assert lib.bwla_workspace_bytes(16, 1024, 1024, 16, 5) == 0        # bits
    assert lib.bwla_status_string(0) == b"BWLA_OK"
    assert lib.bwla_status_string(-5) == b"BWLA_ERR_DEVICE_TIMEOUT"
    assert lib.bwla_force_path(7) == -1 and lib.bwla_force_path(0) == 0
    # invalid arguments are rejected before anything is launched (NULL pointers, bad sizes)
    lib.bwla_pack_signs.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p]
    assert lib.bwla_pack_signs(None, 0, 4, 33, 33, None, None) == -1
    assert lib.bwla_pack_signs(None, 0, 4, 64, 64, None, None) == -1
    assert lib.bwla_pack_signs(None, 0, 0, 64, 64, None, None) == 0    # empty problem
    lib.bwla_rotate_quant_act.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_int,
                                          C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
    assert lib.bwla_rotate_quant_act(None, 1, 64, 64, None, 8, None, 9, 6, None, None, None) == -1   # 8*9 != 64


def test_compute_refuses_without_sm100():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2605_00422_b200 import build
    lib = C.CDLL(build.build())
    lib.bwla_pack_signs.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p]
    buf = (C.c_float * 64)()
    out = (C.c_uint32 * 2)()
    assert lib.bwla_pack_signs(buf, 0, 1, 64, 64, out, None) == -2     # BWLA_ERR_UNSUPPORTED, nothing ran
