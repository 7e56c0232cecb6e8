"""The C-ABI library loads and exports every entry point that include/espo.h declares (CPU only)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    src = open(os.path.join(ROOT, "include", "espo.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(espo_[a-z_0-9]+)\s*\(", src)))


@pytest.fixture(scope="module")
def lib():
    from paper_2605_29860_b200 import build
    return ctypes.CDLL(build.build())


def test_header_declares_the_documented_entry_points():
    names = _declared_functions()
    for must in ("espo_init_state", "espo_step", "espo_advantages", "espo_reset_state", "espo_free_state",
                 "espo_state_view", "espo_compact_active", "espo_state_status", "espo_strerror"):
        assert must in names


def test_every_declared_symbol_is_exported(lib):
    for name in _declared_functions():
        assert hasattr(lib, name), f"{name} is declared in espo.h but not exported by libespo.so"


def test_argument_errors_are_reported_without_a_device(lib):
    # these paths return before any CUDA call is made
    lib.espo_strerror.restype = ctypes.c_char_p
    assert lib.espo_strerror(0) == b"ok"
    for code in range(-7, 0):
        assert lib.espo_strerror(code) and b"unknown error code" not in lib.espo_strerror(code)
    assert b"unknown error code" in lib.espo_strerror(-99)
    lib.espo_init_state.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_uint64,
                                    ctypes.c_uint64, ctypes.c_void_p]
    assert lib.espo_init_state(None, 1, 1, 0, 0, None) == -1                    # NULL out pointer
    h = ctypes.c_void_p()
    assert lib.espo_init_state(ctypes.byref(h), 0, 10, 0, 0, None) == -3         # capacity < 1
    assert lib.espo_init_state(ctypes.byref(h), 4, 0, 0, 0, None) == -3          # V < 1
    assert lib.espo_init_state(ctypes.byref(h), 4, 10, 0, 1 << 30, None) == -7   # batch_id too large
    assert lib.espo_step(None, 0, 0, None, 0, None, 0, None, None, None, None, None) == -1
    assert lib.espo_reset_state(None, 0, None) == -1
    assert lib.espo_state_status(None, None, None) == -1
    assert lib.espo_compact_active(None, None, None, None) == -1
    assert lib.espo_advantages_status(None, None) == -1
    lib.espo_free_state(None)                                                    # ignored


def test_python_binding_mirrors_the_abi():
    import paper_2605_29860_b200 as espo
    for name in _declared_functions():
        if name == "espo_strerror" or name == "espo_last_cuda_error":
            continue
        assert hasattr(espo, name), f"binding lacks {name}"
    assert ctypes.sizeof(espo.espo_params) == 76
