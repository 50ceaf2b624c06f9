"""The C-ABI library builds, loads and exports every symbol include/*.h declares (no GPU needed)."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    from paper_1708_08917_b200 import build
    return ctypes.CDLL(str(build.build()))


def declared_functions(headers=("circ.h", "circ_debug.h")):
    names = set()
    for header in headers:
        text = (ROOT / "include" / header).read_text()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(circ_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_header_declares_the_four_calls():
    names = declared_functions(("circ.h",))
    for must in ("circ_fc_create", "circ_fc_forward", "circ_conv_forward", "circ_destroy"):
        assert must in names
    # timing and test aids live in their own header, under their own prefix
    assert not [n for n in names if n.startswith("circ_debug_")]
    assert all(n.startswith("circ_debug_") for n in declared_functions(("circ_debug.h",)))


def test_every_declared_symbol_is_exported(lib):
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} declared in circ.h but not exported by libcirc.so"


def test_binding_mirrors_header(lib):
    from paper_1708_08917_b200 import binding
    assert sorted(binding.SIGNATURES) == declared_functions()
    for name in declared_functions():
        assert callable(getattr(binding, name))


def test_argument_errors_need_no_gpu(lib):
    # shape / argument validation happens before any CUDA call
    lib.circ_fc_create.restype = ctypes.c_void_p
    lib.circ_last_error.restype = ctypes.c_char_p
    buf = (ctypes.c_float * 64)()
    assert lib.circ_fc_create(8, 8, 3, buf) is None and lib.circ_last_code() == -2       # k does not divide m
    assert lib.circ_fc_create(8, 8, 2048, buf) is None and lib.circ_last_code() == -2     # k out of range
    assert lib.circ_fc_create(513, 513, 513, buf) is None and lib.circ_last_code() == -2  # 2k - 1 points exceed the largest transform
    assert lib.circ_fc_create(8, 8, 0, buf) is None and lib.circ_last_code() == -2        # k < 1
    assert lib.circ_fc_create(10, 8, 4, buf) is None and lib.circ_last_code() == -2      # k does not divide m
    assert lib.circ_fc_create(8, 8, 4, None) is None and lib.circ_last_code() == -1      # NULL weights
    assert b"k=" in lib.circ_last_error() or b"NULL" in lib.circ_last_error()
    lib.circ_conv_create.restype = ctypes.c_void_p
    assert lib.circ_conv_create(8, 8, 9, 1, 4, buf) is None and lib.circ_last_code() == -2
    assert lib.circ_fc_forward(None, None, None, 1, None) == -1
    assert lib.circ_set_activation(None, 1) == -1
    lib.circ_destroy(None)                                                               # NULL is a no-op
    assert lib.circ_debug_inject(None, 1) == -1 and lib.circ_debug_last_kernels(None, None) == -1
    assert lib.circ_debug_forward_repeat(None, None, None, 1, 1, 1, 0, 2, None) == -1
    lib.circ_debug_launch_count.restype = ctypes.c_long
    assert lib.circ_debug_launch_count() == 0                                            # nothing was launched


def test_injected_allocation_failure_is_reported_without_a_gpu(lib):
    # the hook makes the next device allocation fail before the runtime is asked; on a machine without a
    # device the create call fails earlier (no device), on one with a device it must report CIRC_ERR_ALLOC
    lib.circ_fc_create.restype = ctypes.c_void_p
    buf = (ctypes.c_float * 64)()
    assert lib.circ_debug_fail_alloc_after(1) == 0
    h = lib.circ_fc_create(8, 8, 4, buf)
    assert h is None and lib.circ_last_code() in (-3, -4)
    assert lib.circ_debug_fail_alloc_after(0) == 0
