"""CPU-side checks of the C-ABI library: it builds, loads without a GPU, and exports every
function that include/polymorph.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "polymorph.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pm_[a-z_0-9]+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    from paper_2507_14959_b200 import build
    path = build.build()
    return ctypes.CDLL(path)


def test_header_declares_the_four_calls():
    names = declared_functions()
    for n in ("pm_create", "pm_register_adapter", "pm_forward", "pm_select"):
        assert n in names


def test_every_declared_symbol_is_exported(lib):
    from paper_2507_14959_b200 import binding
    for name in declared_functions():
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTS) == declared_functions()


def test_argument_errors_need_no_gpu(lib):
    # NULL arguments are rejected before any CUDA call
    assert lib.pm_create(None, None, None) == -1
    assert lib.pm_forward(None, None, 0, None, None, None, None, None) == -1
    assert lib.pm_linear_create(64, 64, None, None, 0, 0, 0, 1, 1, 0, 0, None) == -1
    lib.pm_last_error.restype = ctypes.c_char_p
    assert lib.pm_last_error(None) == b"NULL handle"
