"""The C-ABI library loads and exports every entry point that include/gwq.h declares.
No compute call is made here (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib_path():
    from paper_2411_00850_b200 import build
    return build.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "gwq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gwq_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_four_calls():
    names = _declared()
    for need in ("gwq_select_outliers", "gwq_pack", "gwq_linear", "gwq_free"):
        assert need in names


def test_library_exports_every_declared_symbol(lib_path):
    lib = ctypes.CDLL(lib_path)
    for name in _declared():
        assert hasattr(lib, name), name


def test_binding_lists_the_same_names(lib_path):
    from paper_2411_00850_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()
    lib = binding.load_library()
    assert lib.gwq_status_string(0) == b"GWQ_OK"
    assert lib.gwq_status_string(4) == b"GWQ_ERR_NONFINITE"
    lib.gwq_free(None)  # NULL is a no-op


def test_struct_layout_matches_header():
    from paper_2411_00850_b200 import binding
    # x86-64 / LP64 layout of the two public structs
    assert ctypes.sizeof(binding.gwq_outliers) == 48
    assert binding.gwq_outliers.nnz.offset == 16 and binding.gwq_outliers.row_ptr.offset == 24
    assert ctypes.sizeof(binding.gwq_packed) == 64
    assert binding.gwq_packed.codes.offset == 24 and binding.gwq_packed.priv.offset == 56
