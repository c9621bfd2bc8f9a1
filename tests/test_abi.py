"""Host-side checks of the C ABI: the library loads, exports every declared symbol, and rejects
bad arguments before launching anything (no GPU needed)."""
import ctypes as C
import os
import re

import pytest

from paper_2602_06183_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "sparseffn.h")).read()
    declared = set(re.findall(r"SF_API\s+(?:const\s+char\*|int)\s+(sf_\w+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(binding.EXPORTED_SYMBOLS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    assert binding.status_string(0) == "SF_OK"
    for code in range(-8, 0):
        assert binding.status_string(code).startswith("SF_ERR_")


def test_size_queries_and_shape_errors(lib):
    assert binding.sf_prune24_sizes(128, 256, 1) == (128 * 256, 128 * 256 // 8)
    a, b = C.c_size_t(), C.c_size_t()
    assert lib.sf_prune24_sizes(128, 250, 1, C.byref(a), C.byref(b)) == binding.SF_ERR_SHAPE
    assert lib.sf_prune24_sizes(128, 256, 2, C.byref(a), C.byref(b)) == binding.SF_ERR_SHAPE
    assert lib.sf_prune24_sizes(128, 256, 1, None, C.byref(b)) == binding.SF_ERR_NULL
    assert binding.sf_vnm_sizes(128, 256, 64, 2, 8) == (128 * 64 * 2, 128 * 8 * 2, 2 * 32 * 4)
    c = C.c_size_t()
    assert lib.sf_vnm_sizes(128, 256, 64, 1, 8, C.byref(a), C.byref(b), C.byref(c)) == binding.SF_ERR_UNSUPPORTED
    assert lib.sf_vnm_sizes(100, 256, 64, 2, 8, C.byref(a), C.byref(b), C.byref(c)) == binding.SF_ERR_SHAPE
    assert lib.sf_vnm_sizes(128, 256, 64, 2, 12, C.byref(a), C.byref(b), C.byref(c)) == binding.SF_ERR_SHAPE


def test_null_and_alignment_rejected_before_launch(lib):
    # shapes fine, pointers NULL -> SF_ERR_NULL without touching a device
    assert lib.sf_prune24_compress(None, 128, 256, 256, 1, 0, None, None, None, None) == binding.SF_ERR_NULL
    fake = C.c_void_p(0x1008)   # 8-byte aligned only
    ok = C.c_void_p(0x1000)
    assert lib.sf_prune24_compress(fake, 128, 256, 256, 1, 0, ok, ok, None, None) == binding.SF_ERR_ALIGN
    assert lib.sf_prune24_compress(ok, 128, 256, 100, 1, 0, ok, ok, None, None) == binding.SF_ERR_ALIGN
    assert lib.sf_vnm_sparsify_act(None, 128, 256, 256, 64, 2, 8, 1, None, None, None, None, None, None) == binding.SF_ERR_NULL
    # empty inputs are a no-op
    assert lib.sf_prune24_compress(None, 0, 256, 256, 1, 0, None, None, None, None) == binding.SF_OK
