"""Host-side checks that need no GPU: the library loads, exports every symbol the header
declares, and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import pytest

import paper_2304_04237_b200 as sa
from paper_2304_04237_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2304_04237_b200 import build
    build.build()
    return binding.load()


def test_library_exports_every_declared_symbol(lib):
    hdr = open(os.path.join(ROOT, "include", "slide_attn.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(slide_attn_[a-z_]+)\s*\(", hdr))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_status_strings(lib):
    seen = {sa.slide_attn_status_string(s) for s in range(10)}
    assert len(seen) == 10 and "ok" in seen and "unknown status" not in seen
    assert sa.slide_attn_status_string(99) == "unknown status"


@pytest.mark.parametrize("args,status", [
    ((0, 4, 4, 1, 32, 3, 0, 0), sa.ERR_INVALID_ARG),
    ((1, 0, 4, 1, 32, 3, 0, 0), sa.ERR_INVALID_ARG),
    ((1, 4, -1, 1, 32, 3, 0, 0), sa.ERR_INVALID_ARG),
    ((1, 4, 4, 0, 32, 3, 0, 0), sa.ERR_INVALID_ARG),
    ((1, 4, 4, 1, 32, 3, 7, 0), sa.ERR_INVALID_ARG),      # unknown dtype
    ((1, 4, 4, 1, 32, 0, 0, 0), sa.ERR_INVALID_ARG),
    ((1, 4, 4, 1, 32, 4, 0, 0), sa.ERR_UNSUPPORTED),      # even window
    ((1, 4, 4, 1, 32, 17, 0, 0), sa.ERR_UNSUPPORTED),     # window too large
    ((1, 4, 4, 1, 12, 3, 0, 0), sa.ERR_UNSUPPORTED),      # head_dim not a multiple of 8
    ((1, 4, 4, 1, 512, 3, 0, 0), sa.ERR_UNSUPPORTED),
])
def test_create_rejects_bad_shapes_before_any_device_call(lib, args, status):
    h = ctypes.c_void_p()
    assert lib.slide_attn_create(ctypes.byref(h), *args) == status
    assert h.value is None


def test_null_handles(lib):
    assert lib.slide_attn_create(None, 1, 4, 4, 1, 32, 3, 0, 0) == sa.ERR_INVALID_ARG
    assert lib.slide_attn_destroy(None) == sa.OK
    assert lib.slide_attn_forward(None, *([None] * 8)) == sa.ERR_INVALID_ARG
    assert lib.slide_attn_forward_host(None, *([None] * 8)) == sa.ERR_INVALID_ARG
    assert lib.slide_attn_set_variant(None, 1) == sa.ERR_INVALID_ARG
    assert lib.slide_attn_query_status(None, None) == sa.ERR_INVALID_ARG


def test_create_without_a_device_fails_cleanly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    h = ctypes.c_void_p()
    assert lib.slide_attn_create(ctypes.byref(h), 1, 4, 4, 1, 32, 3, 0, 0) == sa.ERR_CUDA
    assert h.value is None


def test_product_package_does_not_import_the_oracle():
    """The library side must never route through the CPU oracle."""
    pkg = os.path.join(ROOT, "paper_2304_04237_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src, f
                assert "slide_attn_oracle" not in src, f
