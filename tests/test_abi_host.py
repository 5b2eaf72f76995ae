"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the header
declares, and argument errors are reported as status codes before any CUDA work."""
import ctypes
import os
import re

import numpy as np
import pytest
import torch

from paper_2609_22441_b200 import binding as B
from paper_2609_22441_b200 import build as builder

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    builder.build()
    return B.lib()


def test_library_exports_every_declared_symbol(L):
    header = open(os.path.join(ROOT, "include", "ccr.h")).read()
    declared = set(re.findall(r"^(?:ccr_status|size_t|int64_t|int|const char\*)\s+(ccr_[a-z_]+)\s*\(", header, re.M))
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name
    assert L.ccr_version() >= 100
    assert L.ccr_status_str(B.CCR_ERR_VALIDATION) == b"input validation failed"


def test_desc_struct_matches_header_layout():
    assert ctypes.sizeof(B.ccr_docstore_desc) == 48
    assert B.ccr_docstore_desc.reduce_sum_mask.offset == 40


def test_bad_handles_and_null_arguments(L):
    assert L.ccr_docstore_free(None) == B.CCR_ERR_BAD_HANDLE
    assert L.ccr_out_row_bytes(None, 0) == 0
    assert L.ccr_docstore_launch_count(None) == -1
    assert L.ccr_docstore_create(None, None) == B.CCR_ERR_INVALID_ARG
    h = ctypes.c_void_p()
    assert L.ccr_docstore_create(None, ctypes.byref(h)) == B.CCR_ERR_INVALID_ARG
    junk = (ctypes.c_uint64 * 64)()
    assert L.ccr_docstore_free(ctypes.cast(junk, ctypes.c_void_p)) == B.CCR_ERR_BAD_HANDLE
    assert L.ccr_join_batch(ctypes.cast(junk, ctypes.c_void_p), 1, 1, 1, None, None, None, None, None, None,
                            None, None, 0, None) == B.CCR_ERR_BAD_HANDLE
    assert L.ccr_workspace_free(None) == B.CCR_ERR_BAD_HANDLE


@pytest.mark.parametrize("field,value,want", [
    ("n_docs", -1, B.CCR_ERR_INVALID_ARG),
    ("doc_dim", 0, B.CCR_ERR_INVALID_ARG),
    ("doc_dtype", 7, B.CCR_ERR_INVALID_ARG),
    ("edge_dim", 3, B.CCR_ERR_UNSUPPORTED),       # 6 bytes: not a multiple of 16
    ("max_actors", 5, B.CCR_ERR_UNSUPPORTED),
    ("n_docs", 2**31, B.CCR_ERR_UNSUPPORTED),     # positions are int32
    ("device", -1, B.CCR_ERR_INVALID_ARG),
])
def test_create_rejects_bad_descriptors_before_touching_cuda(L, field, value, want):
    d = B.ccr_docstore_desc(1000, 64, B.CCR_F32, 32, B.CCR_F16, 0, B.CCR_F32, 0, 0, 0)
    setattr(d, field, value)
    h = ctypes.c_void_p()
    assert L.ccr_docstore_create(ctypes.byref(d), ctypes.byref(h)) == want
    assert not h


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device behaviour")
def test_no_device_means_an_error_not_a_fallback(L):
    d = B.ccr_docstore_desc(1000, 64, B.CCR_F32, 32, B.CCR_F16, 0, B.CCR_F32, 0, 0, 0)
    h = ctypes.c_void_p()
    assert L.ccr_docstore_create(ctypes.byref(d), ctypes.byref(h)) == B.CCR_ERR_CUDA
    with pytest.raises(B.CcrError):
        B.Docstore(10, 64, np.float32, 32)
