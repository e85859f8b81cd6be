"""The C-ABI library loads without a GPU and exports every function include/s3.h declares; argument
checks that need no device work from the host."""
import ctypes as C
import os
import re

import pytest

import paper_2601_17702_b200 as S
from paper_2601_17702_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "s3.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(s3_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2601_17702_b200.build import build
    build()
    lib = B.lib()
    declared = _declared_functions()
    assert len(declared) >= 20
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in include/s3.h but not exported"
    assert sorted(B.EXPORTS) == declared
    assert S.s3_version() >= 100


def test_struct_layouts_match_header():
    assert C.sizeof(B.PostingsItem) == 64
    assert C.sizeof(B.CsrView) == 16
    assert C.sizeof(B.ScoreParams) == 32
    assert C.sizeof(B.IndexStats) == 48


def test_host_side_argument_checks():
    lib = B.lib()
    assert lib.s3_sae_prepared_bytes(0, 16, B.S3_BF16) == 0
    assert lib.s3_sae_prepared_bytes(1024, 16384, B.S3_BF16) >= 1024 * 16384 * 2 + 16384 * 4
    h = C.c_void_p()
    assert lib.s3_sae_create(C.byref(h), None, None, None, 8, 8, 0, None, 0, None) == B.S3_ERR_INVALID_ARG
    assert b"null" in lib.s3_last_error()
    assert lib.s3_index_create(None, 1, 8, 0) == B.S3_ERR_INVALID_ARG
    assert lib.s3_index_append(None, 0, None, None, None, 0, 1, 0, None, None) == B.S3_ERR_INVALID_ARG
    item = B.PostingsItem(None, None, 4, 70000, 8, 0, 0, None, None, None)
    arr = (B.PostingsItem * 1)(item)
    ws = C.create_string_buffer(64)
    assert lib.s3_postings_build_batched(arr, 1, ws, 64, None) in (B.S3_ERR_INVALID_ARG, B.S3_ERR_UNSUPPORTED)
    assert lib.s3_postings_build_batched(arr, 33, ws, 64, None) == B.S3_ERR_UNSUPPORTED
    item = B.PostingsItem(1, None, 4, 2, (1 << 20) + 8, 0, 0, 1, 1, None)
    arr = (B.PostingsItem * 1)(item)
    assert lib.s3_postings_build_batched(arr, 1, ws, 64, None) == B.S3_ERR_UNSUPPORTED       # d_sae limit
    item = B.PostingsItem(1, None, 4, 2, 64, 0, 2**31 - 2, 1, 1, None)
    arr = (B.PostingsItem * 1)(item)
    assert lib.s3_postings_build_batched(arr, 1, ws, 64, None) == B.S3_ERR_CAPACITY           # int32 positions
    p = B.ScoreParams(0, 1, 0, 4, 1.0, 0.0, 0)
    v = (B.CsrView * 1)(B.CsrView(1, 1))
    assert lib.s3_coactivation_score_topspans(v, 1, 8, 100, None, None, 1, 1, 1, C.byref(p), None, 0, None, None,
                                              None, ws, 64, None) == B.S3_ERR_INVALID_ARG       # width 0
    p = B.ScoreParams(4, 4, 0, 100, 1.0, 0.0, 0)
    assert lib.s3_coactivation_score_topspans(v, 1, 8, 100, None, None, 1, 1, 1, C.byref(p), None, 0, None, None,
                                              None, ws, 64, None) == B.S3_ERR_UNSUPPORTED       # s > 64
