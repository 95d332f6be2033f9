"""Host-side checks that need no GPU: the library loads, exports every symbol the header
declares, and rejects bad arguments before touching a device."""
import ctypes as C
import os
import re

import pytest

from paper_2601_00644_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "flexspec.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(flexspec_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_symbols()
    assert len(names) >= 14
    for n in names:
        assert hasattr(B.LIB, n), n
    assert set(B.EXPORTS) <= set(names)


def test_version_and_error_strings():
    assert b"sm_100a" in B.LIB.flexspec_version()
    seen = set()
    for code in range(0, -9, -1):
        s = B.LIB.flexspec_strerror(code)
        assert s and s != b"unknown error"
        seen.add(s)
    assert len(seen) == 9
    assert B.LIB.flexspec_strerror(-99) == b"unknown error"


def test_create_rejects_bad_arguments_without_a_device():
    h = C.c_void_p()
    good = dict(n_q_heads=8, n_kv_heads=2, head_dim=64, vocab=4096, page_size=16, max_batch=1,
                k_max=4, max_kv_len=256, mode=0, device=0, flags=0)

    def create(w=256, **kw):
        cfg = B.Config(**{**good, **kw})
        return B.LIB.flexspec_create(C.byref(cfg), C.c_void_p(w), C.byref(h))

    assert B.LIB.flexspec_create(None, C.c_void_p(256), C.byref(h)) == B.ERR_INVALID_ARG
    assert create(w=0) == B.ERR_INVALID_ARG
    assert create(w=264) == B.ERR_INVALID_ARG                      # not 16-byte aligned
    assert create(n_kv_heads=3) == B.ERR_INVALID_ARG               # does not divide the query heads
    assert create(vocab=0) == B.ERR_INVALID_ARG
    assert create(mode=7) == B.ERR_INVALID_ARG
    assert create(max_kv_len=3) == B.ERR_INVALID_ARG               # smaller than k_max + 1
    assert create(head_dim=96) == B.ERR_UNSUPPORTED
    assert create(page_size=32) == B.ERR_UNSUPPORTED
    assert create(k_max=64) == B.ERR_UNSUPPORTED
    assert create(max_batch=5000) == B.ERR_UNSUPPORTED
    assert h.value is None


def test_null_handle_calls_are_errors_not_crashes():
    assert B.LIB.flexspec_destroy(None) == B.OK
    assert B.LIB.flexspec_status(None, None) == B.ERR_INVALID_ARG
    assert B.LIB.flexspec_last_launches(None) == B.ERR_INVALID_ARG
    assert B.LIB.flexspec_lm_head(None, None, 1, None, None) == B.ERR_INVALID_ARG
    assert B.LIB.flexspec_get_debug(None, None) == B.ERR_INVALID_ARG


@pytest.mark.skipif(__import__("torch").cuda.is_available(), reason="only meaningful without a GPU")
def test_create_without_gpu_reports_no_device():
    h = C.c_void_p()
    cfg = B.Config(8, 2, 64, 4096, 16, 1, 4, 256, 0, 0, 0)
    assert B.LIB.flexspec_create(C.byref(cfg), C.c_void_p(256), C.byref(h)) == B.ERR_NO_DEVICE
