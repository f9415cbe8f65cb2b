"""Host-side checks of the C-ABI library: it loads, exports every symbol include/tm.h declares, and
rejects bad arguments before anything is launched.  No GPU needed (no compute call succeeds here)."""
from __future__ import annotations

import ctypes
import os
import re

import pytest

import paper_2102_08124_b200 as tm
from paper_2102_08124_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2102_08124_b200 import build
    build.build()
    return tm.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "tm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tm_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = _declared_functions()
    assert {"tm_find_mask", "tm_find_mask_bf16", "tm_find_mask_batched", "tm_find_mask_host", "tm_mask_words",
            "tm_workspace_bytes", "tm_status_string", "tm_version", "tm_device_status"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_python_binding_has_the_same_names():
    for n in _declared_functions():
        assert hasattr(tm, n), n


def test_version_and_sizes(lib):
    assert tm.tm_version() == 100
    assert tm.tm_mask_words_per_row(0) == 0 and tm.tm_mask_words_per_row(1) == 1 and tm.tm_mask_words_per_row(32) == 1
    assert tm.tm_mask_words_per_row(33) == 2 and tm.tm_mask_words(8, 148) == 8 * 5 and tm.tm_mask_words(0, 64) == 0
    assert tm.tm_workspace_bytes(1) > 0 and tm.tm_workspace_bytes(96) > tm.tm_workspace_bytes(1)
    assert tm.tm_workspace_bytes(1) % 256 == 0


def test_status_strings(lib):
    seen = {tm.tm_status_string(c) for c in range(10)}
    assert len(seen) == 10 and "ok" in seen
    assert tm.tm_status_string(12345) == "unknown status"


A = 0x10000  # a fake, well-aligned, never dereferenced device address


@pytest.mark.parametrize("args,code", [
    (dict(N=2, M=5), 3), (dict(N=0, M=4), 3), (dict(N=4, M=4), 3), (dict(N=3, M=8), 3), (dict(N=0, M=0), 3), (dict(N=1, M=2), 3),
    (dict(method=3), 4), (dict(method=-1), 4),
    (dict(rows=-4), 2), (dict(rows=6), 2), (dict(cols=6), 2), (dict(rows=4, cols=4, N=4, M=8), 2),
    (dict(W=0), 1), (dict(mask=0), 1),
    (dict(W=A + 4), 6), (dict(masked=A + 8), 6), (dict(mask=A + 2), 6), (dict(obj=A + 4), 6),
])
def test_plain_call_rejects_bad_arguments(lib, args, code):
    a = dict(W=A, rows=8, cols=8, N=2, M=4, method=1, mask=A, masked=A, obj=A)
    a.update(args)
    rc = lib.tm_find_mask(a["W"], a["rows"], a["cols"], a["N"], a["M"], a["method"], a["mask"], a["masked"], a["obj"])
    assert rc == code, tm.tm_status_string(rc)


def test_bf16_alignment_is_one_block_row(lib):
    assert lib.tm_find_mask_bf16(A + 8, 8, 8, 2, 4, 1, A, None, None) in (0, 7)        # 8-byte aligned rows are fine for 2:4
    assert lib.tm_find_mask_bf16(A + 4, 8, 8, 2, 4, 1, A, None, None) == 6
    assert lib.tm_find_mask_bf16(A + 8, 8, 8, 4, 8, 1, A, None, None) == 6             # 4:8 rows are 16 bytes


def _prob(**kw):
    p = binding.tm_problem()
    p.W = kw.get("W", A); p.rows = kw.get("rows", 8); p.cols = kw.get("cols", 8); p.ld = kw.get("ld", p.cols)
    p.dtype = kw.get("dtype", 0); p.mask_out = kw.get("mask", A); p.masked_w_out = kw.get("masked", None)
    p.objective_out = kw.get("obj", None)
    return p


@pytest.mark.parametrize("prob,ws,wsbytes,code", [
    (dict(dtype=7), A, 1 << 30, 5), (dict(ld=4), A, 1 << 30, 2), (dict(ld=10), A, 1 << 30, 6),
    (dict(), 0, 1 << 30, 8), (dict(), A + 16, 1 << 30, 8), (dict(), A, 16, 8), (dict(W=0), A, 1 << 30, 1),
])
def test_batched_call_rejects_bad_arguments(lib, prob, ws, wsbytes, code):
    arr = (binding.tm_problem * 1)(_prob(**prob))
    rc = lib.tm_find_mask_batched(arr, 1, 2, 4, 1, ws, wsbytes, None, None)
    assert rc == code, tm.tm_status_string(rc)


def test_batched_trivial_cases(lib):
    assert lib.tm_find_mask_batched(None, 0, 2, 4, 1, None, 0, None, None) == 0
    assert lib.tm_find_mask_batched(None, -1, 2, 4, 1, None, 0, None, None) == 2
    assert lib.tm_find_mask_batched(None, 2, 2, 4, 1, A, 1 << 30, None, None) == 1


def test_host_call_rejects_bad_arguments(lib):
    obj = ctypes.c_double(1.0); st = ctypes.c_int(5)
    f = lib.tm_find_mask_host
    assert f(A, 0, 8, 8, 2, 5, 1, A, None, ctypes.byref(obj), ctypes.byref(st)) == 3
    assert f(A, 9, 8, 8, 2, 4, 1, A, None, ctypes.byref(obj), ctypes.byref(st)) == 5
    assert f(A, 0, 8, 6, 2, 4, 1, A, None, ctypes.byref(obj), ctypes.byref(st)) == 2
    assert f(None, 0, 8, 8, 2, 4, 1, A, None, ctypes.byref(obj), ctypes.byref(st)) == 1
    assert f(A, 0, 0, 8, 2, 4, 1, A, None, ctypes.byref(obj), ctypes.byref(st)) == 0      # empty matrix: nothing to do
    assert obj.value == 0.0 and st.value == 0


def test_no_cpu_fallback_without_a_device(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    assert lib.tm_find_mask(A, 8, 8, 2, 4, 1, A, None, None) == 7                          # TM_ERR_CUDA, never a CPU result
    with pytest.raises(tm.TmError):
        tm.tm_find_mask(torch.zeros(8, 8), 2, 4, tm.TM_APPROX)


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2102_08124_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f
    assert "paper_2102_08124_b200" not in open(os.path.join(ROOT, "oracle", "tm_oracle.py")).read()
    assert "paper_2102_08124_b200" not in open(os.path.join(ROOT, "oracle", "tm_oracle.c")).read()
