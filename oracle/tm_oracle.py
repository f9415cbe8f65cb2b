"""ctypes front end of the CPU oracle (``oracle/tm_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
CPU-baseline leg of the benchmark.  It never imports the CUDA package, and the
CUDA package never imports it.  Arrays are numpy; bf16 tensors travel as their
uint16 bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

EXACT, APPROX, APPROX_COVER, EXACT_MCF, EXACT_ENUM = 0, 1, 2, 3, 4
F32, BF16 = 0, 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tm_oracle.c")
_LIB = os.path.join(_HERE, "libtm_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP over block rows for the timed baseline)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-Wall", "-Wextra",
                               "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
        lib.tmo_find_mask.argtypes = [vp, i32, i64, i64, i64, i32, i32, i32, i32, vp, vp, vp, vp]
        lib.tmo_find_mask.restype = i32
        lib.tmo_block_cover.argtypes = [vp, i32, i32, vp, vp, vp]
        lib.tmo_block_approx.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp]
        lib.tmo_block_approx_trace.argtypes = [vp, i32, i32, vp, vp, vp, vp]
        lib.tmo_block_exact_enum.argtypes = [vp, i32, i32, vp, vp]
        lib.tmo_block_exact_bruteforce.argtypes = [vp, i32, i32, vp, vp]
        lib.tmo_block_exact_mcf.argtypes = [vp, i32, i32, vp, vp, vp, vp]
        lib.tmo_nm_mask_1d.argtypes = [vp, i32, i64, i64, i64, i32, i32, i32, vp, vp, vp, vp]
        lib.tmo_mask_violations.argtypes = [vp, i32, i64, i64, i64, vp, vp]
        lib.tmo_compress_2_4.argtypes = [vp, i32, i64, i64, i64, vp, vp, vp, vp, vp, vp]
        lib.tmo_max_threads.restype = i32
        _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().tmo_max_threads())


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def magnitude_bits(block) -> np.ndarray:
    """fp32 bit patterns with the sign cleared, from an fp32 array or uint16 bf16 patterns."""
    a = np.ascontiguousarray(block)
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) & np.uint32(0x7FFF)) << np.uint32(16)
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32) & np.uint32(0x7FFFFFFF)


def _block_u(block, M):
    u = np.ascontiguousarray(magnitude_bits(block).reshape(-1), dtype=np.uint32)
    assert u.size == M * M
    return u


def block_cover(block, N, M):
    """Algorithm 1 on one M x M block -> (kept[M,M] uint8, accepted positions in pick order)."""
    u = _block_u(block, M)
    kept = np.zeros(M * M, np.uint8); acc = np.zeros(M * M, np.int32); n = ctypes.c_int(0)
    rc = _load().tmo_block_cover(_ptr(u), N, M, _ptr(kept), _ptr(acc), ctypes.byref(n))
    assert rc == 0
    return kept.reshape(M, M), acc[: n.value].copy()


def block_approx(block, N, M):
    """Algorithm 1 + completion -> dict(kept, after_a, after_b, n_fill, n_swap)."""
    u = _block_u(block, M)
    kept = np.zeros(M * M, np.uint8); a = np.zeros(M * M, np.uint8); b = np.zeros(M * M, np.uint8)
    nf, ns = ctypes.c_int(0), ctypes.c_int(0)
    rc = _load().tmo_block_approx(_ptr(u), N, M, _ptr(kept), _ptr(a), _ptr(b), ctypes.byref(nf), ctypes.byref(ns))
    assert rc == 0, "completion failed"
    return dict(kept=kept.reshape(M, M), after_a=a.reshape(M, M), after_b=b.reshape(M, M),
                n_fill=nf.value, n_swap=ns.value)


def block_approx_trace(block, N, M):
    """Algorithm 1 + completion -> (after_b, [kept set after every swap of step C]); the last one is the result."""
    u = _block_u(block, M)
    kept = np.zeros(M * M, np.uint8); b = np.zeros(M * M, np.uint8); ns = ctypes.c_int(0)
    trace = np.zeros((N * N // 4 + 1, M * M), np.uint8)
    rc = _load().tmo_block_approx_trace(_ptr(u), N, M, _ptr(kept), _ptr(b), _ptr(trace), ctypes.byref(ns))
    assert rc == 0, "completion failed"
    states = [trace[k].reshape(M, M).copy() for k in range(ns.value)]
    assert ns.value == 0 or np.array_equal(states[-1], kept.reshape(M, M))
    return b.reshape(M, M), states


def block_exact_enum(block, N, M):
    u = _block_u(block, M)
    kept = np.zeros(M * M, np.uint8); n = ctypes.c_int64(0)
    rc = _load().tmo_block_exact_enum(_ptr(u), N, M, _ptr(kept), ctypes.byref(n))
    assert rc == 0
    return kept.reshape(M, M), n.value


def block_exact_bruteforce(block, N, M):
    u = _block_u(block, M)
    kept = np.zeros(M * M, np.uint8); n = ctypes.c_int64(0)
    rc = _load().tmo_block_exact_bruteforce(_ptr(u), N, M, _ptr(kept), ctypes.byref(n))
    assert rc == 0
    return kept.reshape(M, M), n.value


def block_exact_mcf(block, N, M):
    """-> (kept, dict(nodes, edges, units)) for the Fig. 3 network."""
    u = _block_u(block, M)
    kept = np.zeros(M * M, np.uint8); nn, ne, nu = ctypes.c_int(0), ctypes.c_int(0), ctypes.c_int(0)
    rc = _load().tmo_block_exact_mcf(_ptr(u), N, M, _ptr(kept), ctypes.byref(nn), ctypes.byref(ne), ctypes.byref(nu))
    assert rc == 0
    return kept.reshape(M, M), dict(nodes=nn.value, edges=ne.value, units=nu.value)


def find_mask(W, N, M, method, threads: int = 1, want_masked: bool = True):
    """Whole matrix.  W: 2-D float32 array or uint16 bf16 patterns (C-contiguous).

    Returns dict(mask=uint32[rows, ceil(cols/32)], masked=same dtype/shape as W or None,
    objective=float, nonfinite=int)."""
    W = np.ascontiguousarray(W)
    assert W.ndim == 2 and W.dtype in (np.float32, np.uint16)
    dtype = F32 if W.dtype == np.float32 else BF16
    rows, cols = W.shape
    wpr = (cols + 31) // 32
    mask = np.zeros((rows, wpr), np.uint32)
    masked = np.empty_like(W) if want_masked else None
    obj = ctypes.c_double(0.0); bad = ctypes.c_int64(0)
    rc = _load().tmo_find_mask(_ptr(W), dtype, rows, cols, cols, N, M, method, threads,
                               _ptr(mask), _ptr(masked), ctypes.byref(obj), ctypes.byref(bad))
    if rc != 0:
        raise ValueError("tmo_find_mask rejected its arguments")
    return dict(mask=mask, masked=masked, objective=obj.value, nonfinite=bad.value)


def nm_mask_1d(W, N, M, absorb_mean: bool = False):
    """1-D N:M magnitude pruning along rows (N kept per group of M).  -> dict(mask, masked, objective, violations)."""
    W = np.ascontiguousarray(W)
    dtype = F32 if W.dtype == np.float32 else BF16
    rows, cols = W.shape
    mask = np.zeros((rows, (cols + 31) // 32), np.uint32); masked = np.empty_like(W)
    obj = ctypes.c_double(0.0); viol = ctypes.c_int64(0)
    rc = _load().tmo_nm_mask_1d(_ptr(W), dtype, rows, cols, cols, N, M, int(absorb_mean), _ptr(mask), _ptr(masked),
                                ctypes.byref(obj), ctypes.byref(viol))
    if rc != 0:
        raise ValueError("tmo_nm_mask_1d rejected its arguments")
    return dict(mask=mask, masked=masked, objective=obj.value, violations=viol.value)


def mask_violations(W, mask) -> int:
    W = np.ascontiguousarray(W); mask = np.ascontiguousarray(mask, dtype=np.uint32)
    viol = ctypes.c_int64(0)
    rc = _load().tmo_mask_violations(_ptr(W), F32 if W.dtype == np.float32 else BF16, W.shape[0], W.shape[1], W.shape[1], _ptr(mask), ctypes.byref(viol))
    assert rc == 0
    return viol.value


def compress_2_4(W, mask):
    """-> dict(values[rows, cols/2], meta[rows, wpr], values_t[cols, rows/2], meta_t[cols, wpr_t], bad_groups)."""
    W = np.ascontiguousarray(W); mask = np.ascontiguousarray(mask, dtype=np.uint32)
    rows, cols = W.shape
    values = np.zeros((rows, cols // 2), W.dtype); values_t = np.zeros((cols, rows // 2), W.dtype)
    meta = np.zeros((rows, (cols + 31) // 32), np.uint32); meta_t = np.zeros((cols, (rows + 31) // 32), np.uint32)
    bad = ctypes.c_int64(0)
    rc = _load().tmo_compress_2_4(_ptr(W), F32 if W.dtype == np.float32 else BF16, rows, cols, cols, _ptr(mask), _ptr(values), _ptr(meta),
                                  _ptr(values_t), _ptr(meta_t), ctypes.byref(bad))
    if rc != 0:
        raise ValueError("tmo_compress_2_4 rejected its arguments")
    return dict(values=values, meta=meta, values_t=values_t, meta_t=meta_t, bad_groups=bad.value)


def unpack_mask(mask: np.ndarray, cols: int) -> np.ndarray:
    """uint32[rows, wpr] -> uint8[rows, cols] of 0/1."""
    bits = np.unpackbits(np.ascontiguousarray(mask).view(np.uint8), axis=1, bitorder="little")
    return bits[:, :cols]
