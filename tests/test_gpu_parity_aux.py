"""GPU parity of the neighbouring operations (1-D N:M pruning with violation count and mean absorption, mask
violations, 2:4 operand compression) against the CPU oracle: everything bit-exact, objective within 1e-6."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import paper_2102_08124_b200 as tm
import workloads
from oracle import tm_oracle as orc
from tests.gpu_util import to_device, to_host_bits

pytestmark = pytest.mark.gpu


def _case(dtype, rows, cols, seed, ties=False):
    if ties:
        W = np.random.Generator(np.random.PCG64(seed)).integers(-2, 3, size=(rows, cols)).astype(np.float32)
    else:
        W = workloads.normal_f32(rows, cols, 0.02, seed)
        W[np.random.Generator(np.random.PCG64(seed + 1)).random(W.shape) < 0.3] = 0.0      # an "unstructured sparse" tensor
    return workloads.f32_to_bf16_bits(W) if dtype == "bf16" else W


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("N,M", [(2, 4), (4, 8), (1, 4), (1, 2), (3, 4), (2, 8), (6, 8), (0, 4), (4, 4)])
@pytest.mark.parametrize("absorb", [False, True])
def test_nm_1d(dtype, N, M, absorb):
    for rows, cols, seed, ties in [(7, 8 * 33 + M, 3, False), (16, 1024, 4, True), (1, M, 5, False), (5, 2048 + 8, 6, False)]:
        W = _case(dtype, rows, cols - cols % M, seed, ties)
        want = orc.nm_mask_1d(W, N, M, absorb_mean=absorb)
        mask, masked, obj, viol, status = tm.tm_nm_mask_1d(to_device(W), N, M, absorb_mean=absorb)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert np.array_equal(to_host_bits(mask), want["mask"])
        assert np.array_equal(to_host_bits(masked), want["masked"].view(np.uint16 if dtype == "bf16" else np.uint32))
        assert int(viol.item()) == want["violations"]
        assert abs(float(obj.item()) - want["objective"]) <= 1e-6 * abs(want["objective"]) + 1e-300


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("N,M", [(1, 4), (2, 4), (3, 4), (1, 8), (3, 8), (4, 8), (5, 8), (7, 8)])
def test_nm_1d_groups_on_the_bandwidth_kernels_edge_values(dtype, N, M):
    """Shapes the bandwidth kernels take (16-byte aligned rows), groups of four and of eight: zeros of both signs, subnormals,
    equal magnitudes, an odd number of rows, several column chunks; then Inf and NaN, which must be ordered by bit pattern and flagged."""
    rows, cols = 13, 776
    rng = np.random.Generator(np.random.PCG64(50 + N))
    W = workloads.normal_f32(rows, cols, 0.02, 51)
    W[rng.random(W.shape) < 0.25] = 0.0
    W[rng.random(W.shape) < 0.05] = -0.0
    W[rng.random(W.shape) < 0.05] = np.float32(1e-40)
    W[:, 100:140] = np.float32(0.5) * np.sign(W[:, 100:140] + 1e-9)
    if dtype == "bf16":
        W = workloads.f32_to_bf16_bits(W)
    for nonfinite in (False, True):
        if nonfinite:
            if dtype == "bf16":
                W[2, 5] = 0x7F80; W[3, 300] = 0xFFC1; W[3, 301] = 0x7FC0; W[12, 775] = 0xFF80
            else:
                W[2, 5] = np.inf; W[3, 300] = np.nan; W[3, 301] = -np.nan; W[12, 775] = -np.inf
        want = orc.nm_mask_1d(W, N, M)
        mask, masked, obj, viol, status = tm.tm_nm_mask_1d(to_device(W), N, M)
        torch.cuda.synchronize()
        assert int(status.item()) == (tm.TM_DEV_NONFINITE if nonfinite else 0)
        assert np.array_equal(to_host_bits(mask), want["mask"])
        assert np.array_equal(to_host_bits(masked), want["masked"].view(np.uint16 if dtype == "bf16" else np.uint32))
        assert int(viol.item()) == want["violations"]
        if not nonfinite:
            assert abs(float(obj.item()) - want["objective"]) <= 1e-6 * abs(want["objective"]) + 1e-300


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("N", [1, 2, 3])
def test_nm_1d_mean_absorption_edge_values(dtype, N):
    """Mean absorption on the bandwidth kernel where the rounding matters: sums that land between two bf16 values or on a
    tie, results that round up to Inf, subnormal results, zeros of both signs, and rows that hold Inf or NaN."""
    rows, cols = 12, 1544
    rng = np.random.Generator(np.random.PCG64(70 + N))
    W = workloads.normal_f32(rows, cols, 0.02, 71)
    W[rng.random(W.shape) < 0.2] = 0.0
    W[rng.random(W.shape) < 0.05] = -0.0
    W[:, 64:128] = rng.choice(np.array([1.0, 1.00390625, 1.0078125, -1.0, 0.99609375], np.float32), size=(rows, 64))   # one bf16 step apart
    W[:, 128:192] = rng.choice(np.array([3.3e38, -3.3e38, 3.38e38, 1e38], np.float32), size=(rows, 64))               # sums overflow
    W[:, 192:256] = rng.choice(np.array([1e-39, -2e-39, 9.2e-41, 1.2e-38], np.float32), size=(rows, 64))              # subnormal range
    if dtype == "bf16":
        W = workloads.f32_to_bf16_bits(W)
    for nonfinite in (False, True):
        if nonfinite:
            if dtype == "bf16":
                W[2, 5] = 0x7F80; W[3, 300] = 0xFFC1; W[3, 301] = 0x7FC0; W[7, 900] = 0x7F81; W[11, 1543] = 0xFF80
            else:
                W[2, 5] = np.inf; W[3, 300] = np.nan; W[3, 301] = -np.nan; W[11, 1543] = -np.inf
        want = orc.nm_mask_1d(W, N, 4, absorb_mean=True)
        mask, masked, obj, viol, status = tm.tm_nm_mask_1d(to_device(W), N, 4, absorb_mean=True)
        torch.cuda.synchronize()
        assert np.array_equal(to_host_bits(mask), want["mask"])
        got, exp = to_host_bits(masked), want["masked"].view(np.uint16 if dtype == "bf16" else np.uint32)
        # a NaN that went through the fp64 addition carries the sign and payload its processor chose: NaN must meet NaN, all else bit for bit
        is_nan = (lambda a: (a & 0x7FFF) > 0x7F80) if dtype == "bf16" else (lambda a: (a & 0x7FFFFFFF) > 0x7F800000)
        assert np.array_equal(is_nan(got), is_nan(exp))
        assert np.array_equal(got[~is_nan(exp)], exp[~is_nan(exp)])
        assert int(viol.item()) == want["violations"]


def test_nm_1d_strided_rows_and_unaligned_pitch():
    base = to_device(_case("bf16", 12, 100, 7))                  # 200-byte pitch: rows are only 8-byte aligned
    W = base[:, :92]                                             # a strided view
    want = orc.nm_mask_1d(np.ascontiguousarray(to_host_bits(W.contiguous())), 2, 4)
    mask, masked, obj, viol, status = tm.tm_nm_mask_1d(W, 2, 4)
    torch.cuda.synchronize()
    assert np.array_equal(to_host_bits(mask), want["mask"])
    assert np.array_equal(to_host_bits(masked.contiguous()), want["masked"])
    assert int(viol.item()) == want["violations"]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_mask_violations(dtype):
    W = _case(dtype, 40, 520, 11)
    Wd = to_device(W)
    for N, M in [(2, 4), (4, 8)]:
        res = orc.find_mask(W, N, M, orc.APPROX)
        got = tm.tm_mask_violations(Wd, torch.from_numpy(res["mask"].view(np.int32)).cuda())
        torch.cuda.synchronize()
        assert int(got.item()) == orc.mask_violations(W, res["mask"])
    zero = torch.zeros((40, 17), dtype=torch.int32, device="cuda")
    assert int(tm.tm_mask_violations(Wd, zero).item()) == int((workloads.bf16_bits_to_f32(W) != 0).sum() if dtype == "bf16" else (W != 0).sum())


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_compress_2_4(dtype):
    # bf16 shapes whose mask rows are multiples of 16 bytes take the streaming kernel (items of 32 rows x 128 columns): single
    # and ragged items, rows that allow 16-byte stores of the column form (rows % 16 == 0) and of its metadata (rows % 128 == 0)
    # and rows that do not, several items per warp down one column tile and across tiles
    for rows, cols, seed in [(4, 4, 21), (36, 132, 22), (64, 512, 23), (100, 260, 24), (272, 384, 25), (2180, 2560, 26),
                             (36, 128, 27), (512, 256, 28), (1024, 384, 29), (4096, 1280, 30), (1156, 3968, 32)]:
        W = _case(dtype, rows, cols, seed)
        Wd = to_device(W)
        fn = tm.tm_find_mask_bf16 if dtype == "bf16" else tm.tm_find_mask
        mask, _, _ = fn(Wd, 2, 4, tm.TM_APPROX)
        values, meta, values_t, meta_t, status = tm.tm_compress_2_4(Wd, mask)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        want = orc.compress_2_4(W, to_host_bits(mask))
        assert want["bad_groups"] == 0
        assert np.array_equal(to_host_bits(values), want["values"].view(np.uint16 if dtype == "bf16" else np.uint32))
        assert np.array_equal(to_host_bits(meta), want["meta"])
        assert np.array_equal(to_host_bits(values_t), want["values_t"].view(np.uint16 if dtype == "bf16" else np.uint32))
        assert np.array_equal(to_host_bits(meta_t), want["meta_t"])
    # a mask that is not transposable is flagged, and the bad groups come out as zeros like the oracle's
    W = _case("f32", 16, 64, 31); Wd = to_device(W)
    one_d, _, _, _, _ = tm.tm_nm_mask_1d(Wd, 2, 4)
    values, meta, values_t, meta_t, status = tm.tm_compress_2_4(Wd, one_d)
    torch.cuda.synchronize()
    assert int(status.item()) == tm.TM_DEV_BADMASK
    want = orc.compress_2_4(W, to_host_bits(one_d))
    assert np.array_equal(to_host_bits(values_t), want["values_t"].view(np.uint32)) and np.array_equal(to_host_bits(meta_t), want["meta_t"])
    assert np.array_equal(to_host_bits(values), want["values"].view(np.uint32))
    # the same through the streaming bf16 kernel: bad groups inside full items and inside a ragged one
    for rows, cols in [(64, 256), (100, 128)]:
        W = _case("bf16", rows, cols, 33); Wd = to_device(W)
        one_d, _, _, _, _ = tm.tm_nm_mask_1d(Wd, 2, 4)
        values, meta, values_t, meta_t, status = tm.tm_compress_2_4(Wd, one_d)
        torch.cuda.synchronize()
        assert int(status.item()) == tm.TM_DEV_BADMASK
        want = orc.compress_2_4(W, to_host_bits(one_d))
        assert want["bad_groups"] > 0
        assert np.array_equal(to_host_bits(values_t), want["values_t"].view(np.uint16)) and np.array_equal(to_host_bits(meta_t), want["meta_t"])
        assert np.array_equal(to_host_bits(values), want["values"].view(np.uint16)) and np.array_equal(to_host_bits(meta), want["meta"])
