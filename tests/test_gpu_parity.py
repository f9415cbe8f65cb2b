"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element, on the same
seeded inputs.  Masks and masked weights must be bit-identical; the objective within 1e-6 relative."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import paper_2102_08124_b200 as tm
import workloads
from bench import quality_numbers
from oracle import tm_oracle as orc
from tests.gpu_util import assert_parity, gpu_find_mask, to_device, to_host_bits

pytestmark = pytest.mark.gpu

METHODS = [tm.TM_EXACT, tm.TM_APPROX, tm.TM_APPROX_COVER]


@pytest.mark.parametrize("method", METHODS)
@pytest.mark.parametrize("N,M", [(2, 4), (4, 8)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_small_ragged_shapes(N, M, method, dtype):
    # several work items per block row, a ragged last item, a partial last mask word
    for rows, cols, seed in [(5 * M, 70 * M, 1), (M, M, 2), (3 * M, 33 * M, 3), (2 * M, 32 * M, 4), (7 * M, 301 * M, 5)]:
        W = workloads.normal_f32(rows, cols, 0.02, seed)
        if dtype == "bf16":
            W = workloads.f32_to_bf16_bits(W)
        assert_parity(W, N, M, method)


@pytest.mark.parametrize("method", METHODS)
@pytest.mark.parametrize("N,M", [(1, 4), (3, 4), (2, 8), (6, 8)])
def test_other_n_m_pairs(N, M, method):
    """Transposable masks with N != M/2 kept entries per line (generic kernels)."""
    W = workloads.normal_f32(3 * M, 40 * M, 0.02, 70 + N + M)
    assert_parity(W, N, M, method)
    assert_parity(workloads.f32_to_bf16_bits(W), N, M, method)
    rng = np.random.Generator(np.random.PCG64(71))
    assert_parity(rng.integers(-2, 3, size=(2 * M, 36 * M)).astype(np.float32), N, M, method)


@pytest.mark.parametrize("method", METHODS)
def test_config1(method):
    assert_parity(workloads.config1()[0], 2, 4, method)


@pytest.mark.parametrize("method", METHODS)
@pytest.mark.parametrize("N,M", [(2, 4), (4, 8)])
def test_ties_everywhere(N, M, method):
    rng = np.random.Generator(np.random.PCG64(7))
    W = rng.integers(-2, 3, size=(8 * M, 48 * M)).astype(np.float32)
    assert_parity(W, N, M, method)
    assert_parity(workloads.f32_to_bf16_bits(W), N, M, method)
    assert_parity(workloads.quantised_bf16(8 * M, 64 * M, 0.02, 5), N, M, method)


@pytest.mark.parametrize("method", METHODS)
@pytest.mark.parametrize("N,M", [(2, 4), (4, 8)])
def test_adversarial_blocks(N, M, method):
    blocks = workloads.adversarial_blocks_f32(M)                       # [n, M, M]
    W = np.ascontiguousarray(blocks.transpose(1, 0, 2).reshape(M, -1))
    assert_parity(W, N, M, method)
    assert_parity(np.zeros((2 * M, 40 * M), np.float32), N, M, method)
    assert_parity(np.full((2 * M, 40 * M), -1.5, np.float32), N, M, method)


@pytest.mark.parametrize("N,M", [(2, 4), (4, 8)])
def test_extreme_exponent_spread_uses_exact_sums(N, M):
    rng = np.random.Generator(np.random.PCG64(9))
    W = np.ldexp(rng.standard_normal((4 * M, 40 * M)), rng.integers(-125, 120, size=(4 * M, 40 * M))).astype(np.float32)
    W[::3, ::5] = (rng.integers(0, 50, size=W[::3, ::5].shape).astype(np.uint32)).view(np.float32)   # subnormals
    assert_parity(W, N, M, tm.TM_EXACT)


def test_near_tie_block_needs_exact_sums():
    B, u = np.float32(2.0 ** 40), np.float32(2.0 ** -23)
    blk = np.array([[B, 0, 0, 0], [0, B, 0, 0], [B, 0, np.float32(1.0) + u, 1], [0, B, 1, 1]], np.float32)
    W = np.tile(blk, (3, 50))
    assert_parity(W, 2, 4, tm.TM_EXACT)


@pytest.mark.parametrize("N,M", [(2, 4), (4, 8)])
def test_nonfinite_inputs_raise_the_status_bit(N, M):
    W = workloads.normal_f32(2 * M, 40 * M, 0.02, 11)
    W[1, 3] = np.inf; W[M + 1, 7 * M] = np.nan; W[0, 39 * M + 1] = -np.inf
    for method in METHODS:
        assert_parity(W, N, M, method, rel=None)                        # outputs follow the bit-pattern order; the sum is Inf/NaN


@pytest.mark.parametrize("N,M", [(2, 4), (4, 8)])
def test_bf16_nonfinite_inputs_follow_the_bit_pattern_order(N, M):
    """Inf and several NaN patterns inside bf16 data: the packed-subtraction comparisons must give way to the
    integer ones for the whole warp, before and after the first such value is met."""
    W = workloads.normal_bf16(6 * M, 300 * M, 0.02, 31)
    W[1, 3] = 0x7F80; W[2, 5] = 0xFF80; W[M + 1, 7 * M] = 0x7FC0; W[M + 1, 7 * M + 1] = 0x7F81; W[M + 2, 7 * M + 1] = 0xFFFF
    W[5 * M + 3, 299 * M + 2] = 0x7FFF; W[5 * M + 2, 299 * M + 2] = 0x7FA0
    for method in (tm.TM_APPROX, tm.TM_APPROX_COVER):
        assert_parity(W, N, M, method, rel=None)


@pytest.mark.parametrize("N,M", [(2, 4), (4, 8)])
def test_bf16_subnormals_and_extremes_compare_exactly(N, M):
    """Subnormal, smallest-normal and largest finite bf16 magnitudes, many of them equal or one step apart."""
    rng = np.random.Generator(np.random.PCG64(32))
    rows, cols = 4 * M, 160 * M
    W = rng.integers(0, 0x0100, size=(rows, cols)).astype(np.uint16)            # subnormals and the first normals
    W[:, ::3] = rng.integers(0x7000, 0x7080, size=W[:, ::3].shape).astype(np.uint16)     # large values, close together
    W[::2, ::5] = rng.integers(0, 4, size=W[::2, ::5].shape).astype(np.uint16)
    W |= (rng.integers(0, 2, size=W.shape).astype(np.uint16) << 15)
    V = W.copy()
    V[1::3, 1::7] = rng.integers(0x7F70, 0x7F80, size=V[1::3, 1::7].shape).astype(np.uint16)   # up to the largest finite value
    for method in (tm.TM_APPROX, tm.TM_APPROX_COVER):
        assert_parity(W, N, M, method, rel=1e-6)
        assert_parity(V, N, M, method, rel=None)                        # fp32 partial sums may overflow here


def test_exact_2_4_bf16_narrow_blocks_take_the_32_bit_scorer():
    """Quantised bf16 (every block spans few binades, ties everywhere): the 32-bit scorer must give the optimum and
    break ties by the mask code exactly as the 64-bit one; a second matrix mixes in blocks it cannot take."""
    W = workloads.quantised_bf16(64, 1024, 0.02, 41)
    assert_parity(W, 2, 4, tm.TM_EXACT)
    Z = W.copy()
    Z[:, :] = Z[:, :] & np.uint16(0x8003) | np.uint16(0x3C00)          # four magnitudes only: ties in every block
    assert_parity(Z, 2, 4, tm.TM_EXACT)
    V = W.copy()
    V[5, 100] = 0x0001; V[40, 777] = 0x7F00; V[41, 20] = 0x0080         # blocks with a wide exponent spread
    assert_parity(V, 2, 4, tm.TM_EXACT)
    # the same on the staged kernel (above a million weights): most work items take the 32-bit scorer as a whole, a few
    # hold one block that cannot and are scored again by the later tiers, and one item has such blocks in both halves
    B = workloads.quantised_bf16(260, 4104, 0.02, 42)
    assert_parity(B, 2, 4, tm.TM_EXACT)
    B[9, 300] = 0x0001; B[130, 2048] = 0x7F00; B[131, 2050] = 0x0003; B[200, 10] = 0x0080; B[201, 400] = 0x7F7F
    B[258, 4100] = 0x0002; B[64, 0:512] = 0                              # a ragged item, and a row of zeros across one item
    assert_parity(B, 2, 4, tm.TM_EXACT)


def test_exact_2_4_bf16_changes_tier_along_a_warps_items():
    """The staged exact kernel starts a warp on the 32-bit scorer and moves it to the 64-bit one when its items leave the first
    often: quantised rows (never leave it), then continuous rows (nearly every item does), with blocks that no in-loop tier
    takes (subnormals beside large values, Inf) before and after the change -- those are scored after the loop; in place too."""
    rows, cols = 4096, 8200                                       # about six items per warp, the last item of a row ragged
    W = workloads.quantised_bf16(rows, cols, 0.02, 91)
    W[:, 2048:] = workloads.normal_bf16(rows, cols - 2048, 0.02, 92)      # four quantised items, then thirteen continuous ones, per block row
    W[8, 16] = 0x0001; W[9, 17] = 0x7F00; W[500, 5000] = 0x0002; W[501, 5001] = 0x7E80; W[4092, 8196] = 0x0003; W[4093, 8197] = 0x7F7F
    W[700:704, 2048:2052] = 0; W[2000:2004, 4096:4608] = 0
    assert_parity(W, 2, 4, tm.TM_EXACT)
    V = W.copy(); V[600, 40] = 0x7F80; V[601, 41] = 0xFFC1
    assert_parity(V, 2, 4, tm.TM_EXACT, rel=None)
    want = orc.find_mask(W, 2, 4, orc.EXACT)
    Wd = to_device(W)
    mask, masked, obj = tm.tm_find_mask_bf16(Wd, 2, 4, tm.TM_EXACT, masked_w_out=Wd)        # in place
    torch.cuda.synchronize()
    assert np.array_equal(to_host_bits(Wd), want["masked"].view(np.uint16))
    assert np.array_equal(to_host_bits(mask), want["mask"])
    assert abs(float(obj.item()) - want["objective"]) <= 1e-6 * abs(want["objective"])


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_exact_2_4_on_the_bandwidth_kernel(dtype):
    """16-byte aligned matrices take the staged kernel for the exact 2:4 search too: several 512-column items and a ragged
    last one, mask only, in place, and (bf16) Inf and NaN patterns, which the scorer must order by bit pattern."""
    rows, cols = 204, 5144 if dtype == "f32" else 5144 + 8             # above a million weights: smaller exact calls stay on the generic kernel
    W = workloads.normal_f32(rows, cols, 0.02, 71) if dtype == "f32" else workloads.normal_bf16(rows, cols, 0.02, 71)
    assert_parity(W, 2, 4, tm.TM_EXACT)
    want = orc.find_mask(W, 2, 4, orc.EXACT)
    got = gpu_find_mask(W, 2, 4, tm.TM_EXACT, want_masked=False, want_objective=False)
    assert got["masked"] is None and np.array_equal(got["mask"], want["mask"])
    Wd = to_device(W)
    fn = tm.tm_find_mask_bf16 if dtype == "bf16" else tm.tm_find_mask
    mask, masked, obj = fn(Wd, 2, 4, tm.TM_EXACT, masked_w_out=Wd)        # in place
    torch.cuda.synchronize()
    assert np.array_equal(to_host_bits(Wd), want["masked"].view(np.uint16 if dtype == "bf16" else np.uint32))
    assert np.array_equal(to_host_bits(mask), want["mask"])
    V = W.copy()
    if dtype == "bf16":
        V[1, 3] = 0x7F80; V[2, 5] = 0xFF80; V[5, 28] = 0x7FC0; V[5, 29] = 0x7F81; V[6, 29] = 0xFFFF; V[43, cols - 2] = 0x7FA0
    else:
        V[1, 3] = np.inf; V[5, 28] = np.nan; V[43, cols - 2] = -np.inf
    assert_parity(V, 2, 4, tm.TM_EXACT, rel=None)


@pytest.mark.parametrize("N,M", [(2, 4), (4, 8)])
def test_optional_outputs_and_in_place(N, M):
    W = workloads.normal_f32(4 * M, 45 * M, 0.02, 13)
    want = orc.find_mask(W, N, M, orc.APPROX)
    got = gpu_find_mask(W, N, M, tm.TM_APPROX, want_masked=False, want_objective=False)
    assert got["masked"] is None and got["objective"] is None and np.array_equal(got["mask"], want["mask"])
    Wd = to_device(W)
    mask, masked, obj = tm.tm_find_mask(Wd, N, M, tm.TM_APPROX, masked_w_out=Wd)      # in place
    torch.cuda.synchronize()
    assert masked.data_ptr() == Wd.data_ptr()
    assert np.array_equal(to_host_bits(Wd), want["masked"].view(np.uint32))
    assert np.array_equal(to_host_bits(mask), want["mask"])


def test_empty_matrices():
    for rows, cols in [(0, 64), (64, 0), (0, 0)]:
        W = torch.empty((rows, cols), device="cuda")
        mask, masked, obj = tm.tm_find_mask(W, 2, 4, tm.TM_APPROX)
        torch.cuda.synchronize()
        assert float(obj.item()) == 0.0 and mask.numel() == rows * ((cols + 31) // 32)


def test_same_input_same_bits():
    W = workloads.normal_f32(512, 1024, 0.02, 17)
    a = gpu_find_mask(W, 2, 4, tm.TM_APPROX); b = gpu_find_mask(W, 2, 4, tm.TM_APPROX)
    assert np.array_equal(a["mask"], b["mask"]) and np.array_equal(a["masked"], b["masked"])
    assert a["objective"] == b["objective"]                              # fixed-order reduction


def _batched_parity(mats, N, M, method, strided=False):
    Ws = []
    for m in mats:
        d = to_device(m)
        if strided:                                                      # rows embedded in a wider buffer
            wide = torch.zeros((d.shape[0], d.shape[1] + 16), dtype=d.dtype, device="cuda")
            wide[:, : d.shape[1]] = d
            d = wide[:, : d.shape[1]]
        Ws.append(d)
    masks, maskeds, objs, status, ws = tm.tm_find_mask_batched(Ws, N, M, method)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for k, m in enumerate(mats):
        want = orc.find_mask(m, N, M, method, threads=orc.max_threads())
        assert np.array_equal(to_host_bits(masks[k]), want["mask"]), k
        wmasked = want["masked"].view(np.uint16 if m.dtype == np.uint16 else np.uint32)
        assert np.array_equal(to_host_bits(maskeds[k].contiguous()), wmasked), k
        assert abs(float(objs[k].item()) - want["objective"]) <= 1e-6 * want["objective"] + 1e-300, k


@pytest.mark.parametrize("method", [tm.TM_APPROX, tm.TM_EXACT])
def test_batched_mixed_dtypes_and_strides(method):
    mats = [workloads.normal_f32(16, 148, 0.1, 21), workloads.normal_bf16(64, 264, 0.02, 22),
            workloads.normal_f32(4, 4, 1.0, 23), workloads.normal_bf16(8, 4096, 0.02, 24), np.zeros((0, 64), np.float32)]
    _batched_parity(mats[:4], 2, 4, method)
    _batched_parity(mats[:4], 2, 4, method, strided=True)


def test_batched_cover_deals_items_round_robin():
    """Algorithm 1 alone takes the work items of a call round-robin over the warps of the grid, so one step of a warp may leave
    a matrix, skip several small ones and land in the middle of another.  Many matrices of a few items each (fp32 and bf16 in one
    call, ragged last items, one matrix of a single block; more items than warps, so every warp steps), then the 54 matrices of the ResNet-50-shaped model."""
    mats = []
    for k in range(240):                       # about 1700 items for the 888 warps of the fp32 launch
        mats.append(workloads.normal_f32(4 * (1 + k % 5), 4 * (1 + (k * 37) % 331), 0.05, 300 + k))
    for k in range(120):                       # about 3600 items for the 1776 warps of the bf16 launch
        mats.append(workloads.normal_bf16(32 + 4 * (k % 9), 8 * (120 + (k * 29) % 140), 0.02, 600 + k))
    mats.append(workloads.normal_f32(4, 4, 1.0, 399))
    _batched_parity(mats, 2, 4, tm.TM_APPROX_COVER)
    _batched_parity(mats, 2, 4, tm.TM_APPROX)
    _batched_parity(workloads.config2(), 2, 4, tm.TM_APPROX_COVER)


@pytest.mark.parametrize("seed", [1, 2])
def test_random_shapes_dtypes_methods_and_batches(seed):
    """Seeded random calls: 2:4 and 4:8, every method, fp32 and bf16 in one call, one to thirty matrices of up to 300 block
    rows and 6000 columns, values with and without ties, contiguous rows or rows inside a wider buffer."""
    rng = np.random.Generator(np.random.PCG64(seed))

    def matrix(M, big):
        rows = M * int(rng.integers(1, 300 if big else 40)); cols = M * int(rng.integers(1, 1500 if big else 700))
        bf16 = rng.random() < 0.5
        if bf16 and rng.random() < 0.7:
            cols = 8 * max(1, cols // 8)
        kind = int(rng.integers(0, 3))
        if kind == 0:
            W = workloads.normal_f32(rows, cols, 0.02, int(rng.integers(1 << 30)))
        elif kind == 1:
            W = (rng.integers(-3, 4, size=(rows, cols)) * 0.25).astype(np.float32)
        else:
            W = workloads.laplace_f32(rows, cols, 0.05, int(rng.integers(1 << 30)))
        return workloads.f32_to_bf16_bits(W) if bf16 else W

    for _ in range(24):
        N, M = (2, 4) if rng.random() < 0.7 else (4, 8)
        method = METHODS[int(rng.integers(0, 3))]
        count = int(rng.choice([1, 1, 2, 5, 30]))
        mats = [matrix(M, count <= 2 and rng.random() < 0.3) for _ in range(count)]
        if method == tm.TM_EXACT and M == 8:
            mats = [np.ascontiguousarray(m[: 4 * M, : 40 * M]) for m in mats]      # the flow solver is slow on the CPU side
        _batched_parity(mats, N, M, method, strided=rng.random() < 0.3)


def test_prepared_batch_object():
    mats = [workloads.normal_f32(32, 264, 0.05, 61), workloads.normal_bf16(16, 520, 0.02, 62)]
    batch = tm.TmBatch([to_device(m) for m in mats])
    for method in (tm.TM_APPROX, tm.TM_EXACT, tm.TM_APPROX):          # the same descriptors serve repeated calls
        masks, maskeds, objs, status = batch.run(2, 4, method)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        for k, m in enumerate(mats):
            want = orc.find_mask(m, 2, 4, method)
            assert np.array_equal(to_host_bits(masks[k]), want["mask"]), k
            assert abs(float(objs[k].item()) - want["objective"]) <= 1e-6 * want["objective"], k


def test_batched_4_8():
    mats = [workloads.laplace_f32(32, 264, 0.05, 31), workloads.normal_bf16(16, 520, 0.02, 32)]
    for method in METHODS:
        _batched_parity(mats, 4, 8, method)
    # fp32 with the full search runs on the kernel that splits a block over two lanes (items of 8 x 128): many small
    # matrices in one call, ragged last items, rows inside a wider buffer, ties everywhere
    rng = np.random.Generator(np.random.PCG64(33))
    small = [workloads.laplace_f32(8 * (1 + k % 4), 8 * (1 + (k * 13) % 61), 0.05, 340 + k) for k in range(40)]
    small.append(rng.integers(-2, 3, size=(24, 392)).astype(np.float32))
    small.append(np.zeros((8, 136), np.float32))
    _batched_parity(small, 4, 8, tm.TM_APPROX)
    _batched_parity(small, 4, 8, tm.TM_APPROX, strided=True)


def test_config2_whole_model_approx():
    _batched_parity(workloads.config2(), 2, 4, tm.TM_APPROX)


def test_config2_whole_model_exact():
    """All 54 ResNet-50-shaped matrices, exact 2:4, one batched call: every matrix compared with the oracle in full."""
    mats = workloads.config2()
    Ws = [to_device(m) for m in mats]
    masks, maskeds, objs, status, ws = tm.tm_find_mask_batched(Ws, 2, 4, tm.TM_EXACT)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for k, m in enumerate(mats):
        want = orc.find_mask(m, 2, 4, orc.EXACT, threads=orc.max_threads())
        assert np.array_equal(to_host_bits(masks[k]), want["mask"]), k
        assert np.array_equal(to_host_bits(maskeds[k]), want["masked"].view(np.uint32)), k
        assert abs(float(objs[k].item()) - want["objective"]) <= 1e-6 * want["objective"], k


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_host_buffer_entry_point(dtype):
    W = workloads.normal_f32(72, 520, 0.02, 41)
    if dtype == "bf16":
        Wb = workloads.f32_to_bf16_bits(W)
        Wt = torch.from_numpy(Wb.view(np.int16)).view(torch.bfloat16).pin_memory()
        ref = Wb
    else:
        Wt = torch.from_numpy(W).pin_memory(); ref = W
    for (N, M) in [(2, 4), (4, 8)]:
        for method in METHODS:
            want = orc.find_mask(ref, N, M, method)
            mask, masked, obj, status = tm.tm_find_mask_host(Wt, N, M, method)
            assert status == 0
            assert np.array_equal(mask.numpy().view(np.uint32), want["mask"])
            got_masked = masked.view(torch.int16).numpy().view(np.uint16) if dtype == "bf16" else masked.numpy().view(np.uint32)
            assert np.array_equal(got_masked, want["masked"].view(got_masked.dtype))
            assert abs(obj - want["objective"]) <= 1e-6 * want["objective"]


# ----------------------------------------------------------------------------------------------
# Full-size workloads, in the launch configuration the benchmark times
# ----------------------------------------------------------------------------------------------
def _check_line_sums(bits, N, M):
    r, c = bits.shape
    b = bits.reshape(r // M, M, c // M, M)
    assert (b.sum(axis=1) == N).all() and (b.sum(axis=3) == N).all()


def test_config5_full_size_whole_matrix():
    """12288 x 49152 bf16 (the benchmark's workload, in the launch configuration the benchmark times): mask, masked weights
    and objective of the whole matrix against the oracle (its OpenMP loop over block rows; results do not depend on the
    thread count)."""
    W = workloads.config5()[0]
    Wd = to_device(W)
    mask, masked, obj = tm.tm_find_mask_bf16(Wd, 2, 4, tm.TM_APPROX)
    torch.cuda.synchronize()
    assert tm.tm_device_status() == 0
    want = orc.find_mask(W, 2, 4, orc.APPROX, threads=orc.max_threads())
    got_mask = to_host_bits(mask)
    assert np.array_equal(got_mask, want["mask"]), "mask differs in %d words" % int((got_mask != want["mask"]).sum())
    assert np.array_equal(to_host_bits(masked), want["masked"].view(np.uint16))
    assert abs(float(obj.item()) - want["objective"]) <= 1e-6 * want["objective"]
    _check_line_sums(orc.unpack_mask(got_mask[:2048], 49152), 2, 4)


def test_config3_full_size_whole_model():
    """96 BERT-large-shaped bf16 matrices in one batched call; every matrix checked against the oracle."""
    mats = workloads.config3()
    Ws = [to_device(m) for m in mats]
    masks, maskeds, objs, status, ws = tm.tm_find_mask_batched(Ws, 2, 4, tm.TM_APPROX)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for k, m in enumerate(mats):
        want = orc.find_mask(m, 2, 4, orc.APPROX, threads=orc.max_threads(), want_masked=False)
        assert np.array_equal(to_host_bits(masks[k]), want["mask"]), k
        assert abs(float(objs[k].item()) - want["objective"]) <= 1e-6 * want["objective"], k
    # a later simulated step: the perturbed weights give different masks, still bit-identical to the oracle
    mats2 = workloads.config3_perturbed(mats[:4], 1)
    Ws2 = [to_device(m) for m in mats2]
    masks2, _, _, status2, _ = tm.tm_find_mask_batched(Ws2, 2, 4, tm.TM_APPROX)
    torch.cuda.synchronize()
    for k, m in enumerate(mats2):
        want = orc.find_mask(m, 2, 4, orc.APPROX, threads=orc.max_threads(), want_masked=False)
        assert np.array_equal(to_host_bits(masks2[k]), want["mask"]), k
        assert not np.array_equal(to_host_bits(masks2[k]), to_host_bits(masks[k]))


def test_config4_full_size_4_8(capsys):
    """8192 x 8192 fp32 Laplace, 4:8: approximate AND exact masks of the whole matrix against the oracle (the exact one is
    the min-cost flow of Fig. 3 on every one of the 1 048 576 blocks); then the quality of the approximation per block."""
    W = workloads.config4()[0]
    Wd = to_device(W)
    am, amasked, aobj = tm.tm_find_mask(Wd, 4, 8, tm.TM_APPROX)
    em, emasked, eobj = tm.tm_find_mask(Wd, 4, 8, tm.TM_EXACT)
    cm, _, _ = tm.tm_find_mask(Wd, 4, 8, tm.TM_APPROX_COVER, want_masked=False)
    torch.cuda.synchronize()
    assert tm.tm_device_status() == 0
    want = orc.find_mask(W, 4, 8, orc.APPROX, threads=orc.max_threads())
    assert np.array_equal(to_host_bits(am), want["mask"])
    assert np.array_equal(to_host_bits(amasked), want["masked"].view(np.uint32))
    assert abs(float(aobj.item()) - want["objective"]) <= 1e-6 * want["objective"]
    want_e = orc.find_mask(W, 4, 8, orc.EXACT, threads=orc.max_threads())
    got_e = to_host_bits(em)
    assert np.array_equal(got_e, want_e["mask"]), "exact mask differs in %d words" % int((got_e != want_e["mask"]).sum())
    assert np.array_equal(to_host_bits(emasked), want_e["masked"].view(np.uint32))
    assert abs(float(eobj.item()) - want_e["objective"]) <= 1e-6 * want_e["objective"]
    want_c = orc.find_mask(W, 4, 8, orc.APPROX_COVER, threads=orc.max_threads(), want_masked=False)
    assert np.array_equal(to_host_bits(cm), want_c["mask"])
    ebits, abits, cbits = (orc.unpack_mask(to_host_bits(m), 8192) for m in (em, am, cm))
    _check_line_sums(ebits, 4, 8); _check_line_sums(abits, 4, 8)
    q = quality_numbers(W, cbits, abits, ebits, 8)
    with capsys.disabled():
        print("\nconfig4 quality (4:8, 8192 x 8192 Laplace):", q)
    assert q["cover_ratio_max"] <= 2.0 + 1e-9                    # the Lemma, on every block
    assert 1.1 <= q["cover_ratio_mean"] <= 1.3                   # "on average within a factor of 1.2"
    assert q["kept_gap_max"] >= 0 and q["kept_gap_mean"] >= 0 and q["approx_ratio_max"] <= 2.0 + 1e-9


def test_config1_quality_2_4(capsys):
    W = workloads.config1()[0]
    Wd = to_device(W)
    bits = []
    for method in (tm.TM_APPROX_COVER, tm.TM_APPROX, tm.TM_EXACT):
        m, _, _ = tm.tm_find_mask(Wd, 2, 4, method, want_masked=False)
        torch.cuda.synchronize()
        bits.append(orc.unpack_mask(to_host_bits(m), 256))
    q = quality_numbers(W, bits[0], bits[1], bits[2], 4)
    with capsys.disabled():
        print("\nconfig1 quality (2:4, 256 x 256 normal):", q)
    assert q["cover_ratio_max"] <= 2.0 + 1e-9 and 1.1 <= q["cover_ratio_mean"] <= 1.35
