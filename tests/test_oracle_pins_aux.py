"""Pins for the oracle's neighbouring operations (Section 5 of the paper and the operand compression the
transposable mask exists for): checked against numpy's sort, the paper's Eq. 3, closed forms and round trips."""
from __future__ import annotations

from fractions import Fraction
from math import comb

import numpy as np
import pytest

import workloads
from oracle import tm_oracle as orc


def _values(W):
    return workloads.bf16_bits_to_f32(W) if W.dtype == np.uint16 else W


@pytest.mark.parametrize("N,M", [(2, 4), (4, 8), (1, 4), (1, 2), (3, 4), (2, 8), (6, 8)])
@pytest.mark.parametrize("kind", ["normal", "ties", "bf16"])
def test_nm_1d_keeps_the_n_largest_of_every_group(N, M, kind):
    rng = np.random.Generator(np.random.PCG64(5 + N + M))
    if kind == "normal": W = workloads.normal_f32(24, 16 * M, 0.02, 7)
    elif kind == "ties": W = rng.integers(-2, 3, size=(24, 16 * M)).astype(np.float32)
    else: W = workloads.quantised_bf16(24, 16 * M, 0.02, 9)
    res = orc.nm_mask_1d(W, N, M)
    bits = orc.unpack_mask(res["mask"], W.shape[1]).reshape(24, -1, M)
    mag = np.abs(_values(W).astype(np.float64)).reshape(24, -1, M)
    assert (bits.sum(axis=2) == N).all()
    # numpy's stable sort on |w|: among equals the later position is heavier, so the N last of the order are kept
    order = np.argsort(mag, axis=2, kind="stable")
    want = np.zeros_like(bits)
    np.put_along_axis(want, order[:, :, M - N:], 1, axis=2)
    assert np.array_equal(bits, want)
    v = _values(W).reshape(24, -1, M)
    assert res["violations"] == int(((want == 0) & (v != 0)).sum())
    assert res["objective"] == pytest.approx(float((mag * want).sum()), rel=1e-12)
    kept_vals = _values(res["masked"]).reshape(24, -1, M)
    assert np.array_equal(kept_vals, np.where(want == 1, v, 0).astype(np.float32))


def test_pattern_violation_probability_matches_eq_3():
    """Eq. 3: P(a block of M with i.i.d. prunable-probability rho is N:M sparse) = sum_{i>=N} C(M,i) rho^i (1-rho)^(M-i).
    Here 'N' of Eq. 3 counts prunable (zero) entries; a block has no pattern-violation iff it holds >= M - kept zeros."""
    rng = np.random.Generator(np.random.PCG64(33))
    rho, M = 0.6, 8
    W = workloads.normal_f32(512, 1024, 1.0, 31)
    W[rng.random(W.shape) < rho] = 0.0
    for kept in (2, 4, 6):
        res = orc.nm_mask_1d(W, kept, M)
        bits = orc.unpack_mask(res["mask"], 1024).reshape(512, -1, M)
        viol_per_block = ((bits == 0) & (W.reshape(512, -1, M) != 0)).sum(axis=2)
        assert res["violations"] == int(viol_per_block.sum())
        frac_sparse = float((viol_per_block == 0).mean())
        p = sum(comb(M, i) * rho ** i * (1 - rho) ** (M - i) for i in range(M - kept, M + 1))
        n = viol_per_block.size
        assert abs(frac_sparse - p) < 5 * np.sqrt(p * (1 - p) / n) + 1e-3
        assert orc.mask_violations(W, res["mask"]) == res["violations"]
    assert orc.mask_violations(W, np.zeros((512, 32), np.uint32)) == int((W != 0).sum())
    assert orc.mask_violations(W, np.full((512, 32), 0xFFFFFFFF, np.uint32)) == 0


@pytest.mark.parametrize("N,M", [(2, 4), (4, 8)])
def test_mean_absorption_preserves_the_group_sum(N, M):
    """With as many pruned as kept entries, adding the mean of the pruned weights to every kept weight moves
    exactly the pruned mass onto the kept ones: the group sum is unchanged up to the final fp32 roundings."""
    W = workloads.normal_f32(64, 32 * M, 0.05, 41)
    plain = orc.nm_mask_1d(W, N, M)
    res = orc.nm_mask_1d(W, N, M, absorb_mean=True)
    assert np.array_equal(res["mask"], plain["mask"]) and res["objective"] == plain["objective"]
    before = W.astype(np.float64).reshape(64, -1, M).sum(axis=2)
    after = res["masked"].astype(np.float64).reshape(64, -1, M).sum(axis=2)
    scale = np.abs(W).reshape(64, -1, M).max(axis=2)
    assert (np.abs(before - after) <= N * scale * 2.0 ** -22).all()
    bits = orc.unpack_mask(res["mask"], W.shape[1])
    assert (res["masked"][bits == 0] == 0).all()
    # a hand-checked group: kept 4 and -3 (the later of the equal magnitudes 3), pruned 1 and 3 -> mean 2
    g = np.array([[1.0, 3.0, -3.0, 4.0]], np.float32)
    out = orc.nm_mask_1d(g, 2, 4, absorb_mean=True)["masked"]
    assert out.tolist() == [[0.0, 0.0, -1.0, 6.0]]
    gb = workloads.f32_to_bf16_bits(np.array([[1.0, 3.0, -3.0, 4.0, 0.5, 0.25, 100.0, 0.001]], np.float32))
    outb = workloads.bf16_bits_to_f32(orc.nm_mask_1d(gb, 2, 4, absorb_mean=True)["masked"])
    assert outb[0, :4].tolist() == [0.0, 0.0, -1.0, 6.0] and outb[0, 5] == 0.0 and outb[0, 7] == 0.0


def _bf16_nearest_even(x: Fraction) -> int:
    """Bit pattern of the bf16 number nearest to the positive rational x (ties to the even pattern), worked out with
    exact fractions: no float arithmetic, no bit tricks shared with the oracle.  Normal range only."""
    assert x > 0
    e = 0
    while Fraction(2) ** (e + 1) <= x: e += 1
    while Fraction(2) ** e > x: e -= 1
    ulp = Fraction(2) ** (e - 7)                      # bf16: 8 significant bits
    lo = (x // ulp) * ulp
    hi = lo + ulp
    def pattern(v):
        ee = e if v < Fraction(2) ** (e + 1) else e + 1
        frac = int(v / (Fraction(2) ** (ee - 7))) - 128
        return ((ee + 127) << 7) | frac
    if x - lo < hi - x: return pattern(lo)
    if x - lo > hi - x: return pattern(hi)
    return pattern(lo) if pattern(lo) % 2 == 0 else pattern(hi)


def _bf16(v: float) -> int:
    b = workloads.f32_to_bf16_bits(np.array([v], np.float32))
    assert workloads.bf16_bits_to_f32(b)[0] == np.float32(v), "test value must be exact in bf16"
    return int(b[0])


@pytest.mark.parametrize("case", ["below", "above", "tie_even_low", "tie_odd_low", "carry", "exact"])
def test_mean_absorption_rounds_bf16_to_nearest_even(case):
    """Groups (p1, p2, k1, k2) with |p| < |k|: the pruned mean mu = (p1 + p2) / 2 is added to the kept entries, and the
    sum -- exact in fp64 and in fp32 for these values -- must be rounded to bf16 to nearest, ties to even.  Expected
    patterns come from exact fractions.  Truncation, round-half-up or a missing carry each fail one of the cases."""
    u = 2.0 ** -7                                                   # bf16 spacing in [1, 2)
    k1 = {"below": 1.0, "above": 1.0, "tie_even_low": 1.0, "tie_odd_low": 1.0 + u, "carry": 2.0 - u, "exact": 1.0}[case]
    # mu chosen so that k1 + mu lies a quarter, three quarters or exactly half an ulp above k1 (all exact in fp32)
    mu = {"below": u / 4, "above": 3 * u / 4, "tie_even_low": u / 2, "tie_odd_low": u / 2, "carry": u / 2, "exact": u}[case]
    k2 = 1.5
    g = np.array([[mu, mu, k1, k2]], np.float32)                    # the two light entries are pruned: their mean is mu
    gb = np.array([[_bf16(mu), _bf16(mu), _bf16(k1), _bf16(k2)]], np.uint16)
    res = orc.nm_mask_1d(gb, 2, 4, absorb_mean=True)
    assert orc.unpack_mask(res["mask"], 4).tolist() == [[0, 0, 1, 1]]
    want1 = _bf16_nearest_even(Fraction(k1) + Fraction(mu)); want2 = _bf16_nearest_even(Fraction(k2) + Fraction(mu))
    assert [int(v) for v in res["masked"][0]] == [0, 0, want1, want2]
    if case == "tie_even_low": assert want1 == _bf16(1.0)          # halfway between 1 and 1 + u: the even pattern is the lower one
    if case == "tie_odd_low": assert want1 == _bf16(1.0 + 2 * u)   # halfway between 1 + u and 1 + 2u: the even one is the upper
    if case == "carry": assert want1 == _bf16(2.0)                 # the rounding carries into the exponent
    if case == "below": assert want1 == _bf16(1.0)
    if case == "above": assert want1 == _bf16(1.0 + u)
    # the same group in fp32 keeps the unrounded sum
    assert orc.nm_mask_1d(g, 2, 4, absorb_mean=True)["masked"][0].tolist() == [0.0, 0.0, float(np.float32(k1 + mu)), float(np.float32(k2 + mu))]


def test_mean_absorption_keeps_nan_a_nan_in_bf16():
    gb = np.array([[_bf16(0.25), _bf16(0.5), 0x7FC1, _bf16(1.0)]], np.uint16)          # a NaN counts as the heaviest
    out = orc.nm_mask_1d(gb, 2, 4, absorb_mean=True)["masked"][0]
    assert out[0] == 0 and out[1] == 0
    assert (int(out[2]) & 0x7F80) == 0x7F80 and (int(out[2]) & 0x7F) != 0             # still a NaN, not an Inf
    assert int(out[3]) == _bf16(1.375)                                                # 1 + (0.25 + 0.5) / 2


@pytest.mark.parametrize("N,M,group,want", [
    # N kept of M.  mu = (sum of the pruned weights) / (number of pruned weights) -- the reading of Section 5's "mean of
    # the pruned weights" taken by this build; spreading the pruned sum over the kept entries instead would give the
    # values in the comments, which differ whenever N != M / 2.
    (1, 4, [1.0, 2.0, 3.0, 8.0], [0.0, 0.0, 0.0, 10.0]),                                  # mean 6 / 3 = 2      (spread: 14)
    (3, 4, [1.0, 2.0, 3.0, 8.0], [0.0, 3.0, 4.0, 9.0]),                                   # mean 1 / 1 = 1      (spread: 1/3 each)
    (2, 8, [1.0, 2.0, 3.0, 4.0, 5.0, 6.0, 16.0, 32.0], [0.0] * 6 + [19.5, 35.5]),         # mean 21 / 6 = 3.5   (spread: 10.5)
    (6, 8, [1.0, 3.0, 4.0, 5.0, 6.0, 7.0, 16.0, 32.0], [0.0, 0.0, 6.0, 7.0, 8.0, 9.0, 18.0, 34.0]),   # mean 4 / 2 = 2 (spread: 2/3)
    (2, 4, [1.0, -5.0, 8.0, 16.0], [0.0, 0.0, 6.0, 14.0]),                                # mean (1 - 5) / 2 = -2: signs count
])
def test_mean_absorption_divides_by_the_number_of_pruned_weights(N, M, group, want):
    g = np.array([group], np.float32)
    assert orc.nm_mask_1d(g, N, M, absorb_mean=True)["masked"][0].tolist() == want
    gb = workloads.f32_to_bf16_bits(g)                                                    # all values are exact in bf16
    assert workloads.bf16_bits_to_f32(orc.nm_mask_1d(gb, N, M, absorb_mean=True)["masked"])[0].tolist() == want


def _decompress(values, meta, cols):
    rows = values.shape[0]
    out = np.zeros((rows, cols), values.dtype)
    for r in range(rows):
        for g in range(cols // 4):
            nib = (int(meta[r, g // 8]) >> (4 * (g % 8))) & 0xF
            out[r, 4 * g + (nib & 3)] = values[r, 2 * g]
            out[r, 4 * g + (nib >> 2)] = values[r, 2 * g + 1]
    return out


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_compression_round_trip_for_w_and_its_transpose(dtype):
    W = workloads.normal_f32(24, 72, 0.02, 51)
    if dtype == "bf16":
        W = workloads.f32_to_bf16_bits(W)
    res = orc.find_mask(W, 2, 4, orc.APPROX)
    c = orc.compress_2_4(W, res["mask"])
    assert c["bad_groups"] == 0
    assert np.array_equal(_decompress(c["values"], c["meta"], 72), res["masked"])
    assert np.array_equal(_decompress(c["values_t"], c["meta_t"], 24), np.ascontiguousarray(res["masked"].T))
    nib = (c["meta"][:, :, None] >> (4 * np.arange(8))) & 0xF
    nib = nib.reshape(24, -1)[:, : 72 // 4]
    assert ((nib & 3) < (nib >> 2)).all()                      # indices ascend inside a group
    # a 1-D mask is not transposable: its column groups are reported, not silently compressed
    one_d = orc.nm_mask_1d(W, 2, 4)["mask"]
    assert orc.compress_2_4(W, one_d)["bad_groups"] > 0
