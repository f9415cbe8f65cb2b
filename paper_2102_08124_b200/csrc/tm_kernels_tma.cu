// Bandwidth kernels of the 2:4 search (TM_APPROX / TM_APPROX_COVER and, with the 90-pattern scorer in place of
// steps A to C, TM_EXACT; M = 4).
//
// Every warp runs its own software pipeline over work items (4 rows x 512 columns of one matrix: one
// block row, 128 blocks, in two halves of 256 columns) -- a contiguous range for the full search,
// every n-th item for the variants that only wait for memory:
//   1. lane 0 keeps the bulk-tensor (TMA) load of the next item in flight into the other of the warp's
//      two private shared-memory stages;
//   2. each lane reads its two 4x4 blocks of either block row with 128-bit shared loads and runs steps
//      A and B of the search bit-parallel in registers (tm_core24.cuh); the rounds of step B are
//      warp-uniform (a vote decides whether any lane still has candidates); the two halves give
//      the scheduler two independent instruction streams;
//   3. the blocks that need step C (about one in six) are queued in shared memory and fixed by as
//      many lanes at once as there are queued blocks, each reading the six magnitudes it must compare
//      straight from the stage;
//   4. the lanes write the masked weights back into the stage, lane 0 sends it out with one TMA store,
//      mask bytes meet in shared memory and leave as whole 32-bit words.
// An item that reaches past the last column (or, for the 1-D pruning, past the last row) is zero-filled by
// the copy on the way in and clipped on the way out, and its surplus mask words are not written.  Row segments of 1 KB (bf16) or 2 KB (fp32) keep
// the DRAM pages busier than narrower, taller items of the same size.
// Apart from one barrier after the lane-mask table is built, no CTA-wide synchronisation exists; every
// wait is bounded.
#include "tm_core24.cuh"
#include "tm_launch.h"
#include "tm_pair_bf16.cuh"
#include "tm_solvers.cuh"
#include "tm_tma.cuh"
#include "tm_tma_items.cuh"

#include <cstring>
#include <type_traits>

namespace tmask {

namespace {

constexpr int kItemRows = 4;               // one block row per item
constexpr int kHalves = 2;                 // processed as two halves of 256 columns: a lane owns two adjacent blocks of either
constexpr int kItemCols = 512;
constexpr int kHalfCols = kItemCols / kHalves;

// Warps per CTA (one CTA per SM) and stages per warp.  The full search is bound by integer issue and wants many
// warps: for bf16, 24 warps at 80 registers per thread fill the shared memory with two stages each (a deeper ring
// with fewer warps measured no faster).  Algorithm 1 alone and the 1-D pruning only wait for memory, and the memory
// system is at its best with about 96 KB of stages per SM: 12 warps for bf16 (0.387 ms on the 12288 x 49152 matrix
// against 0.418 / 0.427 / 0.449 ms with 10 / 14 / 16 warps), 6 for fp32.
template <int DT, int METHOD> struct Geometry {
    static constexpr int kElem = DT == kF32 ? 4 : 2;
    static constexpr bool kHeavy = METHOD == kMethodApprox || METHOD == kMethodRowsAbsorb || METHOD == kMethodExact;      // bound by arithmetic, not by memory
    // the exact scorer wants registers: 20 warps (96 registers a thread) measured best for bf16 (1.12 ms on the 12288 x 49152
    // matrix against 1.16 / 1.20 ms with 16 / 12 warps)
    static constexpr int kWarps = METHOD == kMethodExact ? (DT == kF32 ? 12 : 20) : (kHeavy ? (DT == kF32 ? 12 : 24) : (DT == kF32 ? 6 : 12));
    static constexpr int kStages = 2;
    static constexpr int kRowPitch = kItemCols * kElem;        // bytes between rows inside a stage
    static constexpr int kHalfBytes = kHalfCols * kElem;       // from the first half of a row to the second
    static constexpr int kStageBytes = kItemRows * kRowPitch;
    // exact search: one bit per item of the warp, set when the item is set aside for the out-of-line scorer after the loop
    static constexpr int kAsideBytes = METHOD == kMethodExact ? 2048 : 0;
    static constexpr int kAsideItems = kAsideBytes * 8;
    // stages | mask bytes [half][4][32] | kept [2][32] | queue [128] | barriers | set-aside bits
    static constexpr int kWarpBytes = kStages * kStageBytes + 256 + 256 + 128 + 128 + kAsideBytes;
    static constexpr int kSmemBytes = kWarps * kWarpBytes + (DT == kBF16 ? kLaneLutBytes : 0);
    static_assert(kSmemBytes <= 232448, "at most 227 KB of shared memory per CTA");
    static_assert(kWarpBytes % 128 == 0, "stages stay 128-byte aligned");
};

// ------------------------------------------------------------------------------------------
// per-dtype front end: relation masks of the lane's two blocks; largest magnitude seen
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t max_u16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.u16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// NZ: also return the pair mask of the non-zero entries (for the pattern-violation count)
template <int DT, bool NZ>
__device__ __forceinline__ void front_end(const unsigned char* stage, int lane, Rel24& rel, uint32_t& worst, uint32_t& nonzero) {
    constexpr int kPitch = kItemCols * (DT == kF32 ? 4 : 2);
    if constexpr (DT == kBF16) {
        uint4 v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] = *reinterpret_cast<const uint4*>(stage + i * kPitch + lane * 16);
        PairKeys pk;
        interleave_keys<true>(v, pk);
        // Inf / NaN watch.  The OR of the sixteen words can only show an all-ones exponent where some magnitude has the top
        // exponent bit set (|w| >= 2): for ordinary weights this cheap test settles it; otherwise the packed maximum
        // decides exactly.  `worst` stays as it is once it holds an Inf or NaN, so the warp keeps to the integer form.
        uint32_t any_bits = worst;
#pragma unroll
        for (int i = 0; i < 4; ++i) any_bits |= (pk.x[i][0] | pk.x[i][1]) | (pk.x[i][2] | pk.x[i][3]);
        bool integer_form = false;
        if (__any_sync(0xFFFFFFFFu, nonfinite_bf16x2(any_bits))) {
            uint32_t m[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) m[i] = max_u16x2(max_u16x2(pk.x[i][0], pk.x[i][1]), max_u16x2(pk.x[i][2], pk.x[i][3]));
            worst = max_u16x2(worst, max_u16x2(max_u16x2(m[0], m[1]), max_u16x2(m[2], m[3])));
            integer_form = __any_sync(0xFFFFFFFFu, nonfinite_bf16x2(worst));
        }
        if (integer_form) {                                            // Inf or NaN met: integer keys, bit-pattern order
            interleave_keys<false>(v, pk);
            relations_bf16<false>(pk, rel);
        }
        else relations_bf16<true>(pk, rel);
        if constexpr (NZ) {                    // x + 0x7FFF sets the top bit of a 15-bit magnitude iff x != 0 (a NaN kept its sign: still set)
            uint32_t p[8];
#pragma unroll
            for (int b = 0; b < 8; ++b) {
                const int i = (7 - b) >> 2, j = (7 - b) & 3;
                p[b] = pick((pk.x[i][j] & 0x7FFF7FFFu) + 0x7FFF7FFFu, (pk.x[i + 2][j] & 0x7FFF7FFFu) + 0x7FFF7FFFu);
            }
            nonzero = gather8<0u>(p);
        }
    } else {
        uint32_t ka[16], kb[16];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint4 a = *reinterpret_cast<const uint4*>(stage + i * kPitch + lane * 32);
            const uint4 b = *reinterpret_cast<const uint4*>(stage + i * kPitch + lane * 32 + 16);
            ka[4 * i] = a.x & 0x7FFFFFFFu; ka[4 * i + 1] = a.y & 0x7FFFFFFFu; ka[4 * i + 2] = a.z & 0x7FFFFFFFu; ka[4 * i + 3] = a.w & 0x7FFFFFFFu;
            kb[4 * i] = b.x & 0x7FFFFFFFu; kb[4 * i + 1] = b.y & 0x7FFFFFFFu; kb[4 * i + 2] = b.z & 0x7FFFFFFFu; kb[4 * i + 3] = b.w & 0x7FFFFFFFu;
        }
        rel = Rel24{0, 0, 0, 0, 0, 0};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t (&k)[16] = h ? kb : ka;
            const int shift = 16 * h;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t a = k[4 * i], b = k[4 * i + 1], c = k[4 * i + 2], d = k[4 * i + 3];
                rel.hr1 |= ((b >= a ? 1u : 0u) | (c >= b ? 2u : 0u) | (d >= c ? 4u : 0u) | (a > d ? 8u : 0u)) << (4 * i + shift);
                rel.hr2 |= ((c >= a ? 1u : 0u) | (d >= b ? 2u : 0u)) << (4 * i + shift);
                const uint32_t e = k[i], f = k[4 + i], g = k[8 + i], hh = k[12 + i];
                rel.hc1 |= ((f >= e ? 0x1u : 0u) | (g >= f ? 0x10u : 0u) | (hh >= g ? 0x100u : 0u) | (e > hh ? 0x1000u : 0u)) << (i + shift);
                rel.hc2 |= ((g >= e ? 0x1u : 0u) | (hh >= f ? 0x10u : 0u)) << (i + shift);
            }
        }
        complete_relations(rel);
        {   // Inf / NaN watch (for the status flag): the OR of the magnitudes shows an all-ones exponent only if some
            // |w| >= 2; the exact maximum is taken only then
            uint32_t any_bits = 0;
#pragma unroll
            for (int p = 0; p < 16; ++p) any_bits |= ka[p] | kb[p];
            if (any_bits >= 0x7F800000u) {
#pragma unroll
                for (int p = 0; p < 16; ++p) worst = max(worst, max(ka[p], kb[p]));
            }
        }
        if constexpr (NZ) {
            nonzero = 0;
#pragma unroll
            for (int p = 0; p < 16; ++p) nonzero |= (ka[p] ? 1u : 0u) << p | (kb[p] ? 1u : 0u) << (16 + p);
        }
    }
}

// Step C on a block whose magnitudes sit in shared memory (natural layout): entry p = 4i + j lies i rows and j elements on.
template <int DT>
__device__ __forceinline__ bool swap_apply_smem(const unsigned char* blk, uint32_t& kept16) {
    constexpr int kElemBytes = DT == kF32 ? 4 : 2;
    constexpr int kRowStep = kItemCols * kElemBytes / 4 - kElemBytes;      // offset(p) = p * elem + (p & 12) * kRowStep
    return swap_apply_2_4<DT == kBF16>(kept16, [blk](int p) -> uint32_t {
        const unsigned char* at = blk + p * kElemBytes + (p & 12) * kRowStep;
        if constexpr (DT == kBF16) return *reinterpret_cast<const unsigned short*>(at) & 0x7FFFu;
        else return *reinterpret_cast<const uint32_t*>(at) & 0x7FFFFFFFu;
    });
}

// Exact search, after the item loop: the items that were set aside because some block of theirs does not fit the first tier
// of the scorer (bit `it` of `aside` for the warp's item number `it`; the warp's items start at `first`).  Nothing of such an
// item has been written.  They are few, so they go the plain way: every lane reads its four blocks of the item from the
// matrix, scores them with exact_2_4_any() -- every tier, out of line -- and stores masked weights and mask words itself; the
// warp's sum goes on top of the partial it has already stored for the item's matrix.
template <int DT>
static __device__ __noinline__ void exact_aside_pass(const TmaEntry* tab, int count, long long first, int n_items, const uint32_t* aside,
                                                      double* partials, long long pstride, long long pbase) {
    constexpr int kWords = DT == kF32 ? 4 : 2;                     // 32-bit words of a block's row
    const int lane = threadIdx.x & 31;
    const int words = ((n_items < Geometry<DT, kMethodExact>::kAsideItems ? n_items : Geometry<DT, kMethodExact>::kAsideItems) + 31) >> 5;
    for (int w = 0; w < words; ++w) {
        uint32_t bits = aside[w];                                  // the same word for every lane
        while (bits) {
            const int it = w * 32 + __ffs((int)bits) - 1;
            bits &= bits - 1;
            Cursor c;
            c.seek(tab, count, first + it);
            const DevProblem& P = tab[c.k].p;
            const long long r0 = (long long)c.bi * kItemRows;
            const size_t pitch = (size_t)P.ld * (DT == kF32 ? 4 : 2);
            float sum = 0.f;
            for (int h = 0; h < kHalves; ++h) {
                const long long c0 = (long long)c.cj * kItemCols + h * kHalfCols + lane * 8;
                uint32_t nib[4] = {0, 0, 0, 0};                    // row i: block A's keep nibble, block B's above it
                for (int b = 0; b < 2; ++b) {
                    const long long cb = c0 + 4 * b;
                    const bool present = cb < P.cols;              // cols % 4 == 0: a block is inside or outside as a whole
                    uint32_t raw[4][kWords], u[16];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const unsigned char* src = static_cast<const unsigned char*>(P.W) + (size_t)(r0 + i) * pitch + (size_t)cb * (DT == kF32 ? 4 : 2);
                        if constexpr (DT == kF32) {
                            const uint4 v = present ? *reinterpret_cast<const uint4*>(src) : make_uint4(0, 0, 0, 0);
                            raw[i][0] = v.x; raw[i][1] = v.y; raw[i][2] = v.z; raw[i][3] = v.w;
#pragma unroll
                            for (int j = 0; j < 4; ++j) u[4 * i + j] = raw[i][j] & 0x7FFFFFFFu;
                        } else {
                            const uint2 v = present ? *reinterpret_cast<const uint2*>(src) : make_uint2(0, 0);
                            raw[i][0] = v.x; raw[i][1] = v.y;
                            u[4 * i] = (v.x << 16) & 0x7FFFFFFFu; u[4 * i + 1] = v.x & 0x7FFF0000u;
                            u[4 * i + 2] = (v.y << 16) & 0x7FFFFFFFu; u[4 * i + 3] = v.y & 0x7FFF0000u;
                        }
                    }
                    uint32_t code = exact_2_4_any(u, DT == kBF16 ? 16 : 0);      // all 32 lanes call
                    if (!present) code = 0;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t n = (code >> (4 * i)) & 15u;
                        nib[i] |= n << (4 * b);
#pragma unroll
                        for (int j = 0; j < 4; ++j) sum += ((n >> j) & 1u) ? __uint_as_float(u[4 * i + j]) : 0.f;
                        if (P.masked && present) {
                            unsigned char* dst = static_cast<unsigned char*>(P.masked) + (size_t)(r0 + i) * pitch + (size_t)cb * (DT == kF32 ? 4 : 2);
                            if constexpr (DT == kF32) {
                                *reinterpret_cast<uint4*>(dst) = make_uint4((n & 1u) ? raw[i][0] : 0u, (n & 2u) ? raw[i][1] : 0u, (n & 4u) ? raw[i][2] : 0u, (n & 8u) ? raw[i][3] : 0u);
                            } else {
                                const uint32_t m0 = ((n & 1u) ? 0x0000FFFFu : 0u) | ((n & 2u) ? 0xFFFF0000u : 0u);
                                const uint32_t m1 = ((n & 4u) ? 0x0000FFFFu : 0u) | ((n & 8u) ? 0xFFFF0000u : 0u);
                                *reinterpret_cast<uint2*>(dst) = make_uint2(raw[i][0] & m0, raw[i][1] & m1);
                            }
                        }
                    }
                }
                // four lanes share a mask word
                const long long word = c0 >> 5;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint32_t wbits = nib[i] << (8 * (lane & 3));
                    wbits |= __shfl_xor_sync(0xFFFFFFFFu, wbits, 1);
                    wbits |= __shfl_xor_sync(0xFFFFFFFFu, wbits, 2);
                    if ((lane & 3) == 0 && word < P.wpr) P.mask[(r0 + i) * P.wpr + word] = wbits;
                }
            }
            double t = (double)sum;
            for (int o = 16; o; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
            if (lane == 0) partials[(long long)c.k * pstride + pbase] += t;
        }
    }
}

// Masked weights back into the stage, mask bytes, objective contribution of the lane's two blocks.
template <int DT, bool HAS_OUT>
__device__ __forceinline__ float back_end(unsigned char* stage, unsigned char* mrow /* [4][32] */, const uint4* lut, int lane, uint32_t kept) {
    constexpr int kPitch = kItemCols * (DT == kF32 ? 4 : 2);
    float s4 = 0.f;
    const uint32_t mb4 = mask_bytes_2_4(kept);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t mb = i == 0 ? (mb4 & 0xFFu) : prmt(mb4, 0u, 0x4440 + i);
        if constexpr (DT == kBF16) {
            const uint4 r = *reinterpret_cast<const uint4*>(stage + i * kPitch + lane * 16);
            const uint4 mm = lut[mb];
            const uint32_t raw[4] = {r.x, r.y, r.z, r.w}, m[4] = {mm.x, mm.y, mm.z, mm.w};
            uint32_t o[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                o[q] = raw[q] & m[q];
                const uint32_t ab = abs_bf16x2(o[q]);
                unsigned short lo, hi;
                asm("mov.b32 {%0,%1}, %2;" : "=h"(lo), "=h"(hi) : "r"(ab));
                asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(s4) : "h"(lo));        // fp32 accumulator + bf16 addend
                asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(s4) : "h"(hi));
            }
            if constexpr (HAS_OUT) *reinterpret_cast<uint4*>(stage + i * kPitch + lane * 16) = make_uint4(o[0], o[1], o[2], o[3]);
        } else {
            const uint4 ra = *reinterpret_cast<const uint4*>(stage + i * kPitch + lane * 32);
            const uint4 rb = *reinterpret_cast<const uint4*>(stage + i * kPitch + lane * 32 + 16);
            const uint32_t raw[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
            uint32_t o[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                o[q] = ((mb >> q) & 1u) ? raw[q] : 0u;
                s4 += fabsf(__uint_as_float(o[q]));
            }
            if constexpr (HAS_OUT) {
                *reinterpret_cast<uint4*>(stage + i * kPitch + lane * 32) = make_uint4(o[0], o[1], o[2], o[3]);
                *reinterpret_cast<uint4*>(stage + i * kPitch + lane * 32 + 16) = make_uint4(o[4], o[5], o[6], o[7]);
            }
        }
        mrow[i * 32 + lane] = (unsigned char)mb;
    }
    return s4;
}

// Back end of the 1-D pruning with mean absorption (Section 5): every kept weight of a group of four receives
// the mean of the group's pruned weights -- their sum in position order in fp64, divided by their number, added
// in fp64, rounded once to fp32 and from there (bf16 tensors) to bf16, nearest even.  The row rule keeps exactly
// n_keep entries of every group, so the divisor is the same for the whole call.  The objective stays the sum of
// the kept magnitudes before absorption.
template <int DT>
__device__ __forceinline__ float back_end_absorb(unsigned char* stage, unsigned char* mrow /* [4][32] */, const uint4* lut, int lane, uint32_t kept, int n_keep) {
    constexpr int kPitch = kItemCols * (DT == kF32 ? 4 : 2);
    float s4 = 0.f;
    const uint32_t mb4 = mask_bytes_2_4(kept);
    const double pruned = (double)(4 - n_keep);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t mb = (mb4 >> (8 * i)) & 0xFFu;
        uint32_t raw[8];
        uint4 r = make_uint4(0, 0, 0, 0);
        if constexpr (DT == kBF16) {
            r = *reinterpret_cast<const uint4*>(stage + i * kPitch + lane * 16);
            raw[0] = r.x << 16; raw[1] = r.x & 0xFFFF0000u; raw[2] = r.y << 16; raw[3] = r.y & 0xFFFF0000u;
            raw[4] = r.z << 16; raw[5] = r.z & 0xFFFF0000u; raw[6] = r.w << 16; raw[7] = r.w & 0xFFFF0000u;
        } else {
            const uint4 ra = *reinterpret_cast<const uint4*>(stage + i * kPitch + lane * 32);
            const uint4 rb = *reinterpret_cast<const uint4*>(stage + i * kPitch + lane * 32 + 16);
            raw[0] = ra.x; raw[1] = ra.y; raw[2] = ra.z; raw[3] = ra.w; raw[4] = rb.x; raw[5] = rb.y; raw[6] = rb.z; raw[7] = rb.w;
        }
        uint32_t o[8];
        float v8[8];
#pragma unroll
        for (int g = 0; g < 2; ++g) {                    // block A, block B: one group of four each
            double psum = 0.0;
#pragma unroll
            for (int j = 0; j < 4; ++j) psum += ((mb >> (4 * g + j)) & 1u) ? 0.0 : (double)__uint_as_float(raw[4 * g + j]);
            // a block past the last column (kept = 0 everywhere) is all zeros: its mean is 0 whatever the divisor
            const double mu = n_keep == 2 ? psum * 0.5 : (n_keep == 3 ? psum : __ddiv_rn(psum, pruned));
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const bool k = (mb >> (4 * g + j)) & 1u;
                const float v = (float)((double)__uint_as_float(raw[4 * g + j]) + mu);
                v8[4 * g + j] = v;
                if constexpr (DT == kF32) {
                    o[4 * g + j] = k ? __float_as_uint(v) : 0u;
                    s4 += k ? fabsf(__uint_as_float(raw[4 * g + j])) : 0.f;
                }
            }
        }
        if constexpr (DT == kBF16) {
            // pairs rounded to bf16 by the packed conversion (nearest even); the rounding rule of this library lets a NaN keep
            // its payload bits, so a row that holds one takes the integer form; pruned entries are cleared by the lane masks
            const uint4 mm = lut[mb];
            const uint32_t rw[4] = {r.x, r.y, r.z, r.w}, m4[4] = {mm.x, mm.y, mm.z, mm.w};
            const float chk = ((v8[0] + v8[1]) + (v8[2] + v8[3])) + ((v8[4] + v8[5]) + (v8[6] + v8[7]));
            uint32_t pk[4];
            if (chk == chk) {
#pragma unroll
                for (int c = 0; c < 4; ++c) asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(pk[c]) : "f"(v8[2 * c + 1]), "f"(v8[2 * c]));
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c) pk[c] = float_to_bf16_bits(v8[2 * c]) | (float_to_bf16_bits(v8[2 * c + 1]) << 16);
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                pk[c] &= m4[c];
                const uint32_t ab = abs_bf16x2(rw[c] & m4[c]);
                unsigned short lo, hi;
                asm("mov.b32 {%0,%1}, %2;" : "=h"(lo), "=h"(hi) : "r"(ab));
                asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(s4) : "h"(lo));
                asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(s4) : "h"(hi));
            }
            *reinterpret_cast<uint4*>(stage + i * kPitch + lane * 16) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        } else {
            *reinterpret_cast<uint4*>(stage + i * kPitch + lane * 32) = make_uint4(o[0], o[1], o[2], o[3]);
            *reinterpret_cast<uint4*>(stage + i * kPitch + lane * 32 + 16) = make_uint4(o[4], o[5], o[6], o[7]);
        }
        mrow[i * 32 + lane] = (unsigned char)mb;
    }
    return s4;
}

template <int DT, int METHOD, bool HAS_OUT>
__global__ void __launch_bounds__(Geometry<DT, METHOD>::kWarps * 32, 1)
tma24_kernel(const __grid_constant__ TmaEntry single, const TmaEntry* __restrict__ table, int count, long long total_items,
             double* __restrict__ partials, int* __restrict__ status_out, int n_keep, unsigned long long* __restrict__ vpartials,
             unsigned int* __restrict__ done) {
    using G = Geometry<DT, METHOD>;
    constexpr bool kRows = METHOD == kMethodRows || METHOD == kMethodRowsAbsorb;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned char* stages = smem_raw + (size_t)warp * G::kWarpBytes;
    unsigned char* mbytes = stages + G::kStages * G::kStageBytes;
    uint32_t* kbuf = reinterpret_cast<uint32_t*>(mbytes + 256);
    unsigned char* queue = reinterpret_cast<unsigned char*>(kbuf + kHalves * 32);
    uint64_t* bars = reinterpret_cast<uint64_t*>(queue + 128);
    uint32_t* aside = reinterpret_cast<uint32_t*>(queue + 256);            // exact search only
    if constexpr (METHOD == kMethodExact) {
        for (int w = lane; w < G::kAsideBytes / 4; w += 32) aside[w] = 0u;
    }
    uint4* lut = reinterpret_cast<uint4*>(smem_raw + (size_t)G::kWarps * G::kWarpBytes);
    if constexpr (DT == kBF16) {           // the only CTA-wide step: the lane-mask table
        fill_lane_lut(lut, threadIdx.x, G::kWarps * 32);
        __syncthreads();
    }

    const long long gw = (long long)blockIdx.x * G::kWarps + warp, nwarps = (long long)gridDim.x * G::kWarps;
    // where this warp's objective partial for matrix k goes: k * pstride + pbase (a launch over several matrices that reduces
    // its own objectives packs them: slot = the warp's place in the deal + k, see finish_objectives_ranged)
    const bool ranged = done != nullptr && count > 1;
    const long long pstride = ranged ? 1 : nwarps, pbase = ranged ? (long long)warp * gridDim.x + blockIdx.x : gw;
    // A fixed deal of the items, so the objective's partial sums are reproducible.  Where the kernel waits for memory
    // (Algorithm 1 alone, the 1-D pruning) the warps take the items round-robin -- first, first + nwarps, ... -- so that the
    // whole grid works on one dense window of the matrix (3 % faster there); the full search, which also waits for the
    // integer pipe, is indifferent to the order and 2 % faster with the plain cursor of a contiguous range.
    constexpr bool kRoundRobin = !G::kHeavy;
    int n_items;
    long long first;
    if constexpr (kRoundRobin) {       // the same order as even_share(): surplus items fall on different SMs
        first = (long long)warp * gridDim.x + blockIdx.x;
        n_items = first < total_items ? (int)((total_items - first + nwarps - 1) / nwarps) : 0;
    } else {
        first = even_share(total_items, G::kWarps, n_items);
    }
    const TmaEntry* tab = table ? table : &single;

    if (lane == 0) {
        for (int s = 0; s < G::kStages; ++s) mbar_init(&bars[s], 1);
        fence_mbar_init();
    }
    __syncwarp();

    typename std::conditional<kRoundRobin, StrideCursor, Cursor>::type ld, cur;      // next item to request / item in process
    if constexpr (kRoundRobin) ld.seek(tab, count, first, (int)nwarps); else ld.seek(tab, count, first);
    cur = ld;
    int loaded = 0;
    auto issue_next = [&](int s) {         // all lanes track the cursor, lane 0 issues the copy
        if (lane == 0) {
            mbar_expect_tx(&bars[s], G::kStageBytes);
            tma_load_2d(stages + s * G::kStageBytes, &tab[ld.k].in, ld.cj * kTmaBoxUnits, ld.bi * kItemRows, &bars[s]);
        }
        ld.advance(tab, count);
        ++loaded;
    };
    for (int g = 0; g < G::kStages - 1 && loaded < n_items; ++g) issue_next(g);

    int status = 0, acc_k = -1;
    float facc = 0.f; double acc = 0.0;
    uint32_t worst = 0;                                                  // largest magnitude pattern seen (per 16-bit lane for bf16)
    const uint32_t lt = (1u << lane) - 1u;
    bool alive = true;
    // the matrix in process: the fields every item needs
    int p_cols = 0, p_wpr = 0, p_rows = 0;
    uint32_t* p_mask = nullptr;
    // an item's mask words: 4 rows x 16 words, lane -> word (lane & 15) of rows (lane >> 4) and (lane >> 4) + 2
    const int mw = lane & 15, mr = lane >> 4;
    const unsigned char* msrc = mbytes + (mw >> 3) * 128 + mr * 32 + (mw & 7) * 4;
    unsigned long long viol = 0;                                         // kMethodRows: non-zero entries pruned by this lane

    // The item loop.  The exact search on bf16 has it twice: with the 32-bit first tier of the scorer and, for a warp whose
    // items leave that tier often (ordinary continuous data does, quantised data never), with the 64-bit one; a warp
    // starts with the first and may change over once, between two items (the pipeline's state is the captured variables).
    constexpr bool kTwoTiers = METHOD == kMethodExact && DT == kBF16;
    auto run_items = [&](auto wide_mode, int it_begin) -> int {
    constexpr bool kWideTier = decltype(wide_mode)::value;
    int it = it_begin, recent_aside = 0;
    for (; it < n_items && alive; ++it) {
        const int s = it % G::kStages;
        const uint32_t parity = (uint32_t)((it / G::kStages) & 1);
        unsigned char* stage = stages + s * G::kStageBytes;
        // a copy that never landed: stop before anything is computed on, or stored from, the unfilled stage
        if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(&bars[s], parity))) { status |= kDevInternal; alive = false; break; }
        int qn = 0;
        bool redo = false;                                      // exact search: some block of the item is outside the first tier (warp-uniform)
        if (cur.k != acc_k) {                                   // a new matrix starts: flush the objective partial
            if (acc_k >= 0) {
                acc += (double)facc;
                for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
                if (lane == 0) partials[(long long)acc_k * pstride + pbase] = acc;
            }
            acc = 0.0; facc = 0.f; acc_k = cur.k;
            const DevProblem& P = tab[cur.k].p;
            p_cols = (int)P.cols; p_wpr = P.wpr; p_rows = (int)P.rows; p_mask = P.mask;
        }
        // does the item lie inside the matrix? (warp-uniform; otherwise the copy zero-filled the rest)
        const bool inside_cols = cur.cj < p_cols / kItemCols, inside = inside_cols && cur.bi < p_rows / kItemRows;
        // ---- steps A and B on both halves ---------------------------------------------------------
#pragma unroll
        for (int h = 0; h < kHalves; ++h) {
            Rel24 rel;
            uint32_t nonzero = 0;
            uint32_t k;
            if constexpr (METHOD == kMethodExact) {
                // the optimum of Eq. 1 for either of the lane's two blocks: all 90 patterns, exact integer sums
                k = 0;
#pragma unroll
                for (int b = 0; b < 2; ++b) {
                    const unsigned char* blk = stage + h * G::kHalfBytes + lane * (8 * G::kElem) + b * (4 * G::kElem);
                    uint32_t u[16];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        if constexpr (DT == kBF16) {
                            const uint2 v = *reinterpret_cast<const uint2*>(blk + i * G::kRowPitch);
                            u[4 * i] = (v.x << 16) & 0x7FFFFFFFu; u[4 * i + 1] = v.x & 0x7FFF0000u;
                            u[4 * i + 2] = (v.y << 16) & 0x7FFFFFFFu; u[4 * i + 3] = v.y & 0x7FFF0000u;
                        } else {
                            const uint4 v = *reinterpret_cast<const uint4*>(blk + i * G::kRowPitch);
                            u[4 * i] = v.x & 0x7FFFFFFFu; u[4 * i + 1] = v.y & 0x7FFFFFFFu; u[4 * i + 2] = v.z & 0x7FFFFFFFu; u[4 * i + 3] = v.w & 0x7FFFFFFFu;
                        }
                    }
                    bool bad = false;
#pragma unroll
                    for (int p = 0; p < 16; ++p) bad |= (u[p] >> 23) == 0xFFu;
                    if (bad) status |= kDevNonFinite;
                    uint64_t code = 0;
                    if (!redo) redo = !exact_2_4_first<DT == kBF16, kWideTier>(u, code);       // once set, the whole item is scored again after the loop
                    k |= (uint32_t)code << (16 * b);
                }
            } else {
            front_end<DT, kRows>(stage + h * G::kHalfBytes, lane, rel, worst, nonzero);
            if constexpr (kRows) {
                // N of 4 along rows: kept iff fewer than N entries of the row are heavier
                const int nk = n_keep;
                k = nk == 2 ? ~maj3(rel.hr1, rel.hr2, rel.hr3) : (nk == 1 ? ~(rel.hr1 | rel.hr2 | rel.hr3) : ~(rel.hr1 & rel.hr2 & rel.hr3));
                const int c0 = cur.cj * kItemCols + h * kHalfCols + lane * 8;
                const uint32_t in_cols = c0 >= p_cols ? 0u : (c0 + 4 >= p_cols ? 0xFFFFu : 0xFFFFFFFFu);
                viol += (unsigned)__popc(~k & nonzero & in_cols);
            } else {
                k = cover_2_4(rel);
            }
            }
            if constexpr (METHOD == kMethodApprox) {
                LineFill f = line_fill(k);
                uint32_t cand = open_candidates(k, f);
                // two full rounds are needed by every warp of ordinary data (some block of its 64 has candidates left after
                // the first): they run without asking; after them a block that still has candidates has, as a rule, one
#pragma unroll
                for (int round = 0; round < 2; ++round) {
                    k |= fill_accept(rel, k, cand);
                    f = line_fill(k);
                    cand = open_candidates(k, f);
                }
                if (__any_sync(0xFFFFFFFFu, cand != 0)) {
                    k |= lone_candidates(cand);
                    f = line_fill(k);
                    cand = open_candidates(k, f);
                    int rounds = 2;
                    while (__any_sync(0xFFFFFFFFu, cand != 0)) {
                        if (++rounds > 4) { status |= kDevInternal; break; }    // a block lacks at most four entries
                        k |= fill_accept(rel, k, cand);
                        f = line_fill(k);
                        cand = open_candidates(k, f);
                    }
                }
                const uint32_t sb = short_blocks(f);
                {   // some block of the 64 needs step C in all but a few warps: no vote first
#pragma unroll
                    for (int b = 0; b < 2; ++b) {
                        const bool need = (sb >> b) & 1;
                        const uint32_t m = __ballot_sync(0xFFFFFFFFu, need);
                        if (need) queue[qn + __popc(m & lt)] = (unsigned char)((h << 6) | (b << 5) | lane);
                        qn += __popc(m);
                    }
                }
            }
            kbuf[h * 32 + lane] = k;
            if (h == 0 && loaded < n_items) {       // refill the stage of the previous item: its store was issued one item ago
                if constexpr (HAS_OUT) { if (lane == 0 && it > 0) tma_wait_read<0>(); }
                issue_next((s + G::kStages - 1) % G::kStages);
            }
        }
        __syncwarp();
        // ---- step C on the queued blocks ---------------------------------------------------------
        if constexpr (METHOD == kMethodApprox) {
            for (int q0 = 0; q0 < qn; q0 += 32) {
                if (q0 + lane < qn) {
                    const uint32_t e = queue[q0 + lane];
                    const int h = e >> 6, b = (e >> 5) & 1, ln = e & 31;
                    unsigned short* kh = reinterpret_cast<unsigned short*>(kbuf + h * 32 + ln) + b;
                    uint32_t k16 = *kh;
                    const unsigned char* blk = stage + h * G::kHalfBytes + ln * (8 * G::kElem) + b * (4 * G::kElem);
                    if (!swap_apply_smem<DT>(blk, k16)) status |= kDevInternal;
                    *kh = (unsigned short)k16;
                }
            }
            __syncwarp();
        }
        // ---- outputs ---------------------------------------------------------------------------
        if (METHOD == kMethodExact && redo) {
            // set aside: nothing of this item is written here (in place, its weights stay as they are); exact_aside_pass() does it
            if (it >= G::kAsideItems) status |= kDevInternal;              // the launcher refuses calls whose warps would get that many items
            else if (lane == 0) aside[it >> 5] |= 1u << (it & 31);
            ++recent_aside;
        } else {
        // blocks past the last column (zero-filled by the copy) contribute nothing
        uint32_t colmask[kHalves] = {0xFFFFFFFFu, 0xFFFFFFFFu};
        if (!inside_cols) {
#pragma unroll
            for (int h = 0; h < kHalves; ++h) {
                const int col0 = cur.cj * kItemCols + h * kHalfCols + lane * 8;
                colmask[h] = col0 >= p_cols ? 0u : (col0 + 4 >= p_cols ? 0xFFFFu : 0xFFFFFFFFu);
            }
        }
        if constexpr (METHOD == kMethodRowsAbsorb && HAS_OUT) {
#pragma unroll
            for (int h = 0; h < kHalves; ++h)
                facc += back_end_absorb<DT>(stage + h * G::kHalfBytes, mbytes + h * 128, lut, lane, kbuf[h * 32 + lane] & colmask[h], n_keep);
        } else {
#pragma unroll
            for (int h = 0; h < kHalves; ++h)
                facc += back_end<DT, HAS_OUT>(stage + h * G::kHalfBytes, mbytes + h * 128, lut, lane, kbuf[h * 32 + lane] & colmask[h]);
        }
        if constexpr (HAS_OUT) fence_proxy_async_smem();
        __syncwarp();
        if constexpr (HAS_OUT) {
            if (lane == 0) { tma_store_2d(&tab[cur.k].out, cur.cj * kTmaBoxUnits, cur.bi * kItemRows, stage); tma_commit(); }
        }
        {   // mask words: 64 bytes per row
            const uint32_t w0 = *reinterpret_cast<const uint32_t*>(msrc), w1 = *reinterpret_cast<const uint32_t*>(msrc + 64);
            const int word = cur.cj * (kItemCols / 32) + mw, row = cur.bi * kItemRows + mr;
            uint32_t* dst = p_mask + (long long)row * p_wpr + word;
            if (inside) { dst[0] = w0; dst[2 * (long long)p_wpr] = w1; }
            else if (word < p_wpr) {                                    // the 1-D pruning takes any number of rows
                if (row < p_rows) dst[0] = w0;
                if (row + 2 < p_rows) dst[2 * (long long)p_wpr] = w1;
            }
        }
        }
        cur.advance(tab, count);
        if ((it & 31) == 31) { acc += (double)facc; facc = 0.f; }           // keep the fp32 partial short
        __syncwarp();
        if constexpr (kTwoTiers && !kWideTier) {
            if (recent_aside >= 2) { ++it; break; }                         // two items set aside within a window of four: the wider tier from here on
            if (((it - it_begin) & 3) == 3) recent_aside = 0;
        }
    }
    return it;
    };
    {
        const int reached = run_items(std::false_type{}, 0);
        if constexpr (kTwoTiers) { if (reached < n_items && alive) run_items(std::true_type{}, reached); }
    }
    if (!alive && lane == 0) {
        // a copy never landed: give the copies still in flight a bounded chance to finish before the stages die
        for (int s = 0; s < G::kStages; ++s) { mbar_wait_bounded(&bars[s], 0, 1u << 14); mbar_wait_bounded(&bars[s], 1, 1u << 14); }
    }
    if (lane == 0) tma_wait_all<0>();
    if (acc_k >= 0 || (done && count == 1)) {  // a single-matrix launch that reduces its own objective wants a partial (a zero) from idle warps too
        acc += (double)facc;
        for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        if (lane == 0) partials[(long long)(acc_k >= 0 ? acc_k : 0) * pstride + pbase] = acc;
    }
    if constexpr (METHOD == kMethodExact) {
        __syncwarp();
        if (alive) exact_aside_pass<DT>(tab, count, first, n_items, aside, partials, pstride, pbase);
    }
    if constexpr (DT == kF32) { if (worst >= 0x7F800000u) status |= kDevNonFinite; }
    else { if (nonfinite_bf16x2(worst)) status |= kDevNonFinite; }
    for (int o = 16; o; o >>= 1) status |= __shfl_xor_sync(0xFFFFFFFFu, status, o);
    if (lane == 0 && status && status_out) atomicOr(status_out, status);
    if (done) {                                // the launch reduces its own objectives; the stages are idle by now
        const long long nw = (long long)gridDim.x * G::kWarps;
        if (count > 1) finish_objectives_ranged(done, partials, tab, count, total_items, nw, reinterpret_cast<double*>(smem_raw));
        else finish_objective(done, partials, nw, tab[0].p.objective, reinterpret_cast<double*>(smem_raw));
    }
    if constexpr (kRows) {
        for (int o = 16; o; o >>= 1) viol += __shfl_xor_sync(0xFFFFFFFFu, viol, o);
        if (lane == 0 && vpartials) vpartials[gw] = viol;
    }
}

// objective[k] = sum of the problem's partials in a fixed order (one CTA per problem)
__global__ void __launch_bounds__(256)
reduce_tma_kernel(const __grid_constant__ TmaEntry single, const TmaEntry* __restrict__ table, const double* __restrict__ partials, long long stride) {
    const DevProblem& P = table ? table[blockIdx.x].p : single.p;
    __shared__ double sm[256];
    double s = 0.0;
    for (long long i = threadIdx.x; i < stride; i += 256) s += partials[(long long)blockIdx.x * stride + i];
    sm[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o; o >>= 1) {
        if ((int)threadIdx.x < o) sm[threadIdx.x] += sm[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0 && P.objective) *P.objective = sm[0];
}

template <int DT, int METHOD, bool HAS_OUT>
cudaError_t launch_one(const TmaLaunch& a, const TmaEntry& single, const TmaEntry* table) {
    using G = Geometry<DT, METHOD>;
    const size_t smem = G::kSmemBytes;
    auto kern = tma24_kernel<DT, METHOD, HAS_OUT>;
    static PerDeviceOnce configured;       // per instantiation
    const cudaError_t e = configured.run([&] { return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); });
    if (e != cudaSuccess) return e;
    kern<<<a.ctas, G::kWarps * 32, smem, a.stream>>>(single, table, a.count, a.total_items, a.partials, a.status, a.n_keep, a.vpartials, a.done);
    return cudaGetLastError();
}

}  // namespace

size_t tma_entry_bytes() { return sizeof(TmaEntry); }
int tma_warps_per_cta(int dtype, int M, int method) {
    if (M == 8) return tma48_warps_per_cta(dtype, method);
    const bool heavy = method == kMethodApprox || method == kMethodRowsAbsorb;
    if (method == kMethodExact) return dtype == kF32 ? Geometry<kF32, kMethodExact>::kWarps : Geometry<kBF16, kMethodExact>::kWarps;
    if (dtype == kF32) return heavy ? Geometry<kF32, kMethodApprox>::kWarps : Geometry<kF32, kMethodCover>::kWarps;
    return heavy ? Geometry<kBF16, kMethodApprox>::kWarps : Geometry<kBF16, kMethodCover>::kWarps;
}

bool tma_eligible(const DevProblem& p, int N, int M, int method) {
    if (method == kMethodRows || method == kMethodRowsAbsorb) {
        // groups of four with or without the mean absorption, groups of eight without
        if (!((M == 4 && N >= 1 && N <= 3) || (M == 8 && N >= 1 && N <= 7 && method == kMethodRows))) return false;
    }
    else if (method == kMethodExact) { if (N != 2 || M != 4) return false; }
    else if (!((N == 2 && M == 4) || (N == 4 && M == 8)) || (method != kMethodApprox && method != kMethodCover)) return false;
    const size_t elem = p.dtype == kF32 ? 4 : 2;
    if ((uintptr_t)p.W % 16 || ((size_t)p.ld * elem) % 16) return false;
    if (p.masked && (uintptr_t)p.masked % 16) return false;
    if (p.rows >= (1ll << 31) || p.cols >= (1ll << 31) - kItemCols || (size_t)p.ld * elem >= (1ull << 40)) return false;
    if ((p.rows / M) * ((p.cols + kItemCols - 1) / kItemCols) >= (1ll << 30)) return false;
    return encode_fn() != nullptr;
}

// Fills `entries_host` (count TmaEntry records) for problems that all passed tma_eligible() and share a dtype; an item is
// one block row of 4 x 512 (M = 4) or 8 x 256 (M = 8; 8 x 128 where fp32 runs the split kernel) elements.
bool tma_build_entries(const DevProblem* probs, int count, void* entries_host, long long* total_items, int M, int method) {
    if (M == 8) return build_entries(probs, count, static_cast<TmaEntry*>(entries_host), total_items, 8, tma48_item_cols(count > 0 ? probs[0].dtype : kF32, method));
    return build_entries(probs, count, static_cast<TmaEntry*>(entries_host), total_items, kItemRows, kItemCols);
}

cudaError_t tma_reduce(const void* entries_host, const void* entries_dev, int count, const double* partials, long long stride, cudaStream_t stream) {
    const TmaEntry* host = static_cast<const TmaEntry*>(entries_host);
    reduce_tma_kernel<<<count, 256, 0, stream>>>(host[0], static_cast<const TmaEntry*>(entries_dev), partials, stride);
    return cudaGetLastError();
}

// All problems of one launch share dtype and the presence of masked_w_out (the caller groups them).
// With a counter word at hand (a_in.done) a single matrix, or several under a full search, is one launch: the search kernel
// reduces its own objectives.  Everything else: partials cleared, search, reduction kernel.
cudaError_t launch_tma(const TmaLaunch& a_in) {
    TmaLaunch a = a_in;
    const bool rows_method = a.method == kMethodRows || a.method == kMethodRowsAbsorb;
    // several matrices only where the warps hold contiguous item ranges (the full searches; Algorithm 1 alone deals round-robin)
    const bool contiguous = a.method == kMethodApprox || (a.method == kMethodExact && a.M == 4);
    if (!((a.count == 1 || contiguous) && a.total_items > 0 && !rows_method)) a.done = nullptr;
    if (a.M == 8) return launch_tma48(a);
    const int wpc = tma_warps_per_cta(a.dtype, 4, a.method);
    // the exact search keeps one bit per item of a warp (16 384 of them: more than 180 GB of weights on a full grid)
    if (a.method == kMethodExact && (a.total_items + (long long)a.ctas * wpc - 1) / ((long long)a.ctas * wpc) > Geometry<kBF16, kMethodExact>::kAsideItems)
        return cudaErrorInvalidValue;
    cudaError_t err = cudaSuccess;
    if (!a.done) err = cudaMemsetAsync(a.partials, 0, sizeof(double) * (size_t)a.count * (size_t)a.ctas * wpc, a.stream);
    if (err != cudaSuccess) return err;
    const TmaEntry* host = static_cast<const TmaEntry*>(a.entries_host);
    const TmaEntry* table = static_cast<const TmaEntry*>(a.entries_dev);   // nullptr when count == 1
    if (a.total_items > 0) {
#define TM_DISPATCH(DT, METHOD)                                                                                   \
    err = a.has_out ? launch_one<DT, METHOD, true>(a, host[0], table) : launch_one<DT, METHOD, false>(a, host[0], table)
        if (a.dtype == kF32) { if (a.method == kMethodExact) TM_DISPATCH(kF32, kMethodExact); else if (a.method == kMethodApprox) TM_DISPATCH(kF32, kMethodApprox); else if (a.method == kMethodRows) TM_DISPATCH(kF32, kMethodRows); else if (a.method == kMethodRowsAbsorb) TM_DISPATCH(kF32, kMethodRowsAbsorb); else TM_DISPATCH(kF32, kMethodCover); }
        else { if (a.method == kMethodExact) TM_DISPATCH(kBF16, kMethodExact); else if (a.method == kMethodApprox) TM_DISPATCH(kBF16, kMethodApprox); else if (a.method == kMethodRows) TM_DISPATCH(kBF16, kMethodRows); else if (a.method == kMethodRowsAbsorb) TM_DISPATCH(kBF16, kMethodRowsAbsorb); else TM_DISPATCH(kBF16, kMethodCover); }
#undef TM_DISPATCH
        if (err != cudaSuccess) return err;
    }
    if (rows_method) return cudaSuccess;       // the caller sums objective and violation partials together
    if (a.done) return cudaSuccess;            // the search kernel has written the objective
    reduce_tma_kernel<<<a.count, 256, 0, a.stream>>>(host[0], table, a.partials, (long long)a.ctas * wpc);
    return cudaGetLastError();
}

}  // namespace tmask
