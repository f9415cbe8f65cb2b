// Packed bf16 front and back ends of the bit-parallel 2:4 search: two 4x4 blocks per thread.
//
// Input: the thread's 4 rows x 8 bf16 (block A = columns 0..3, block B = columns 4..7) as four
// 128-bit words.  The sixteen magnitudes of both blocks are interleaved into sixteen registers
// X[i][j] = (|a_ij|, |b_ij|) (16-bit lanes), so that every comparison the search needs -- entries
// sharing a row or a column -- is one 32-bit instruction deciding the same pair in both blocks.
// Two forms of that instruction exist:
//   arithmetic  X_q - X_p as a packed bf16 subtraction: the sign of either lane says "q lighter than
//               p" (a difference of two finite bf16 numbers never rounds to zero or across zero).  It
//               runs on the floating-point pipe, which the search leaves idle; it is used while every
//               magnitude seen is finite;
//   integer     X_q - X_p + 0x80008000 has bit 15 / bit 31 set iff q >= p (15-bit magnitudes: no
//               borrow crosses the lanes).  It orders any bit patterns, Inf and NaN included, and takes
//               over as soon as a warp has met one.
// The 48 decisions are then collected into the relation masks of tm_core24.cuh: a byte permute in
// sign-replicating mode turns every decision into a whole byte of equal bits, so a tree of bit
// selects with constant masks places them without shifts; decisions that arrive negated (the
// arithmetic form of ">=") are turned in the first level of the tree at no cost.
#pragma once
#include "tm_core24.cuh"

namespace tmask {

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}
// bits of a where m is set, bits of b elsewhere
__device__ __forceinline__ uint32_t bitsel(uint32_t a, uint32_t b, uint32_t m) {
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, 0xCA;" : "=r"(r) : "r"(m), "r"(a), "r"(b));   // m ? a : b
    return r;
}
// the same with a and / or b complemented first
template <bool NA, bool NB>
__device__ __forceinline__ uint32_t bitsel_n(uint32_t a, uint32_t b, uint32_t m) {
    constexpr int lut = (0xF0 & (NA ? 0x33 : 0xCC)) | (0x0F & (NB ? 0x55 : 0xAA));
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, %4;" : "=r"(r) : "r"(m), "r"(a), "r"(b), "n"(lut));
    return r;
}

struct PairKeys {
    uint32_t x[4][4];   // (|a_ij|, |b_ij|)
};

// |x| of both lanes on the floating-point pipe; bit-exact for every finite value and Inf (a NaN may
// come back with another payload, which the integer path below never sees)
__device__ __forceinline__ uint32_t abs_bf16x2(uint32_t a) {
    uint32_t r;
    asm("abs.bf16x2 %0, %1;" : "=r"(r) : "r"(a));
    return r;
}

// ARITH = false clears the sign bits with integer logic instead (exact for every bit pattern)
template <bool ARITH>
__device__ __forceinline__ void interleave_keys(const uint4 (&v)[4], PairKeys& k) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t a = prmt(v[i].x, v[i].z, 0x5410), b = prmt(v[i].x, v[i].z, 0x7632);
        const uint32_t c = prmt(v[i].y, v[i].w, 0x5410), d = prmt(v[i].y, v[i].w, 0x7632);
        if constexpr (ARITH) { k.x[i][0] = abs_bf16x2(a); k.x[i][1] = abs_bf16x2(b); k.x[i][2] = abs_bf16x2(c); k.x[i][3] = abs_bf16x2(d); }
        else { k.x[i][0] = a & 0x7FFF7FFFu; k.x[i][1] = b & 0x7FFF7FFFu; k.x[i][2] = c & 0x7FFF7FFFu; k.x[i][3] = d & 0x7FFF7FFFu; }
    }
}

// Decision words.  ARITH = false: the top bit of either 16-bit lane says "q heavier than p".
// ARITH = true: later_heavier() returns the negated decision (sign of X_q - X_p = "q lighter"),
// earlier_heavier() the plain one (sign of X_p - X_q = "p lighter").
__device__ __forceinline__ uint32_t sub_bf16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
// q > p in position: ties go to q
template <bool ARITH> __device__ __forceinline__ uint32_t later_heavier(uint32_t xq, uint32_t xp) {
    if constexpr (ARITH) return sub_bf16x2(xq, xp); else return xq - xp + 0x80008000u;
}
// q < p in position: a strictly larger magnitude is needed
template <bool ARITH> __device__ __forceinline__ uint32_t earlier_heavier(uint32_t xq, uint32_t xp) {
    if constexpr (ARITH) return sub_bf16x2(xp, xq); else return xq - xp + 0x7FFF7FFFu;
}

// byte 0/1 <- decisions of dx/dy for block A, byte 2/3 <- for block B; every byte is 0x00 or 0xFF
__device__ __forceinline__ uint32_t pick(uint32_t dx, uint32_t dy) { return prmt(dx, dy, 0xFBD9); }

// p[b] (bytes of equal bits) carries the decision destined for bit 7-b of every byte, negated where bit b of NEG is set.
// As an integer, a word of 0x00 / 0xFF bytes is 255 times the word of 0 / 1 bytes, so the weighted sum 128 p[0] + 64 p[1] +
// ... + p[7] is 255 times the gathered word (modulo 2^32, carries between bytes and all), and the factor leaves by a
// multiplication with the inverse of 255 modulo 2^32, -0x01010101: eight integer multiply-adds on the multiply-add pipe,
// which has room, instead of seven bit selects on the logic pipe, which has none.  The factors sit in constant memory so
// that the compiler keeps the multiply-adds.
__constant__ uint32_t g_gather_mul[2] = {2u, 0xFEFEFEFFu};
__device__ __forceinline__ uint32_t imad(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t r;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}
template <unsigned NEG>
__device__ __forceinline__ uint32_t gather8(const uint32_t (&p)[8]) {
    const uint32_t two = g_gather_mul[0];
    uint32_t acc = imad(p[0], two, p[1]);
#pragma unroll
    for (int b = 2; b < 8; ++b) acc = imad(acc, two, p[b]);
    acc *= g_gather_mul[1];
    uint32_t turn = 0;
#pragma unroll
    for (int b = 0; b < 8; ++b) turn |= ((NEG >> b) & 1u) ? (0x01010101u << (7 - b)) : 0u;
    return NEG ? acc ^ turn : acc;
}

template <bool ARITH>
__device__ __forceinline__ void relations_bf16(const PairKeys& k, Rel24& r) {
    const uint32_t (&x)[4][4] = k.x;
    uint32_t p[8];
    // hr1: bit 4i+j <- pair (j, j+1 mod 4) of row i; byte 0 holds rows 0,1 and byte 1 rows 2,3
#pragma unroll
    for (int b = 0; b < 8; ++b) {
        const int i = (7 - b) >> 2, j = (7 - b) & 3;
        const uint32_t dx = j < 3 ? later_heavier<ARITH>(x[i][j + 1], x[i][j]) : earlier_heavier<ARITH>(x[i][0], x[i][3]);
        const uint32_t dy = j < 3 ? later_heavier<ARITH>(x[i + 2][j + 1], x[i + 2][j]) : earlier_heavier<ARITH>(x[i + 2][0], x[i + 2][3]);
        p[b] = pick(dx, dy);
    }
    r.hr1 = gather8<ARITH ? 0xEEu : 0u>(p);                           // j = 3 (b = 0 and 4) compares with an earlier entry
    // hc1: bit 4i+j <- pair (i, i+1 mod 4) of column j
#pragma unroll
    for (int b = 0; b < 8; ++b) {
        const int i = (7 - b) >> 2, j = (7 - b) & 3;                  // i in {0,1}; the partner byte holds i+2
        const uint32_t dx = later_heavier<ARITH>(x[i + 1][j], x[i][j]);
        uint32_t dy;
        if (i + 2 < 3) dy = later_heavier<ARITH>(x[(i + 3) & 3][j], x[i + 2][j]);
        else { dy = earlier_heavier<ARITH>(x[0][j], x[3][j]); if constexpr (ARITH) dy ^= 0x80008000u; }    // same sense as dx
        p[b] = pick(dx, dy);
    }
    r.hc1 = gather8<ARITH ? 0xFFu : 0u>(p);
    // hr2 (columns 0,1 only): bits 4i+j, j in {0,1}
    {
        const uint32_t q7 = pick(later_heavier<ARITH>(x[0][2], x[0][0]), later_heavier<ARITH>(x[2][2], x[2][0]));
        const uint32_t q6 = pick(later_heavier<ARITH>(x[0][3], x[0][1]), later_heavier<ARITH>(x[2][3], x[2][1]));
        const uint32_t q3 = pick(later_heavier<ARITH>(x[1][2], x[1][0]), later_heavier<ARITH>(x[3][2], x[3][0]));
        const uint32_t q2 = pick(later_heavier<ARITH>(x[1][3], x[1][1]), later_heavier<ARITH>(x[3][3], x[3][1]));
        r.hr2 = bitsel(bitsel_n<ARITH, ARITH>(q7, q6, 0x01010101u), bitsel_n<ARITH, ARITH>(q3, q2, 0x10101010u), 0x0F0F0F0Fu);   // bits 2,3 of a nibble: don't care
    }
    // hc2 (rows 0,1 only): bit 4i+j, i in {0,1}; gathered as (row 0 -> byte 0, row 1 -> byte 1), then packed
    {
        uint32_t q[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) q[j] = pick(later_heavier<ARITH>(x[2][j], x[0][j]), later_heavier<ARITH>(x[3][j], x[1][j]));
        const uint32_t g = bitsel(bitsel_n<ARITH, ARITH>(q[0], q[1], 0x01010101u), bitsel_n<ARITH, ARITH>(q[2], q[3], 0x04040404u), 0x03030303u);
        r.hc2 = bitsel(g, g >> 4, 0x0F0F0F0Fu);
    }
    r.hr3 = 0; r.hc3 = 0;
    complete_relations(r);
}

// Some 16-bit lane of `worst` (a running maximum of magnitudes) is Inf or NaN.  The sign bits are
// ignored: the arithmetic |x| may hand a NaN back with its sign still set.
__device__ __forceinline__ bool nonfinite_bf16x2(uint32_t worst) { return (((worst & 0x7FFF7FFFu) + 0x00800080u) & 0x80008000u) != 0; }

// Keep flags as 16-bit lane masks, by table: entry e of the 256-entry table holds four words whose
// 16-bit lane j is all ones iff bit j of e is set.  The kernels build it in shared memory once per CTA.
constexpr int kLaneLutBytes = 256 * 16;
__device__ __forceinline__ void fill_lane_lut(uint4* lut, int tid, int nthreads) {
    for (int e = tid; e < 256; e += nthreads) {
        uint32_t w[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) w[c] = (((e >> (2 * c)) & 1) ? 0x0000FFFFu : 0u) | (((e >> (2 * c + 1)) & 1) ? 0xFFFF0000u : 0u);
        lut[e] = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

// Keep flags of a row of eight fp32 entries as eight words of 0 or 1: entry e of the 256-entry table (two 16-byte halves).
__device__ __forceinline__ void fill_keep_lut32(uint4* lut, int tid, int nthreads) {
    for (int e = tid; e < 256; e += nthreads) {
        lut[2 * e] = make_uint4(e & 1, (e >> 1) & 1, (e >> 2) & 1, (e >> 3) & 1);
        lut[2 * e + 1] = make_uint4((e >> 4) & 1, (e >> 5) & 1, (e >> 6) & 1, (e >> 7) & 1);
    }
}

// The four mask bytes of a pair mask, byte i = (row i of block B) << 4 | (row i of block A): the layout
// of the packed mask for the thread's eight columns.
__device__ __forceinline__ uint32_t mask_bytes_2_4(uint32_t kept) {
    const uint32_t t = kept & 0x0F0F0F0Fu, u = (kept >> 4) & 0x0F0F0F0Fu;      // rows 0,2 / rows 1,3 (A in bytes 0,1; B in bytes 2,3)
    return prmt(t | (t >> 12), u | (u >> 12), 0x5140);
}

}  // namespace tmask
