// Packed bf16 front and back ends of the bit-parallel 2:4 search: two 4x4 blocks per thread.
//
// Input: the thread's 4 rows x 8 bf16 (block A = columns 0..3, block B = columns 4..7) as four
// 128-bit words.  The sixteen magnitudes of both blocks are interleaved into sixteen registers
// X[i][j] = (|a_ij|, |b_ij|) (16-bit lanes), so that every comparison the search needs -- entries
// sharing a row or a column -- is one 32-bit subtraction deciding the same pair in both blocks:
//   X_q - X_p + 0x80008000  has bit 15 / bit 31 set iff  q >= p  in block A / block B
// (15-bit magnitudes: no borrow crosses the lanes).  The 48 decisions are then collected into the
// relation masks of tm_core24.cuh: a byte permute in sign-replicating mode turns every decision into a
// whole byte of equal bits, so a tree of bit selects with constant masks places them without shifts.
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

struct PairKeys {
    uint32_t x[4][4];   // (|a_ij|, |b_ij|)
};

__device__ __forceinline__ void interleave_keys(const uint4 (&v)[4], PairKeys& k) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        k.x[i][0] = prmt(v[i].x, v[i].z, 0x5410) & 0x7FFF7FFFu;
        k.x[i][1] = prmt(v[i].x, v[i].z, 0x7632) & 0x7FFF7FFFu;
        k.x[i][2] = prmt(v[i].y, v[i].w, 0x5410) & 0x7FFF7FFFu;
        k.x[i][3] = prmt(v[i].y, v[i].w, 0x7632) & 0x7FFF7FFFu;
    }
}

// decision words: "q heavier than p" for positions q > p (ties go to the later position) ...
__device__ __forceinline__ uint32_t later_heavier(uint32_t xq, uint32_t xp) { return xq - xp + 0x80008000u; }
// ... and for q < p (strictly larger magnitude needed)
__device__ __forceinline__ uint32_t earlier_heavier(uint32_t xq, uint32_t xp) { return xq - xp + 0x7FFF7FFFu; }

// byte 0/1 <- decisions of dx/dy for block A, byte 2/3 <- for block B; every byte is 0x00 or 0xFF
__device__ __forceinline__ uint32_t pick(uint32_t dx, uint32_t dy) { return prmt(dx, dy, 0xFBD9); }

// p[b] (bytes of equal bits) carries the decisions destined for bit 7-b of every byte
__device__ __forceinline__ uint32_t gather8(const uint32_t (&p)[8]) {
    const uint32_t t01 = bitsel(p[0], p[1], 0x80808080u), t23 = bitsel(p[2], p[3], 0x20202020u);
    const uint32_t t45 = bitsel(p[4], p[5], 0x08080808u), t67 = bitsel(p[6], p[7], 0x02020202u);
    return bitsel(bitsel(t01, t23, 0xC0C0C0C0u), bitsel(t45, t67, 0x0C0C0C0Cu), 0xF0F0F0F0u);
}

__device__ __forceinline__ void relations_bf16(const PairKeys& k, Rel24& r) {
    const uint32_t (&x)[4][4] = k.x;
    uint32_t p[8];
    // hr1: bit 4i+j <- pair (j, j+1 mod 4) of row i; byte 0 holds rows 0,1 and byte 1 rows 2,3
#pragma unroll
    for (int b = 0; b < 8; ++b) {
        const int i = (7 - b) >> 2, j = (7 - b) & 3;
        const uint32_t dx = j < 3 ? later_heavier(x[i][j + 1], x[i][j]) : earlier_heavier(x[i][0], x[i][3]);
        const uint32_t dy = j < 3 ? later_heavier(x[i + 2][j + 1], x[i + 2][j]) : earlier_heavier(x[i + 2][0], x[i + 2][3]);
        p[b] = pick(dx, dy);
    }
    r.hr1 = gather8(p);
    // hc1: bit 4i+j <- pair (i, i+1 mod 4) of column j
#pragma unroll
    for (int b = 0; b < 8; ++b) {
        const int i = (7 - b) >> 2, j = (7 - b) & 3;                  // i in {0,1}; the partner byte holds i+2
        const uint32_t dx = later_heavier(x[i + 1][j], x[i][j]);
        const uint32_t dy = (i + 2 < 3) ? later_heavier(x[(i + 3) & 3][j], x[i + 2][j]) : earlier_heavier(x[0][j], x[3][j]);
        p[b] = pick(dx, dy);
    }
    r.hc1 = gather8(p);
    // hr2 (columns 0,1 only): bits 4i+j, j in {0,1}
    {
        const uint32_t q7 = pick(later_heavier(x[0][2], x[0][0]), later_heavier(x[2][2], x[2][0]));
        const uint32_t q6 = pick(later_heavier(x[0][3], x[0][1]), later_heavier(x[2][3], x[2][1]));
        const uint32_t q3 = pick(later_heavier(x[1][2], x[1][0]), later_heavier(x[3][2], x[3][0]));
        const uint32_t q2 = pick(later_heavier(x[1][3], x[1][1]), later_heavier(x[3][3], x[3][1]));
        r.hr2 = bitsel(bitsel(q7, q6, 0x01010101u), bitsel(q3, q2, 0x10101010u), 0x0F0F0F0Fu);      // bits 2,3 of a nibble: don't care
    }
    // hc2 (rows 0,1 only): bit 4i+j, i in {0,1}; gathered as (row 0 -> byte 0, row 1 -> byte 1), then packed
    {
        uint32_t q[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) q[j] = pick(later_heavier(x[2][j], x[0][j]), later_heavier(x[3][j], x[1][j]));
        const uint32_t g = bitsel(bitsel(q[0], q[1], 0x01010101u), bitsel(q[2], q[3], 0x04040404u), 0x03030303u);
        r.hc2 = bitsel(g, g >> 4, 0x0F0F0F0Fu);
    }
    r.hr3 = 0; r.hc3 = 0;
    complete_relations(r);
}

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

// The four mask bytes of a pair mask, byte i = (row i of block B) << 4 | (row i of block A): the layout
// of the packed mask for the thread's eight columns.
__device__ __forceinline__ uint32_t mask_bytes_2_4(uint32_t kept) {
    const uint32_t t = kept & 0x0F0F0F0Fu, u = (kept >> 4) & 0x0F0F0F0Fu;      // rows 0,2 / rows 1,3 (A in bytes 0,1; B in bytes 2,3)
    return prmt(t | (t >> 12), u | (u >> 12), 0x5140);
}

}  // namespace tmask
