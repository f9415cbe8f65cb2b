// 2:4 operand compression of W and of W^T from one transposable mask (Section 1, Fig. 2): the streaming form for
// bf16 matrices whose rows, and whose mask rows, start on 16-byte boundaries.  Two kernels:
//
// compress24_meta_kernel    mask -> meta, meta_t.  The metadata nibble idx0 | idx1 << 2 of a group is a function of the
//   group's keep nibble alone, so both metadata arrays come from the packed mask without a look at W.  A warp takes a
//   unit of 256 rows x 256 columns, 32 rows at a time.  A word of eight keep nibbles becomes eight metadata nibbles by
//   three logic operations; for the transposed metadata the nibbles of a column's eight block rows have to meet in one
//   word, a 32 x 32 bit transpose across the warp.  Units inside the matrix hold four rows per lane, which makes the
//   column groups' nibbles come out bit-sliced and leaves only three of the transpose's five steps to shuffles
//   (meta_rows_fast); units on an edge, and rows with a bad group, take the plainer lane-per-row form (meta_rows).  The
//   transposed words wait in the warp's shared buffer until the unit's 256 rows are done and leave as 32-byte runs.  The
//   same pass checks that every group keeps exactly two and raises the bad-mask status otherwise.
//
// compress24_values_kernel  W, mask -> values, values_t.  Every warp is a pipeline of its own over work items of 32 rows
//   x 128 columns.  An item arrives as two halves of 16 rows (4 KB of weights and 256 bytes of mask words each, two
//   bulk-tensor copies per half) through the warp's ring of three stages, one half in work and two in flight (a ring of
//   six stages of 8 rows measured the same time with a fifth more instructions).  No CTA-wide step after the start.  Lane = block
//   column: a lane owns the four columns 4*lane .. 4*lane+3 of the item and walks down its eight block rows.
//     row form     the kept pair of a row of a block is one 32-bit word, picked out of the row's two loaded words by ONE
//                  byte permute; its selector is computed from the row's metadata nibble by two multiplications, for
//                  two rows at once (no table: shared-memory instructions are what this kernel has least room for);
//                  a warp writes 128 contiguous bytes per row.
//     column form  stays in registers: the lane builds the kept pair of each of its four columns per block row (the
//                  column's four values as two words by byte permutes, then the same selectors from the column's
//                  nibble) and after eight block rows holds 16 values = 32 bytes per column, a full DRAM sector;
//                  nothing is transposed through shared memory.
//   Keep nibbles arrive as bytes: the four mask words of a block's rows are narrowed to the lane's nibble by three byte
//   permutes, a shift and a mask (byte i = row i); two exchange steps turn them (byte j = column j).
//   The common variant assumes that every group keeps exactly two and that the matrix is a whole number of items; the
//   careful variant tests every group (zeros for a bad one) and every edge.  Which one runs is decided on the device from
//   the status word the first kernel has just written.
//
// Granularity is what both are built around: a store instruction that leaves part of a 32-byte sector unwritten makes
// the memory system read the sector first, and a 16-byte read of a line that nobody else touches soon costs a whole
// line.  So neighbouring lanes share the writing of a sector (for the even lane's data the even lane stores the first 16
// bytes and the odd lane the second, then likewise for the odd lane's), and the warps of a CTA work side by side on
// neighbouring items, so that the 16 bytes of mask words per row an item needs are found in L2 by seven warps out of eight
// (see warp_items()).
#include <cstring>

#include "tm_launch.h"
#include "tm_tma.cuh"
#include "tm_tma_items.cuh"

namespace tmask {

namespace {

__device__ __forceinline__ uint32_t cprmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}

struct CompressArgs {
    long long rows, cols;
    int wpr, wpr_t;
    long long tiles_c, groups_r, total_items;     // values kernel: column tiles, row groups, strip items (eight tiles x 32 rows)
    long long units_c, total_units;     // metadata kernel: units of 256 x 256, row-major
    const uint32_t* mask;
    uint32_t* values;                   // [rows][cols / 4] words
    uint32_t* meta;
    unsigned char* values_t;            // [cols][rows / 2] bf16
    uint32_t* meta_t;
    int vec_t, vec_mt;                  // 16-byte stores possible for values_t / for meta_t
    int ragged;                         // rows % 32 or cols % 128: the values kernel takes its careful variant
};

// A CTA's share of `total` consecutive work items; inside it a warp takes the local indices warp, warp + nwarps, ...
// (the warps of a CTA work on neighbouring items at the same time).
__device__ __forceinline__ long long cta_share(long long total, long long& count) {
    const long long q = total / gridDim.x, rem = total - q * gridDim.x, b = blockIdx.x;
    count = q + (b < rem ? 1 : 0);
    return b * q + (b < rem ? b : rem);
}

// ---- metadata -------------------------------------------------------------------------------------------------------

// The eight metadata nibbles of a word of eight keep nibbles: for a nibble b3 b2 b1 b0 with exactly two bits set,
// idx0 = index of the lower one, idx1 = index of the upper one, nibble = idx0 | idx1 << 2:
//   bit 0 = ~b0 & b1, bit 1 = ~b0 & ~b1, bit 2 = b3 | ~b2, bit 3 = b3 | b2.
// With l = x << 1 and r = x >> 1 every bit sees its lower neighbour in l and its upper one in r: bits 0 and 2 are functions
// of (x, r), bits 1 and 3 of (x, l), and a constant mask tells the two members of either pair apart -- three three-input
// logic operations in all.
template <int LUT> __device__ __forceinline__ uint32_t lop3(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, %4;" : "=r"(r) : "r"(a), "r"(b), "r"(c), "n"(LUT));
    return r;
}
// truth-table byte of f(a, b, c): bit (a << 2 | b << 1 | c)
constexpr int lut3(bool (*f)(bool, bool, bool)) {
    int t = 0;
    for (int i = 0; i < 8; ++i) t |= (f((i >> 2) & 1, (i >> 1) & 1, i & 1) ? 1 : 0) << i;
    return t;
}
constexpr bool f_even(bool x, bool r, bool m) { return m ? (!x && r) : (r || !x); }     // bit 0 where m, bit 2 elsewhere
constexpr bool f_odd(bool x, bool l, bool m) { return m ? (!l && !x) : (l || x); }      // bit 1 where m, bit 3 elsewhere
constexpr bool f_sel(bool a, bool b, bool m) { return m ? a : b; }
__device__ __forceinline__ uint32_t meta_of(uint32_t x) {
    const uint32_t l = x << 1, r = x >> 1;
    const uint32_t even = lop3<lut3(f_even)>(x, r, 0x11111111u), odd = lop3<lut3(f_odd)>(x, l, 0x22222222u);
    return lop3<lut3(f_sel)>(even, odd, 0x55555555u);
}
// number of kept entries per nibble
__device__ __forceinline__ uint32_t nibble_counts(uint32_t x) {
    const uint32_t s = x - ((x >> 1) & 0x55555555u);
    return (s & 0x33333333u) + ((s >> 2) & 0x33333333u);
}
// metadata with zeros for the nibbles that do not keep exactly two
__device__ __forceinline__ uint32_t meta_of_checked(uint32_t x) {
    uint32_t v = nibble_counts(x) ^ 0x22222222u;          // zero nibble <=> two kept
    v |= v >> 1; v |= v >> 2;
    return meta_of(x) & ((~v & 0x11111111u) * 15u);
}
// 32 x 32 bit transpose across the warp: lane r gives row r, lane c receives column c (bit r = row r's bit c).
// Step j exchanges the off-diagonal j x j blocks of every 2j x 2j block: a lane whose index has bit j clear keeps its bits
// with column bit j clear and receives, moved up by j, its partner's; the other lane the other way round.  Moving up by j
// under a mask is a rotation by j, moving down a rotation by 32 - j (what the rotation wraps around the mask removes).
struct TransposePlan {
    uint32_t keep[5];       // the bits the lane keeps in step 16, 8, 4, 2, 1
    int rot[5];             // how far its partner's word is rotated left
};
__device__ __forceinline__ TransposePlan transpose_plan(int lane) {
    TransposePlan p;
#pragma unroll
    for (int k = 0; k < 5; ++k) {
        const int j = 16 >> k;
        const uint32_t m = j == 16 ? 0x0000FFFFu : (j == 8 ? 0x00FF00FFu : (j == 4 ? 0x0F0F0F0Fu : (j == 2 ? 0x33333333u : 0x55555555u)));
        p.keep[k] = (lane & j) ? ~m : m;
        p.rot[k] = (lane & j) ? 32 - j : j;
    }
    return p;
}
__device__ __forceinline__ uint32_t transpose32(uint32_t x, const TransposePlan& p) {
#pragma unroll
    for (int k = 0; k < 5; ++k) {
        const uint32_t y = __shfl_xor_sync(0xFFFFFFFFu, x, 16 >> k);
        x = lop3<lut3(f_sel)>(x, __funnelshift_l(y, y, p.rot[k]), p.keep[k]);
    }
    return x;
}

constexpr int kMWarps = 4;
constexpr int kMParkWords = 8 * 256;                    // [8 row groups][256 columns]

struct MetaUnit {
    long long ur, uc, word0;    // unit row, unit column, first mask word of its columns
    int groups_left;            // groups of four columns from word0 on that lie inside the matrix, at most 64
};

// 32 rows of a unit: lane = row.  a, b: the row's eight mask words.  FULL: the unit lies wholly inside the matrix.
// Returns true if some group, along a row or down a column, does not keep exactly two.
template <bool FULL>
__device__ __forceinline__ bool meta_rows(const CompressArgs& A, const MetaUnit& U, int g, uint4 a, uint4 b, const TransposePlan& plan, uint32_t* park, int lane) {
    const long long row = U.ur * 256 + g * 32 + lane;
    const bool row_in = FULL || row < A.rows;
    const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    bool bad = false;
    // ---- row form: my row's eight metadata words ----
    uint32_t mrow[8], rbad = 0;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        mrow[q] = meta_of(w[q]);
        uint32_t in = 0xFFFFFFFFu;
        if constexpr (!FULL) {
            const int ng = U.groups_left - 8 * q;                      // groups of this word inside the matrix
            in = ng >= 8 ? 0xFFFFFFFFu : (ng <= 0 ? 0u : (1u << (4 * ng)) - 1u);
        }
        rbad |= (nibble_counts(w[q]) ^ 0x22222222u) & in;
    }
    if (!row_in) rbad = 0;
    const bool rows_bad = __any_sync(0xFFFFFFFFu, rbad != 0);
    bad |= rows_bad;
    if (rows_bad || (!FULL && U.groups_left < 64)) {          // also past the last column: the padding nibbles of a word are zero
#pragma unroll
        for (int q = 0; q < 8; ++q) mrow[q] = meta_of_checked(w[q]);
    }
    {   // a row's 32 bytes are one sector: neighbouring lanes share the writing of it
        const bool odd = lane & 1;
        uint32_t recv[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) recv[q] = __shfl_xor_sync(0xFFFFFFFFu, odd ? mrow[q] : mrow[4 + q], 1);
        const long long prow = odd ? row - 1 : row + 1;
        uint32_t* mine = A.meta + row * A.wpr + U.word0 + (odd ? 4 : 0);
        uint32_t* theirs = A.meta + prow * A.wpr + U.word0 + (odd ? 4 : 0);
        const bool half_in = FULL || U.word0 + (odd ? 4 : 0) < A.wpr;
        const bool mine_in = half_in && row_in, theirs_in = half_in && (FULL || prow < A.rows);
        const uint4 own = odd ? make_uint4(mrow[4], mrow[5], mrow[6], mrow[7]) : make_uint4(mrow[0], mrow[1], mrow[2], mrow[3]);
        const uint4 got = make_uint4(recv[0], recv[1], recv[2], recv[3]);
        // first the even lane's row, then the odd lane's
        if (odd) { if (theirs_in) *reinterpret_cast<uint4*>(theirs) = got; } else { if (mine_in) *reinterpret_cast<uint4*>(mine) = own; }
        if (odd) { if (mine_in) *reinterpret_cast<uint4*>(mine) = own; } else { if (theirs_in) *reinterpret_cast<uint4*>(theirs) = got; }
    }
    // ---- column form: transpose the eight bit tiles; lane = column ----
    int rows_here = 32;
    if constexpr (!FULL) rows_here = (int)min((long long)32, A.rows - (U.ur * 256 + g * 32));            // a multiple of 4
    const uint32_t rin = rows_here >= 32 ? 0xFFFFFFFFu : (1u << rows_here) - 1u;                        // nibble b covers rows 4b .. 4b+3
    uint32_t cbad = 0, t[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        t[q] = transpose32(w[q], plan);
        const bool col_in = FULL || (U.word0 + q) * 32 + lane < A.cols;
        cbad |= col_in ? (nibble_counts(t[q]) ^ 0x22222222u) & rin : 0u;
    }
    const bool cols_bad = __any_sync(0xFFFFFFFFu, cbad != 0);
    bad |= cols_bad;
    const bool careful = cols_bad || rows_here < 32;      // also below the last row: the padding nibbles of a word are zero
#pragma unroll
    for (int q = 0; q < 8; ++q) park[g * 256 + q * 32 + lane] = careful ? meta_of_checked(t[q]) : meta_of(t[q]);
    return bad;
}

// The same 32 rows for a unit that lies wholly inside the matrix, with four rows per lane: lane = (block row b = lane & 7,
// word pair q = lane >> 3) holds rows 4b .. 4b+3 of words 2q, 2q+1.  A column group's four keep bits then sit in the same
// bit of the lane's four words, so the group's metadata nibble comes out bit-sliced (four words of "bit n of the nibble of
// column c") with four logic operations for 32 columns, and the 32 x 32 transpose that gathers a column's eight nibbles
// starts with its two finest steps inside the lane; only the three coarse steps cross lanes (12 shuffles per 32 columns
// instead of 40).  The row form needs no exchange at all: four lanes write the 32 bytes of a row in one instruction.
// r[i][t]: row 4b + i, word 2q + t.  Returns false, having written nothing, if some group does not keep exactly two.
__device__ __forceinline__ bool meta_rows_fast(const CompressArgs& A, const MetaUnit& U, int g, const uint2 (&r)[4], uint32_t* park, int lane) {
    const int b = lane & 7, q = lane >> 3;
    uint32_t bad = 0;
    uint2 mrow[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        mrow[i] = make_uint2(meta_of(r[i].x), meta_of(r[i].y));
        bad |= (nibble_counts(r[i].x) ^ 0x22222222u) | (nibble_counts(r[i].y) ^ 0x22222222u);
    }
    uint32_t t4[2][4];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const uint32_t b0 = t ? r[0].y : r[0].x, b1 = t ? r[1].y : r[1].x, b2 = t ? r[2].y : r[2].x, b3 = t ? r[3].y : r[3].x;
        // exactly two of the four: the pairs (b0, b1) and (b2, b3) hold one each, or one holds both and the other none
        const uint32_t a = b0 ^ b1, p = b0 & b1, c = b2 ^ b3, d = b2 & b3;
        bad |= ~((a & c) | ((p ^ d) & ~(a | c)));
        uint32_t x0 = ~b0 & b1, x1 = ~b0 & ~b1, x2 = b3 | ~b2, x3 = b3 | b2;      // bit n of the columns' metadata nibbles
        // transpose steps 1 and 2: rows 4b + n of the bit matrix are the lane's own four words
        uint32_t e = ((x0 >> 1) ^ x1) & 0x55555555u; x1 ^= e; x0 ^= e << 1;
        e = ((x2 >> 1) ^ x3) & 0x55555555u; x3 ^= e; x2 ^= e << 1;
        e = ((x0 >> 2) ^ x2) & 0x33333333u; x2 ^= e; x0 ^= e << 2;
        e = ((x1 >> 2) ^ x3) & 0x33333333u; x3 ^= e; x1 ^= e << 2;
        t4[t][0] = x0; t4[t][1] = x1; t4[t][2] = x2; t4[t][3] = x3;
    }
    if (__any_sync(0xFFFFFFFFu, bad != 0)) return false;
    // steps 4, 8, 16 across the lanes b ^ 1, b ^ 2, b ^ 4
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        const int j = 4 << k, lb = 1 << k;
        const uint32_t m = j == 16 ? 0x0000FFFFu : (j == 8 ? 0x00FF00FFu : 0x0F0F0F0Fu);
        const uint32_t keep = (b & lb) ? ~m : m;
        const int rot = (b & lb) ? 32 - j : j;
#pragma unroll
        for (int t = 0; t < 2; ++t)
#pragma unroll
            for (int n = 0; n < 4; ++n) {
                const uint32_t y = __shfl_xor_sync(0xFFFFFFFFu, t4[t][n], lb);
                t4[t][n] = lop3<lut3(f_sel)>(t4[t][n], __funnelshift_l(y, y, rot), keep);
            }
    }
    // word n of the lane now belongs to column 4b + n of its 32: eight nibbles, one per block row
    const long long row = U.ur * 256 + g * 32 + 4 * b;
#pragma unroll
    for (int i = 0; i < 4; ++i) *reinterpret_cast<uint2*>(A.meta + (row + i) * A.wpr + U.word0 + 2 * q) = mrow[i];
#pragma unroll
    for (int t = 0; t < 2; ++t)
        *reinterpret_cast<uint4*>(park + g * 256 + 64 * q + 32 * t + 4 * b) = make_uint4(t4[t][0], t4[t][1], t4[t][2], t4[t][3]);
    return true;
}

__global__ void __launch_bounds__(kMWarps * 32, 6)
compress24_meta_kernel(const __grid_constant__ CompressArgs A, int* __restrict__ status_out) {
    __shared__ uint32_t park_all[kMWarps][kMParkWords];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t* park = park_all[warp];
    long long n_cta;
    const long long first = cta_share(A.total_units, n_cta);
    bool bad = false;
    const TransposePlan plan = transpose_plan(lane);
    for (long long k = warp; k < n_cta; k += kMWarps) {
        MetaUnit U;
        const long long u = first + k;
        U.ur = u / A.units_c; U.uc = u - U.ur * A.units_c; U.word0 = U.uc * 8;
        U.groups_left = (int)min((long long)64, (A.cols - U.word0 * 32) / 4);
        const int n_g = (int)min((long long)8, (A.rows - U.ur * 256 + 31) / 32);
        const bool full = U.groups_left == 64 && U.ur * 256 + 256 <= A.rows;
        if (full) {
            // four rows per lane; the rows are read one group ahead of their use
            const int b = lane & 7, q = lane >> 3;
            auto load4 = [&](int g, uint2 (&r)[4]) {
                const uint32_t* src = A.mask + (U.ur * 256 + g * 32 + 4 * b) * A.wpr + U.word0 + 2 * q;
#pragma unroll
                for (int i = 0; i < 4; ++i) r[i] = __ldg(reinterpret_cast<const uint2*>(src + (long long)i * A.wpr));
            };
            uint2 next[4];
            load4(0, next);
#pragma unroll 1
            for (int g = 0; g < 8; ++g) {
                uint2 r[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) r[i] = next[i];
                if (g + 1 < 8) load4(g + 1, next);
                if (!meta_rows_fast(A, U, g, r, park, lane)) {
                    // a bad group somewhere in these rows: the lane-per-row form, which writes zeros for it
                    const long long row = U.ur * 256 + g * 32 + lane;
                    const uint4* src = reinterpret_cast<const uint4*>(A.mask + row * A.wpr + U.word0);
                    bad |= meta_rows<true>(A, U, g, __ldg(src), __ldg(src + 1), plan, park, lane);
                }
            }
        } else {
            // the rows are read one group ahead of their use
            auto load = [&](int g, uint4& a, uint4& b) {
                const long long row = U.ur * 256 + g * 32 + lane;
                const uint4* src = reinterpret_cast<const uint4*>(A.mask + row * A.wpr + U.word0);
                a = make_uint4(0, 0, 0, 0); b = a;
                if (row < A.rows && U.word0 < A.wpr) a = __ldg(src);
                if (row < A.rows && U.word0 + 4 < A.wpr) b = __ldg(src + 1);
            };
            uint4 na, nb;
            load(0, na, nb);
#pragma unroll 1
            for (int g = 0; g < n_g; ++g) {
                const uint4 a = na, b = nb;
                if (g + 1 < n_g) load(g + 1, na, nb);
                bad |= meta_rows<false>(A, U, g, a, b, plan, park, lane);
            }
        }
        // ---- the unit's transposed metadata: eight words per column ----
        __syncwarp();
        if (A.vec_mt && n_g == 8) {
            // two lanes per column, 16 bytes each: every store instruction carries whole sectors
#pragma unroll 4
            for (int kk = 0; kk < 16; ++kk) {
                const int c = kk * 16 + (lane >> 1), h = lane & 1;
                const long long col = U.uc * 256 + c;
                if (col >= A.cols) continue;
                const uint32_t* src = park + h * 4 * 256 + c;
                reinterpret_cast<uint4*>(A.meta_t + col * A.wpr_t + U.ur * 8)[h] = make_uint4(src[0], src[256], src[512], src[768]);
            }
        } else {
            for (int kk = 0; kk < 8; ++kk) {
                const int c = kk * 32 + lane;
                const long long col = U.uc * 256 + c;
                if (col >= A.cols) continue;
                for (int g = 0; g < n_g; ++g) A.meta_t[col * A.wpr_t + U.ur * 8 + g] = park[g * 256 + c];
            }
        }
        __syncwarp();
    }
    if (bad && lane == 0 && status_out) atomicOr(status_out, kDevBadMask);
}

// ---- values ---------------------------------------------------------------------------------------------------------

constexpr int kCRows = 32, kCCols = 128;                // a work item
constexpr int kCParts = 2, kCPartRows = kCRows / kCParts;   // an item arrives in halves of 16 rows, one pair of bulk-tensor copies each
constexpr int kCWarps = 16, kCStages = 3;                // a warp's ring of half-item stages: one in work, two in flight
static_assert(kCParts == 2, "values_warp() names the two halves");
constexpr int kCStageW = kCPartRows * kCCols * 2, kCStageM = kCPartRows * 16, kCStageBytes = kCStageW + kCStageM;
constexpr int kCWarpBytes = kCStages * kCStageBytes + 128;
static_assert(kCStageBytes % 128 == 0 && kCWarpBytes % 128 == 0, "stages stay 128-byte aligned");
constexpr int kCSmemBytes = kCWarps * kCWarpBytes;
static_assert(kCSmemBytes <= 232448, "at most 227 KB of shared memory per CTA");

// The byte-permute selectors that pick the kept pair (halfwords idx0, idx1) out of two words holding four 16-bit values,
// for two groups at once: byte 0 and byte 2 of t hold the groups' metadata nibbles idx0 | idx1 << 2.  t + (t << 6), masked,
// leaves idx0 in a group's low byte and idx1 in the byte above; times 0x22 turns an index i into 2i | 2i << 4, and 0x10
// on top makes it the selector byte of halfword i, 2i | (2i + 1) << 4.  The low 16 bits of the result serve the first
// group, the high 16 bits the second.
__device__ __forceinline__ uint32_t pair_selectors(uint32_t t) { return ((t * 65u) & 0x03030303u) * 0x22u + 0x10101010u; }

// The keep nibbles of a block, one per byte (byte i = row i), turned: byte j = column j (bit i = row i).
__device__ __forceinline__ uint32_t transpose_nibbles(uint32_t x) {
    uint32_t t = (x ^ (x >> 7)) & 0x000A000Au;
    x ^= t ^ (t << 7);
    t = (x ^ (x >> 14)) & 0x00000C0Cu;
    return x ^ t ^ (t << 14);
}

// One half of an item: block rows 4 * PART .. 4 * PART + 3 into the row form and into acc (the kept pairs of the lane's
// four columns, eight block rows each).  stage: weights [16][128] bf16, then mask words [16][4].
template <bool CAREFUL, int PART>
__device__ __forceinline__ void pack_half(const unsigned char* stage, uint32_t (&acc)[4][8], const CompressArgs& A, long long tc, long long g, int lane) {
    const int l7 = lane & 7, wsel = lane >> 3;
    const uint32_t selm = (uint32_t)(l7 >> 1) | ((4u + (uint32_t)(l7 >> 1)) << 4);
    const int nsh = 4 * (l7 & 1);
    const long long c0 = tc * kCCols + lane * 4, row0 = g * kCRows + PART * kCPartRows;
    const bool col_in = c0 < A.cols;
    const int stride = (int)(A.cols / 4);                              // words per row of `values`
    uint32_t* vrow = A.values + row0 * stride + tc * 32 + lane;
#pragma unroll
    for (int hb = 0; hb < kCPartRows / 4; ++hb) {
        const bool active = col_in && row0 + hb * 4 < A.rows;     // rows % 4 == 0: a block row is inside or outside as a whole
        uint2 raw[4];
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            raw[i] = *reinterpret_cast<const uint2*>(stage + (hb * 4 + i) * (kCCols * 2) + lane * 8);
            w[i] = *reinterpret_cast<const uint32_t*>(stage + kCStageW + (hb * 4 + i) * 16 + wsel * 4);
        }
        // byte i = keep nibble of row i
        uint32_t mb = (cprmt(cprmt(w[0], w[1], selm), cprmt(w[2], w[3], selm), 0x5410u) >> nsh) & 0x0F0F0F0Fu;
        if constexpr (CAREFUL) { if (!active) mb = 0; }
        // ---- row form: the rows' metadata nibbles (one per byte), from them the selectors ----
        {
            const uint32_t nibs = (CAREFUL ? meta_of_checked(mb) : meta_of(mb)) & 0x0F0F0F0Fu;      // the empty upper nibbles give no metadata
            const uint32_t s01 = pair_selectors(cprmt(nibs, 0u, 0x4140u)), s23 = pair_selectors(cprmt(nibs, 0u, 0x4342u));
            uint32_t pair[4] = {cprmt(raw[0].x, raw[0].y, s01), cprmt(raw[1].x, raw[1].y, s01 >> 16),
                                cprmt(raw[2].x, raw[2].y, s23), cprmt(raw[3].x, raw[3].y, s23 >> 16)};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if constexpr (CAREFUL) {
                    if (!((nibs >> (8 * i)) & 0xFu)) pair[i] = 0;
                    if (active) vrow[(hb * 4 + i) * stride] = pair[i];
                } else {
                    vrow[(hb * 4 + i) * stride] = pair[i];
                }
            }
        }
        // ---- column form: the same on the turned nibbles; a column's four values as two words by byte permutes ----
        {
            const uint32_t cb = transpose_nibbles(mb);
            const uint32_t nibs = (CAREFUL ? meta_of_checked(cb) : meta_of(cb)) & 0x0F0F0F0Fu;
            const uint32_t s01 = pair_selectors(cprmt(nibs, 0u, 0x4140u)), s23 = pair_selectors(cprmt(nibs, 0u, 0x4342u));
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t sel = (j & 1) ? 0x7632u : 0x5410u;
                const uint32_t c01 = j < 2 ? cprmt(raw[0].x, raw[1].x, sel) : cprmt(raw[0].y, raw[1].y, sel);
                const uint32_t c23 = j < 2 ? cprmt(raw[2].x, raw[3].x, sel) : cprmt(raw[2].y, raw[3].y, sel);
                uint32_t pair = cprmt(c01, c23, (j < 2 ? s01 : s23) >> (16 * (j & 1)));
                if constexpr (CAREFUL) { if (!((nibs >> (8 * j)) & 0xFu)) pair = 0; }
                acc[j][(kCPartRows / 4) * PART + hb] = pair;
            }
        }
    }
}

// After both halves: the columns' 16 values each, one 32-byte sector per column.
template <bool CAREFUL>
__device__ __forceinline__ void store_columns(const uint32_t (&acc)[4][8], const CompressArgs& A, long long tc, long long g, int lane) {
    const long long c0 = tc * kCCols + lane * 4, half_r = A.rows / 2, v0 = g * 16;
    const bool odd = lane & 1;
    if (A.vec_t && (!CAREFUL || v0 + 16 <= half_r)) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t recv[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) recv[q] = __shfl_xor_sync(0xFFFFFFFFu, odd ? acc[j][q] : acc[j][4 + q], 1);
            // own column: my half of it; the partner's column (four columns on or back): the half I received
            unsigned char* mine = A.values_t + ((c0 + j) * half_r + v0) * 2 + (odd ? 16 : 0);
            unsigned char* theirs = A.values_t + ((c0 + j + (odd ? -4 : 4)) * half_r + v0) * 2 + (odd ? 16 : 0);
            const bool mine_in = !CAREFUL || c0 + j < A.cols, theirs_in = !CAREFUL || c0 + j + (odd ? -4 : 4) < A.cols;
            const uint4 own = odd ? make_uint4(acc[j][4], acc[j][5], acc[j][6], acc[j][7]) : make_uint4(acc[j][0], acc[j][1], acc[j][2], acc[j][3]);
            const uint4 got = make_uint4(recv[0], recv[1], recv[2], recv[3]);
            // first the even lane's column, then the odd lane's
            if (odd) { if (theirs_in) *reinterpret_cast<uint4*>(theirs) = got; } else { if (mine_in) *reinterpret_cast<uint4*>(mine) = own; }
            if (odd) { if (mine_in) *reinterpret_cast<uint4*>(mine) = own; } else { if (theirs_in) *reinterpret_cast<uint4*>(theirs) = got; }
        }
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (c0 + j >= A.cols) continue;
            unsigned char* dst = A.values_t + ((c0 + j) * half_r + v0) * 2;
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if (v0 + 2 * k < half_r) reinterpret_cast<uint32_t*>(dst)[k] = acc[j][k];
        }
    }
}

// The order of the work.  Strips of eight column tiles (1024 columns: a row's 128 bytes of mask words) are walked down
// 32 rows at a time; "strip items" (strip, row group) are numbered strip by strip, a CTA takes a run of consecutive
// ones, and its sixteen warps stand side by side on two consecutive strip items: warp w on column tile w % 8 of strip
// item w / 8, then of strip item w / 8 + 2, and so on.  So a warp walks down its columns (the 32-byte sectors it writes
// into a line of the column form follow one another closely), and the eight warps of a strip item ask for the same mask
// lines at about the same time.
struct WarpItems {
    long long si0;      // the warp's first strip item
    int count;          // how many of its strip items fall on an existing column tile
    int tile;           // its column tile inside a strip
};
__device__ __forceinline__ WarpItems warp_items(const CompressArgs& A, int warp) {
    long long n_cta;
    const long long first = cta_share(A.total_items, n_cta), end = first + n_cta;    // total_items counts strip items
    WarpItems wi;
    wi.tile = warp & 7;
    wi.si0 = first + (warp >> 3);
    // in the last strip the tiles past the last column do not exist: for this warp its strip items end there
    const long long strips = (A.tiles_c + 7) / 8, last0 = (strips - 1) * A.groups_r;
    const long long stop = (strips - 1) * 8 + wi.tile >= A.tiles_c && last0 < end ? last0 : end;
    wi.count = wi.si0 < stop ? (int)((stop - wi.si0 + 1) / 2) : 0;
    return wi;
}

// The warp's items through its ring.  Returns false if a copy did not land within its bounded wait.
template <bool CAREFUL>
__device__ __forceinline__ bool values_warp(unsigned char* stages, uint64_t* bars, const CompressArgs& A, const CUtensorMap* wmap,
                                            const CUtensorMap* mmap, const WarpItems& wi, int lane) {
    const int n_parts = kCParts * wi.count;
    auto issue = [&](int hi) {                 // lane 0: both copies of the warp's part number hi into its ring slot
        const long long si = wi.si0 + 2 * (long long)(hi / kCParts), strip = si / A.groups_r, g = si - strip * A.groups_r, tc = strip * 8 + wi.tile;
        const int s = hi % kCStages, y = (int)(g * kCRows) + (hi % kCParts) * kCPartRows;
        mbar_expect_tx(&bars[s], kCStageBytes);
        tma_load_2d(stages + s * kCStageBytes, wmap, (int)(tc * kCCols), y, &bars[s]);
        tma_load_2d(stages + s * kCStageBytes + kCStageW, mmap, (int)(tc * 4), y, &bars[s]);
    };
    if (lane == 0)
        for (int hi = 0; hi < kCStages - 1 && hi < n_parts; ++hi) issue(hi);
    int hi = 0;
    for (int it = 0; it < wi.count; ++it) {
        const long long si = wi.si0 + 2 * (long long)it, strip = si / A.groups_r, g = si - strip * A.groups_r, tc = strip * 8 + wi.tile;
        uint32_t acc[4][8];
#pragma unroll
        for (int part = 0; part < kCParts; ++part, ++hi) {
            const int s = hi % kCStages;
            // the slot of the part before this one was last read before the warp-wide barrier that ended that part
            if (lane == 0 && hi + kCStages - 1 < n_parts) issue(hi + kCStages - 1);
            if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(&bars[s], (uint32_t)((hi / kCStages) & 1)))) return false;
            const unsigned char* stage = stages + s * kCStageBytes;
            if (part == 0) pack_half<CAREFUL, 0>(stage, acc, A, tc, g, lane);
            else pack_half<CAREFUL, 1>(stage, acc, A, tc, g, lane);
            __syncwarp();
        }
        store_columns<CAREFUL>(acc, A, tc, g, lane);
    }
    return true;
}

__global__ void __launch_bounds__(kCWarps * 32, 1)
compress24_values_kernel(const __grid_constant__ CompressArgs A, int* __restrict__ status_out, const __grid_constant__ CUtensorMap wmap,
                         const __grid_constant__ CUtensorMap mmap) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned char* stages = smem_raw + (size_t)warp * kCWarpBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(stages + kCStages * kCStageBytes);
    if (lane == 0) {
        for (int s = 0; s < kCStages; ++s) mbar_init(&bars[s], 1);
        fence_mbar_init();
    }
    __syncthreads();
    // the metadata kernel ran before this one on the same stream and has flagged a mask with a bad group
    const bool careful = A.ragged || !status_out || (*reinterpret_cast<volatile int*>(status_out) & kDevBadMask);
    const WarpItems wi = warp_items(A, warp);
    const bool ok = careful ? values_warp<true>(stages, bars, A, &wmap, &mmap, wi, lane)
                            : values_warp<false>(stages, bars, A, &wmap, &mmap, wi, lane);
    if (!ok) {
        // a copy never landed: give the ones that may still be in flight a bounded chance to finish before the stages die
        if (lane == 0) {
            for (int s = 0; s < kCStages; ++s) { mbar_wait_bounded(&bars[s], 0, 1u << 14); mbar_wait_bounded(&bars[s], 1, 1u << 14); }
            if (status_out) atomicOr(status_out, kDevInternal);
        }
    }
}

}  // namespace

bool compress24_stream_eligible(const AuxProblem& P, const void* values, const void* meta, const void* meta_t) {
    return P.dtype == kBF16 && (uintptr_t)P.W % 16 == 0 && ((size_t)P.ld * 2) % 16 == 0 && (uintptr_t)P.mask % 16 == 0 && P.wpr % 4 == 0 &&
           P.rows % 4 == 0 && P.cols % 4 == 0 && (uintptr_t)values % 4 == 0 && (uintptr_t)meta % 16 == 0 && (uintptr_t)meta_t % 4 == 0 &&
           P.rows < (1ll << 31) && P.cols < (1ll << 31) && encode_fn() != nullptr;
}

cudaError_t launch_compress24_stream(const AuxProblem& P, void* values, uint32_t* meta, void* values_t, uint32_t* meta_t, int* status,
                                     int sms, cudaStream_t stream) {
    CUtensorMap wmap, mmap;
    memset(&wmap, 0, sizeof wmap); memset(&mmap, 0, sizeof mmap);
    EncodeTiledFn fn = encode_fn();
    const cuuint64_t wd[2] = {(cuuint64_t)P.cols, (cuuint64_t)P.rows}, ws[1] = {(cuuint64_t)P.ld * 2};
    const cuuint64_t md[2] = {(cuuint64_t)P.wpr, (cuuint64_t)P.rows}, ms[1] = {(cuuint64_t)P.wpr * 4};
    const cuuint32_t wb[2] = {kCCols, kCPartRows}, mb[2] = {4, kCPartRows}, es[2] = {1, 1};
    if (fn(&wmap, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, const_cast<void*>(P.W), wd, ws, wb, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
        fn(&mmap, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, P.mask, md, ms, mb, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
           CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    CompressArgs A;
    A.rows = P.rows; A.cols = P.cols; A.wpr = P.wpr; A.wpr_t = (int)((P.rows + 31) / 32);
    A.tiles_c = (P.cols + kCCols - 1) / kCCols;
    A.groups_r = (P.rows + kCRows - 1) / kCRows;
    A.total_items = ((A.tiles_c + 7) / 8) * A.groups_r;
    A.units_c = (P.cols + 255) / 256;
    A.total_units = A.units_c * ((P.rows + 255) / 256);
    A.mask = P.mask;
    A.values = static_cast<uint32_t*>(values); A.meta = meta; A.values_t = static_cast<unsigned char*>(values_t); A.meta_t = meta_t;
    A.vec_t = (uintptr_t)values_t % 16 == 0 && P.rows % 16 == 0;          // a column's run of P.rows / 2 values starts on 16 bytes
    A.vec_mt = (uintptr_t)meta_t % 16 == 0 && A.wpr_t % 4 == 0;
    A.ragged = P.rows % kCRows != 0 || P.cols % kCCols != 0;
    {
        const long long want = (A.total_units + kMWarps - 1) / kMWarps;
        const long long cap = (long long)sms * 6;
        compress24_meta_kernel<<<(int)(want < cap ? want : cap), kMWarps * 32, 0, stream>>>(A, status);
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    static PerDeviceOnce configured;
    const cudaError_t e = configured.run([&] { return cudaFuncSetAttribute(compress24_values_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kCSmemBytes); });
    if (e != cudaSuccess) return e;
    const long long want = (A.total_items + 1) / 2;           // a CTA stands on two strip items at a time
    compress24_values_kernel<<<(int)(want < sms ? want : sms), kCWarps * 32, kCSmemBytes, stream>>>(A, status, wmap, mmap);
    return cudaGetLastError();
}

}  // namespace tmask
