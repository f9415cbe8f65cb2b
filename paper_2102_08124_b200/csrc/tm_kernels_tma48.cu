// Bandwidth kernels of the approximate 4:8 search (TM_APPROX / TM_APPROX_COVER, M = 8).
//
// Same pipeline idea as the 2:4 kernels: every warp walks a contiguous range of work items (8 rows x
// 256 columns of one matrix) with bulk-tensor (TMA) loads running ahead into a private ring of
// shared-memory stages and TMA stores draining it; a lane owns one 8x8 block of the item.
// The search itself is the bit-parallel core of tm_core48.cuh on 64-bit sets:
//   front end  the 448 row/column comparisons of the block, collected into relation masks
//              (bf16: two comparisons per 32-bit subtraction on packed magnitudes; fp32: scalar);
//   step A     two bit-sliced counts;
//   step B     warp-uniform rounds (a vote decides whether any lane still has candidates);
//   step C     per lane: candidates from the relation masks, then the few magnitudes that must be
//              compared are read back from the stage;
//   back end   masked weights written into the stage and stored by TMA, mask bytes through shared
//              memory as whole words, objective in fp32 per lane / fp64 across.
#include "tm_core48.cuh"
#include "tm_launch.h"
#include "tm_pair_bf16.cuh"
#include "tm_tma.cuh"
#include "tm_tma_items.cuh"

#include <type_traits>

namespace tmask {

namespace {

constexpr int kRows8 = 8;
constexpr int kCols8 = 256;

// Warps per CTA and stages per warp.  Algorithm 1 alone on bf16 runs best with 12 warps x 3 stages (0.465 ms on the
// 12288 x 49152 matrix against 0.500 with 16 x 3 and 0.537 with 12 x 2); for fp32 fewer than 12 warps only lose.
template <int DT, int METHOD> struct Geo48 {
    static constexpr int kElem = DT == kF32 ? 4 : 2;
    static constexpr int kWarps = METHOD == kMethodApprox ? (DT == kF32 ? 12 : 16) : (DT == kF32 ? 12 : 12);
    static constexpr int kStages = METHOD == kMethodApprox ? (DT == kF32 ? 2 : 3) : (DT == kF32 ? 2 : 3);
    static constexpr int kRowPitch = kCols8 * kElem;
    static constexpr int kStageBytes = kRows8 * kRowPitch;
    static constexpr int kWarpBytes = kStages * kStageBytes + 256 /* mask bytes [8][32] */ + 64 /* barriers */ + 64;
    static constexpr int kLutBytes = DT == kBF16 ? kLaneLutBytes : 256 * 32;     // keep flags of a row as lane masks (bf16) or as 0/1 words (fp32)
};

__device__ __forceinline__ uint32_t max_u16x2_(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.u16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// p[b] (bytes of equal bits) carries the decisions destined for bit 7-b of every byte (see gather8);
// only bits 0..3 are wanted, the upper four come out as copies of p4
template <bool NEG>                              // NEG: the four arrive negated
__device__ __forceinline__ uint32_t gather4_low(uint32_t p7, uint32_t p6, uint32_t p5, uint32_t p4) {
    return bitsel(bitsel_n<NEG, NEG>(p7, p6, 0x01010101u), bitsel_n<NEG, NEG>(p5, p4, 0x04040404u), 0x03030303u);
}

// ---- bf16: packed comparisons ----------------------------------------------------------------
// hr[K] from the row-paired magnitudes Y[i'][j] = (|x_2i',j|, |x_2i'+1,j|); for K = 4 only columns 0..3
template <bool ARITH, int K>
__device__ __forceinline__ u64 row_relation(const uint32_t (&Y)[4][8]) {
    uint32_t word[2];
#pragma unroll
    for (int w = 0; w < 2; ++w) {
        uint32_t pj[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (K == 4 && j >= 4) { pj[j] = 0; continue; }
            const uint32_t d0 = (j + K <= 7) ? later_heavier<ARITH>(Y[2 * w][(j + K) & 7], Y[2 * w][j]) : earlier_heavier<ARITH>(Y[2 * w][(j + K) & 7], Y[2 * w][j]);
            const uint32_t d1 = (j + K <= 7) ? later_heavier<ARITH>(Y[2 * w + 1][(j + K) & 7], Y[2 * w + 1][j]) : earlier_heavier<ARITH>(Y[2 * w + 1][(j + K) & 7], Y[2 * w + 1][j]);
            pj[j] = prmt(d0, d1, 0xFDB9);      // bytes (0x00 / 0xFF) = rows 4w .. 4w+3 of column j
        }
        if constexpr (K == 4) {
            word[w] = gather4_low<ARITH>(pj[0], pj[1], pj[2], pj[3]);
        } else {
            const uint32_t p[8] = {pj[7], pj[6], pj[5], pj[4], pj[3], pj[2], pj[1], pj[0]};
            word[w] = gather8<ARITH ? (0xFFu & ~((1u << K) - 1u)) : 0u>(p);            // p[b] = column 7-b: a later partner iff b >= K
        }
    }
    return (u64)word[0] | ((u64)word[1] << 32);
}

// R[i][c] = (|x_i,2c|, |x_i,2c+1|) of the lane's block.  ARITH selects the form of the comparison (see
// tm_pair_bf16.cuh): packed bf16 subtraction for finite data, integer subtraction for any bit pattern.
template <bool ARITH>
__device__ __forceinline__ void relations48_bf16(const uint32_t (&R)[8][4], Rel48& rel) {
    // column relations hc[k]: bit (i,j) <- rows (i, i+k mod 8) of column j.  One subtraction decides two
    // adjacent columns; byte permutes line the decisions up as (byte = row, all bits equal), a select tree packs them.
#pragma unroll
    for (int k = 1; k <= 4; ++k) {
        uint32_t word[2] = {0, 0};
#pragma unroll
        for (int w = 0; w < 2; ++w) {
            if (k == 4 && w == 1) continue;        // rows 4..7 of hc[4] follow by antisymmetry
            uint32_t cw[8];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t d[4];
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const int i = 4 * w + r;
                    d[r] = (i + k <= 7) ? later_heavier<ARITH>(R[(i + k) & 7][c], R[i][c]) : earlier_heavier<ARITH>(R[(i + k) & 7][c], R[i][c]);
                }
                const uint32_t q0 = prmt(d[0], d[1], 0xFBD9), q1 = prmt(d[2], d[3], 0xFBD9);      // decisions as whole bytes
                cw[2 * c] = prmt(q0, q1, 0x5410);
                cw[2 * c + 1] = prmt(q0, q1, 0x7632);
            }
            const uint32_t p[8] = {cw[7], cw[6], cw[5], cw[4], cw[3], cw[2], cw[1], cw[0]};
            word[w] = gather8<ARITH ? 0xFFu : 0u>(p);
            // rows that wrap around (i + k > 7) compare with an earlier entry: their decisions were not negated
            if constexpr (ARITH) { if (w == 1) word[w] ^= 0xFFFFFFFFu << (8 * (4 - k)); }
        }
        rel.hc[k] = (u64)word[0] | ((u64)word[1] << 32);
    }
    // row relations hr[k]: rows 2i', 2i'+1 are paired, Y[i'][j] = (|x_2i',j|, |x_2i'+1,j|)
    uint32_t Y[4][8];
#pragma unroll
    for (int ip = 0; ip < 4; ++ip)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            Y[ip][2 * c] = prmt(R[2 * ip][c], R[2 * ip + 1][c], 0x5410);
            Y[ip][2 * c + 1] = prmt(R[2 * ip][c], R[2 * ip + 1][c], 0x7632);
        }
    rel.hr[1] = row_relation<ARITH, 1>(Y); rel.hr[2] = row_relation<ARITH, 2>(Y);
    rel.hr[3] = row_relation<ARITH, 3>(Y); rel.hr[4] = row_relation<ARITH, 4>(Y);
    complete_relations8(rel);
}

// The row relations alone (1-D pruning along rows needs no column relation)
template <bool ARITH>
__device__ __forceinline__ void row_relations48_bf16(const uint32_t (&R)[8][4], Rel48& rel) {
    uint32_t Y[4][8];
#pragma unroll
    for (int ip = 0; ip < 4; ++ip)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            Y[ip][2 * c] = prmt(R[2 * ip][c], R[2 * ip + 1][c], 0x5410);
            Y[ip][2 * c + 1] = prmt(R[2 * ip][c], R[2 * ip + 1][c], 0x7632);
        }
    rel.hr[1] = row_relation<ARITH, 1>(Y); rel.hr[2] = row_relation<ARITH, 2>(Y);
    rel.hr[3] = row_relation<ARITH, 3>(Y); rel.hr[4] = row_relation<ARITH, 4>(Y);
    complete_row_relations8(rel);
}

// ---- fp32: scalar comparisons ------------------------------------------------------------------
__device__ __forceinline__ void relations48_f32(const unsigned char* blk, Rel48& rel, uint32_t& worst) {
    uint32_t u[64];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint4 a = *reinterpret_cast<const uint4*>(blk + i * 1024), b = *reinterpret_cast<const uint4*>(blk + i * 1024 + 16);
        u[8 * i] = a.x & 0x7FFFFFFFu; u[8 * i + 1] = a.y & 0x7FFFFFFFu; u[8 * i + 2] = a.z & 0x7FFFFFFFu; u[8 * i + 3] = a.w & 0x7FFFFFFFu;
        u[8 * i + 4] = b.x & 0x7FFFFFFFu; u[8 * i + 5] = b.y & 0x7FFFFFFFu; u[8 * i + 6] = b.z & 0x7FFFFFFFu; u[8 * i + 7] = b.w & 0x7FFFFFFFu;
    }
#pragma unroll
    for (int p = 0; p < 64; ++p) worst = max(worst, u[p]);
#pragma unroll
    for (int k = 1; k <= 4; ++k) {
        uint32_t rw[2] = {0, 0}, cw[2] = {0, 0};
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int bit = 8 * (i & 3) + j;
                if (!(k == 4 && j >= 4)) {
                    const int jj = (j + k) & 7;          // later position: ties count as heavier
                    const bool h = (j + k <= 7) ? (u[8 * i + jj] >= u[8 * i + j]) : (u[8 * i + jj] > u[8 * i + j]);
                    rw[i >> 2] |= (h ? 1u : 0u) << bit;
                }
                if (!(k == 4 && i >= 4)) {
                    const int ii = (i + k) & 7;
                    const bool h = (i + k <= 7) ? (u[8 * ii + j] >= u[8 * i + j]) : (u[8 * ii + j] > u[8 * i + j]);
                    cw[i >> 2] |= (h ? 1u : 0u) << bit;
                }
            }
        rel.hr[k] = (u64)rw[0] | ((u64)rw[1] << 32);
        rel.hc[k] = (u64)cw[0] | ((u64)cw[1] << 32);
    }
    complete_relations8(rel);
}

// ---- fp32, finite data: subtractions on the floating-point pipe ------------------------------------
// The sign of |q| - |p| decides "q lighter than p" exactly (a difference of two finite floats is zero only for equal
// operands and never changes sign in rounding; denormals are kept).  One subtraction per comparison runs on the
// multiply-add pipe, one funnel shift pushes its sign bit into the relation word: half the logic-pipe work of a
// compare-and-set pair.  A partner at a later position is heavier on ties, so for it the pushed bit is the complement
// of the relation (turned by one constant per word at the end); a partner at an earlier position (the line wrapped
// around) needs a strictly larger magnitude, and |p| - |q| gives the relation itself.
__device__ __forceinline__ uint32_t push_sign(uint32_t acc, float d) { return __funnelshift_l(__float_as_uint(d), acc, 1); }

__device__ __forceinline__ void relations48_f32_arith(const float (&f)[64], Rel48& rel) {
#pragma unroll
    for (int k = 1; k <= 4; ++k) {
        uint32_t rw[2], cw[2] = {0, 0};
        // rows: bit 8r + j of word w <- entry (4w + r, j) against (4w + r, j + k mod 8); k = 4: columns 0..3 only
#pragma unroll
        for (int w = 0; w < 2; ++w) {
            uint32_t acc = 0;
#pragma unroll
            for (int r = 3; r >= 0; --r) {
                const int i = 4 * w + r;
                if (k == 4 && r != 3) acc <<= 4;
#pragma unroll
                for (int j = (k == 4 ? 3 : 7); j >= 0; --j) {
                    const int jj = (j + k) & 7;
                    const float a = fabsf(f[8 * i + jj]), b = fabsf(f[8 * i + j]);
                    acc = push_sign(acc, (j + k <= 7) ? a - b : b - a);
                }
            }
            const uint32_t later = k == 4 ? 0x0F0F0F0Fu : 0x01010101u * ((1u << (8 - k)) - 1u);      // partners that did not wrap
            rw[w] = acc ^ later;
        }
        // columns: bit 8r + j of word w <- entry (4w + r, j) against (4w + r + k mod 8, j); k = 4: rows 0..3 only
#pragma unroll
        for (int w = 0; w < 2; ++w) {
            if (k == 4 && w == 1) continue;
            uint32_t acc = 0, later = 0;
#pragma unroll
            for (int r = 3; r >= 0; --r) {
                const int i = 4 * w + r, ii = (i + k) & 7;
                if (i + k <= 7) later |= 0xFFu << (8 * r);
#pragma unroll
                for (int j = 7; j >= 0; --j) {
                    const float a = fabsf(f[8 * ii + j]), b = fabsf(f[8 * i + j]);
                    acc = push_sign(acc, (i + k <= 7) ? a - b : b - a);
                }
            }
            cw[w] = acc ^ later;
        }
        rel.hr[k] = (u64)rw[0] | ((u64)rw[1] << 32);
        rel.hc[k] = (u64)cw[0] | ((u64)cw[1] << 32);
    }
    complete_relations8(rel);
}

// The row relations alone, finite fp32 data (see relations48_f32_arith)
__device__ __forceinline__ void row_relations48_f32_arith(const float (&f)[64], Rel48& rel) {
#pragma unroll
    for (int k = 1; k <= 4; ++k) {
        uint32_t rw[2];
#pragma unroll
        for (int w = 0; w < 2; ++w) {
            uint32_t acc = 0;
#pragma unroll
            for (int r = 3; r >= 0; --r) {
                const int i = 4 * w + r;
                if (k == 4 && r != 3) acc <<= 4;
#pragma unroll
                for (int j = (k == 4 ? 3 : 7); j >= 0; --j) {
                    const int jj = (j + k) & 7;
                    const float a = fabsf(f[8 * i + jj]), b = fabsf(f[8 * i + j]);
                    acc = push_sign(acc, (j + k <= 7) ? a - b : b - a);
                }
            }
            const uint32_t later = k == 4 ? 0x0F0F0F0Fu : 0x01010101u * ((1u << (8 - k)) - 1u);
            rw[w] = acc ^ later;
        }
        rel.hr[k] = (u64)rw[0] | ((u64)rw[1] << 32);
    }
    complete_row_relations8(rel);
}

// magnitude pattern of entry p of the lane's block, read back from the stage
template <int DT>
__device__ __forceinline__ uint32_t key_at(const unsigned char* blk, int p) {
    if constexpr (DT == kBF16) return *reinterpret_cast<const unsigned short*>(blk + (p >> 3) * 512 + (p & 7) * 2) & 0x7FFFu;
    else return *reinterpret_cast<const uint32_t*>(blk + (p >> 3) * 1024 + (p & 7) * 4) & 0x7FFFFFFFu;
}

// Step C, scalar half (see swap_apply8): set bits are visited in ascending position.
template <int DT>
__device__ __forceinline__ bool swap_apply8_smem(const unsigned char* blk, u64& kept, u64 cands, u64 free_a, u64 free_b) {
    if (!cands) return false;
    int x = -1; uint32_t best = 0;
    for (int n = 0; n < 64 && cands; ++n) {
        const int p = __ffsll((long long)cands) - 1;
        cands &= cands - 1;
        const uint32_t kp = key_at<DT>(blk, p);
        if (x < 0 || kp < best) { x = p; best = kp; }
    }
    const int r2 = x >> 3, c2 = x & 7;
    u64 ca = free_a & (0x0101010101010101ull << c2), cb = free_b & (0xFFull << (8 * r2));
    int a = -1, b = -1; uint32_t ka = 0, kb = 0;
    for (int n = 0; n < 8 && ca; ++n) {
        const int e = __ffsll((long long)ca) - 1; ca &= ca - 1;
        const uint32_t k = key_at<DT>(blk, e);
        if (a < 0 || k >= ka) { a = e; ka = k; }
    }
    for (int n = 0; n < 8 && cb; ++n) {
        const int e = __ffsll((long long)cb) - 1; cb &= cb - 1;
        const uint32_t k = key_at<DT>(blk, e);
        if (b < 0 || k >= kb) { b = e; kb = k; }
    }
    if (a < 0 || b < 0) return false;
    kept = (kept & ~(1ull << x)) | (1ull << a) | (1ull << b);
    return true;
}

// Masked weights back into the stage, mask bytes, objective contribution of the lane's block.
template <int DT, bool HAS_OUT>
__device__ __forceinline__ float back_end48(unsigned char* blk, unsigned char* mrow /* [8][32] */, const uint4* lut, int lane, u64 kept) {
    float s8 = 0.f;
    const uint32_t kw[2] = {(uint32_t)kept, (uint32_t)(kept >> 32)};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t word = kw[i >> 2];
        const uint32_t mb = (i & 3) == 0 ? (word & 0xFFu) : prmt(word, 0u, 0x4440 + (i & 3));      // the row's mask byte
        if constexpr (DT == kBF16) {
            const uint4 r = *reinterpret_cast<const uint4*>(blk + i * 512);
            const uint4 mm = lut[mb];                  // 16-bit lane masks of the row's eight keep flags
            const uint32_t raw[4] = {r.x, r.y, r.z, r.w}, m4[4] = {mm.x, mm.y, mm.z, mm.w};
            uint32_t o[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t m = m4[c];
                o[c] = raw[c] & m;
                const uint32_t ab = abs_bf16x2(o[c]);
                unsigned short lo, hi;
                asm("mov.b32 {%0,%1}, %2;" : "=h"(lo), "=h"(hi) : "r"(ab));
                asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(s8) : "h"(lo));
                asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(s8) : "h"(hi));
            }
            if constexpr (HAS_OUT) *reinterpret_cast<uint4*>(blk + i * 512) = make_uint4(o[0], o[1], o[2], o[3]);
        } else {
            const uint4 ra = *reinterpret_cast<const uint4*>(blk + i * 1024), rb = *reinterpret_cast<const uint4*>(blk + i * 1024 + 16);
            const uint4 ka = lut[2 * mb], kb = lut[2 * mb + 1];          // the row's keep flags as words of 0 or 1
            const uint32_t raw[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w}, k01[8] = {ka.x, ka.y, ka.z, ka.w, kb.x, kb.y, kb.z, kb.w};
            uint32_t o[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                o[q] = raw[q] * k01[q];                                  // the bits themselves or +0: an integer product, off the logic pipe
                s8 += fabsf(__uint_as_float(o[q]));
            }
            if constexpr (HAS_OUT) {
                *reinterpret_cast<uint4*>(blk + i * 1024) = make_uint4(o[0], o[1], o[2], o[3]);
                *reinterpret_cast<uint4*>(blk + i * 1024 + 16) = make_uint4(o[4], o[5], o[6], o[7]);
            }
        }
        mrow[i * 32 + lane] = (unsigned char)mb;
    }
    return s8;
}

template <int DT, int METHOD, bool HAS_OUT>
__global__ void __launch_bounds__(Geo48<DT, METHOD>::kWarps * 32, 1)
tma48_kernel(const __grid_constant__ TmaEntry single, const TmaEntry* __restrict__ table, int count, long long total_items,
             double* __restrict__ partials, int* __restrict__ status_out, unsigned int* __restrict__ done, int n_keep,
             unsigned long long* __restrict__ vpartials) {
    using G = Geo48<DT, METHOD>;
    constexpr bool kRows = METHOD == kMethodRows;        // 1-D n_keep of 8 along rows: row relations only, no steps A to C
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned char* stages = smem_raw + (size_t)warp * G::kWarpBytes;
    unsigned char* mbytes = stages + G::kStages * G::kStageBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(mbytes + 256);
    uint4* lut = reinterpret_cast<uint4*>(smem_raw + (size_t)G::kWarps * G::kWarpBytes);
    // the only CTA-wide step: the table of keep flags
    if constexpr (DT == kBF16) fill_lane_lut(lut, threadIdx.x, G::kWarps * 32); else fill_keep_lut32(lut, threadIdx.x, G::kWarps * 32);
    __syncthreads();

    const long long gw = (long long)blockIdx.x * G::kWarps + warp, nwarps = (long long)gridDim.x * G::kWarps;
    // where this warp's objective partial for matrix k goes: k * pstride + pbase (a launch over several matrices that reduces
    // its own objectives packs them: slot = the warp's place in the deal + k, see finish_objectives_ranged)
    const bool ranged = done != nullptr && count > 1;
    const long long pstride = ranged ? 1 : nwarps, pbase = ranged ? (long long)warp * gridDim.x + blockIdx.x : gw;
    // Algorithm 1 alone takes its items round-robin over the warps of the grid (one dense window of the matrix at a time),
    // the full search contiguous ranges (see the 2:4 kernel)
    constexpr bool kRoundRobin = METHOD != kMethodApprox;
    int n_items;
    long long begin;
    if constexpr (kRoundRobin) {
        begin = (long long)warp * gridDim.x + blockIdx.x;
        n_items = begin < total_items ? (int)((total_items - begin + nwarps - 1) / nwarps) : 0;
    } else {
        begin = even_share(total_items, G::kWarps, n_items);
    }
    const TmaEntry* tab = table ? table : &single;

    if (lane == 0) {
        for (int s = 0; s < G::kStages; ++s) mbar_init(&bars[s], 1);
        fence_mbar_init();
    }
    __syncwarp();

    typename std::conditional<kRoundRobin, StrideCursor, Cursor>::type ld, cur;
    if constexpr (kRoundRobin) ld.seek(tab, count, begin, (int)nwarps); else ld.seek(tab, count, begin);
    cur = ld;
    int loaded = 0;
    auto issue_next = [&]() {              // all lanes track the cursor, lane 0 issues the copy
        const int s = loaded % G::kStages;
        if (lane == 0) {
            mbar_expect_tx(&bars[s], G::kStageBytes);
            tma_load_2d(stages + s * G::kStageBytes, &tab[ld.k].in, ld.cj * kCols8, ld.bi * kRows8, &bars[s]);
        }
        ld.advance(tab, count);
        ++loaded;
    };
    for (int g = 0; g < G::kStages - 1 && loaded < n_items; ++g) issue_next();

    int status = 0, acc_k = -1;
    float facc = 0.f; double acc = 0.0;
    uint32_t worst = 0;
    // the matrix in process: the fields every item needs
    int p_cols = 0, p_wpr = 0, p_rows = 0;
    uint32_t* p_mask = nullptr;
    unsigned long long viol = 0;                         // kRows: non-zero entries pruned by this lane
    u64 nonzero = 0;

    for (int it = 0; it < n_items; ++it) {
        const int s = it % G::kStages;
        const uint32_t parity = (uint32_t)((it / G::kStages) & 1);
        if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(&bars[s], parity))) {
            status |= kDevInternal;
            if (lane == 0)                 // give the copies still in flight a bounded chance to land before the stages die
                for (int j = it + 1; j < loaded; ++j) mbar_wait_bounded(&bars[j % G::kStages], (uint32_t)((j / G::kStages) & 1), 1u << 14);
            break;
        }
        unsigned char* stage = stages + s * G::kStageBytes;
        unsigned char* blk = stage + lane * (8 * G::kElem);

        Rel48 rel;
        if constexpr (DT == kBF16) {
            uint32_t R[8][4];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint4 v = *reinterpret_cast<const uint4*>(blk + i * 512);
                R[i][0] = abs_bf16x2(v.x); R[i][1] = abs_bf16x2(v.y); R[i][2] = abs_bf16x2(v.z); R[i][3] = abs_bf16x2(v.w);
                worst = max_u16x2_(worst, max_u16x2_(max_u16x2_(R[i][0], R[i][1]), max_u16x2_(R[i][2], R[i][3])));
            }
            if (__any_sync(0xFFFFFFFFu, nonfinite_bf16x2(worst))) {        // Inf or NaN met: integer keys, bit-pattern order
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const uint4 v = *reinterpret_cast<const uint4*>(blk + i * 512);
                    R[i][0] = v.x & 0x7FFF7FFFu; R[i][1] = v.y & 0x7FFF7FFFu; R[i][2] = v.z & 0x7FFF7FFFu; R[i][3] = v.w & 0x7FFF7FFFu;
                }
                if constexpr (kRows) row_relations48_bf16<false>(R, rel); else relations48_bf16<false>(R, rel);
            } else {
                if constexpr (kRows) row_relations48_bf16<true>(R, rel); else relations48_bf16<true>(R, rel);
            }
            if constexpr (kRows) {                       // x + 0x7FFF sets the top bit of a 15-bit magnitude iff x != 0
                uint32_t nz[2] = {0, 0};
#pragma unroll
                for (int i = 0; i < 8; ++i)
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const uint32_t t = (R[i][c] & 0x7FFF7FFFu) + 0x7FFF7FFFu;
                        nz[i >> 2] |= (((t >> 15) & 1u) | ((t >> 30) & 2u)) << (8 * (i & 3) + 2 * c);
                    }
                nonzero = (u64)nz[0] | ((u64)nz[1] << 32);
            }
        } else {
            float f[64];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float4 a = *reinterpret_cast<const float4*>(blk + i * 1024), b = *reinterpret_cast<const float4*>(blk + i * 1024 + 16);
                f[8 * i] = a.x; f[8 * i + 1] = a.y; f[8 * i + 2] = a.z; f[8 * i + 3] = a.w;
                f[8 * i + 4] = b.x; f[8 * i + 5] = b.y; f[8 * i + 6] = b.z; f[8 * i + 7] = b.w;
            }
            // Inf / NaN watch on the multiply-add pipe: x * 0 + acc stays 0 for finite data and turns NaN otherwise
            float watch = 0.f;
#pragma unroll
            for (int p = 0; p < 64; ++p) watch = fmaf(f[p], 0.f, watch);
            if (__any_sync(0xFFFFFFFFu, watch != watch)) relations48_f32(blk, rel, worst);       // integer keys, bit-pattern order
            else if constexpr (kRows) row_relations48_f32_arith(f, rel);
            else relations48_f32_arith(f, rel);
            if constexpr (kRows) {
                uint32_t nz[2] = {0, 0};
#pragma unroll
                for (int p = 0; p < 64; ++p) nz[p >> 5] |= ((__float_as_uint(f[p]) & 0x7FFFFFFFu) ? 1u : 0u) << (p & 31);
                nonzero = (u64)nz[0] | ((u64)nz[1] << 32);
            }
        }
        // refill the stage of the previous item -- its store, issued one item ago, has long been read -- so that the copy
        // runs under the rest of this item
        if (loaded < n_items) {
            if constexpr (HAS_OUT) { if (lane == 0 && it > 0) tma_wait_read<0>(); }
            __syncwarp();
            issue_next();
        }
        u64 kept = kRows ? keep_rows_8(rel, n_keep) : cover_4_8(rel);
        if constexpr (METHOD == kMethodApprox) {
            Short48 L = line_short(kept);
            u64 cand = open_candidates8(kept, L);
            // three full rounds are needed by every warp of ordinary data (some block of its 32 still has candidates):
            // they run without asking
#pragma unroll 1                                                           // one copy of the round's code: the loop body is large
            for (int round = 0; round < 3; ++round) {
                kept |= fill_accept8(rel, kept, cand);
                L = line_short(kept);
                cand = open_candidates8(kept, L);
            }
            if (__any_sync(0xFFFFFFFFu, cand != 0)) {
                // a block that still has candidates has, as a rule, exactly one: it has no rival in its row or column and
                // is taken as it stands
                if ((cand & (cand - 1)) == 0) kept |= cand;
                L = line_short(kept);
                cand = open_candidates8(kept, L);
                int rounds = 3;
                while (__any_sync(0xFFFFFFFFu, cand != 0)) {
                    if (++rounds > 16) { status |= kDevInternal; break; }  // a block lacks at most sixteen entries
                    kept |= fill_accept8(rel, kept, cand);
                    L = line_short(kept);
                    cand = open_candidates8(kept, L);
                }
            }
            int swaps = 0;
            while (__any_sync(0xFFFFFFFFu, L.row_short != 0)) {
                if (++swaps > 5) { status |= kDevInternal; break; }       // at most N*N/4 = 4 swaps per block
                if (L.row_short) {
                    u64 fa, fb;
                    const u64 c = swap_candidates8(rel, L, kept, fa, fb);
                    if (!swap_apply8_smem<DT>(blk, kept, c, fa, fb)) { status |= kDevInternal; L.row_short = 0; }
                    else L = line_short(kept);
                }
            }
        }
        if (cur.k != acc_k) {                                              // a new matrix starts: flush the objective partial
            if (acc_k >= 0) {
                acc += (double)facc;
                for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
                if (lane == 0) partials[(long long)acc_k * pstride + pbase] = acc;
            }
            acc = 0.0; facc = 0.f; acc_k = cur.k;
            const DevProblem& P = tab[cur.k].p;
            p_cols = (int)P.cols; p_wpr = P.wpr; p_mask = P.mask; p_rows = (int)P.rows;
        }
        if (cur.cj * kCols8 + lane * 8 >= p_cols) kept = 0;               // blocks past the last column (zero-filled by the copy)
        if constexpr (kRows) {
            // pruned non-zero entries; rows past the last one (the 1-D pruning takes any number of rows) and blocks past the
            // last column were zero-filled by the copy and count nothing
            if (cur.cj * kCols8 + lane * 8 < p_cols) viol += (unsigned)__popcll(~kept & nonzero);
        }
        facc += back_end48<DT, HAS_OUT>(blk, mbytes, lut, lane, kept);
        if constexpr (HAS_OUT) fence_proxy_async_smem();
        __syncwarp();
        if constexpr (HAS_OUT) {
            if (lane == 0) { tma_store_2d(&tab[cur.k].out, cur.cj * kCols8, cur.bi * kRows8, stage); tma_commit(); }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {                                      // 8 rows x 8 words of mask
            const int idx = lane + 32 * h, row = idx >> 3, word = cur.cj * 8 + (idx & 7);
            const uint32_t w = *reinterpret_cast<const uint32_t*>(mbytes + row * 32 + (idx & 7) * 4);
            if (word < p_wpr && (!kRows || cur.bi * kRows8 + row < p_rows)) p_mask[((long long)cur.bi * kRows8 + row) * p_wpr + word] = w;
        }
        cur.advance(tab, count);
        if ((it & 15) == 15) { acc += (double)facc; facc = 0.f; }           // keep the fp32 partial short
        __syncwarp();
    }
    if (lane == 0) tma_wait_all<0>();
    if (acc_k >= 0 || (done && count == 1)) {  // a single-matrix launch that reduces its own objective wants a partial (a zero) from idle warps too
        acc += (double)facc;
        for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        if (lane == 0) partials[(long long)(acc_k >= 0 ? acc_k : 0) * pstride + pbase] = acc;
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

template <int DT, int METHOD, bool HAS_OUT>
cudaError_t launch_one48(const TmaLaunch& a, const TmaEntry& single, const TmaEntry* table) {
    using G = Geo48<DT, METHOD>;
    const size_t smem = (size_t)G::kWarps * G::kWarpBytes + G::kLutBytes;
    auto kern = tma48_kernel<DT, METHOD, HAS_OUT>;
    static PerDeviceOnce configured;       // per instantiation
    const cudaError_t e = configured.run([&] { return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); });
    if (e != cudaSuccess) return e;
    kern<<<a.ctas, G::kWarps * 32, smem, a.stream>>>(single, table, a.count, a.total_items, a.partials, a.status, a.done, a.n_keep, a.vpartials);
    return cudaGetLastError();
}

}  // namespace

// fp32 with the full search runs on the kernel that splits a block over two lanes (tm_kernels_tma48s.cu)
static bool takes_split_kernel(int dtype, int method) { return dtype == kF32 && method == kMethodApprox; }
int tma48_item_cols(int dtype, int method) { return takes_split_kernel(dtype, method) ? tma48s_item_cols() : kCols8; }

int tma48_warps_per_cta(int dtype, int method) {
    if (takes_split_kernel(dtype, method)) return tma48s_warps_per_cta();
    if (method == kMethodApprox) return dtype == kF32 ? Geo48<kF32, kMethodApprox>::kWarps : Geo48<kBF16, kMethodApprox>::kWarps;
    return dtype == kF32 ? Geo48<kF32, kMethodCover>::kWarps : Geo48<kBF16, kMethodCover>::kWarps;
}

cudaError_t launch_tma48(const TmaLaunch& a) {
    const int wpc = tma48_warps_per_cta(a.dtype, a.method);
    // a.done (set only for a single matrix with work items): the search kernel is the whole call
    cudaError_t err = cudaSuccess;
    if (!a.done) err = cudaMemsetAsync(a.partials, 0, sizeof(double) * (size_t)a.count * (size_t)a.ctas * wpc, a.stream);
    if (err != cudaSuccess) return err;
    const TmaEntry* host = static_cast<const TmaEntry*>(a.entries_host);
    const TmaEntry* table = static_cast<const TmaEntry*>(a.entries_dev);
    if (a.total_items > 0) {
#define TM_DISPATCH(DT, METHOD)                                                                                   \
    err = a.has_out ? launch_one48<DT, METHOD, true>(a, host[0], table) : launch_one48<DT, METHOD, false>(a, host[0], table)
        if (takes_split_kernel(a.dtype, a.method)) err = launch_tma48s(a);
        else if (a.dtype == kF32) { if (a.method == kMethodRows) TM_DISPATCH(kF32, kMethodRows); else TM_DISPATCH(kF32, kMethodCover); }
        else { if (a.method == kMethodApprox) TM_DISPATCH(kBF16, kMethodApprox); else if (a.method == kMethodRows) TM_DISPATCH(kBF16, kMethodRows); else TM_DISPATCH(kBF16, kMethodCover); }
#undef TM_DISPATCH
        if (err != cudaSuccess) return err;
    }
    if (a.done) return cudaSuccess;
    if (a.method == kMethodRows) return cudaSuccess;          // the caller sums objective and violation partials together
    return tma_reduce(a.entries_host, a.entries_dev, a.count, a.partials, (long long)a.ctas * wpc, a.stream);
}

}  // namespace tmask
