// Approximate 4:8 search on fp32 matrices (TM_APPROX, M = 8): an 8x8 block split over two lanes.
//
// The one-lane-per-block kernel (tm_kernels_tma48.cu) holds a block's sets as 64-bit masks and its 14 relation
// masks in 28 registers; on fp32 data its 8 KB work items leave room for 12 warps per SM, and the long dependent
// chains of the search then wait on one another.  Here lane 2b + h of a warp owns rows 4h .. 4h+3 of block b of the
// item (8 rows x 128 columns, 16 blocks, 4 KB): every set is one 32-bit word per lane (byte r = row 4h + r), row
// operations stay inside the lane, column operations fetch the partner's word with one shuffle and splice the rows
// with one byte permute.  The instruction count per block is about the same; the state per thread halves, 24 warps
// fit an SM, and the code per item is half as long.
//
//   front end  |q| - |p| on the floating-point pipe, the sign funnel-shifted into the relation word (see
//              tm_kernels_tma48.cu); a lane compares its rows with one another and with the four rows that follow
//              them cyclically.  For the upper half those rows wrap around to the block's first rows, i.e. to earlier
//              positions, where a tie counts the other way: the difference passes through d * s + 0 with s = -1, which
//              turns the sign and leaves a tie at +0.
//   steps A, B, C and the back end as in the one-lane kernel, on half sets (tm_core48.cuh names the rules).
#include "tm_core48.cuh"
#include "tm_launch.h"
#include "tm_pair_bf16.cuh"
#include "tm_tma.cuh"
#include "tm_tma_items.cuh"

namespace tmask {

namespace {

constexpr int kSRows = 8, kSCols = 128;
constexpr int kSWarps = 24, kSStages = 2;
constexpr int kSRowPitch = kSCols * 4, kSStageBytes = kSRows * kSRowPitch;
// stages | mask bytes [8 rows][16 blocks] | barriers (stages stay 128-byte aligned)
constexpr int kSWarpBytes = kSStages * kSStageBytes + 128 + 128;
static_assert(kSWarpBytes % 128 == 0, "stages stay 128-byte aligned");
constexpr int kSLutBytes = 256 * 32;
constexpr unsigned kAll = 0xFFFFFFFFu;

__device__ __forceinline__ uint32_t maj3w(uint32_t a, uint32_t b, uint32_t c) { return (a & b) | (c & (a | b)); }
__device__ __forceinline__ uint32_t four_of_seven_w(uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t e, uint32_t f, uint32_t g) {
    const uint32_t s1 = a ^ b ^ c, k1 = maj3w(a, b, c), s2 = d ^ e ^ f, k2 = maj3w(d, e, f);
    return maj3w(k1, k2, maj3w(s1, s2, g));
}
// every byte rotated right by K: result bit (r, j) = x bit (r, (j + K) mod 8)
template <int K> __device__ __forceinline__ uint32_t rot_row_w(uint32_t x) {
    constexpr uint32_t lo = 0x01010101u * ((1u << (8 - K)) - 1u);
    return ((x >> K) & lo) | ((x << (8 - K)) & ~lo);
}
// the block's rows moved up by K: my row r receives row (4h + r + K) mod 8 -- from my own word or the partner's
template <int K> __device__ __forceinline__ uint32_t rot_col_w(uint32_t mine) {
    const uint32_t other = __shfl_xor_sync(kAll, mine, 1);
    if constexpr (K == 4) return other;
    constexpr int k = K < 4 ? K : K - 4;
    constexpr uint32_t sel = k | ((k + 1) << 4) | ((k + 2) << 8) | ((k + 3) << 12);
    return K < 4 ? prmt(mine, other, sel) : prmt(other, mine, sel);
}

struct RelHalf {
    uint32_t hr[8], hc[8];      // index 1..7: my four rows of the block's relation masks
};

__device__ __forceinline__ uint32_t push_sign_w(uint32_t acc, float d) { return __funnelshift_l(__float_as_uint(d), acc, 1); }

// Relations of my rows from the stage.  blk: the block's first row; h: my half.  Finite data only.
__device__ __forceinline__ void relations_half(const unsigned char* blk, int h, RelHalf& rel) {
    float g[4][8];                                       // my rows
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const float4 a = *reinterpret_cast<const float4*>(blk + (4 * h + r) * kSRowPitch), b = *reinterpret_cast<const float4*>(blk + (4 * h + r) * kSRowPitch + 16);
        g[r][0] = fabsf(a.x); g[r][1] = fabsf(a.y); g[r][2] = fabsf(a.z); g[r][3] = fabsf(a.w);
        g[r][4] = fabsf(b.x); g[r][5] = fabsf(b.y); g[r][6] = fabsf(b.z); g[r][7] = fabsf(b.w);
    }
    // rows: entry (r, j) against (r, j + k mod 8); k = 4 for columns 0..3 only (the rest by antisymmetry)
#pragma unroll
    for (int k = 1; k <= 4; ++k) {
        uint32_t acc = 0;
#pragma unroll
        for (int r = 3; r >= 0; --r) {
            if (k == 4 && r != 3) acc <<= 4;
#pragma unroll
            for (int j = (k == 4 ? 3 : 7); j >= 0; --j) {
                const int jj = (j + k) & 7;
                acc = push_sign_w(acc, (j + k <= 7) ? g[r][jj] - g[r][j] : g[r][j] - g[r][jj]);
            }
        }
        rel.hr[k] = acc ^ (k == 4 ? 0x0F0F0F0Fu : 0x01010101u * ((1u << (8 - k)) - 1u));     // later partners: the pushed bit was the complement
    }
    // columns: entry (r, j) against the row k further on (cyclically), k = 1..4.  Rows r + k <= 3 are mine; the others are
    // the partner's, read from the stage.  For the upper half they lie earlier in the block: sign turned, tie kept at +0.
    const float turn = h ? -1.f : 1.f;
    uint32_t acc[5] = {0, 0, 0, 0, 0};
#pragma unroll
    for (int r = 3; r >= 0; --r) {
#pragma unroll
        for (int k = 1; k <= 4; ++k) {
            float q[8];
            if (r + k <= 3) {
#pragma unroll
                for (int j = 0; j < 8; ++j) q[j] = g[r + k][j];
            } else {
                const unsigned char* src = blk + ((4 * h + r + k) & 7) * kSRowPitch;
                const float4 a = *reinterpret_cast<const float4*>(src), b = *reinterpret_cast<const float4*>(src + 16);
                q[0] = fabsf(a.x); q[1] = fabsf(a.y); q[2] = fabsf(a.z); q[3] = fabsf(a.w);
                q[4] = fabsf(b.x); q[5] = fabsf(b.y); q[6] = fabsf(b.z); q[7] = fabsf(b.w);
            }
#pragma unroll
            for (int j = 7; j >= 0; --j) {
                const float d = q[j] - g[r][j];
                acc[k] = push_sign_w(acc[k], (r + k <= 3) ? d : fmaf(d, turn, 0.f));
            }
        }
    }
#pragma unroll
    for (int k = 1; k <= 4; ++k) {
        // bits of rows whose partner is a later position hold the complement of the relation; for the upper half the rows
        // with r + k > 3 compared with an earlier position and hold the relation itself
        uint32_t later_upper = 0;
#pragma unroll
        for (int r = 0; r < 4; ++r) if (r + k <= 3) later_upper |= 0xFFu << (8 * r);
        rel.hc[k] = acc[k] ^ (h ? later_upper : 0xFFFFFFFFu);
    }
    // the remaining distances by antisymmetry: h[8-k] bit (i, j + k) = not h[k] bit (i, j)
    rel.hr[4] = (rel.hr[4] & 0x0F0F0F0Fu) | ((~rel.hr[4] << 4) & 0xF0F0F0F0u);
    rel.hr[7] = ~rot_row_w<7>(rel.hr[1]); rel.hr[6] = ~rot_row_w<6>(rel.hr[2]); rel.hr[5] = ~rot_row_w<5>(rel.hr[3]);
    rel.hc[7] = ~rot_col_w<7>(rel.hc[1]); rel.hc[6] = ~rot_col_w<6>(rel.hc[2]); rel.hc[5] = ~rot_col_w<5>(rel.hc[3]);
}

// Integer keys for data with Inf or NaN (bit-pattern order): my rows against all rows, the plain way.
__device__ __forceinline__ void relations_half_int(const unsigned char* blk, int h, RelHalf& rel) {
#pragma unroll
    for (int k = 1; k <= 7; ++k) { rel.hr[k] = 0; rel.hc[k] = 0; }
    for (int r = 0; r < 4; ++r) {
        const int i = 4 * h + r;
        for (int j = 0; j < 8; ++j) {
            const uint32_t p = *reinterpret_cast<const uint32_t*>(blk + i * kSRowPitch + 4 * j) & 0x7FFFFFFFu;
#pragma unroll
            for (int k = 1; k <= 7; ++k) {
                const int jj = (j + k) & 7, ii = (i + k) & 7;
                const uint32_t qr = *reinterpret_cast<const uint32_t*>(blk + i * kSRowPitch + 4 * jj) & 0x7FFFFFFFu;
                const uint32_t qc = *reinterpret_cast<const uint32_t*>(blk + ii * kSRowPitch + 4 * j) & 0x7FFFFFFFu;
                const bool hr = jj > j ? qr >= p : qr > p, hc = ii > i ? qc >= p : qc > p;        // the later of equals is the heavier
                rel.hr[k] |= (hr ? 1u : 0u) << (8 * r + j);
                rel.hc[k] |= (hc ? 1u : 0u) << (8 * r + j);
            }
        }
    }
}

struct ShortHalf { uint32_t row_short, col_short; };
// Lines that still lack entries (hold fewer than four), replicated over the line's entries of my rows.
__device__ __forceinline__ ShortHalf line_short_w(uint32_t kept) {
    ShortHalf L;
    {   // rows: popcount of every byte; 4 is the only count with bit 2 set (no row ever holds more)
        uint32_t c = kept - ((kept >> 1) & 0x55555555u);
        c = (c & 0x33333333u) + ((c >> 2) & 0x33333333u);
        c += c >> 4;
        L.row_short = ~(((c >> 2) & 0x01010101u) * 255u);
    }
    {   // columns: my four rows as a 3-bit count per column, added to the partner's; a column never holds more than four
        const uint32_t b0 = kept, b1 = kept >> 8, b2 = kept >> 16, b3 = kept >> 24;
        const uint32_t s = b0 ^ b1 ^ b2, c = maj3w(b0, b1, b2);
        const uint32_t ones = (s ^ b3) & 0xFFu, c2 = s & b3, twos = (c ^ c2) & 0xFFu, fours = (c & c2) & 0xFFu;
        const uint32_t mine = ones | (twos << 8) | (fours << 16), other = __shfl_xor_sync(kAll, mine, 1);
        const uint32_t c0 = mine & other;                                  // carries of the ones (byte 0), twos (byte 1)
        const uint32_t t = (mine ^ other) >> 8, carry1 = ((mine & other) >> 8) | (t & c0);      // byte 0: twos' sum bit / carry into the fours
        const uint32_t four = (((mine ^ other) >> 16) ^ carry1) & 0xFFu;   // the count's bit 2
        L.col_short = ~(four * 0x01010101u);
    }
    return L;
}

__device__ __forceinline__ uint32_t fill_accept_w(const RelHalf& r, uint32_t kept, uint32_t cand) {
    const uint32_t row_blocked = four_of_seven_w(
        rot_row_w<1>(kept | (cand & ~r.hr[7])), rot_row_w<2>(kept | (cand & ~r.hr[6])), rot_row_w<3>(kept | (cand & ~r.hr[5])),
        rot_row_w<4>(kept | (cand & ~r.hr[4])), rot_row_w<5>(kept | (cand & ~r.hr[3])), rot_row_w<6>(kept | (cand & ~r.hr[2])),
        rot_row_w<7>(kept | (cand & ~r.hr[1])));
    const uint32_t col_blocked = four_of_seven_w(
        rot_col_w<1>(kept | (cand & ~r.hc[7])), rot_col_w<2>(kept | (cand & ~r.hc[6])), rot_col_w<3>(kept | (cand & ~r.hc[5])),
        rot_col_w<4>(kept | (cand & ~r.hc[4])), rot_col_w<5>(kept | (cand & ~r.hc[3])), rot_col_w<6>(kept | (cand & ~r.hc[2])),
        rot_col_w<7>(kept | (cand & ~r.hc[1])));
    return cand & ~(row_blocked | col_blocked);
}

__device__ __forceinline__ uint32_t lighter_in_row_w(const RelHalf& r, uint32_t set) {
    return (rot_row_w<1>(set) & ~r.hr[1]) | (rot_row_w<2>(set) & ~r.hr[2]) | (rot_row_w<3>(set) & ~r.hr[3]) | (rot_row_w<4>(set) & ~r.hr[4]) |
           (rot_row_w<5>(set) & ~r.hr[5]) | (rot_row_w<6>(set) & ~r.hr[6]) | (rot_row_w<7>(set) & ~r.hr[7]);
}
__device__ __forceinline__ uint32_t lighter_in_col_w(const RelHalf& r, uint32_t set) {
    return (rot_col_w<1>(set) & ~r.hc[1]) | (rot_col_w<2>(set) & ~r.hc[2]) | (rot_col_w<3>(set) & ~r.hc[3]) | (rot_col_w<4>(set) & ~r.hc[4]) |
           (rot_col_w<5>(set) & ~r.hc[5]) | (rot_col_w<6>(set) & ~r.hc[6]) | (rot_col_w<7>(set) & ~r.hc[7]);
}
// "some bit of the column is set" over all eight rows, spread over my rows / "some bit of the row" over the row
__device__ __forceinline__ uint32_t any_in_col_w(uint32_t x) {
    x |= x >> 16; x |= x >> 8; x &= 0xFFu;
    x |= __shfl_xor_sync(kAll, x, 1);
    return x * 0x01010101u;
}
__device__ __forceinline__ uint32_t any_in_row_w(uint32_t x) { x |= x >> 4; x |= x >> 2; x |= x >> 1; return (x & 0x01010101u) * 255u; }

__device__ __forceinline__ uint32_t key_at_w(const unsigned char* blk, int h, int p) {       // p: position in my rows, 8 r + j
    return *reinterpret_cast<const uint32_t*>(blk + (4 * h + (p >> 3)) * kSRowPitch + (p & 7) * 4) & 0x7FFFFFFFu;
}

// One swap of step C for the pair's block (both lanes call it; `need`: the block has a short row).  cands: the local minima
// among my eligible entries; free_a / free_b: my free entries of short rows / of short columns.  Returns false on an unexpected
// shape (the mask stays as it is).
__device__ __forceinline__ bool swap_apply_w(const unsigned char* blk, int h, bool need, uint32_t& kept, uint32_t cands, uint32_t free_a, uint32_t free_b) {
    // the lightest marked entry of the block, the earliest of equals: my best first (ascending positions), then the partner's
    uint32_t best = 0xFFFFFFFFu; int x = -1;
    for (uint32_t c = need ? cands : 0u; c; c &= c - 1) {
        const int p = __ffs((int)c) - 1;
        const uint32_t kp = key_at_w(blk, h, p);
        if (kp < best) { best = kp; x = p; }
    }
    const uint32_t obest = __shfl_xor_sync(kAll, best, 1);
    const int ox = __shfl_xor_sync(kAll, x, 1);
    // positions in the block: mine 32 h + x, the partner's 32 (1 - h) + ox
    const bool mine_wins = x >= 0 && (ox < 0 || best < obest || (best == obest && h == 0));
    const bool found = x >= 0 || ox >= 0;
    const int gx = mine_wins ? 32 * h + x : 32 * (1 - h) + ox;              // meaningful when found
    const int r2 = (gx >> 3) & 7, c2 = gx & 7;
    // a: the heaviest free entry of column c2 in a short row (any of the eight rows), the latest of equals
    uint32_t wa = 0; int a = -1;
    for (uint32_t c = (need && found) ? (free_a & (0x01010101u << c2)) : 0u; c; c &= c - 1) {
        const int p = __ffs((int)c) - 1;
        const uint32_t kp = key_at_w(blk, h, p);
        if (kp >= wa) { wa = kp; a = p; }
    }
    const uint32_t owa = __shfl_xor_sync(kAll, wa, 1);
    const int oa = __shfl_xor_sync(kAll, a, 1);
    const bool a_mine = a >= 0 && (oa < 0 || wa > owa || (wa == owa && h == 1));
    const bool a_found = a >= 0 || oa >= 0;
    // b: the heaviest free entry of row r2 in a short column: the lane that owns the row looks
    const bool owner = (r2 >> 2) == h;
    uint32_t wb = 0; int b = -1;
    for (uint32_t c = (need && found && owner) ? (free_b & (0xFFu << (8 * (r2 & 3)))) : 0u; c; c &= c - 1) {
        const int p = __ffs((int)c) - 1;
        const uint32_t kp = key_at_w(blk, h, p);
        if (kp >= wb) { wb = kp; b = p; }
    }
    const int ob = __shfl_xor_sync(kAll, b, 1);
    const bool b_found = owner ? b >= 0 : ob >= 0;
    const bool ok = found && a_found && b_found;
    if (need && ok) {
        if (mine_wins) kept &= ~(1u << x);
        if (a_mine) kept |= 1u << a;
        if (owner) kept |= 1u << b;
    }
    return !need || ok;
}

// Masked weights of my four rows back into the stage, their mask bytes, my share of the objective.
template <bool HAS_OUT>
__device__ __forceinline__ float back_end_w(unsigned char* blk, int h, unsigned char* mrow /* [8][16] */, const uint4* lut, int b, uint32_t kept) {
    float s = 0.f;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const uint32_t mb = r == 0 ? (kept & 0xFFu) : prmt(kept, 0u, 0x4440 + r);
        unsigned char* row = blk + (4 * h + r) * kSRowPitch;
        const uint4 ra = *reinterpret_cast<const uint4*>(row), rb = *reinterpret_cast<const uint4*>(row + 16);
        const uint4 ka = lut[2 * mb], kb = lut[2 * mb + 1];                  // the row's keep flags as words of 0 or 1
        const uint32_t raw[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w}, k01[8] = {ka.x, ka.y, ka.z, ka.w, kb.x, kb.y, kb.z, kb.w};
        uint32_t o[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            o[q] = raw[q] * k01[q];                                          // the bits themselves or +0
            s += fabsf(__uint_as_float(o[q]));
        }
        if constexpr (HAS_OUT) {
            *reinterpret_cast<uint4*>(row) = make_uint4(o[0], o[1], o[2], o[3]);
            *reinterpret_cast<uint4*>(row + 16) = make_uint4(o[4], o[5], o[6], o[7]);
        }
        mrow[(4 * h + r) * 16 + b] = (unsigned char)mb;
    }
    return s;
}

template <bool HAS_OUT>
__global__ void __launch_bounds__(kSWarps * 32, 1)
tma48s_kernel(const __grid_constant__ TmaEntry single, const TmaEntry* __restrict__ table, int count, long long total_items,
              double* __restrict__ partials, int* __restrict__ status_out, unsigned int* __restrict__ done) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int b = lane >> 1, h = lane & 1;               // my block of the item, my half of its rows
    unsigned char* stages = smem_raw + (size_t)warp * kSWarpBytes;
    unsigned char* mbytes = stages + kSStages * kSStageBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(mbytes + 128);
    uint4* lut = reinterpret_cast<uint4*>(smem_raw + (size_t)kSWarps * kSWarpBytes);
    fill_keep_lut32(lut, threadIdx.x, kSWarps * 32);     // the only CTA-wide step
    __syncthreads();

    const long long gw = (long long)blockIdx.x * kSWarps + warp, nwarps = (long long)gridDim.x * kSWarps;
    // where this warp's objective partial for matrix k goes: k * pstride + pbase (a launch over several matrices that reduces
    // its own objectives packs them: slot = the warp's place in the deal + k, see finish_objectives_ranged)
    const bool ranged = done != nullptr && count > 1;
    const long long pstride = ranged ? 1 : nwarps, pbase = ranged ? (long long)warp * gridDim.x + blockIdx.x : gw;
    int n_items;
    const long long begin = even_share(total_items, kSWarps, n_items);
    const TmaEntry* tab = table ? table : &single;
    if (lane == 0) {
        for (int s = 0; s < kSStages; ++s) mbar_init(&bars[s], 1);
        fence_mbar_init();
    }
    __syncwarp();

    Cursor ld, cur;
    ld.seek(tab, count, begin);
    cur = ld;
    int loaded = 0;
    auto issue_next = [&]() {              // all lanes track the cursor, lane 0 issues the copy
        const int s = loaded % kSStages;
        if (lane == 0) {
            mbar_expect_tx(&bars[s], kSStageBytes);
            tma_load_2d(stages + s * kSStageBytes, &tab[ld.k].in, ld.cj * kTmaBoxUnits, ld.bi * kSRows, &bars[s]);
        }
        ld.advance(tab, count);
        ++loaded;
    };
    if (n_items > 0) issue_next();

    int status = 0, acc_k = -1;
    float facc = 0.f; double acc = 0.0;
    bool nonfinite = false;
    int p_cols = 0, p_wpr = 0;
    uint32_t* p_mask = nullptr;

    for (int it = 0; it < n_items; ++it) {
        const int s = it % kSStages;
        const uint32_t parity = (uint32_t)((it / kSStages) & 1);
        if (!__all_sync(kAll, mbar_wait_bounded(&bars[s], parity))) {       // a copy that never landed: stop before the unfilled stage is used
            status |= kDevInternal;
            if (lane == 0)
                for (int j = it + 1; j < loaded; ++j) mbar_wait_bounded(&bars[j % kSStages], (uint32_t)((j / kSStages) & 1), 1u << 14);
            break;
        }
        unsigned char* stage = stages + s * kSStageBytes;
        unsigned char* blk = stage + b * 32;

        // Inf / NaN watch over my rows on the multiply-add pipe (x * 0 + acc turns NaN); the pair decides together
        RelHalf rel;
        {
            float watch = 0.f;
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const float4 a = *reinterpret_cast<const float4*>(blk + (4 * h + r) * kSRowPitch), c = *reinterpret_cast<const float4*>(blk + (4 * h + r) * kSRowPitch + 16);
                watch = fmaf(a.x, 0.f, watch); watch = fmaf(a.y, 0.f, watch); watch = fmaf(a.z, 0.f, watch); watch = fmaf(a.w, 0.f, watch);
                watch = fmaf(c.x, 0.f, watch); watch = fmaf(c.y, 0.f, watch); watch = fmaf(c.z, 0.f, watch); watch = fmaf(c.w, 0.f, watch);
            }
            if (__any_sync(kAll, watch != watch)) {
                nonfinite = true;
                relations_half_int(blk, h, rel);
            } else {
                relations_half(blk, h, rel);
            }
        }
        // refill the stage of the previous item -- its store, issued one item ago, has long been read
        if (loaded < n_items) {
            if constexpr (HAS_OUT) { if (lane == 0 && it > 0) tma_wait_read<0>(); }
            __syncwarp();
            issue_next();
        }
        // step A: fewer than four heavier in the row and in the column
        uint32_t kept = ~(four_of_seven_w(rel.hr[1], rel.hr[2], rel.hr[3], rel.hr[4], rel.hr[5], rel.hr[6], rel.hr[7]) |
                          four_of_seven_w(rel.hc[1], rel.hc[2], rel.hc[3], rel.hc[4], rel.hc[5], rel.hc[6], rel.hc[7]));
        ShortHalf L = line_short_w(kept);
        uint32_t cand = ~kept & L.row_short & L.col_short;
        // step B: three rounds that every warp of ordinary data needs, then by vote
#pragma unroll 1
        for (int round = 0; round < 3; ++round) {
            kept |= fill_accept_w(rel, kept, cand);
            L = line_short_w(kept);
            cand = ~kept & L.row_short & L.col_short;
        }
        if (__any_sync(kAll, cand != 0)) {
            {   // a block with exactly one candidate left takes it as it stands (no rival in its row or column)
                const uint32_t mine = cand == 0 ? 0u : ((cand & (cand - 1)) == 0 ? 1u : 2u), other = __shfl_xor_sync(kAll, mine, 1);
                if (mine + other == 1) kept |= cand;
            }
            L = line_short_w(kept);
            cand = ~kept & L.row_short & L.col_short;
            int rounds = 3;
            while (__any_sync(kAll, cand != 0)) {
                if (++rounds > 16) { status |= kDevInternal; break; }      // a block lacks at most sixteen entries
                kept |= fill_accept_w(rel, kept, cand);
                L = line_short_w(kept);
                cand = ~kept & L.row_short & L.col_short;
            }
        }
        // step C: 2-for-1 swaps while a row of the block is short
        {
            int swaps = 0;
            for (;;) {
                const bool need = (L.row_short | __shfl_xor_sync(kAll, L.row_short, 1)) != 0;
                if (!__any_sync(kAll, need)) break;
                if (++swaps > 5) { status |= kDevInternal; break; }        // at most N*N/4 = 4 swaps per block
                const uint32_t free_a = ~kept & L.row_short, free_b = ~kept & L.col_short;
                const uint32_t elig = kept & any_in_col_w(free_a) & any_in_row_w(free_b);
                const uint32_t cands = elig & ~lighter_in_row_w(rel, elig) & ~lighter_in_col_w(rel, elig);
                if (!swap_apply_w(blk, h, need, kept, cands, free_a, free_b)) { status |= kDevInternal; break; }
                L = line_short_w(kept);
            }
        }

        if (cur.k != acc_k) {                                              // a new matrix starts: flush the objective partial
            if (acc_k >= 0) {
                acc += (double)facc;
                for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(kAll, acc, o);
                if (lane == 0) partials[(long long)acc_k * pstride + pbase] = acc;
            }
            acc = 0.0; facc = 0.f; acc_k = cur.k;
            const DevProblem& P = tab[cur.k].p;
            p_cols = (int)P.cols; p_wpr = P.wpr; p_mask = P.mask;
        }
        if (cur.cj * kSCols + b * 8 >= p_cols) kept = 0;                   // blocks past the last column (zero-filled by the copy)
        facc += back_end_w<HAS_OUT>(blk, h, mbytes, lut, b, kept);
        if constexpr (HAS_OUT) fence_proxy_async_smem();
        __syncwarp();
        if constexpr (HAS_OUT) {
            if (lane == 0) { tma_store_2d(&tab[cur.k].out, cur.cj * kTmaBoxUnits, cur.bi * kSRows, stage); tma_commit(); }
        }
        {   // 8 rows x 4 words of mask, one word per lane
            const int row = lane >> 2, word = cur.cj * 4 + (lane & 3);
            const uint32_t w = *reinterpret_cast<const uint32_t*>(mbytes + row * 16 + (lane & 3) * 4);
            if (word < p_wpr) p_mask[((long long)cur.bi * kSRows + row) * p_wpr + word] = w;
        }
        cur.advance(tab, count);
        if ((it & 15) == 15) { acc += (double)facc; facc = 0.f; }           // keep the fp32 partial short
        __syncwarp();
    }
    if (lane == 0) tma_wait_all<0>();
    if (acc_k >= 0 || (done && count == 1)) {  // a single-matrix launch that reduces its own objective wants a partial (a zero) from idle warps too
        acc += (double)facc;
        for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(kAll, acc, o);
        if (lane == 0) partials[(long long)(acc_k >= 0 ? acc_k : 0) * pstride + pbase] = acc;
    }
    if (nonfinite) status |= kDevNonFinite;
    for (int o = 16; o; o >>= 1) status |= __shfl_xor_sync(kAll, status, o);
    if (lane == 0 && status && status_out) atomicOr(status_out, status);
    if (done) {                                // the launch reduces its own objectives; the stages are idle by now
        const long long nw = (long long)gridDim.x * kSWarps;
        if (count > 1) finish_objectives_ranged(done, partials, tab, count, total_items, nw, reinterpret_cast<double*>(smem_raw));
        else finish_objective(done, partials, nw, tab[0].p.objective, reinterpret_cast<double*>(smem_raw));
    }
}

template <bool HAS_OUT>
cudaError_t launch_one48s(const TmaLaunch& a, const TmaEntry& single, const TmaEntry* table) {
    const size_t smem = (size_t)kSWarps * kSWarpBytes + kSLutBytes;
    auto kern = tma48s_kernel<HAS_OUT>;
    static PerDeviceOnce configured;       // per instantiation
    const cudaError_t e = configured.run([&] { return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); });
    if (e != cudaSuccess) return e;
    kern<<<a.ctas, kSWarps * 32, smem, a.stream>>>(single, table, a.count, a.total_items, a.partials, a.status, a.done);
    return cudaGetLastError();
}

}  // namespace

int tma48s_warps_per_cta() { return kSWarps; }
int tma48s_item_cols() { return kSCols; }

// The search kernel only (launch_tma48 clears the partials before and reduces them after, unless a.done makes the kernel do it).
cudaError_t launch_tma48s(const TmaLaunch& a) {
    const TmaEntry* host = static_cast<const TmaEntry*>(a.entries_host);
    const TmaEntry* table = static_cast<const TmaEntry*>(a.entries_dev);
    return a.has_out ? launch_one48s<true>(a, host[0], table) : launch_one48s<false>(a, host[0], table);
}

}  // namespace tmask
