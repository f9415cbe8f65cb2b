// Per-block solvers of the transposable N:M mask search, one thread per M x M block (the flow solver: one
// block per lane, a whole warp in step).
//
// Every routine takes the block as M*M magnitudes u[p] (fp32 bit pattern of |w|, p = i*M + j) and
// returns the kept set as a bit mask (bit p = S_ij of Eq. 1).  The order of entries is (u, p):
// among equal magnitudes the earlier position is the lighter one.
//
//   cover_mask      Algorithm 1 through its closed form: the pruned list is the union of the M-N
//                   lightest entries of every row and of every column (an entry among its row's
//                   M-N lightest meets row degree < M-N when the sorted scan reaches it; an entry in
//                   neither set finds both degrees full).
//   complete_mask   this library's completion: greedy fill heavy -> light, then 2-for-1 swaps.
//   exact_2_4       the optimum of Eq. 1 for M = 4 by scoring all 90 valid patterns.
//   exact_ssp       the optimum for any M <= 8 by shortest augmenting paths on the flow network of
//                   Fig. 3 (rows supply M-N units, columns demand M-N, unit-capacity coefficient
//                   edges; a unit on (i,j) prunes W_ij), started from a row-feasible pseudo-flow:
//                   exact_flow_warp (128-bit costs, warp-uniform) and exact_flow_run (384-bit costs,
//                   scalar, for blocks spanning more than 26 binades).
//
// Exact arithmetic.  |w_p| = sig_p * 2^(E_p - 150); with Emin the smallest exponent among the
// block's non-zero entries, q_p = sig_p << (E_p - Emin) is an integer proportional to |w_p|.  When
// the block's exponent spread is small the sums fit native integers; otherwise the same code runs
// on a 384-bit integer type, so that masks are always compared as exact real numbers.
#pragma once
#include "tm_device.cuh"

namespace tmask {

// ------------------------------------------------------------------------------------------
// order helpers
// ------------------------------------------------------------------------------------------
template <int M>
__device__ __forceinline__ void line_counts(uint64_t kept, int* rk, int* ck) {
    constexpr uint64_t rowm = (M == 8) ? 0xFFull : 0xFull;
    constexpr uint64_t colm = (M == 8) ? 0x0101010101010101ull : 0x1111ull;
#pragma unroll
    for (int i = 0; i < M; ++i) {
        rk[i] = __popcll(kept & (rowm << (i * M)));
        ck[i] = __popcll(kept & (colm << i));
    }
}

// ------------------------------------------------------------------------------------------
// Algorithm 1 (closed form)
// ------------------------------------------------------------------------------------------
template <int N, int M>
__device__ __forceinline__ uint64_t cover_mask(const uint32_t (&u)[M * M]) {
    // number of heavier entries in the same row / column, from each unordered pair compared once
    unsigned char rh[M * M], ch[M * M];
#pragma unroll
    for (int p = 0; p < M * M; ++p) { rh[p] = 0; ch[p] = 0; }
#pragma unroll
    for (int i = 0; i < M; ++i) {
#pragma unroll
        for (int a = 0; a < M; ++a) {
#pragma unroll
            for (int b = a + 1; b < M; ++b) {
                // row i: positions i*M+a < i*M+b  -> b heavier iff u_b >= u_a
                const bool bh = u[i * M + b] >= u[i * M + a];
                rh[i * M + a] += bh; rh[i * M + b] += !bh;
                // column i: positions a*M+i < b*M+i
                const bool dh = u[b * M + i] >= u[a * M + i];
                ch[a * M + i] += dh; ch[b * M + i] += !dh;
            }
        }
    }
    uint64_t kept = 0;
#pragma unroll
    for (int p = 0; p < M * M; ++p)
        if (rh[p] < N && ch[p] < N) kept |= 1ull << p;   // not among the M-N lightest of its row nor of its column
    return kept;
}

// ------------------------------------------------------------------------------------------
// Completion (steps B and C)
// ------------------------------------------------------------------------------------------
template <int N, int M>
__device__ __noinline__ uint64_t complete_mask(const uint32_t (&u)[M * M], uint64_t kept, int& status) {
    uint32_t ul[M * M];                       // dynamically indexed copy
#pragma unroll
    for (int p = 0; p < M * M; ++p) ul[p] = u[p];
    int rk[M], ck[M];
    // B: heaviest free entry whose row and column are both short, until none is left
    for (int it = 0; it < M * M; ++it) {
        line_counts<M>(kept, rk, ck);
        int best = -1; uint32_t bu = 0;
        for (int p = 0; p < M * M; ++p) {
            if (((kept >> p) & 1) || rk[p / M] >= N || ck[p % M] >= N) continue;
            if (best < 0 || ul[p] >= bu) { best = p; bu = ul[p]; }   // ascending p: ties go to the later one
        }
        if (best < 0) break;
        kept |= 1ull << best;
    }
    // C: 2-for-1 swaps while a row is short (at most N*N/4 of them)
    for (int it = 0; it <= (N * N) / 4; ++it) {
        line_counts<M>(kept, rk, ck);
        bool any_short = false;
        for (int i = 0; i < M; ++i) any_short |= rk[i] < N;
        if (!any_short) return kept;
        if (it == (N * N) / 4) break;
        int x = -1, xa = -1, xb = -1; uint32_t xu = 0;
        for (int p = 0; p < M * M; ++p) {      // lightest eligible kept entry
            if (!((kept >> p) & 1)) continue;
            if (x >= 0 && ul[p] >= xu) continue;
            const int r2 = p / M, c2 = p % M;
            int a = -1, b = -1;
            for (int r = 0; r < M; ++r) {
                const int e = r * M + c2;
                if (rk[r] < N && !((kept >> e) & 1) && (a < 0 || ul[e] >= ul[a])) a = e;
            }
            for (int c = 0; c < M; ++c) {
                const int e = r2 * M + c;
                if (ck[c] < N && !((kept >> e) & 1) && (b < 0 || ul[e] >= ul[b])) b = e;
            }
            if (a >= 0 && b >= 0) { x = p; xu = ul[p]; xa = a; xb = b; }
        }
        if (x < 0) break;
        kept = (kept & ~(1ull << x)) | (1ull << xa) | (1ull << xb);
    }
    status |= kDevInternal;
    return kept;
}

// ------------------------------------------------------------------------------------------
// exact integer images
// ------------------------------------------------------------------------------------------
struct Wide {                      // 384-bit two's-complement integer, little-endian limbs
    unsigned long long w[6];
};
__device__ __forceinline__ Wide wide_zero() { Wide r; for (int i = 0; i < 6; ++i) r.w[i] = 0; return r; }
__device__ __forceinline__ Wide wide_add(const Wide& a, const Wide& b) {
    Wide r; unsigned long long carry = 0;
    for (int i = 0; i < 6; ++i) {
        const unsigned long long s = a.w[i] + b.w[i];
        const unsigned long long c1 = s < a.w[i];
        r.w[i] = s + carry;
        carry = c1 | (r.w[i] < s);
    }
    return r;
}
__device__ __forceinline__ Wide wide_neg(const Wide& a) {
    Wide r; unsigned long long carry = 1;
    for (int i = 0; i < 6; ++i) { r.w[i] = ~a.w[i] + carry; carry = (carry && r.w[i] == 0) ? 1 : 0; }
    return r;
}
__device__ __forceinline__ bool wide_less(const Wide& a, const Wide& b) {   // signed a < b
    const bool sa = a.w[5] >> 63, sb = b.w[5] >> 63;
    if (sa != sb) return sa;
    for (int i = 5; i >= 0; --i) if (a.w[i] != b.w[i]) return a.w[i] < b.w[i];
    return false;
}
__device__ __forceinline__ Wide wide_shl(unsigned long long v, unsigned shift) {
    Wide r = wide_zero();
    const unsigned limb = shift >> 6, off = shift & 63;
    r.w[limb] = v << off;
    if (off && limb + 1 < 6) r.w[limb + 1] = v >> (64 - off);
    return r;
}

// Uniform access to the two cost types.
template <class T> struct CostOps;
template <> struct CostOps<long long> {
    static __device__ __forceinline__ long long zero() { return 0; }
    static __device__ __forceinline__ long long add(long long a, long long b) { return a + b; }
    static __device__ __forceinline__ bool less(long long a, long long b) { return a < b; }
    static __device__ __forceinline__ long long image(uint32_t sig, int shift) { return (long long)sig << shift; }
};
template <> struct CostOps<Wide> {
    static __device__ __forceinline__ Wide zero() { return wide_zero(); }
    static __device__ __forceinline__ Wide add(const Wide& a, const Wide& b) { return wide_add(a, b); }
    static __device__ __forceinline__ bool less(const Wide& a, const Wide& b) { return wide_less(a, b); }
    static __device__ __forceinline__ Wide image(uint32_t sig, int shift) { return wide_shl(sig, (unsigned)shift); }
};

__device__ __forceinline__ void split_float(uint32_t u, uint32_t& sig, int& E) {
    const uint32_t e = u >> 23, m = u & 0x7FFFFFu;
    sig = e ? (m | 0x800000u) : m;
    E = e ? (int)e : 1;
}
// smallest / largest exponent among the non-zero entries; returns false for an all-zero block
template <int CNT>
__device__ __forceinline__ bool exponent_range(const uint32_t (&u)[CNT], int& Emin, int& Emax) {
    Emin = 1 << 20; Emax = 0;
#pragma unroll
    for (int p = 0; p < CNT; ++p) {
        uint32_t sig; int E; split_float(u[p], sig, E);
        if (sig) { Emin = min(Emin, E); Emax = max(Emax, E); }
    }
    return Emax != 0;
}

// ------------------------------------------------------------------------------------------
// Exact, M = 4, N = 2: the 90 valid patterns
// ------------------------------------------------------------------------------------------
// A row keeps 2 of 4 columns: six choices, as nibbles in ascending value.
struct Patterns24 {
    unsigned char k[90][4];     // choice index of rows 0..3, patterns in ascending code order
    int count;
};
constexpr unsigned char kRowChoice[6] = {0x3, 0x5, 0x6, 0x9, 0xA, 0xC};
constexpr Patterns24 make_patterns24() {
    Patterns24 t{};
    int n = 0;
    // code = row3:row2:row1:row0 nibbles, so ascending code = lexicographic in (row3, row2, row1, row0)
    for (int k3 = 0; k3 < 6; ++k3) for (int k2 = 0; k2 < 6; ++k2) for (int k1 = 0; k1 < 6; ++k1) for (int k0 = 0; k0 < 6; ++k0) {
        bool ok = true;
        for (int c = 0; c < 4; ++c) {
            const int s = ((kRowChoice[k0] >> c) & 1) + ((kRowChoice[k1] >> c) & 1) + ((kRowChoice[k2] >> c) & 1) + ((kRowChoice[k3] >> c) & 1);
            if (s != 2) ok = false;
        }
        if (ok) { t.k[n][0] = (unsigned char)k0; t.k[n][1] = (unsigned char)k1; t.k[n][2] = (unsigned char)k2; t.k[n][3] = (unsigned char)k3; ++n; }
    }
    t.count = n;
    return t;
}
constexpr Patterns24 kPatterns24 = make_patterns24();
static_assert(kPatterns24.count == 90, "a 4x4 block has 90 masks with two ones per row and column");

template <int n> struct Pattern24 {
    static constexpr int k0 = kPatterns24.k[n][0], k1 = kPatterns24.k[n][1], k2 = kPatterns24.k[n][2], k3 = kPatterns24.k[n][3];
    static constexpr uint32_t code = (uint32_t)kRowChoice[k0] | ((uint32_t)kRowChoice[k1] << 4) |
                                     ((uint32_t)kRowChoice[k2] << 8) | ((uint32_t)kRowChoice[k3] << 12);
};

// patterns n, n+1, ... in ascending code order: ">=" lets the larger code win ties
template <class T, int n>
__device__ __forceinline__ void score_patterns24(const T (&lo)[6][6], const T (&hi)[6][6], T& best, uint32_t& best_code) {
    if constexpr (n < 90) {
        using P = Pattern24<n>;
        const T s = CostOps<T>::add(lo[P::k0][P::k1], hi[P::k2][P::k3]);
        if (n == 0 || !CostOps<T>::less(s, best)) { best = s; best_code = P::code; }
        score_patterns24<T, n + 1>(lo, hi, best, best_code);
    }
}

template <class T>
__device__ __forceinline__ uint64_t exact_2_4_scored(const uint32_t (&u)[16], int Emin) {
    using Ops = CostOps<T>;
    // sums of the two kept entries of a row, then of two rows, then the 90 totals
    T rs[4][6];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        T q[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t sig; int E; split_float(u[i * 4 + j], sig, E);
            q[j] = sig ? Ops::image(sig, E - Emin) : Ops::zero();
        }
        // same order as kRowChoice: columns {0,1} {0,2} {1,2} {0,3} {1,3} {2,3}
        rs[i][0] = Ops::add(q[0], q[1]); rs[i][1] = Ops::add(q[0], q[2]); rs[i][2] = Ops::add(q[1], q[2]);
        rs[i][3] = Ops::add(q[0], q[3]); rs[i][4] = Ops::add(q[1], q[3]); rs[i][5] = Ops::add(q[2], q[3]);
    }
    T lo[6][6], hi[6][6];
#pragma unroll
    for (int a = 0; a < 6; ++a)
#pragma unroll
        for (int b = 0; b < 6; ++b) { lo[a][b] = Ops::add(rs[0][a], rs[1][b]); hi[a][b] = Ops::add(rs[2][a], rs[3][b]); }
    T best = Ops::zero(); uint32_t best_code = 0;
    score_patterns24<T, 0>(lo, hi, best, best_code);
    return best_code;
}

static __device__ __noinline__ uint64_t exact_2_4_wide(const uint32_t (&u)[16], int Emin) { return exact_2_4_scored<Wide>(u, Emin); }
static __device__ __noinline__ uint64_t exact_2_4_int64(const uint32_t (&u)[16], int Emin) { return exact_2_4_scored<long long>(u, Emin); }

// Fast scorer.  A row keeps one of six column pairs {a,b} (index b(b-1)/2 + a, the order of
// kRowChoice).  value(row i, pair) = (q_a + q_b) * 2^16 + (nibble << 4i): the mask code rides in the
// low 16 bits, so one integer maximum implements "larger sum, then larger code".  The 90 patterns
// split by what rows 0,1 leave for rows 2,3:
//   both rows take the same pair k        -> rows 2,3 both take the complementary pair      (6 cases)
//   they take complementary pairs         -> rows 2,3 take any complementary pairs          (1 case, 6 x 6)
//   they share column c and skip column d -> rows 2,3 share d and skip c                    (12 cases, 2 x 2)
// so 19 sums of a best upper half and a best lower half cover everything.
__host__ __device__ constexpr int pair_index(int a, int b) { return a < b ? b * (b - 1) / 2 + a : a * (a - 1) / 2 + b; }
// the n-th (n = 0, 1) column that is neither c nor d
__host__ __device__ constexpr int other_column(int c, int d, int n) {
    int x = 0;
    for (int k = 0; k < 4; ++k)
        if (k != c && k != d) { if (n == 0) { x = k; break; } --n; }
    return x;
}

template <int C, int D>
__device__ __forceinline__ unsigned long long shared_column_case(const unsigned long long (&v)[4][6]) {
    constexpr int a = other_column(C, D, 0), b = other_column(C, D, 1);
    constexpr int ca = pair_index(C, a), cb = pair_index(C, b), da = pair_index(D, a), db = pair_index(D, b);
    const unsigned long long up = max(v[0][ca] + v[1][cb], v[0][cb] + v[1][ca]);
    const unsigned long long lo = max(v[2][da] + v[3][db], v[2][db] + v[3][da]);
    return up + lo;
}

__device__ __forceinline__ uint64_t exact_2_4_classes(const uint32_t (&u)[16], int Emin, int drop_bits) {
    unsigned long long v[4][6];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        unsigned long long q[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t sig; int E; split_float(u[i * 4 + j], sig, E);
            q[j] = sig ? ((unsigned long long)(sig >> drop_bits) << (E - Emin + 16)) : 0ull;
        }
#pragma unroll
        for (int b = 1; b < 4; ++b)
#pragma unroll
            for (int a = 0; a < b; ++a)
                v[i][pair_index(a, b)] = q[a] + q[b] + ((unsigned long long)((1u << a) | (1u << b)) << (4 * i));
    }
    unsigned long long best = 0;
    // same pair twice / complementary pairs
    unsigned long long up_c = 0, lo_c = 0;
#pragma unroll
    for (int k = 0; k < 6; ++k) {
        best = max(best, v[0][k] + v[1][k] + v[2][5 - k] + v[3][5 - k]);
        up_c = max(up_c, v[0][k] + v[1][5 - k]);
        lo_c = max(lo_c, v[2][k] + v[3][5 - k]);
    }
    best = max(best, up_c + lo_c);
    // shared column c, skipped column d
    best = max(best, max(max(shared_column_case<0, 1>(v), shared_column_case<0, 2>(v)), shared_column_case<0, 3>(v)));
    best = max(best, max(max(shared_column_case<1, 0>(v), shared_column_case<1, 2>(v)), shared_column_case<1, 3>(v)));
    best = max(best, max(max(shared_column_case<2, 0>(v), shared_column_case<2, 1>(v)), shared_column_case<2, 3>(v)));
    best = max(best, max(max(shared_column_case<3, 0>(v), shared_column_case<3, 1>(v)), shared_column_case<3, 2>(v)));
    return best & 0xFFFFull;
}

// The same 19 classes in 32-bit arithmetic, for blocks whose sums leave room: value(row i, pair) =
// (q_a + q_b) * 2^12 + (pair index << 3i).  The pair index (0..5) grows with the row's nibble, so the twelve
// low bits order the patterns exactly as the 16-bit mask code does.  Needs 8-bit significands (bf16) and an
// exponent spread of at most 9: 8 + 9 + 3 bits of sum above 12 bits of code.
template <int C, int D>
__device__ __forceinline__ uint32_t shared_column_case32(const uint32_t (&v)[4][6]) {
    constexpr int a = other_column(C, D, 0), b = other_column(C, D, 1);
    constexpr int ca = pair_index(C, a), cb = pair_index(C, b), da = pair_index(D, a), db = pair_index(D, b);
    return max(v[0][ca] + v[1][cb], v[0][cb] + v[1][ca]) + max(v[2][da] + v[3][db], v[2][db] + v[3][da]);
}
// SCALED: Emin >= 19 (all entries normal numbers or zero), so the integer image is a product: |w| * 2^(146 - Emin) is the
// integer q * 2^12 (at most 29 bits, exact in fp32), one multiplication and one conversion off the logic pipe per entry.
template <bool SCALED>
__device__ __forceinline__ uint64_t exact_2_4_classes32(const uint32_t (&u)[16], int Emin) {
    uint32_t v[4][6];
    const float scale = __uint_as_float((uint32_t)(127 + 146 - Emin) << 23);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint32_t q[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if constexpr (SCALED) {
                q[j] = __float2uint_rz(__uint_as_float(u[i * 4 + j]) * scale);
            } else {
                uint32_t sig; int E; split_float(u[i * 4 + j], sig, E);
                q[j] = sig ? ((sig >> 16) << (E - Emin + 12)) : 0u;
            }
        }
#pragma unroll
        for (int b = 1; b < 4; ++b)
#pragma unroll
            for (int a = 0; a < b; ++a)
                v[i][pair_index(a, b)] = q[a] + q[b] + ((uint32_t)pair_index(a, b) << (3 * i));
    }
    uint32_t best = 0, up_c = 0, lo_c = 0;
#pragma unroll
    for (int k = 0; k < 6; ++k) {
        best = max(best, v[0][k] + v[1][k] + v[2][5 - k] + v[3][5 - k]);
        up_c = max(up_c, v[0][k] + v[1][5 - k]);
        lo_c = max(lo_c, v[2][k] + v[3][5 - k]);
    }
    best = max(best, up_c + lo_c);
    best = max(best, max(max(shared_column_case32<0, 1>(v), shared_column_case32<0, 2>(v)), shared_column_case32<0, 3>(v)));
    best = max(best, max(max(shared_column_case32<1, 0>(v), shared_column_case32<1, 2>(v)), shared_column_case32<1, 3>(v)));
    best = max(best, max(max(shared_column_case32<2, 0>(v), shared_column_case32<2, 1>(v)), shared_column_case32<2, 3>(v)));
    best = max(best, max(max(shared_column_case32<3, 0>(v), shared_column_case32<3, 1>(v)), shared_column_case32<3, 2>(v)));
    // pair indices back to nibbles: 0x3, 0x5, 0x6, 0x9, 0xA, 0xC
    uint32_t code = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) code |= ((0xCA9653u >> (4 * ((best >> (3 * i)) & 7u))) & 0xFu) << (4 * i);
    return code;
}

// drop_bits: low significand bits known to be zero in every entry (16 for widened bf16 inputs).
// Called by all 32 lanes of a warp (the 32-bit scorer is taken when every lane's block fits it).
__device__ __forceinline__ uint64_t exact_2_4(const uint32_t (&u)[16], int drop_bits) {
    if (drop_bits == 16) {
        // bf16 data, the common case first: exponent range from the largest and the smallest non-zero pattern (u - 1 sends
        // zero to the top), no per-entry unpacking
        uint32_t umax = 0, umin1 = 0xFFFFFFFFu;
#pragma unroll
        for (int p = 0; p < 16; ++p) { umax = max(umax, u[p]); umin1 = min(umin1, u[p] - 1u); }
        const int emax = (int)(umax >> 23), emin = (int)((umin1 + 1u) >> 23);
        const bool fits = umax == 0u || (emin >= 19 && emax - emin <= 9);      // all zero: every sum is 0, the largest code wins
        if (__all_sync(0xFFFFFFFFu, fits)) return exact_2_4_classes32<true>(u, umax ? emin : 127);
    }
    int Emin, Emax;
    if (!exponent_range<16>(u, Emin, Emax)) { Emin = 1; Emax = 1; }     // all zero: every sum is 0, the largest code wins
    const int spread = Emax - Emin;
    if (__all_sync(0xFFFFFFFFu, drop_bits == 16 && spread <= 9)) return exact_2_4_classes32<false>(u, Emin);
    // (24 - drop) significand bits + spread + 3 bits for eight terms + 16 code bits must stay below 2^63
    if (spread <= 19 + drop_bits) return exact_2_4_classes(u, Emin, drop_bits);
    if (spread <= 34) return exact_2_4_int64(u, Emin);
    return exact_2_4_wide(u, Emin);
}

// exact_2_4() in two parts for the pipelined kernel, so that the common case pays nothing for the rare one.  With the later
// tiers inlined beside it the first tier's loop spilled 480 bytes a thread at 96 registers; with them behind a call inside
// the loop the values that live across the call went to local memory on the way of every item (46 local loads per item).  So
// the loop holds a first tier only, an item with a block outside it is set aside, and exact_2_4_any() -- out of line --
// scores such items after the loop.  Both are called by all 32 lanes.
// exact_2_4_first: false (nothing computed) unless every lane's block fits the tier:
//   bf16  at most 9 binades between the largest and the smallest non-zero entry, no subnormals: 32-bit class sums;
//   fp32  at most 19 binades: 64-bit class sums.
//   bf16, WIDE  (for data that leaves the 32-bit tier often) at most 35 binades: 64-bit class sums of the 8-bit significands.
template <bool BF16, bool WIDE>
__device__ __forceinline__ bool exact_2_4_first(const uint32_t (&u)[16], uint64_t& code) {
    uint32_t umax = 0, umin1 = 0xFFFFFFFFu;                  // u - 1 sends zero to the top
#pragma unroll
    for (int p = 0; p < 16; ++p) { umax = max(umax, u[p]); umin1 = min(umin1, u[p] - 1u); }
    const int emax = (int)(umax >> 23), emin = (int)((umin1 + 1u) >> 23);
    if constexpr (BF16 && WIDE) {
        const bool fits = umax == 0u || (emin >= 1 && emax - emin <= 35);
        if (!__all_sync(0xFFFFFFFFu, fits)) return false;
        code = exact_2_4_classes(u, umax ? emin : 1, 16);
    } else if constexpr (BF16) {
        const bool fits = umax == 0u || (emin >= 19 && emax - emin <= 9 && emax < 255);      // Inf / NaN patterns take the integer tiers
        if (!__all_sync(0xFFFFFFFFu, fits)) return false;
        code = exact_2_4_classes32<true>(u, umax ? emin : 127);
    } else {
        const bool fits = umax == 0u || (emin >= 1 && emax - emin <= 19);        // normal numbers: the exponent field is split_float()'s E
        if (!__all_sync(0xFFFFFFFFu, fits)) return false;
        code = exact_2_4_classes(u, umax ? emin : 1, 0);
    }
    return true;
}
// every tier, for blocks given as magnitude patterns; drop_bits as for exact_2_4()
static __device__ __noinline__ uint32_t exact_2_4_any(const uint32_t (&u)[16], int drop_bits) { return (uint32_t)exact_2_4(u, drop_bits); }

// ------------------------------------------------------------------------------------------
// Exact, any M <= 8: min-cost flow on the network of Fig. 3
// ------------------------------------------------------------------------------------------
// Cost of the coefficient edge of entry p: q_p * 2^64 + 2^p (the tie rule folded into the cost:
// minimising the pruned cost maximises (sum of kept |w|, code)).
struct CostWide { Wide v; };
template <> struct CostOps<CostWide> {
    static __device__ __forceinline__ CostWide zero() { return CostWide{wide_zero()}; }
    static __device__ __forceinline__ CostWide add(const CostWide& a, const CostWide& b) { return CostWide{wide_add(a.v, b.v)}; }
    static __device__ __forceinline__ CostWide neg(const CostWide& a) { return CostWide{wide_neg(a.v)}; }
    static __device__ __forceinline__ bool less(const CostWide& a, const CostWide& b) { return wide_less(a.v, b.v); }
    static __device__ __forceinline__ CostWide edge(uint32_t sig, int shift, int p) {
        Wide q = wide_shl(sig, (unsigned)shift), c;
        c.w[0] = 1ull << p;
        for (int l = 1; l < 6; ++l) c.w[l] = q.w[l - 1];
        return CostWide{c};
    }
};

// Min-cost flow by repairing a pseudo-flow: start from the state in which every row prunes its M-N
// lightest entries (row supplies met, optimality conditions met with row potentials at the cost of the
// row's (M-N)-th lightest entry), then repair the column imbalances -- a handful of units instead of
// M(M-N) -- by shortest paths from over-subscribed to under-subscribed columns (Dijkstra on reduced
// costs, which stay non-negative).  Costs are the exact integers of Fig. 3's coefficient edges with
// the tie rule folded in, so the result is the unique optimum whatever path is taken among equals.
template <class C, int N, int M>
__device__ __noinline__ uint64_t exact_flow_run(const uint32_t (&u)[M * M], int Emin, int& status) {
    using Ops = CostOps<C>;
    constexpr int P = M - N;
    C cost[M * M], pot[2 * M];
    for (int p = 0; p < M * M; ++p) {
        uint32_t sig; int E; split_float(u[p], sig, E);
        cost[p] = Ops::edge(sig, sig ? E - Emin : 0, p);
    }
    uint64_t pruned = 0;
    int load[M];
    for (int j = 0; j < M; ++j) { load[j] = 0; pot[M + j] = Ops::zero(); }
    for (int i = 0; i < M; ++i) {
        for (int j = 0; j < M; ++j) {
            int heavier = 0;
            for (int k = 0; k < M; ++k)
                heavier += (k != j) && (u[i * M + k] > u[i * M + j] || (u[i * M + k] == u[i * M + j] && k > j));
            if (heavier >= N) { pruned |= 1ull << (i * M + j); load[j]++; }
            if (heavier == N) pot[i] = Ops::neg(cost[i * M + j]);      // reduced cost c + pot[row] - pot[col]: <= 0 pruned, >= 0 kept
        }
    }
    for (int unit = 0; unit <= M * P; ++unit) {
        unsigned reach = 0, done = 0;
        C dist[2 * M]; int pre[2 * M];
        for (int j = 0; j < M; ++j)
            if (load[j] > P) { dist[M + j] = Ops::zero(); pre[M + j] = -1; reach |= 1u << (M + j); }
        if (!reach) break;                                              // every column holds exactly M-N pruned entries
        if (unit == M * P) { status |= kDevInternal; break; }
        int target = -1;
        for (int step = 0; step < 2 * M; ++step) {
            int v = -1;
            for (int n = 0; n < 2 * M; ++n)
                if (((reach & ~done) >> n) & 1) { if (v < 0 || Ops::less(dist[n], dist[v])) v = n; }
            if (v < 0) break;
            done |= 1u << v;
            if (v >= M && load[v - M] < P) { target = v; break; }
            if (v >= M) {                                               // column: un-prune one of its pruned entries
                const int j = v - M;
                for (int i = 0; i < M; ++i) {
                    if (!((pruned >> (i * M + j)) & 1) || ((done >> i) & 1)) continue;
                    const C nd = Ops::add(dist[v], Ops::add(Ops::add(pot[v], Ops::neg(pot[i])), Ops::neg(cost[i * M + j])));
                    if (!((reach >> i) & 1) || Ops::less(nd, dist[i])) { dist[i] = nd; pre[i] = v; reach |= 1u << i; }
                }
            } else {                                                    // row: prune one more of its kept entries
                const int i = v;
                for (int j = 0; j < M; ++j) {
                    if (((pruned >> (i * M + j)) & 1) || ((done >> (M + j)) & 1)) continue;
                    const C nd = Ops::add(dist[v], Ops::add(Ops::add(pot[i], Ops::neg(pot[M + j])), cost[i * M + j]));
                    if (!((reach >> (M + j)) & 1) || Ops::less(nd, dist[M + j])) { dist[M + j] = nd; pre[M + j] = i; reach |= 1u << (M + j); }
                }
            }
        }
        if (target < 0) { status |= kDevInternal; break; }
        const C D = dist[target];
        for (int n = 0; n < 2 * M; ++n)
            pot[n] = Ops::add(pot[n], (((done >> n) & 1) && Ops::less(dist[n], D)) ? dist[n] : D);
        int v = target, steps = 0;
        load[target - M]++;
        while (pre[v] >= 0 && steps++ < 2 * M + 2) {
            const int w = pre[v];
            if (v >= M) pruned |= 1ull << (w * M + (v - M));           // row w -> column v-M
            else pruned &= ~(1ull << (v * M + (w - M)));               // column w-M -> row v
            v = w;
        }
        if (v >= M && pre[v] < 0) load[v - M]--; else { status |= kDevInternal; break; }
    }
    const uint64_t all = (M == 8) ? ~0ull : ((1ull << (M * M)) - 1);
    return ~pruned & all;
}

// The same repair written for a whole warp at once: one block per lane, state in shared memory, and one
// instruction stream for all lanes.  The scalar version above branches on the node it has just settled, so
// the 32 lanes of a warp drift apart and execute one after the other; here every data-dependent choice is a
// select or a predicated store, every loop is uniform (a vote ends it when no lane needs another turn), and
// a settled node's row and column cases share one body.  A thread's edge costs, potentials and distances
// are three strided columns (stride T entries); predecessors and column loads are packed four bits each
// into registers.  Must be called by all 32 lanes; lanes with `enabled` false take part in the votes only.
//
// Two number formats share the routine.  Flow128 carries the full costs q_p * 2^64 + 2^p (recomputed from the
// magnitudes at every use).  Flow64 carries q_p alone, precomputed: half the words in every load, sum and
// comparison.  Without the tie term the optimum it finds is the wanted one only if it is the only one; that is
// certified afterwards (tight_forest below), and a block without the certificate is solved again in full.
// State.  The first pass (exact_flow_warp_reg) keeps potentials and distances in registers and its 64-bit edge costs in
// shared memory: a thread owns the 8-byte cells t, T + t, 2T + t, ... of the CTA's region (T threads; consecutive threads
// touch consecutive cells, so 8-byte accesses do not collide).  The 128-bit pass, which only the blocks without the
// uniqueness certificate take, keeps everything in cells of the thread's local memory (T = 1).  cell(base, k, T) is the
// k-th cell of the thread whose first is base.
constexpr int flow_cells128_per_thread(int M) { return 4 * (2 * M) + M * M / 2; }          // Flow128: two cells per potential / distance, half a cell per magnitude
constexpr int flow_shared_bytes_per_thread(int M) { return 8 * M * M; }                    // shared memory holds the 64-bit edge costs of the first pass only
typedef unsigned long long FlowCell;
__device__ __forceinline__ FlowCell* cell(FlowCell* base, int k, int T) { return base + (size_t)k * T; }

__device__ __forceinline__ __int128 edge_cost128(uint32_t u, int Emin, int p) {
    uint32_t sig; int E; split_float(u, sig, E);
    return ((__int128)((long long)sig << (sig ? E - Emin : 0)) << 64) + ((__int128)1 << p);
}

template <int M> struct Flow128 {
    typedef __int128 V;
    static constexpr bool kTieFree = false;
    static constexpr int kPot = 0, kDist = 2 * (2 * M), kCost = 4 * (2 * M);                // first cell of each array
    static constexpr int kCells = 2;                                                        // cells per potential / distance
    static __device__ __forceinline__ V ld(FlowCell* base, int first, int n, int T) {
        const FlowCell lo = *cell(base, first + 2 * n, T), hi = *cell(base, first + 2 * n + 1, T);
        return (__int128)(((unsigned __int128)hi << 64) | lo);
    }
    static __device__ __forceinline__ void st(FlowCell* base, int first, int n, int T, V x) {
        *cell(base, first + 2 * n, T) = (FlowCell)x; *cell(base, first + 2 * n + 1, T) = (FlowCell)((unsigned __int128)x >> 64);
    }
    static __device__ __forceinline__ V ldp(FlowCell* first, int T) { return (__int128)(((unsigned __int128)first[T] << 64) | first[0]); }
    static __device__ __forceinline__ void stp(FlowCell* first, int T, V x) { first[0] = (FlowCell)x; first[T] = (FlowCell)((unsigned __int128)x >> 64); }
    // what is kept per entry: the magnitude, two to a cell
    static __device__ __forceinline__ void put_cost(FlowCell* base, int p, int T, uint32_t u, int) {
        reinterpret_cast<uint32_t*>(cell(base, kCost + (p >> 1), T))[p & 1] = u;
    }
    static __device__ __forceinline__ V cost(FlowCell* base, int p, int T, int Emin) {
        return edge_cost128(reinterpret_cast<const uint32_t*>(cell(base, kCost + (p >> 1), T))[p & 1], Emin, p);
    }
};
template <int M> struct Flow64 {
    typedef long long V;
    static constexpr bool kTieFree = true;
    static constexpr int kCost = 0, kPot = M * M, kDist = M * M + 2 * M;
    static constexpr int kCells = 1;
    static __device__ __forceinline__ V ld(FlowCell* base, int first, int n, int T) { return (V)*cell(base, first + n, T); }
    static __device__ __forceinline__ void st(FlowCell* base, int first, int n, int T, V x) { *cell(base, first + n, T) = (FlowCell)x; }
    static __device__ __forceinline__ V ldp(FlowCell* first, int) { return (V)*first; }
    static __device__ __forceinline__ void stp(FlowCell* first, int, V x) { *first = (FlowCell)x; }
    // q_p, at most 50 bits (24 significand bits, 26 binades); paths add 4 bits, potentials 5
    static __device__ __forceinline__ void put_cost(FlowCell* base, int p, int T, uint32_t u, int Emin) {
        uint32_t sig; int E; split_float(u, sig, E);
        *cell(base, kCost + p, T) = (FlowCell)sig << (sig ? E - Emin : 0);
    }
    static __device__ __forceinline__ V cost(FlowCell* base, int p, int T, int) { return (V)*cell(base, kCost + p, T); }
};

// Is the bipartite graph of the marked entries (rows and columns as nodes, bit i*M+j an edge) free of cycles?  Leaves are
// stripped until nothing changes: rows with a single edge lose it, then columns with a single edge; what survives lies on
// a cycle.  Called by all 32 lanes (the loop ends on a vote).
template <int M>
__device__ __forceinline__ bool tight_forest(uint64_t edges) {
    uint32_t row[M];
#pragma unroll
    for (int i = 0; i < M; ++i) row[i] = (uint32_t)(edges >> (i * M)) & ((1u << M) - 1u);
    for (int it = 0; it < 2 * M; ++it) {
        bool changed = false;
        uint32_t once = 0, twice = 0;                                   // columns with at least one / at least two edges
#pragma unroll
        for (int i = 0; i < M; ++i) {
            const bool single = row[i] != 0 && (row[i] & (row[i] - 1)) == 0;
            changed |= single;
            row[i] = single ? 0u : row[i];
            twice |= once & row[i]; once |= row[i];
        }
        const uint32_t leaf_cols = once & ~twice;
        changed |= leaf_cols != 0;
#pragma unroll
        for (int i = 0; i < M; ++i) row[i] &= ~leaf_cols;
        if (!__any_sync(0xFFFFFFFFu, changed)) break;
    }
    uint32_t left = 0;
#pragma unroll
    for (int i = 0; i < M; ++i) left |= row[i];
    return left == 0;
}

// certified (Flow64 only): set to true when the optimum found is the only one, so that the tie rule has nothing to decide:
// by complementary slackness every optimal flow agrees with this one outside the entries of reduced cost zero, and when
// those entries form a forest the row and column totals fix the flow on them too.
template <class A, int N, int M, int T>
__device__ __noinline__ uint64_t exact_flow_warp(const uint32_t (&u)[M * M], int Emin, bool enabled, int& status,
                                                 FlowCell* base, bool* certified) {
    typedef typename A::V V;
    constexpr int P = M - N;
    constexpr unsigned kFull = 0xFFFFFFFFu;
    uint64_t pruned = 0;
    uint32_t load = 0;                                                  // nibble j: pruned entries of column j
#pragma unroll
    for (int j = 0; j < M; ++j) A::st(base, A::kPot, M + j, T, 0);
#pragma unroll
    for (int i = 0; i < M; ++i) {
#pragma unroll
        for (int j = 0; j < M; ++j) {
            A::put_cost(base, i * M + j, T, u[i * M + j], Emin);
            int heavier = 0;
#pragma unroll
            for (int k = 0; k < M; ++k)
                heavier += (k != j) && (u[i * M + k] > u[i * M + j] || (u[i * M + k] == u[i * M + j] && k > j));
            if (heavier >= N) { pruned |= 1ull << (i * M + j); load += 1u << (4 * j); }
            if (heavier == N) A::st(base, A::kPot, i, T, -A::cost(base, i * M + j, T, Emin));   // reduced cost c + pot[row] - pot[col]: <= 0 pruned, >= 0 kept
        }
    }
    bool failed = false;
    for (int unit = 0; unit <= M * P; ++unit) {
        unsigned reach = 0, done = 0;
        uint32_t pre_r = 0, pre_c = 0;                                  // nibble k: predecessor of row node k / column node k
#pragma unroll
        for (int j = 0; j < M; ++j) {
            const bool over = enabled && !failed && (int)((load >> (4 * j)) & 15u) > P;
            if (over) A::st(base, A::kDist, M + j, T, 0);
            reach |= (over ? 1u : 0u) << (M + j);
        }
        const unsigned sources = reach;
        const bool active = reach != 0;                                 // this lane's columns are not all at M-N yet
        if (!__any_sync(kFull, active)) break;
        if (unit == M * P) { failed |= active; break; }
        int target = -1;
        for (int step = 0; step < 2 * M; ++step) {
            const bool searching = active && target < 0;
            if (!__any_sync(kFull, searching)) break;
            // settle the open node at the smallest distance
            const unsigned open = searching ? (reach & ~done) : 0u;
            int v = -1; V dv = 0;
#pragma unroll
            for (int n = 0; n < 2 * M; ++n) {
                const V d = A::ld(base, A::kDist, n, T);
                const bool better = ((open >> n) & 1) && (v < 0 || d < dv);
                v = better ? n : v; dv = better ? d : dv;
            }
            const bool has = v >= 0;
            const int vv = has ? v : 0;
            done |= has ? (1u << vv) : 0u;
            const bool iscol = vv >= M;
            const int line = iscol ? vv - M : vv;                       // the settled node's column or row
            const bool hit = has && iscol && (int)((load >> (4 * line)) & 15u) < P;
            target = hit ? vv : target;
            const bool relax = has && !hit;
            // relax its M arcs: a column un-prunes one of its pruned entries, a row prunes one more of its kept ones.
            // Arc k leads to row k (from a column) or to column k (from a row): everything that depends on k alone is a
            // constant offset from what is worked out once per step.
            const V from = dv + A::ld(base, A::kPot, vv, T);
            const uint64_t flags = pruned >> (iscol ? line : line * M); // arc k's pruned flag at bit k*M (column) or k (row)
            FlowCell* const costs = cell(base, A::kCost, T) + (size_t)(iscol ? line : line * M) * (A::kTieFree ? T : 0);
            const unsigned reached = iscol ? reach : reach >> M, settled = iscol ? done : done >> M;
            unsigned taken = 0, spread = 0;                             // arcs that reached or improved their node: bit k / bit 4k
#pragma unroll
            for (int k = 0; k < M; ++k) {
                const bool is_pruned = ((iscol ? flags >> (k * M) : flags >> k) & 1) != 0;
                const bool elig = relax && (is_pruned == iscol) && !((settled >> k) & 1);
                const int p = iscol ? k * M + line : line * M + k;
                const V c = A::kTieFree ? (V)*(iscol ? costs + (size_t)k * M * T : costs + (size_t)k * T) : A::cost(base, p, T, Emin);
                FlowCell* const potk = iscol ? cell(base, A::kPot + A::kCells * k, T) : cell(base, A::kPot + A::kCells * (M + k), T);
                FlowCell* const distk = iscol ? cell(base, A::kDist + A::kCells * k, T) : cell(base, A::kDist + A::kCells * (M + k), T);
                const V nd = from - A::ldp(potk, T) + (iscol ? -c : c);
                const bool better = elig && (!((reached >> k) & 1) || nd < A::ldp(distk, T));
                if (better) A::stp(distk, T, nd);
                taken |= (better ? 1u : 0u) << k;
                spread |= (better ? 1u : 0u) << (4 * k);
            }
            // their predecessor is the settled node
            const uint32_t mask = spread * 15u, fill = spread * (uint32_t)vv;
            pre_r = iscol ? ((pre_r & ~mask) | fill) : pre_r;
            pre_c = iscol ? pre_c : ((pre_c & ~mask) | fill);
            reach |= iscol ? taken : taken << M;
        }
        const bool ok = active && target >= 0;
        failed |= active && target < 0;
        // potentials: settled nodes closer than the target move by their distance, all others by the target's
        const int tt = ok ? target : M;
        const V D = A::ld(base, A::kDist, tt, T);
#pragma unroll
        for (int n = 0; n < 2 * M; ++n) {
            const V d = A::ld(base, A::kDist, n, T);
            const V add = (((done >> n) & 1) && d < D) ? d : D;
            if (ok) A::st(base, A::kPot, n, T, A::ld(base, A::kPot, n, T) + add);
        }
        // flip the arcs of the path back to its source column
        int v = tt;
        load += ok ? (1u << (4 * (tt - M))) : 0u;
#pragma unroll 1
        for (int s = 0; s < 2 * M + 2; ++s) {
            const bool go = ok && !((sources >> v) & 1);
            if (!__any_sync(kFull, go)) break;
            const int w = (int)(((v >= M ? pre_c >> (4 * (v - M)) : pre_r >> (4 * v))) & 15u);
            const uint64_t bit = v >= M ? (1ull << ((w & (M - 1)) * M + (v - M))) : (1ull << (v * M + (w & (M - 1))));
            pruned = go ? (v >= M ? (pruned | bit) : (pruned & ~bit)) : pruned;     // row w -> column v-M prunes; column w-M -> row v un-prunes
            v = go ? w : v;
        }
        const bool home = ok && ((sources >> v) & 1);
        load -= home ? (1u << (4 * (v - M))) : 0u;
        failed |= ok && !home;
    }
    if (failed) status |= kDevInternal;
    if constexpr (A::kTieFree) {
        // the entries of reduced cost zero under the final potentials
        V pr[M], pc[M];
#pragma unroll
        for (int i = 0; i < M; ++i) { pr[i] = A::ld(base, A::kPot, i, T); pc[i] = A::ld(base, A::kPot, M + i, T); }
        uint64_t tight = 0;
#pragma unroll
        for (int i = 0; i < M; ++i)
#pragma unroll
            for (int j = 0; j < M; ++j)
                tight |= (A::cost(base, i * M + j, T, Emin) + pr[i] == pc[j]) ? (1ull << (i * M + j)) : 0ull;
        const bool forest = tight_forest<M>(enabled ? tight : 0ull);
        *certified = enabled && !failed && forest;
    }
    const uint64_t all = (M == 8) ? ~0ull : ((1ull << (M * M)) - 1);
    return ~pruned & all;
}

// The Flow64 pass with potentials and distances in registers.  Every access to them has a position known at compile time
// once the loops over nodes and arcs are unrolled: the scan for the nearest open node walks all of them (and picks up the
// settled node's potential on the way), an arc's far end is node k of one side or node k of the other (a choice of two
// registers), a new distance goes to either by a predicated move, and the target's distance is noted when the target is
// found.  Only the edge costs, which are addressed by the settled node's row or column, stay in the thread's shared cells
// (the Flow64 layout).  Same algorithm, same votes, same results as exact_flow_warp<Flow64<M>, ...>; about a third fewer
// instructions per step and an eighth of its shared-memory traffic.
template <int N, int M, int T>
__device__ __forceinline__ uint64_t exact_flow_warp_reg(const uint32_t (&u)[M * M], int Emin, bool enabled, int& status, FlowCell* base, bool* certified) {
    typedef Flow64<M> A;
    typedef long long V;
    constexpr int P = M - N;
    constexpr unsigned kFull = 0xFFFFFFFFu;
    V pot[2 * M], dist[2 * M];
    uint64_t pruned = 0;
    uint32_t load = 0;                                                  // nibble j: pruned entries of column j
#pragma unroll
    for (int n = 0; n < 2 * M; ++n) { pot[n] = 0; dist[n] = 0; }
#pragma unroll
    for (int i = 0; i < M; ++i) {
#pragma unroll
        for (int j = 0; j < M; ++j) {
            A::put_cost(base, i * M + j, T, u[i * M + j], Emin);
            int heavier = 0;
#pragma unroll
            for (int k = 0; k < M; ++k)
                heavier += (k != j) && (u[i * M + k] > u[i * M + j] || (u[i * M + k] == u[i * M + j] && k > j));
            if (heavier >= N) { pruned |= 1ull << (i * M + j); load += 1u << (4 * j); }
            if (heavier == N) pot[i] = -A::cost(base, i * M + j, T, Emin);      // reduced cost c + pot[row] - pot[col]: <= 0 pruned, >= 0 kept
        }
    }
    bool failed = false;
    for (int unit = 0; unit <= M * P; ++unit) {
        unsigned reach = 0, done = 0;
        uint32_t pre_r = 0, pre_c = 0;                                  // nibble k: predecessor of row node k / column node k
#pragma unroll
        for (int j = 0; j < M; ++j) {
            const bool over = enabled && !failed && (int)((load >> (4 * j)) & 15u) > P;
            dist[M + j] = over ? 0 : dist[M + j];
            reach |= (over ? 1u : 0u) << (M + j);
        }
        const unsigned sources = reach;
        const bool active = reach != 0;                                 // this lane's columns are not all at M-N yet
        if (!__any_sync(kFull, active)) break;
        if (unit == M * P) { failed |= active; break; }
        int target = -1;
        V D = 0;                                                        // the target's distance
        for (int step = 0; step < 2 * M; ++step) {
            const bool searching = active && target < 0;
            if (!__any_sync(kFull, searching)) break;
            // settle the open node at the smallest distance
            const unsigned open = searching ? (reach & ~done) : 0u;
            int v = -1; V dv = 0, pv = 0;
#pragma unroll
            for (int n = 0; n < 2 * M; ++n) {
                const bool better = ((open >> n) & 1) && (v < 0 || dist[n] < dv);
                v = better ? n : v; dv = better ? dist[n] : dv; pv = better ? pot[n] : pv;
            }
            const bool has = v >= 0;
            const int vv = has ? v : 0;
            done |= has ? (1u << vv) : 0u;
            const bool iscol = vv >= M;
            const int line = iscol ? vv - M : vv;                       // the settled node's column or row
            const bool hit = has && iscol && (int)((load >> (4 * line)) & 15u) < P;
            target = hit ? vv : target;
            D = hit ? dv : D;
            const bool relax = has && !hit;
            // relax its M arcs: a column un-prunes one of its pruned entries, a row prunes one more of its kept ones
            const V from = dv + pv;
            const uint64_t flags = pruned >> (iscol ? line : line * M); // arc k's pruned flag at bit k*M (column) or k (row)
            const FlowCell* const costs = cell(base, A::kCost, T) + (size_t)(iscol ? line : line * M) * T;
            const unsigned reached = iscol ? reach : reach >> M, settled = iscol ? done : done >> M;
            unsigned taken = 0, spread = 0;                             // arcs that reached or improved their node: bit k / bit 4k
#pragma unroll
            for (int k = 0; k < M; ++k) {
                const bool is_pruned = ((iscol ? flags >> (k * M) : flags >> k) & 1) != 0;
                const bool elig = relax && (is_pruned == iscol) && !((settled >> k) & 1);
                const V c = (V)*(iscol ? costs + (size_t)k * M * T : costs + (size_t)k * T);
                const V pk = iscol ? pot[k] : pot[M + k], dk = iscol ? dist[k] : dist[M + k];
                const V nd = from - pk + (iscol ? -c : c);
                const bool better = elig && (!((reached >> k) & 1) || nd < dk);
                dist[k] = (better && iscol) ? nd : dist[k];
                dist[M + k] = (better && !iscol) ? nd : dist[M + k];
                taken |= (better ? 1u : 0u) << k;
                spread |= (better ? 1u : 0u) << (4 * k);
            }
            // their predecessor is the settled node
            const uint32_t mask = spread * 15u, fill = spread * (uint32_t)vv;
            pre_r = iscol ? ((pre_r & ~mask) | fill) : pre_r;
            pre_c = iscol ? pre_c : ((pre_c & ~mask) | fill);
            reach |= iscol ? taken : taken << M;
        }
        const bool ok = active && target >= 0;
        failed |= active && target < 0;
        // potentials: settled nodes closer than the target move by their distance, all others by the target's
        const int tt = ok ? target : M;
#pragma unroll
        for (int n = 0; n < 2 * M; ++n) {
            const V add = (((done >> n) & 1) && dist[n] < D) ? dist[n] : D;
            pot[n] += ok ? add : 0;
        }
        // flip the arcs of the path back to its source column
        int v = tt;
        load += ok ? (1u << (4 * (tt - M))) : 0u;
#pragma unroll 1
        for (int s = 0; s < 2 * M + 2; ++s) {
            const bool go = ok && !((sources >> v) & 1);
            if (!__any_sync(kFull, go)) break;
            const int w = (int)(((v >= M ? pre_c >> (4 * (v - M)) : pre_r >> (4 * v))) & 15u);
            const uint64_t bit = v >= M ? (1ull << ((w & (M - 1)) * M + (v - M))) : (1ull << (v * M + (w & (M - 1))));
            pruned = go ? (v >= M ? (pruned | bit) : (pruned & ~bit)) : pruned;     // row w -> column v-M prunes; column w-M -> row v un-prunes
            v = go ? w : v;
        }
        const bool home = ok && ((sources >> v) & 1);
        load -= home ? (1u << (4 * (v - M))) : 0u;
        failed |= ok && !home;
    }
    if (failed) status |= kDevInternal;
    {   // the entries of reduced cost zero under the final potentials
        uint64_t tight = 0;
#pragma unroll
        for (int i = 0; i < M; ++i)
#pragma unroll
            for (int j = 0; j < M; ++j)
                tight |= (A::cost(base, i * M + j, T, Emin) + pot[i] == pot[M + j]) ? (1ull << (i * M + j)) : 0ull;
        const bool forest = tight_forest<M>(enabled ? tight : 0ull);
        *certified = enabled && !failed && forest;
    }
    const uint64_t all = (M == 8) ? ~0ull : ((1ull << (M * M)) - 1);
    return ~pruned & all;
}

// Called by all 32 lanes of a warp.  flow_smem: the CTA's region of flow_shared_bytes_per_thread(M) bytes per thread, T =
// threads per CTA (a constant, so that every cell offset is one), tid = this thread; live: the lane holds a block of the matrix (the others only keep the votes whole).
// turn: run the first pass on the block with rows and columns exchanged (the caller found that its start needs fewer
// paths); the optimum is the same set of entries, and the certificate of uniqueness holds for either view.  The pass that
// decides ties by position always sees the block as it stands.
template <int N, int M, int T>
__device__ __forceinline__ uint64_t exact_ssp(const uint32_t (&u)[M * M], int& status, unsigned char* flow_smem, int tid, bool live, bool turn) {
    int Emin, Emax;
    if (!exponent_range<M * M>(u, Emin, Emax)) { Emin = 1; Emax = 1; }
    // 128-bit costs: 64 tie bits + 24 significand bits + spread; paths (<= 2M arcs) and potentials (<= M(M-N)
    // updates) add 4 + 5 bits, the sign one more; beyond that the block takes the wide integers, on its own
    const bool wide = Emax - Emin > 26;
    FlowCell* base = reinterpret_cast<FlowCell*>(flow_smem) + tid;
    // first without the tie term, in 64-bit words
    bool certified = false;
    uint64_t kept;
    {
        uint32_t ut[M * M];
#pragma unroll
        for (int i = 0; i < M; ++i)
#pragma unroll
            for (int j = 0; j < M; ++j) ut[i * M + j] = turn ? u[j * M + i] : u[i * M + j];
        const uint64_t k1 = exact_flow_warp_reg<N, M, T>(ut, Emin, live && !wide, status, base, &certified);
        uint64_t back = 0;                                              // k1 with rows and columns exchanged
#pragma unroll
        for (int i = 0; i < M; ++i)
#pragma unroll
            for (int j = 0; j < M; ++j) back |= ((k1 >> (j * M + i)) & 1ull) << (i * M + j);
        kept = turn ? back : k1;
    }
    // blocks whose optimum is not certified unique (magnitude ties, as a rule): the full costs decide
    const bool again = live && !wide && !certified;
    if (__any_sync(0xFFFFFFFFu, again)) {
        // its state lives in the thread's local memory (cells one after the other): shared memory is all taken by the first pass
        FlowCell cells[flow_cells128_per_thread(M)];
        const uint64_t k2 = exact_flow_warp<Flow128<M>, N, M, 1>(u, Emin, again, status, cells, nullptr);
        kept = again ? k2 : kept;
    }
    if (live && wide) kept = exact_flow_run<CostWide, N, M>(u, Emin, status);
    return kept;
}

}  // namespace tmask
