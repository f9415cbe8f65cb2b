// Bit-parallel core of the approximate 4:8 search (Algorithm 1 + completion) for 8x8 blocks.
//
// A set of entries is a 64-bit mask, bit p = 8*i + j for entry (i, j): a row is a byte, a column is
// the same bit of every byte.  As for 4x4 blocks the search only compares entries that share a row or
// a column; that order is carried by relation masks
//   hr[k] bit (i,j) = entry (i, (j+k) mod 8) is heavier than entry (i,j)      k = 1..7
//   hc[k] bit (i,j) = entry ((i+k) mod 8, j) is heavier than entry (i,j)      k = 1..7
// ("heavier" in the (|w|, position) order).  Counting is done bit-sliced: the number of set masks
// among seven is a 3-bit number held in three masks.
//
// Step A (Algorithm 1, closed form): kept iff fewer than four entries of the row and fewer than four
//   of the column are heavier.
// Step B (greedy fill heavy -> light) in rounds: a free entry of a short row and short column is
//   taken when fewer than d_row heavier candidates share its row and fewer than d_col its column
//   (d = what the line still lacks).  Exactly the sequential scan, a few rounds per block.
// Step C (2-for-1 swaps while a row is short): the entry to give way is the lightest kept entry
//   (r',c') such that some short row is free in column c' and some short column is free in row r'.
//   It is lighter than every other such entry of its row and of its column, so only the few "local
//   minima" marked by swap_candidates() need their magnitudes compared; the two entries taken instead
//   are the heaviest free ones of column c' in a short row and of row r' in a short column.
#pragma once
#include <cstdint>

#if defined(__CUDACC__)
#define TM_HD __host__ __device__ __forceinline__
#else
#define TM_HD inline
#endif

namespace tmask {

typedef unsigned long long u64;

struct Rel48 {
    u64 hr[8], hc[8];     // index 1..7 used
};

TM_HD u64 maj3_64(u64 a, u64 b, u64 c) { return (a & b) | (c & (a | b)); }

// result bit (i,j) = x bit (i, (j+k) mod 8): every byte rotated right by k
template <int K> TM_HD u64 rot_row8(u64 x) {
    constexpr u64 lo = 0x0101010101010101ull * (u64)((1u << (8 - K)) - 1u);
    return ((x >> K) & lo) | ((x << (8 - K)) & ~lo);
}
// result bit (i,j) = x bit ((i+k) mod 8, j): the word rotated right by k bytes
template <int K> TM_HD u64 rot_col8(u64 x) { return (x >> (8 * K)) | (x << (64 - 8 * K)); }

// hr[1..3], hc[1..3] given in full, hr[4] for columns 0..3, hc[4] for rows 0..3: the rest by antisymmetry
// (hr[8-k] bit (i, j+k) = not hr[k] bit (i, j)).
TM_HD void complete_relations8(Rel48& r) {
    r.hr[4] = (r.hr[4] & 0x0F0F0F0F0F0F0F0Full) | ((~r.hr[4] << 4) & 0xF0F0F0F0F0F0F0F0ull);
    r.hc[4] = (r.hc[4] & 0x00000000FFFFFFFFull) | ((~r.hc[4]) << 32);
    r.hr[7] = ~rot_row8<7>(r.hr[1]); r.hr[6] = ~rot_row8<6>(r.hr[2]); r.hr[5] = ~rot_row8<5>(r.hr[3]);
    r.hc[7] = ~rot_col8<7>(r.hc[1]); r.hc[6] = ~rot_col8<6>(r.hc[2]); r.hc[5] = ~rot_col8<5>(r.hc[3]);
}

// number of set masks among seven, as a 3-bit bit-sliced number
struct Count3 { u64 b0, b1, b2; };
TM_HD Count3 count7(u64 a, u64 b, u64 c, u64 d, u64 e, u64 f, u64 g) {
    const u64 s1 = a ^ b ^ c, k1 = maj3_64(a, b, c), s2 = d ^ e ^ f, k2 = maj3_64(d, e, f);
    const u64 s3 = s1 ^ s2 ^ g, k3 = maj3_64(s1, s2, g);
    Count3 n; n.b0 = s3; n.b1 = k1 ^ k2 ^ k3; n.b2 = maj3_64(k1, k2, k3);
    return n;
}
// bit-sliced "n < d"
TM_HD u64 less3(const Count3& n, const Count3& d) {
    const u64 lt0 = ~n.b0 & d.b0, eq1 = ~(n.b1 ^ d.b1), lt1 = ~n.b1 & d.b1, eq2 = ~(n.b2 ^ d.b2), lt2 = ~n.b2 & d.b2;
    return lt2 | (eq2 & (lt1 | (eq1 & lt0)));
}

// Step A.
TM_HD u64 cover_4_8(const Rel48& r) {
    const Count3 a = count7(r.hr[1], r.hr[2], r.hr[3], r.hr[4], r.hr[5], r.hr[6], r.hr[7]);
    const Count3 b = count7(r.hc[1], r.hc[2], r.hc[3], r.hc[4], r.hc[5], r.hc[6], r.hc[7]);
    return ~(a.b2 | b.b2);          // fewer than four heavier in the row and in the column
}

// What every line still lacks (0..4), bit-sliced and replicated over the line's entries.
struct Lack48 { Count3 row, col; u64 row_short, col_short; };
TM_HD Lack48 line_lack(u64 kept) {
    Lack48 L;
    {   // rows: popcount of every byte (at most 4), then 4 - count
        u64 c = kept - ((kept >> 1) & 0x5555555555555555ull);
        c = (c & 0x3333333333333333ull) + ((c >> 2) & 0x3333333333333333ull);
        c = (c + (c >> 4)) & 0x0F0F0F0F0F0F0F0Full;
        const u64 one = 0x0101010101010101ull;
        const u64 c0 = c & one, c1 = (c >> 1) & one, c2 = (c >> 2) & one;
        const u64 d0 = c0, d1 = c0 ^ c1, d2 = one & ~(c0 | c1 | c2);
        L.row.b0 = (d0 << 8) - d0; L.row.b1 = (d1 << 8) - d1; L.row.b2 = (d2 << 8) - d2;   // x * 255: spread over the byte
    }
    {   // columns: bit-sliced sum of the eight row bytes (at most 4)
        const uint32_t lo = (uint32_t)kept, hi = (uint32_t)(kept >> 32);
        const uint32_t r0 = lo, r1 = lo >> 8, r2 = lo >> 16, r3 = lo >> 24, r4 = hi, r5 = hi >> 8, r6 = hi >> 16, r7 = hi >> 24;
        const uint32_t s1 = r0 ^ r1 ^ r2, k1 = (r0 & r1) | (r2 & (r0 | r1)), s2 = r3 ^ r4 ^ r5, k2 = (r3 & r4) | (r5 & (r3 | r4));
        const uint32_t s3 = r6 ^ r7, k3 = r6 & r7;
        const uint32_t c0 = s1 ^ s2 ^ s3, k4 = (s1 & s2) | (s3 & (s1 | s2));
        const uint32_t t = k1 ^ k2, v = k3 ^ k4;
        const uint32_t c1 = t ^ v, c2 = (k1 & k2) | (k3 & k4) | (t & v);
        const uint32_t d0 = c0 & 0xFFu, d1 = (c0 ^ c1) & 0xFFu, d2 = ~(c0 | c1 | c2) & 0xFFu;
        const u64 rep = 0x0101010101010101ull;
        L.col.b0 = (u64)(d0 * 0x01010101u) * 0x0000000100000001ull; L.col.b1 = (u64)(d1 * 0x01010101u) * 0x0000000100000001ull;
        L.col.b2 = (u64)(d2 * 0x01010101u) * 0x0000000100000001ull;
        (void)rep;
    }
    L.row_short = L.row.b0 | L.row.b1 | L.row.b2;
    L.col_short = L.col.b0 | L.col.b1 | L.col.b2;
    return L;
}
TM_HD u64 open_candidates8(u64 kept, const Lack48& L) { return ~kept & L.row_short & L.col_short; }

// members of `set` heavier than the entry, in its row / column: bit-sliced count
TM_HD Count3 heavier_in_row8(const Rel48& r, u64 set) {
    return count7(r.hr[1] & rot_row8<1>(set), r.hr[2] & rot_row8<2>(set), r.hr[3] & rot_row8<3>(set), r.hr[4] & rot_row8<4>(set),
                  r.hr[5] & rot_row8<5>(set), r.hr[6] & rot_row8<6>(set), r.hr[7] & rot_row8<7>(set));
}
TM_HD Count3 heavier_in_col8(const Rel48& r, u64 set) {
    return count7(r.hc[1] & rot_col8<1>(set), r.hc[2] & rot_col8<2>(set), r.hc[3] & rot_col8<3>(set), r.hc[4] & rot_col8<4>(set),
                  r.hc[5] & rot_col8<5>(set), r.hc[6] & rot_col8<6>(set), r.hc[7] & rot_col8<7>(set));
}
// is some member of `set` lighter than the entry, in its row / column
TM_HD u64 lighter_in_row8(const Rel48& r, u64 set) {
    return (rot_row8<1>(set) & ~r.hr[1]) | (rot_row8<2>(set) & ~r.hr[2]) | (rot_row8<3>(set) & ~r.hr[3]) | (rot_row8<4>(set) & ~r.hr[4]) |
           (rot_row8<5>(set) & ~r.hr[5]) | (rot_row8<6>(set) & ~r.hr[6]) | (rot_row8<7>(set) & ~r.hr[7]);
}
TM_HD u64 lighter_in_col8(const Rel48& r, u64 set) {
    return (rot_col8<1>(set) & ~r.hc[1]) | (rot_col8<2>(set) & ~r.hc[2]) | (rot_col8<3>(set) & ~r.hc[3]) | (rot_col8<4>(set) & ~r.hc[4]) |
           (rot_col8<5>(set) & ~r.hc[5]) | (rot_col8<6>(set) & ~r.hc[6]) | (rot_col8<7>(set) & ~r.hc[7]);
}

// One round of step B: the candidates taken.
TM_HD u64 fill_accept8(const Rel48& r, const Lack48& L, u64 cand) {
    return cand & less3(heavier_in_row8(r, cand), L.row) & less3(heavier_in_col8(r, cand), L.col);
}

// spread "some bit of the column is set" over the column / "some bit of the row" over the row
TM_HD u64 any_in_col8(u64 x) { x |= x >> 32; x |= x >> 16; x |= x >> 8; x &= 0xFFull; return x * 0x0101010101010101ull; }
TM_HD u64 any_in_row8(u64 x) { x |= x >> 4; x |= x >> 2; x |= x >> 1; x &= 0x0101010101010101ull; return (x << 8) - x; }

// Step C, bit-parallel half.  free_a / free_b: the free entries of short rows / short columns (where
// the two new entries can go); returns the local minima among the entries that may give way.
TM_HD u64 swap_candidates8(const Rel48& r, const Lack48& L, u64 kept, u64& free_a, u64& free_b) {
    free_a = ~kept & L.row_short;
    free_b = ~kept & L.col_short;
    const u64 elig = kept & any_in_col8(free_a) & any_in_row8(free_b);
    return elig & ~lighter_in_row8(r, elig) & ~lighter_in_col8(r, elig);
}

// Step C, scalar half for one block: key(p) returns the magnitude pattern of entry p.  Returns false on
// an unexpected shape (no candidate).
template <class KeyFn>
TM_HD bool swap_apply8(u64& kept, u64 cands, u64 free_a, u64 free_b, KeyFn key) {
    if (!cands) return false;
    int x = -1; uint32_t best = 0;
    for (int p = 0; p < 64; ++p) {                               // ascending positions: the earliest of equals wins
        if (!((cands >> p) & 1)) continue;
        const uint32_t kp = key(p);
        if (x < 0 || kp < best) { x = p; best = kp; }
    }
    const int r2 = x >> 3, c2 = x & 7;
    int a = -1, b = -1; uint32_t ka = 0, kb = 0;
    for (int r = 0; r < 8; ++r) {                                // heaviest free entry of column c2 in a short row
        const int e = 8 * r + c2;
        if ((free_a >> e) & 1) { const uint32_t k = key(e); if (a < 0 || k >= ka) { a = e; ka = k; } }
    }
    for (int c = 0; c < 8; ++c) {                                // heaviest free entry of row r2 in a short column
        const int e = 8 * r2 + c;
        if ((free_b >> e) & 1) { const uint32_t k = key(e); if (b < 0 || k >= kb) { b = e; kb = k; } }
    }
    if (a < 0 || b < 0) return false;
    kept = (kept & ~(1ull << x)) | (1ull << a) | (1ull << b);
    return true;
}

}  // namespace tmask
