// Bit-parallel core of the approximate 4:8 search (Algorithm 1 + completion) for 8x8 blocks.
//
// A set of entries is a 64-bit mask, bit p = 8*i + j for entry (i, j): a row is a byte, a column is
// the same bit of every byte.  As for 4x4 blocks the search only compares entries that share a row or
// a column; that order is carried by relation masks
//   hr[k] bit (i,j) = entry (i, (j+k) mod 8) is heavier than entry (i,j)      k = 1..7
//   hc[k] bit (i,j) = entry ((i+k) mod 8, j) is heavier than entry (i,j)      k = 1..7
// ("heavier" in the (|w|, position) order).  Counting is done bit-sliced with carry-save adders on
// whole masks.
//
// Step A (Algorithm 1, closed form): kept iff fewer than four entries of the row and fewer than four
//   of the column are heavier.
// Step B (greedy fill heavy -> light) in rounds: a free entry of a short row and short column is
//   taken when fewer than d_row heavier candidates share its row and fewer than d_col its column
//   (d = what the line still lacks), i.e. when kept entries and heavier candidates together number
//   fewer than four in each.  Exactly the sequential scan, a few rounds per block.
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

// the row half of complete_relations8()
TM_HD void complete_row_relations8(Rel48& r);
// hr[1..3], hc[1..3] given in full, hr[4] for columns 0..3, hc[4] for rows 0..3: the rest by antisymmetry
// (hr[8-k] bit (i, j+k) = not hr[k] bit (i, j)).
TM_HD void complete_relations8(Rel48& r) {
    r.hr[4] = (r.hr[4] & 0x0F0F0F0F0F0F0F0Full) | ((~r.hr[4] << 4) & 0xF0F0F0F0F0F0F0F0ull);
    r.hc[4] = (r.hc[4] & 0x00000000FFFFFFFFull) | ((~r.hc[4]) << 32);
    r.hr[7] = ~rot_row8<7>(r.hr[1]); r.hr[6] = ~rot_row8<6>(r.hr[2]); r.hr[5] = ~rot_row8<5>(r.hr[3]);
    r.hc[7] = ~rot_col8<7>(r.hc[1]); r.hc[6] = ~rot_col8<6>(r.hc[2]); r.hc[5] = ~rot_col8<5>(r.hc[3]);
}

TM_HD void complete_row_relations8(Rel48& r) {
    r.hr[4] = (r.hr[4] & 0x0F0F0F0F0F0F0F0Full) | ((~r.hr[4] << 4) & 0xF0F0F0F0F0F0F0F0ull);
    r.hr[7] = ~rot_row8<7>(r.hr[1]); r.hr[6] = ~rot_row8<6>(r.hr[2]); r.hr[5] = ~rot_row8<5>(r.hr[3]);
}

// at least four of seven masks are set
TM_HD u64 four_of_seven(u64 a, u64 b, u64 c, u64 d, u64 e, u64 f, u64 g) {
    const u64 s1 = a ^ b ^ c, k1 = maj3_64(a, b, c), s2 = d ^ e ^ f, k2 = maj3_64(d, e, f);
    return maj3_64(k1, k2, maj3_64(s1, s2, g));          // count = (s1 ^ s2 ^ g) + 2 * (k1 + k2 + k3)
}

// at least n of seven masks are set, n = 1..7 (the same n for every bit): the count bit-sliced as ones, twos, fours
TM_HD u64 at_least_of_seven(u64 a, u64 b, u64 c, u64 d, u64 e, u64 f, u64 g, int n) {
    const u64 s1 = a ^ b ^ c, k1 = maj3_64(a, b, c), s2 = d ^ e ^ f, k2 = maj3_64(d, e, f);
    const u64 ones = s1 ^ s2 ^ g, k3 = maj3_64(s1, s2, g);
    const u64 twos = k1 ^ k2 ^ k3, fours = maj3_64(k1, k2, k3);
    switch (n) {
        case 1: return ones | twos | fours;
        case 2: return twos | fours;
        case 3: return fours | (twos & ones);
        case 4: return fours;
        case 5: return fours & (twos | ones);
        case 6: return fours & twos;
        default: return fours & twos & ones;
    }
}
// 1-D N:M along rows (no column constraint): kept iff fewer than n_keep entries of the row are heavier; n_keep = 1..7
TM_HD u64 keep_rows_8(const Rel48& r, int n_keep) {
    return ~at_least_of_seven(r.hr[1], r.hr[2], r.hr[3], r.hr[4], r.hr[5], r.hr[6], r.hr[7], n_keep);
}

// Step A.
TM_HD u64 cover_4_8(const Rel48& r) {
    // fewer than four heavier in the row and in the column
    return ~(four_of_seven(r.hr[1], r.hr[2], r.hr[3], r.hr[4], r.hr[5], r.hr[6], r.hr[7]) |
             four_of_seven(r.hc[1], r.hc[2], r.hc[3], r.hc[4], r.hc[5], r.hc[6], r.hc[7]));
}

// Lines that still lack entries (hold fewer than four; no line ever holds more), replicated over the
// line's entries.
struct Short48 { u64 row_short, col_short; };
TM_HD Short48 line_short(u64 kept) {
    Short48 L;
    {   // rows: popcount of every byte; 4 is the only count with bit 2 set
        u64 c = kept - ((kept >> 1) & 0x5555555555555555ull);
        c = (c & 0x3333333333333333ull) + ((c >> 2) & 0x3333333333333333ull);
        c += c >> 4;
        const u64 full = (c >> 2) & 0x0101010101010101ull;
        L.row_short = ~((full << 8) - full);
    }
    {   // columns: carry-save sum of the eight row bytes; the count is 4 iff at least two of the four carries are set
        const uint32_t lo = (uint32_t)kept, hi = (uint32_t)(kept >> 32);
        const uint32_t r0 = lo, r1 = lo >> 8, r2 = lo >> 16, r3 = lo >> 24, r4 = hi, r5 = hi >> 8, r6 = hi >> 16, r7 = hi >> 24;
        const uint32_t s1 = r0 ^ r1 ^ r2, k1 = (r0 & r1) | (r2 & (r0 | r1)), s2 = r3 ^ r4 ^ r5, k2 = (r3 & r4) | (r5 & (r3 | r4));
        const uint32_t s3 = r6 ^ r7, k3 = r6 & r7, k4 = (s1 & s2) | (s3 & (s1 | s2));
        const uint32_t full = ((k1 & k2) | (k3 & k4) | ((k1 | k2) & (k3 | k4))) & 0xFFu;
        const uint32_t w = ~(full * 0x01010101u);
        L.col_short = (u64)w | ((u64)w << 32);
    }
    return L;
}
TM_HD u64 open_candidates8(u64 kept, const Short48& L) { return ~kept & L.row_short & L.col_short; }

// is some member of `set` lighter than the entry, in its row / column
TM_HD u64 lighter_in_row8(const Rel48& r, u64 set) {
    return (rot_row8<1>(set) & ~r.hr[1]) | (rot_row8<2>(set) & ~r.hr[2]) | (rot_row8<3>(set) & ~r.hr[3]) | (rot_row8<4>(set) & ~r.hr[4]) |
           (rot_row8<5>(set) & ~r.hr[5]) | (rot_row8<6>(set) & ~r.hr[6]) | (rot_row8<7>(set) & ~r.hr[7]);
}
TM_HD u64 lighter_in_col8(const Rel48& r, u64 set) {
    return (rot_col8<1>(set) & ~r.hc[1]) | (rot_col8<2>(set) & ~r.hc[2]) | (rot_col8<3>(set) & ~r.hc[3]) | (rot_col8<4>(set) & ~r.hc[4]) |
           (rot_col8<5>(set) & ~r.hc[5]) | (rot_col8<6>(set) & ~r.hc[6]) | (rot_col8<7>(set) & ~r.hc[7]);
}

// One round of step B: the candidates taken.  A candidate is taken when its row holds fewer than four
// entries that are kept or heavier candidates, and its column likewise.  Seen from the other entry
// q = p + k of the line, "q is a heavier candidate than p" reads "q is a candidate and p (8 - k places
// on) is not heavier than q", so one rotation per distance moves a ready-made set.
TM_HD u64 fill_accept8(const Rel48& r, u64 kept, u64 cand) {
    const u64 row_blocked = four_of_seven(
        rot_row8<1>(kept | (cand & ~r.hr[7])), rot_row8<2>(kept | (cand & ~r.hr[6])), rot_row8<3>(kept | (cand & ~r.hr[5])),
        rot_row8<4>(kept | (cand & ~r.hr[4])), rot_row8<5>(kept | (cand & ~r.hr[3])), rot_row8<6>(kept | (cand & ~r.hr[2])),
        rot_row8<7>(kept | (cand & ~r.hr[1])));
    const u64 col_blocked = four_of_seven(
        rot_col8<1>(kept | (cand & ~r.hc[7])), rot_col8<2>(kept | (cand & ~r.hc[6])), rot_col8<3>(kept | (cand & ~r.hc[5])),
        rot_col8<4>(kept | (cand & ~r.hc[4])), rot_col8<5>(kept | (cand & ~r.hc[3])), rot_col8<6>(kept | (cand & ~r.hc[2])),
        rot_col8<7>(kept | (cand & ~r.hc[1])));
    return cand & ~(row_blocked | col_blocked);
}

// spread "some bit of the column is set" over the column / "some bit of the row" over the row
TM_HD u64 any_in_col8(u64 x) { x |= x >> 32; x |= x >> 16; x |= x >> 8; x &= 0xFFull; return x * 0x0101010101010101ull; }
TM_HD u64 any_in_row8(u64 x) { x |= x >> 4; x |= x >> 2; x |= x >> 1; x &= 0x0101010101010101ull; return (x << 8) - x; }

// Step C, bit-parallel half.  free_a / free_b: the free entries of short rows / short columns (where
// the two new entries can go); returns the local minima among the entries that may give way.
TM_HD u64 swap_candidates8(const Rel48& r, const Short48& L, u64 kept, u64& free_a, u64& free_b) {
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
