// Bit-parallel core of the approximate 2:4 search (Algorithm 1 + completion) for 4x4 blocks.
//
// A "pair mask" is a 32-bit word holding one 16-bit set per block for two blocks at once (block A in
// bits 0..15, block B in bits 16..31); inside a half, bit p = 4*i + j stands for entry (i, j).
// Every logic step below costs one instruction for both blocks and all 16 entries.
//
// The search only ever compares entries that share a row or a column, so the whole order it needs
// is carried by six relation masks:
//   hr[k] bit (i,j) = entry (i, (j+k) mod 4) is heavier than entry (i,j)      k = 1,2,3
//   hc[k] bit (i,j) = entry ((i+k) mod 4, j) is heavier than entry (i,j)      k = 1,2,3
// ("heavier" in the (|w|, position) order: among equal magnitudes the later position is heavier).
//
// Step A (Algorithm 1, closed form): an entry stays kept iff fewer than two entries of its row and
// fewer than two entries of its column are heavier.
// Step B (greedy fill heavy -> light) is evaluated in rounds: a free entry whose row and column are
// both short is taken in this round when, among the current candidates, fewer than d_row heavier ones
// share its row and fewer than d_col heavier ones share its column (d = what the line still lacks).
// Such an entry is reached by the sequential scan before its line fills up, so the rounds reproduce
// the scan exactly; every round takes at least one entry per unfinished block, and a block never
// lacks more than four entries.
// Step C (one 2-for-1 swap) is needed by roughly one block in six and is done per block by
// swap_fix_2_4().
#pragma once
#include <cstdint>

#if defined(__CUDACC__)
#define TM_HD __host__ __device__ __forceinline__
#else
#define TM_HD inline
#endif

namespace tmask {

struct Rel24 {
    uint32_t hr1, hr2, hr3, hc1, hc2, hc3;
};

TM_HD uint32_t maj3(uint32_t a, uint32_t b, uint32_t c) { return (a & b) | (c & (a | b)); }

// result bit (i,j) = x bit (i, (j+k) mod 4)
template <int K> TM_HD uint32_t rot_row(uint32_t x) {
    constexpr uint32_t lo = K == 1 ? 0x77777777u : (K == 2 ? 0x33333333u : 0x11111111u);
    return ((x >> K) & lo) | ((x << (4 - K)) & ~lo);
}
// result bit (i,j) = x bit ((i+k) mod 4, j), inside each 16-bit half
template <int K> TM_HD uint32_t rot_col(uint32_t x) {
    constexpr uint32_t lo = K == 1 ? 0x0FFF0FFFu : (K == 2 ? 0x00FF00FFu : 0x000F000Fu);
    return ((x >> (4 * K)) & lo) | ((x << (16 - 4 * K)) & ~lo);
}

// Completes the relation masks from their independent halves:
//   hr1, hc1 are given in full (pairs (j, j+1 mod 4)); hr2, hc2 only for j (resp. i) in {0, 1}.
// The rest follows from antisymmetry: "b heavier than a" is the complement of "a heavier than b".
TM_HD void complete_relations(Rel24& r) {
    r.hr2 = (r.hr2 & 0x33333333u) | ((~r.hr2 << 2) & 0xCCCCCCCCu);
    r.hc2 = (r.hc2 & 0x00FF00FFu) | ((~r.hc2 << 8) & 0xFF00FF00u);
    // hr3 bit (i, j+1) = not hr1 bit (i, j)
    const uint32_t nr = ~r.hr1, nc = ~r.hc1;
    r.hr3 = ((nr << 1) & 0xEEEEEEEEu) | ((nr >> 3) & 0x11111111u);
    r.hc3 = ((nc << 4) & 0xFFF0FFF0u) | ((nc >> 12) & 0x000F000Fu);
}

// Step A.
TM_HD uint32_t cover_2_4(const Rel24& r) {
    return ~(maj3(r.hr1, r.hr2, r.hr3) | maj3(r.hc1, r.hc2, r.hc3));
}

// Lines that already hold two kept entries / at least one, replicated over the line's bits.
TM_HD void line_fill(uint32_t kept, uint32_t& row_full, uint32_t& row_has, uint32_t& col_full, uint32_t& col_has) {
    {
        const uint32_t a = kept, b = kept >> 1, c = kept >> 2, d = kept >> 3, t = a | b | c;
        row_has = ((t | d) & 0x11111111u) * 15u;
        row_full = ((maj3(a, b, c) | (d & t)) & 0x11111111u) * 15u;
    }
    {
        const uint32_t a = kept, b = kept >> 4, c = kept >> 8, d = kept >> 12, t = a | b | c;
        col_has = ((t | d) & 0x000F000Fu) * 0x1111u;
        col_full = ((maj3(a, b, c) | (d & t)) & 0x000F000Fu) * 0x1111u;
    }
}

// One round of step B.  Returns the candidates that were still open when the round began (0 = done).
TM_HD uint32_t fill_round_2_4(const Rel24& r, uint32_t& kept) {
    uint32_t row_full, row_has, col_full, col_has;
    line_fill(kept, row_full, row_has, col_full, col_has);
    const uint32_t cand = ~(kept | row_full | col_full);
    // heavier candidates in the same row: at least one / at least two
    const uint32_t r1 = r.hr1 & rot_row<1>(cand), r2 = r.hr2 & rot_row<2>(cand), r3 = r.hr3 & rot_row<3>(cand);
    const uint32_t row_rej = maj3(r1, r2, r3) | ((r1 | r2 | r3) & row_has);   // a row holding one entry lacks one
    const uint32_t c1 = r.hc1 & rot_col<1>(cand), c2 = r.hc2 & rot_col<2>(cand), c3 = r.hc3 & rot_col<3>(cand);
    const uint32_t col_rej = maj3(c1, c2, c3) | ((c1 | c2 | c3) & col_has);
    kept |= cand & ~(row_rej | col_rej);
    return cand;
}

// Blocks (A: bit 0, B: bit 1) that still have a short row after step B, i.e. need step C.
TM_HD uint32_t short_blocks(uint32_t kept) {
    uint32_t row_full, row_has, col_full, col_has;
    line_fill(kept, row_full, row_has, col_full, col_has);
    return ((row_full & 0xFFFFu) != 0xFFFFu ? 1u : 0u) | ((row_full >> 16) != 0xFFFFu ? 2u : 0u);
}

// Step C for one block: kept16 has exactly one short row r and one short column c (each holding one
// entry, the shared entry (r,c)).  The lightest kept entry (r',c') outside row r and column c gives
// way to (r,c') and (r',c).  key[p] = magnitude pattern of entry p.  Returns false (mask unchanged)
// if the block does not have that shape.
template <class KeyT>
TM_HD bool swap_fix_2_4(const KeyT (&key)[16], uint32_t& kept16) {
    int r = -1, c = -1, nshort = 0;
    for (int i = 0; i < 4; ++i) {
        const uint32_t rowbits = (kept16 >> (4 * i)) & 0xFu, colbits = (kept16 >> i) & 0x1111u;
        const int rc = (int)((rowbits & 1) + ((rowbits >> 1) & 1) + ((rowbits >> 2) & 1) + (rowbits >> 3));
        const int cc = (int)((colbits & 1) + ((colbits >> 4) & 1) + ((colbits >> 8) & 1) + (colbits >> 12));
        if (rc != 2) { r = i; nshort += (rc == 1) ? 1 : 100; }
        if (cc != 2) { c = i; nshort += (cc == 1) ? 1 : 100; }
    }
    if (nshort != 2 || r < 0 || c < 0 || !((kept16 >> (4 * r + c)) & 1)) return false;
    const uint32_t elig = kept16 & ~(0xFu << (4 * r)) & ~(0x1111u << c);
    int x = -1; KeyT best = 0;
    for (int p = 0; p < 16; ++p)
        if (((elig >> p) & 1) && (x < 0 || key[p] < best)) { x = p; best = key[p]; }   // ascending p: earliest of equals
    if (x < 0) return false;
    kept16 = (kept16 & ~(1u << x)) | (1u << (4 * r + (x & 3))) | (1u << ((x & ~3) + c));
    return true;
}

}  // namespace tmask
