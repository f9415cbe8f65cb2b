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
// share its row and fewer than d_col heavier ones share its column (d = what the line still lacks),
// in other words when kept entries and heavier candidates together number fewer than two in each.
// Such an entry is reached by the sequential scan before its line fills up, so the rounds reproduce
// the scan exactly; every round takes at least one entry per unfinished block, and a block never
// lacks more than four entries.
// Step C (one 2-for-1 swap) is needed by roughly one block in six.  After step B such a block has
// exactly one short row r and one short column c, each holding the single entry (r,c); the swap
// removes the lightest kept entry x = (r',c') outside row r (none of them lies in column c) and adds
// (r,c') and (r',c).  Only the flagged blocks do this, each on a lane of its own, comparing the six
// magnitudes directly (marking the local minima from the relation masks first would spare three of the
// comparisons but cost every lane of every item a dozen instructions).
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
#if defined(__CUDA_ARCH__)
    if constexpr (K == 2) { uint32_t r; asm("prmt.b32 %0, %1, %1, 0x2301;" : "=r"(r) : "r"(x)); return r; }   // bytes swapped inside either half
#endif
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

// Lines that already hold two kept entries, replicated over the line's bits.
struct LineFill {
    uint32_t row_full, col_full;
};
TM_HD LineFill line_fill(uint32_t kept) {
    // Left shifts gather a line's four flags in its last entry (the top bit of the nibble, the last row); one right shift
    // brings the verdict back down and a multiplication spreads it over the line.  (Left shifts can run on either of two
    // pipes, right shifts only on the busier one.)
    LineFill f;
    {
        const uint32_t a = kept, b = kept << 1, c = kept << 2, d = kept << 3;
        f.row_full = (((maj3(a, b, c) | (d & (a | b | c))) >> 3) & 0x11111111u) * 15u;
    }
    {
        const uint32_t a = kept, b = kept << 4, c = kept << 8, d = kept << 12;
        f.col_full = (((maj3(a, b, c) | (d & (a | b | c))) >> 12) & 0x000F000Fu) * 0x1111u;
    }
    return f;
}
TM_HD uint32_t open_candidates(uint32_t kept, const LineFill& f) { return ~(kept | f.row_full | f.col_full); }

// entries of `set` that have a heavier member of `set` in their row: at least one / at least two
TM_HD void heavier_in_row(const Rel24& r, uint32_t set, uint32_t& any, uint32_t& two) {
    const uint32_t a = r.hr1 & rot_row<1>(set), b = r.hr2 & rot_row<2>(set), c = r.hr3 & rot_row<3>(set);
    any = a | b | c; two = maj3(a, b, c);
}
TM_HD void heavier_in_col(const Rel24& r, uint32_t set, uint32_t& any, uint32_t& two) {
    const uint32_t a = r.hc1 & rot_col<1>(set), b = r.hc2 & rot_col<2>(set), c = r.hc3 & rot_col<3>(set);
    any = a | b | c; two = maj3(a, b, c);
}

// One round of step B on the candidates `cand` (= open_candidates(kept, f)): returns the entries taken.
// A candidate is taken when its row holds fewer than two entries that are kept or heavier candidates,
// and its column likewise.  Seen from the other entry q = p + k of the line, "q is a heavier candidate
// than p" reads "q is a candidate and p (k places back, i.e. 4 - k places on) is not heavier than q",
// so one rotation per distance moves a ready-made set.
TM_HD uint32_t fill_accept(const Rel24& r, uint32_t kept, uint32_t cand) {
    const uint32_t row_blocked = maj3(rot_row<1>(kept | (cand & ~r.hr3)), rot_row<2>(kept | (cand & ~r.hr2)), rot_row<3>(kept | (cand & ~r.hr1)));
    const uint32_t col_blocked = maj3(rot_col<1>(kept | (cand & ~r.hc3)), rot_col<2>(kept | (cand & ~r.hc2)), rot_col<3>(kept | (cand & ~r.hc1)));
    return cand & ~(row_blocked | col_blocked);
}

// The candidates of blocks that have exactly one: such a candidate has no rival in its row or column, so the scan
// takes it as it stands (and the block has none left afterwards).
TM_HD uint32_t lone_candidates(uint32_t cand) {
#if defined(__CUDA_ARCH__)
    uint32_t less_one;
    asm("add.u16x2 %0, %1, %2;" : "=r"(less_one) : "r"(cand), "r"(0xFFFFFFFFu));      // cand - 1 in either half
#else
    const uint32_t less_one = ((cand - 1u) & 0xFFFFu) | ((cand - 0x10000u) & 0xFFFF0000u);
#endif
    const uint32_t several = cand & less_one;                          // a half is non-zero iff it holds two or more
    return cand & (((several & 0xFFFFu) ? 0u : 0xFFFFu) | ((several >> 16) ? 0u : 0xFFFF0000u));
}

// Blocks (A: bit 0, B: bit 1) that still have a short row after step B, i.e. need step C.
TM_HD uint32_t short_blocks(const LineFill& f) {
    return ((f.row_full & 0xFFFFu) != 0xFFFFu ? 1u : 0u) | ((f.row_full >> 16) != 0xFFFFu ? 2u : 0u);
}

// index of the highest set bit (x != 0)
TM_HD int highest_bit(uint32_t x) {
#if defined(__CUDA_ARCH__)
    return 31 - __clz((int)x);
#else
    int p = 31;
    while (!((x >> p) & 1)) --p;
    return p;
#endif
}

// Step C for one block flagged by short_blocks(): key(p) returns the magnitude pattern of entry p.  The
// entry to give way is the lightest of the six kept entries outside the short row (the earliest of equal
// magnitudes).  SMALL: magnitudes fit in 28 bits, so magnitude and position are compared as one word.
// Returns false (mask unchanged) on an unexpected shape.
template <bool SMALL, class KeyFn>
TM_HD bool swap_apply_2_4(uint32_t& kept16, KeyFn key) {
    const uint32_t a = kept16;
    const uint32_t s = a - ((a >> 1) & 0x5555u);
    const uint32_t t = (s & 0x3333u) + ((s >> 2) & 0x3333u);       // kept entries per row, one nibble each
    const uint32_t rs = t ^ 0x2222u;                               // 3 in the nibble of the row that holds one, 0 where a row holds two
    if (!rs) return false;
    const int r4 = highest_bit(rs) - 1;                            // 4 * short row
    if (r4 < 0 || rs != (3u << r4)) return false;
    const uint32_t only = (a >> r4) & 0xFu;                        // the short row's single entry: it marks the short column
    const int c = highest_bit(only);
    uint32_t cands = a & ~(0xFu << r4);                            // two entries in each of the three other rows
    int x;
    if constexpr (SMALL) {
        uint32_t best = 0xFFFFFFFFu;
#pragma unroll
        for (int n = 0; n < 6; ++n) {
            const int p = highest_bit(cands);
            cands ^= 1u << p;
            const uint32_t kp = key(p) * 16u + (uint32_t)p;
            best = kp < best ? kp : best;
        }
        x = (int)(best & 15u);
    } else {
        uint32_t best = 0xFFFFFFFFu;
        x = 0;
#pragma unroll
        for (int n = 0; n < 6; ++n) {                              // descending positions: of equals the earliest stays
            const int p = highest_bit(cands);
            cands ^= 1u << p;
            const uint32_t kp = key(p);
            if (kp <= best) { best = kp; x = p; }
        }
    }
    kept16 = (a ^ (1u << x)) | (1u << (r4 + (x & 3))) | (1u << ((x & 12) + c));
    return true;
}

}  // namespace tmask
