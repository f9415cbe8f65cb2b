/*
 * tm_oracle.c -- plain CPU oracle for the transposable N:M mask search.
 *
 * TEST INFRASTRUCTURE ONLY.  This file defines what the CUDA library must
 * compute; it is slow on purpose, shares no code with the CUDA path, and is
 * called only from the tests, the smoke check and the CPU-baseline leg of the
 * benchmark.  Nothing in the product path may link or call it.
 *
 * Paper: "Accelerated Sparse Neural Training: A Provable and Efficient Method to
 * Find N:M Transposable Masks" (arXiv 2102.08124), Section 4 (problem statement
 * Eq. 1, the min-cost-flow reduction of Fig. 3, Algorithm 1) and Appendix
 * "Proof of Lemma" (worked 4x4 example).
 *
 * Conventions (the paper is silent on all of them; they are this build's reading)
 *   - A weight matrix W[rows, cols] (row-major, leading dimension ld) is tiled into
 *     independent M x M blocks anchored at (0,0).  Inside a block the entry (i,j)
 *     has the position index p = i*M + j.
 *   - N is the number of KEPT entries per block row and per block column (Eq. 1).
 *   - Magnitudes are handled through their fp32 bit pattern with the sign cleared
 *     (bf16 is widened exactly); for finite values the unsigned integer order of
 *     these patterns is the order of |w|, and -0 equals +0.
 *   - Ties: every magnitude is read as |w_p| + eps * 2^p with eps a positive
 *     infinitesimal.  Two entries compare by (|w|, p); two masks compare by
 *     (sum of kept |w| as an exact number, code(S) = sum_p S_p 2^p), larger wins.
 *   - Exact sums: each |w_p| is turned into an integer q_p = significand << (E_p - Emin)
 *     (Emin = smallest exponent among the block's non-zero entries), carried in a
 *     384-bit integer, so candidate masks are compared as exact real numbers.
 *
 * Parity pins live in tests/test_oracle_pins.py (brute force over all 2^(M*M)
 * masks, the paper's worked example, the Lemma's bound, an LP solve, residual
 * graph optimality certificates, metamorphic relations).  The completion steps
 * B and C of the approximate method are defined by this build, not by the paper:
 * beyond their invariants they are "parity unpinned".
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define TMO_MAXM 8
#define TMO_MAXE (TMO_MAXM * TMO_MAXM)

enum { TMO_EXACT = 0, TMO_APPROX = 1, TMO_APPROX_COVER = 2, TMO_EXACT_MCF = 3, TMO_EXACT_ENUM = 4 };
enum { TMO_F32 = 0, TMO_BF16 = 1 };
enum { TMO_OK = 0, TMO_ERR_ARG = 1 };

/* ------------------------------------------------------------------------- */
/* 384-bit two's-complement integers (little-endian 64-bit limbs)             */
/* ------------------------------------------------------------------------- */
#define WL 6
typedef struct { uint64_t w[WL]; } wide;

static wide wide_zero(void) { wide r; memset(&r, 0, sizeof r); return r; }

static wide wide_add(wide a, wide b) {
    wide r; unsigned __int128 c = 0;
    for (int i = 0; i < WL; ++i) { c += (unsigned __int128)a.w[i] + b.w[i]; r.w[i] = (uint64_t)c; c >>= 64; }
    return r;
}
static wide wide_neg(wide a) {
    wide r; unsigned __int128 c = 1;
    for (int i = 0; i < WL; ++i) { c += (uint64_t)~a.w[i]; r.w[i] = (uint64_t)c; c >>= 64; }
    return r;
}
/* signed comparison: <0, 0, >0 */
static int wide_cmp(wide a, wide b) {
    int sa = (int)(a.w[WL - 1] >> 63), sb = (int)(b.w[WL - 1] >> 63);
    if (sa != sb) return sa ? -1 : 1;
    for (int i = WL - 1; i >= 0; --i) if (a.w[i] != b.w[i]) return a.w[i] < b.w[i] ? -1 : 1;
    return 0;
}
/* v << shift, v < 2^64, shift + 64 <= 384 - 1 */
static wide wide_shl64(uint64_t v, unsigned shift) {
    wide r = wide_zero();
    unsigned limb = shift / 64, off = shift % 64;
    r.w[limb] = v << off;
    if (off && limb + 1 < WL) r.w[limb + 1] = v >> (64 - off);
    return r;
}

/* ------------------------------------------------------------------------- */
/* magnitudes                                                                 */
/* ------------------------------------------------------------------------- */
/* fp32 bit pattern of |w| for element idx of a buffer of the given dtype */
static uint32_t mag_bits(const void* W, int dtype, int64_t idx) {
    if (dtype == TMO_F32) return ((const uint32_t*)W)[idx] & 0x7FFFFFFFu;
    return ((uint32_t)(((const uint16_t*)W)[idx] & 0x7FFFu)) << 16;
}
static int is_nonfinite(uint32_t u) { return (u >> 23) == 0xFFu; }

/* "entry p is lighter than entry q" under the (|w|, position) order */
static int lighter(const uint32_t* u, int p, int q) { return u[p] < u[q] || (u[p] == u[q] && p < q); }

/* exact integer image q_p of |w_p| relative to the block's smallest exponent.
 * |w| = sig * 2^(E-150) with E = max(biased exponent, 1), sig = mantissa (+ hidden bit if normal). */
static void exact_images(const uint32_t* u, int n, wide* q) {
    int Emin = 1 << 30;
    for (int p = 0; p < n; ++p) {
        uint32_t e = u[p] >> 23, m = u[p] & 0x7FFFFFu;
        uint32_t sig = e ? (m | 0x800000u) : m;
        int E = e ? (int)e : 1;
        if (sig && E < Emin) Emin = E;
    }
    for (int p = 0; p < n; ++p) {
        uint32_t e = u[p] >> 23, m = u[p] & 0x7FFFFFu;
        uint32_t sig = e ? (m | 0x800000u) : m;
        int E = e ? (int)e : 1;
        q[p] = sig ? wide_shl64(sig, (unsigned)(E - Emin)) : wide_zero();
    }
}

/* ------------------------------------------------------------------------- */
/* Algorithm 1 (Section 4, "2-Approximation algorithm"), as printed            */
/* ------------------------------------------------------------------------- */
/* order[] receives the entries sorted light -> heavy by (|w|, p). */
static void sort_entries(const uint32_t* u, int n, int* order) {
    for (int p = 0; p < n; ++p) order[p] = p;
    for (int a = 1; a < n; ++a) {               /* insertion sort */
        int x = order[a], b = a - 1;
        while (b >= 0 && lighter(u, x, order[b])) { order[b + 1] = order[b]; --b; }
        order[b + 1] = x;
    }
}

/* Step A.  Visit the coefficient edges light -> heavy; an edge (row i, column j) joins the pruned
 * list P when node i or node j still has fewer than M-N edges in P (the proof's "first M/2 edges
 * adjacent to i" reading of the degree test).  kept[] = complement of P.  If accepted is not NULL it
 * receives the accepted edges in the order they were picked; returns |P|. */
static int alg1_cover(const uint32_t* u, int N, int M, uint8_t* kept, int* accepted) {
    int n = M * M, order[TMO_MAXE], rdeg[TMO_MAXM] = {0}, cdeg[TMO_MAXM] = {0}, np = 0;
    sort_entries(u, n, order);
    for (int p = 0; p < n; ++p) kept[p] = 1;
    for (int k = 0; k < n; ++k) {
        int p = order[k], i = p / M, j = p % M;
        if (rdeg[i] < M - N || cdeg[j] < M - N) {
            kept[p] = 0; rdeg[i]++; cdeg[j]++;
            if (accepted) accepted[np] = p;
            np++;
        }
    }
    return np;
}

/* Step B (this build's completion): visit the pruned entries heavy -> light and keep an entry
 * again when its row and its column both hold fewer than N kept entries.  Returns #entries added. */
static int complete_fill(const uint32_t* u, int N, int M, uint8_t* kept) {
    int n = M * M, order[TMO_MAXE], rk[TMO_MAXM] = {0}, ck[TMO_MAXM] = {0}, added = 0;
    sort_entries(u, n, order);
    for (int p = 0; p < n; ++p) if (kept[p]) { rk[p / M]++; ck[p % M]++; }
    for (int k = n - 1; k >= 0; --k) {
        int p = order[k], i = p / M, j = p % M;
        if (!kept[p] && rk[i] < N && ck[j] < N) { kept[p] = 1; rk[i]++; ck[j]++; added++; }
    }
    return added;
}

/* Step C (this build's completion): while some row is short, take the lightest kept entry
 * x = (r', c') for which a short row r with (r, c') free and a short column c with (r', c) free
 * exist; un-keep x and keep the heaviest such (r, c') and the heaviest such (r', c).
 * Each swap adds one kept entry.  Returns the number of swaps, or -1 if no eligible entry exists
 * or the cap M*M is exceeded (neither can happen; the tests assert it).  If trace is not NULL it
 * receives a copy of kept[] after every swap (M*M bytes each, room for N*N/4 + 1 of them): an
 * observation point for the pins, the steps themselves do not look at it. */
static int complete_swap(const uint32_t* u, int N, int M, uint8_t* kept, uint8_t* trace) {
    int n = M * M, order[TMO_MAXE], swaps = 0;
    sort_entries(u, n, order);
    for (;;) {
        int rk[TMO_MAXM] = {0}, ck[TMO_MAXM] = {0}, shortrow = 0;
        for (int p = 0; p < n; ++p) if (kept[p]) { rk[p / M]++; ck[p % M]++; }
        for (int i = 0; i < M; ++i) if (rk[i] < N) shortrow = 1;
        if (!shortrow) return swaps;
        if (swaps >= n) return -1;
        int done = 0;
        for (int k = 0; k < n && !done; ++k) {
            int x = order[k];
            if (!kept[x]) continue;
            int r2 = x / M, c2 = x % M, a = -1, b = -1;
            for (int r = 0; r < M; ++r)            /* heaviest free (r, c2) in a short row */
                if (rk[r] < N && !kept[r * M + c2] && (a < 0 || lighter(u, a, r * M + c2))) a = r * M + c2;
            for (int c = 0; c < M; ++c)            /* heaviest free (r2, c) in a short column */
                if (ck[c] < N && !kept[r2 * M + c] && (b < 0 || lighter(u, b, r2 * M + c))) b = r2 * M + c;
            if (a >= 0 && b >= 0) {
                kept[x] = 0; kept[a] = 1; kept[b] = 1; done = 1;
                if (trace && swaps <= N * N / 4) memcpy(trace + (size_t)swaps * (size_t)n, kept, (size_t)n);
                swaps++;
            }
        }
        if (!done) return -1;
    }
}

/* ------------------------------------------------------------------------- */
/* Exact: the definition (Eq. 1) by enumeration of every valid pattern         */
/* ------------------------------------------------------------------------- */
typedef struct {
    int N, M; const wide* q;
    uint8_t cur[TMO_MAXE]; int colcnt[TMO_MAXM];
    wide best_sum; uint64_t best_code; int have; uint8_t best[TMO_MAXE]; int64_t count;
} enum_state;

static void enum_rows(enum_state* st, int row, int col, int inrow, wide sum, uint64_t code) {
    int M = st->M, N = st->N;
    if (row == M) {                      /* all rows placed; column sums are checked on the way */
        st->count++;
        int c = st->have ? wide_cmp(sum, st->best_sum) : 1;
        if (c > 0 || (c == 0 && code > st->best_code)) {
            st->best_sum = sum; st->best_code = code; st->have = 1;
            memcpy(st->best, st->cur, (size_t)(M * M));
        }
        return;
    }
    if (col == M) { if (inrow == N) enum_rows(st, row + 1, 0, 0, sum, code); return; }
    if (inrow + (M - col) < N) return;   /* cannot reach N kept in this row any more */
    int p = row * M + col;
    /* leave (row, col) pruned -- allowed only if the column can still reach N */
    if (st->colcnt[col] + (M - 1 - row) >= N) { st->cur[p] = 0; enum_rows(st, row, col + 1, inrow, sum, code); }
    /* keep it */
    if (inrow < N && st->colcnt[col] < N) {
        st->cur[p] = 1; st->colcnt[col]++;
        enum_rows(st, row, col + 1, inrow + 1, wide_add(sum, st->q[p]), code | (1ull << p));
        st->colcnt[col]--; st->cur[p] = 0;
    }
}

/* returns the number of valid patterns visited (90 for N=2, M=4) */
static int64_t exact_enumerate(const uint32_t* u, int N, int M, uint8_t* kept) {
    wide q[TMO_MAXE]; enum_state st; memset(&st, 0, sizeof st);
    exact_images(u, M * M, q);
    st.N = N; st.M = M; st.q = q;
    enum_rows(&st, 0, 0, 0, wide_zero(), 0);
    memcpy(kept, st.best, (size_t)(M * M));
    return st.count;
}

/* Brute force over all 2^(M*M) masks (M <= 4): the ground truth the pins compare against. */
static int64_t exact_bruteforce(const uint32_t* u, int N, int M, uint8_t* kept) {
    int n = M * M; wide q[TMO_MAXE], best_sum = wide_zero(); uint64_t best_code = 0; int have = 0; int64_t valid = 0;
    if (n > 16) return -1;
    exact_images(u, n, q);
    for (uint64_t code = 0; code < (1ull << n); ++code) {
        int ok = 1;
        for (int i = 0; i < M && ok; ++i) { int s = 0; for (int j = 0; j < M; ++j) s += (int)((code >> (i * M + j)) & 1); ok = (s == N); }
        for (int j = 0; j < M && ok; ++j) { int s = 0; for (int i = 0; i < M; ++i) s += (int)((code >> (i * M + j)) & 1); ok = (s == N); }
        if (!ok) continue;
        valid++;
        wide sum = wide_zero();
        for (int p = 0; p < n; ++p) if ((code >> p) & 1) sum = wide_add(sum, q[p]);
        int c = have ? wide_cmp(sum, best_sum) : 1;
        if (c > 0 || (c == 0 && code > best_code)) { best_sum = sum; best_code = code; have = 1; }
    }
    for (int p = 0; p < n; ++p) kept[p] = (uint8_t)((best_code >> p) & 1);
    return valid;
}

/* ------------------------------------------------------------------------- */
/* Exact: min-cost flow on the network of Fig. 3, successive shortest paths    */
/* ------------------------------------------------------------------------- */
/* Nodes: source, M row nodes, M column nodes, sink (2M+2).  Edges: source->row i (capacity M-N,
 * cost 0), row i->column j (capacity 1, cost c_ij = q_ij * 2^64 + 2^p, the tie rule folded into
 * the cost), column j->sink (capacity M-N, cost 0): M*M + 2M edges.  A flow of M*(M-N) units is
 * sent one unit at a time along a cheapest residual path (Bellman-Ford); a unit on (i,j) prunes
 * W_ij.  Minimising the pruned cost maximises the kept (sum |w|, code). */
typedef struct { int from, to, cap; wide cost; } mcf_edge;

static int exact_mcf(const uint32_t* u, int N, int M, uint8_t* kept, int* n_nodes, int* n_edges, int* n_units) {
    int n = M * M, V = 2 * M + 2, S = 0, T = 2 * M + 1, ne = 0;
    mcf_edge e[2 * (TMO_MAXE + 2 * TMO_MAXM)]; wide q[TMO_MAXE];
    exact_images(u, n, q);
#define ADD_EDGE(a, b, c, w) do { e[ne].from = (a); e[ne].to = (b); e[ne].cap = (c); e[ne].cost = (w); ne++; \
                                  e[ne].from = (b); e[ne].to = (a); e[ne].cap = 0;   e[ne].cost = wide_neg(w); ne++; } while (0)
    for (int i = 0; i < M; ++i) ADD_EDGE(S, 1 + i, M - N, wide_zero());
    int first_coef = ne;
    for (int p = 0; p < n; ++p) {
        wide c = wide_zero();                       /* c = q_p * 2^64 + 2^p */
        for (int l = 1; l < WL; ++l) c.w[l] = q[p].w[l - 1];
        c.w[0] = 1ull << p;
        ADD_EDGE(1 + p / M, 1 + M + p % M, 1, c);
    }
    for (int j = 0; j < M; ++j) ADD_EDGE(1 + M + j, T, M - N, wide_zero());
#undef ADD_EDGE
    int units = 0, demand = M * (M - N);
    while (units < demand) {
        wide dist[2 * TMO_MAXM + 2]; int reach[2 * TMO_MAXM + 2] = {0}, pre[2 * TMO_MAXM + 2];
        reach[S] = 1; dist[S] = wide_zero();
        for (int round = 0; round < V; ++round) {
            int changed = 0;
            for (int k = 0; k < ne; ++k) {
                if (e[k].cap <= 0 || !reach[e[k].from]) continue;
                wide d = wide_add(dist[e[k].from], e[k].cost);
                if (!reach[e[k].to] || wide_cmp(d, dist[e[k].to]) < 0) { dist[e[k].to] = d; reach[e[k].to] = 1; pre[e[k].to] = k; changed = 1; }
            }
            if (!changed) break;
        }
        if (!reach[T]) return -1;
        for (int v = T; v != S; v = e[pre[v]].from) { e[pre[v]].cap -= 1; e[pre[v] ^ 1].cap += 1; }
        units++;
    }
    for (int p = 0; p < n; ++p) kept[p] = (uint8_t)(e[first_coef + 2 * p].cap == 1);  /* unsaturated = kept */
    if (n_nodes) *n_nodes = V;
    if (n_edges) *n_edges = ne / 2;
    if (n_units) *n_units = units;
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Block-level entry points (used by the pins)                                 */
/* ------------------------------------------------------------------------- */
static int check_nm(int N, int M) { return M >= 1 && M <= TMO_MAXM && N >= 0 && N <= M; }

/* u: M*M fp32 bit patterns of |w| (sign already cleared).  kept: M*M bytes (1 = kept). */
int tmo_block_cover(const uint32_t* u, int N, int M, uint8_t* kept, int* accepted, int* n_accepted) {
    if (!check_nm(N, M)) return TMO_ERR_ARG;
    int np = alg1_cover(u, N, M, kept, accepted);
    if (n_accepted) *n_accepted = np;
    return TMO_OK;
}

/* Steps A, B, C.  after_a / after_b (optional, M*M bytes) receive the intermediate kept sets. */
int tmo_block_approx(const uint32_t* u, int N, int M, uint8_t* kept, uint8_t* after_a, uint8_t* after_b,
                     int* n_fill, int* n_swap) {
    if (!check_nm(N, M)) return TMO_ERR_ARG;
    alg1_cover(u, N, M, kept, NULL);
    if (after_a) memcpy(after_a, kept, (size_t)(M * M));
    int nb = complete_fill(u, N, M, kept);
    if (after_b) memcpy(after_b, kept, (size_t)(M * M));
    int nc = complete_swap(u, N, M, kept, NULL);
    if (n_fill) *n_fill = nb;
    if (n_swap) *n_swap = nc;
    return nc < 0 ? TMO_ERR_ARG : TMO_OK;
}

/* The same search, also handing back the kept set after every swap of step C (swap_trace: room for
 * N*N/4 + 1 sets of M*M bytes), so that the pins can check a sequence of swaps one rule application at a time. */
int tmo_block_approx_trace(const uint32_t* u, int N, int M, uint8_t* kept, uint8_t* after_b, uint8_t* swap_trace, int* n_swap) {
    if (!check_nm(N, M) || !swap_trace) return TMO_ERR_ARG;
    alg1_cover(u, N, M, kept, NULL);
    complete_fill(u, N, M, kept);
    if (after_b) memcpy(after_b, kept, (size_t)(M * M));
    int nc = complete_swap(u, N, M, kept, swap_trace);
    if (n_swap) *n_swap = nc;
    return nc < 0 ? TMO_ERR_ARG : TMO_OK;
}

int tmo_block_exact_enum(const uint32_t* u, int N, int M, uint8_t* kept, int64_t* n_patterns) {
    if (!check_nm(N, M) || M > 6) return TMO_ERR_ARG;
    int64_t c = exact_enumerate(u, N, M, kept);
    if (n_patterns) *n_patterns = c;
    return TMO_OK;
}

int tmo_block_exact_bruteforce(const uint32_t* u, int N, int M, uint8_t* kept, int64_t* n_valid) {
    if (!check_nm(N, M) || M > 4) return TMO_ERR_ARG;
    int64_t c = exact_bruteforce(u, N, M, kept);
    if (n_valid) *n_valid = c;
    return TMO_OK;
}

int tmo_block_exact_mcf(const uint32_t* u, int N, int M, uint8_t* kept, int* n_nodes, int* n_edges, int* n_units) {
    if (!check_nm(N, M)) return TMO_ERR_ARG;
    return exact_mcf(u, N, M, kept, n_nodes, n_edges, n_units) ? TMO_ERR_ARG : TMO_OK;
}

/* ------------------------------------------------------------------------- */
/* Whole-matrix entry point                                                    */
/* ------------------------------------------------------------------------- */
static void solve_block(const uint32_t* u, int N, int M, int method, uint8_t* kept) {
    switch (method) {
    case TMO_APPROX_COVER: alg1_cover(u, N, M, kept, NULL); break;
    case TMO_APPROX: alg1_cover(u, N, M, kept, NULL); complete_fill(u, N, M, kept); complete_swap(u, N, M, kept, NULL); break;
    case TMO_EXACT_ENUM: exact_enumerate(u, N, M, kept); break;
    case TMO_EXACT_MCF: exact_mcf(u, N, M, kept, NULL, NULL, NULL); break;
    default: /* TMO_EXACT: the definition by enumeration where that is feasible, else Fig. 3's flow */
        if (M <= 4) exact_enumerate(u, N, M, kept); else exact_mcf(u, N, M, kept, NULL, NULL, NULL);
    }
}

/* W, masked_w_out: host buffers of dtype (fp32 or bf16 patterns), row-major, leading dimension ld (elements).
 * mask_out: rows * ceil(cols/32) words; bit (i, j) -> word i*wpr + j/32, bit j%32; padding bits 0.
 * masked_w_out (may be NULL, may alias W): kept entries copied bit for bit, pruned entries +0.
 * objective_out (may be NULL): sum of kept |w| in fp64 (compensated, block-row-major order).
 * nonfinite_out (may be NULL): number of Inf/NaN entries seen.  threads: OpenMP threads over block rows. */
int tmo_find_mask(const void* W, int dtype, int64_t rows, int64_t cols, int64_t ld, int N, int M, int method, int threads,
                  uint32_t* mask_out, void* masked_w_out, double* objective_out, int64_t* nonfinite_out) {
    if (!check_nm(N, M) || rows < 0 || cols < 0 || rows % M || cols % M || ld < cols) return TMO_ERR_ARG;
    if (dtype != TMO_F32 && dtype != TMO_BF16) return TMO_ERR_ARG;
    if (method < TMO_EXACT || method > TMO_EXACT_ENUM) return TMO_ERR_ARG;
    int64_t wpr = (cols + 31) / 32, brows = rows / M, bcols = cols / M;
    if (mask_out) memset(mask_out, 0, (size_t)(rows * wpr) * sizeof(uint32_t));
    double* row_sum = (double*)calloc((size_t)(brows > 0 ? brows : 1), sizeof(double));
    int64_t* row_bad = (int64_t*)calloc((size_t)(brows > 0 ? brows : 1), sizeof(int64_t));
    if (!row_sum || !row_bad) { free(row_sum); free(row_bad); return TMO_ERR_ARG; }
    (void)threads;
#ifdef _OPENMP
#pragma omp parallel for schedule(static) num_threads(threads > 0 ? threads : 1)
#endif
    for (int64_t bi = 0; bi < brows; ++bi) {
        double s = 0.0, comp = 0.0; int64_t bad = 0;
        for (int64_t bj = 0; bj < bcols; ++bj) {
            uint32_t u[TMO_MAXE]; uint8_t kept[TMO_MAXE];
            for (int i = 0; i < M; ++i) for (int j = 0; j < M; ++j) {
                u[i * M + j] = mag_bits(W, dtype, (bi * M + i) * ld + bj * M + j);
                bad += is_nonfinite(u[i * M + j]);
            }
            solve_block(u, N, M, method, kept);
            for (int i = 0; i < M; ++i) for (int j = 0; j < M; ++j) {
                int64_t r = bi * M + i, c = bj * M + j, idx = r * ld + c; int k = kept[i * M + j];
                if (k && mask_out) mask_out[r * wpr + c / 32] |= 1u << (c % 32);
                if (masked_w_out) {
                    if (dtype == TMO_F32) ((uint32_t*)masked_w_out)[idx] = k ? ((const uint32_t*)W)[idx] : 0u;
                    else ((uint16_t*)masked_w_out)[idx] = k ? ((const uint16_t*)W)[idx] : (uint16_t)0;
                }
                if (k) {                                  /* Neumaier-compensated fp64 sum of |w| */
                    union { uint32_t b; float f; } cv; cv.b = u[i * M + j];
                    double x = (double)cv.f, t = s + x;
                    comp += (s >= x || s <= -x) ? ((s - t) + x) : ((x - t) + s);
                    s = t;
                }
            }
        }
        row_sum[bi] = s + comp; row_bad[bi] = bad;
    }
    double total = 0.0, comp = 0.0; int64_t bad = 0;
    for (int64_t bi = 0; bi < brows; ++bi) {
        double x = row_sum[bi], t = total + x;
        comp += (total >= x || total <= -x) ? ((total - t) + x) : ((x - t) + total);
        total = t; bad += row_bad[bi];
    }
    if (objective_out) *objective_out = total + comp;
    if (nonfinite_out) *nonfinite_out = bad;
    free(row_sum); free(row_bad);
    return TMO_OK;
}

/* ------------------------------------------------------------------------- */
/* Neighbouring operations of Section 5 ("Structured sparsity without full training") */
/* ------------------------------------------------------------------------- */
static float bits_to_float(uint32_t b) { union { uint32_t b; float f; } c; c.b = b; return c.f; }
static uint32_t float_to_bits(float f) { union { uint32_t b; float f; } c; c.f = f; return c.b; }
/* raw value of element idx widened to fp32 (bf16 exactly) */
static float elem_value(const void* W, int dtype, int64_t idx) {
    if (dtype == TMO_F32) return ((const float*)W)[idx];
    return bits_to_float(((uint32_t)((const uint16_t*)W)[idx]) << 16);
}
/* fp32 -> bf16, round to nearest even; NaN stays NaN */
static uint16_t float_to_bf16(float f) {
    uint32_t u = float_to_bits(f);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x40u);
    return (uint16_t)((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);
}

/* 1-D N:M magnitude pruning (Section 5, "we prune [the] weights with the lowest magnitude" in every group of M
 * contiguous weights of a row).  N = KEPT per group; order (|w|, position in the group), the later of equals is
 * the heavier one.  violations = pruned entries that are non-zero ("pattern-violations": active weights the
 * pattern removes).  absorb_mean ("mean absorption"): the mean of the group's pruned weights is added to every
 * kept weight: mu = (sum of the pruned weights in position order, fp64) / (their number); kept' = fp64(kept + mu)
 * rounded to fp32 (and then to bf16, nearest even, for bf16 tensors).  objective = sum of kept |w| (before absorption). */
int tmo_nm_mask_1d(const void* W, int dtype, int64_t rows, int64_t cols, int64_t ld, int N, int M, int absorb_mean,
                   uint32_t* mask_out, void* masked_w_out, double* objective_out, int64_t* violations_out) {
    if (M < 1 || M > TMO_MAXM || N < 0 || N > M || rows < 0 || cols < 0 || cols % M || ld < cols) return TMO_ERR_ARG;
    if (dtype != TMO_F32 && dtype != TMO_BF16) return TMO_ERR_ARG;
    int64_t wpr = (cols + 31) / 32, viol = 0;
    double total = 0.0, comp = 0.0;
    if (mask_out) memset(mask_out, 0, (size_t)(rows * wpr) * sizeof(uint32_t));
    for (int64_t r = 0; r < rows; ++r) for (int64_t g = 0; g < cols / M; ++g) {
        uint32_t u[TMO_MAXM]; int kept[TMO_MAXM];
        for (int j = 0; j < M; ++j) u[j] = mag_bits(W, dtype, r * ld + g * M + j);
        for (int j = 0; j < M; ++j) {               /* kept iff fewer than N entries of the group are heavier */
            int heavier = 0;
            for (int k = 0; k < M; ++k) if (k != j && lighter(u, j, k)) heavier++;
            kept[j] = heavier < N;
        }
        double psum = 0.0; int pcnt = 0;
        for (int j = 0; j < M; ++j) if (!kept[j]) { psum += (double)elem_value(W, dtype, r * ld + g * M + j); pcnt++; viol += (u[j] != 0); }
        double mu = (absorb_mean && pcnt) ? psum / (double)pcnt : 0.0;
        for (int j = 0; j < M; ++j) {
            int64_t c = g * M + j, idx = r * ld + c;
            if (kept[j] && mask_out) mask_out[r * wpr + c / 32] |= 1u << (c % 32);
            if (kept[j]) { double x = (double)bits_to_float(u[j]), t = total + x; comp += (total >= x) ? ((total - t) + x) : ((x - t) + total); total = t; }
            if (masked_w_out) {
                if (dtype == TMO_F32) {
                    uint32_t raw = ((const uint32_t*)W)[idx];
                    ((uint32_t*)masked_w_out)[idx] = !kept[j] ? 0u : (absorb_mean ? float_to_bits((float)((double)bits_to_float(raw) + mu)) : raw);
                } else {
                    uint16_t raw = ((const uint16_t*)W)[idx];
                    ((uint16_t*)masked_w_out)[idx] = !kept[j] ? (uint16_t)0 :
                        (absorb_mean ? float_to_bf16((float)((double)bits_to_float((uint32_t)raw << 16) + mu)) : raw);
                }
            }
        }
    }
    if (objective_out) *objective_out = total + comp;
    if (violations_out) *violations_out = viol;
    return TMO_OK;
}

/* Pattern-violations of an arbitrary packed mask: entries whose mask bit is 0 although the weight is non-zero. */
int tmo_mask_violations(const void* W, int dtype, int64_t rows, int64_t cols, int64_t ld, const uint32_t* mask, int64_t* violations_out) {
    if (rows < 0 || cols < 0 || ld < cols || (dtype != TMO_F32 && dtype != TMO_BF16)) return TMO_ERR_ARG;
    int64_t wpr = (cols + 31) / 32, viol = 0;
    for (int64_t r = 0; r < rows; ++r) for (int64_t c = 0; c < cols; ++c)
        if (!((mask[r * wpr + c / 32] >> (c % 32)) & 1u) && mag_bits(W, dtype, r * ld + c) != 0) viol++;
    *violations_out = viol;
    return TMO_OK;
}

/* 2:4 operand compression for W and its transpose from one transposable mask (Section 1 and Fig. 2: the same
 * mask serves Y = W X and dL/dX = W^T dL/dY).  Row form: for every row and every group of 4 columns the two kept
 * values in column order -> values[rows][cols/2]; their column indices inside the group, idx0 | idx1 << 2, as a
 * nibble -> meta[rows][ceil(cols/32)] (group g of a row: bits 4*(g%8) of word g/8).  Column form: the same for
 * W^T (groups of 4 rows of a column) -> values_t[cols][rows/2], meta_t[cols][ceil(rows/32)].
 * A group that does not hold exactly two kept entries gets zeros and is counted in bad_groups. */
int tmo_compress_2_4(const void* W, int dtype, int64_t rows, int64_t cols, int64_t ld, const uint32_t* mask,
                     void* values, uint32_t* meta, void* values_t, uint32_t* meta_t, int64_t* bad_groups) {
    if (rows < 0 || cols < 0 || rows % 4 || cols % 4 || ld < cols || (dtype != TMO_F32 && dtype != TMO_BF16)) return TMO_ERR_ARG;
    int64_t wpr = (cols + 31) / 32, wpr_t = (rows + 31) / 32, bad = 0;
    size_t es = dtype == TMO_F32 ? 4 : 2;
    memset(meta, 0, (size_t)(rows * wpr) * 4); memset(meta_t, 0, (size_t)(cols * wpr_t) * 4);
    memset(values, 0, (size_t)(rows * (cols / 2)) * es); memset(values_t, 0, (size_t)(cols * (rows / 2)) * es);
#define TMO_BIT(r, c) ((mask[(r) * wpr + (c) / 32] >> ((c) % 32)) & 1u)
    for (int64_t r = 0; r < rows; ++r) for (int64_t g = 0; g < cols / 4; ++g) {
        int idx[4], n = 0;
        for (int j = 0; j < 4; ++j) if (TMO_BIT(r, g * 4 + j)) idx[n++] = j;
        if (n != 2) { bad++; continue; }
        for (int k = 0; k < 2; ++k) memcpy((char*)values + (size_t)(r * (cols / 2) + g * 2 + k) * es, (const char*)W + (size_t)(r * ld + g * 4 + idx[k]) * es, es);
        meta[r * wpr + g / 8] |= (uint32_t)(idx[0] | (idx[1] << 2)) << (4 * (g % 8));
    }
    for (int64_t c = 0; c < cols; ++c) for (int64_t g = 0; g < rows / 4; ++g) {
        int idx[4], n = 0;
        for (int i = 0; i < 4; ++i) if (TMO_BIT(g * 4 + i, c)) idx[n++] = i;
        if (n != 2) { bad++; continue; }
        for (int k = 0; k < 2; ++k) memcpy((char*)values_t + (size_t)(c * (rows / 2) + g * 2 + k) * es, (const char*)W + (size_t)((g * 4 + idx[k]) * ld + c) * es, es);
        meta_t[c * wpr_t + g / 8] |= (uint32_t)(idx[0] | (idx[1] << 2)) << (4 * (g % 8));
    }
#undef TMO_BIT
    if (bad_groups) *bad_groups = bad;
    return TMO_OK;
}

int tmo_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
