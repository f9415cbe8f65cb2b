"""Pins for the CPU oracle: everything here checks oracle/tm_oracle.c against something other than
itself -- the paper's worked example, brute force written independently in Python, an LP solver, an
optimality certificate, closed forms and metamorphic relations.  No GPU needed."""
from __future__ import annotations

import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

import workloads
from oracle import tm_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------------------------
# independent helpers (plain Python / numpy; no oracle code)
# ----------------------------------------------------------------------------------------------
def exact_abs(x) -> Fraction:
    return abs(Fraction(float(x)))


def valid_patterns(N, M):
    """All 0/1 M x M matrices with every row sum and column sum equal to N, as (code, matrix)."""
    rows = [c for c in itertools.product((0, 1), repeat=M) if sum(c) == N]
    out = []
    for combo in itertools.product(rows, repeat=M):
        a = np.array(combo, dtype=np.int64)
        if (a.sum(axis=0) == N).all():
            code = sum(int(a[i, j]) << (i * M + j) for i in range(M) for j in range(M))
            out.append((code, a))
    return out


def py_exact(block, N, M, patterns):
    """argmax over valid patterns of (exact sum of kept |w|, code)."""
    best = None
    mags = [[exact_abs(block[i, j]) for j in range(M)] for i in range(M)]
    for code, a in patterns:
        s = sum(mags[i][j] for i in range(M) for j in range(M) if a[i, j])
        if best is None or (s, code) > best[:2]:
            best = (s, code, a)
    return best[2].astype(np.uint8), best[0]


def kept_sum(block, kept) -> Fraction:
    M = block.shape[0]
    return sum((exact_abs(block[i, j]) for i in range(M) for j in range(M) if kept[i, j]), Fraction(0))


def closed_form_cover(block, N, M):
    """kept = complement of (M-N lightest of every row) U (M-N lightest of every column), order (|w|, p)."""
    mag = np.abs(block.astype(np.float64))
    key = lambda p: (mag[p // M, p % M], p)
    pruned = set()
    for i in range(M):
        pruned |= set(sorted((i * M + j for j in range(M)), key=key)[: M - N])
    for j in range(M):
        pruned |= set(sorted((i * M + j for i in range(M)), key=key)[: M - N])
    kept = np.ones((M, M), np.uint8)
    for p in pruned:
        kept[p // M, p % M] = 0
    return kept


def rand_blocks(n, M, seed, kind="normal"):
    rng = np.random.Generator(np.random.PCG64(seed))
    if kind == "normal":
        return (rng.standard_normal((n, M, M)) * 0.02).astype(np.float32)
    if kind == "ties":
        return rng.integers(-3, 4, size=(n, M, M)).astype(np.float32)
    if kind == "laplace":
        return rng.laplace(0, 0.05, size=(n, M, M)).astype(np.float32)
    raise ValueError(kind)


# ----------------------------------------------------------------------------------------------
# Algorithm 1: the paper's worked example (golden file), and its generalisation to M x M
# ----------------------------------------------------------------------------------------------
def _read_golden():
    M = N = None; rows = []; accepted = []; wp = wo = None; inblock = False
    for line in open(os.path.join(GOLDEN, "alg1_worked_example.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0] == "M": M = int(tok[1])
        elif tok[0] == "N": N = int(tok[1])
        elif tok[0] == "block": inblock = True
        elif tok[0] == "accepted":
            inblock = False
            accepted = [tuple(int(v) for v in t.split(",")) for t in tok[1:]]
        elif tok[0] == "weight_P": wp = int(tok[1])
        elif tok[0] == "weight_opt": wo = int(tok[1])
        elif inblock: rows.append([float(v) for v in tok])
    return M, N, np.array(rows, np.float32), accepted, wp, wo


def test_alg1_worked_example_from_paper():
    M, N, block, accepted, wp, wo = _read_golden()
    kept, acc = orc.block_cover(block, N, M)
    got = [(int(p) // M + 1, int(p) % M + 1) for p in acc]
    assert got == accepted                      # seven iterations, all accepted, last one u4 -> v4
    assert len(got) == 7 and got[-1] == (4, 4)
    pruned_weight = sum(block[i - 1, j - 1] for i, j in got)
    assert pruned_weight == wp
    ex, _ = orc.block_exact_enum(block, N, M)   # the optimum prunes exactly the diagonal
    assert np.array_equal(ex, 1 - np.eye(M, dtype=np.uint8))
    assert block[ex == 0].sum() == wo
    assert Fraction(int(pruned_weight), int(wo)) == Fraction(7, 4)


@pytest.mark.parametrize("M", [2, 3, 4, 5, 6, 7, 8])
def test_alg1_tight_family_ratio(M):
    """Same construction on an M x M block: |P| = 2M-1 and W(P)/W* = (2M-1)/M (tightness paragraph)."""
    block = np.full((M, M), 10.0, np.float32)
    for i in range(M):
        block[i, i] = 1.0
        if i + 1 < M:
            block[i, i + 1] = 1.0
    kept, acc = orc.block_cover(block, M - 1, M)
    assert len(acc) == 2 * M - 1
    wp = float(block[kept == 0].sum())
    ex, _ = orc.block_exact_mcf(block, M - 1, M)
    wopt = float(block[ex == 0].sum())
    assert wopt == M and Fraction(int(wp), int(wopt)) == Fraction(2 * M - 1, M)


def test_alg1_degree_test_reading():
    """With 'degree <= M/2' read literally an (M/2+1)-th edge would be accepted at a node; the proof's
    'first M/2 edges' reading stops at M-N.  A block whose first row is uniformly lightest shows it:
    the three lightest entries of row 0 may be pruned only if their columns still need them."""
    block = np.array([[1, 2, 3, 4], [50, 60, 70, 80], [51, 61, 71, 81], [52, 62, 72, 82]], np.float32)
    kept, acc = orc.block_cover(block, 2, 4)
    # row 0: entries 1, 2 are accepted for the row; 3 and 4 are accepted for their columns (column degree < 2)
    assert [int(p) for p in acc[:4]] == [0, 1, 2, 3]
    # afterwards every column needs one more, every other row needs two
    assert (kept.sum(axis=0) <= 2).all() and (kept.sum(axis=1) <= 2).all()
    assert ((1 - kept).sum(axis=0) >= 2).all() and ((1 - kept).sum(axis=1) >= 2).all()


@pytest.mark.parametrize("N,M,kind", [(2, 4, "normal"), (2, 4, "ties"), (4, 8, "normal"), (4, 8, "ties"),
                                      (1, 4, "ties"), (3, 4, "normal"), (2, 8, "laplace"), (3, 6, "ties")])
def test_alg1_equals_closed_form(N, M, kind):
    """P = (M-N lightest per row) U (M-N lightest per column): an entry among its row's M-N lightest
    meets row degree < M-N when visited; an entry in neither set finds both degrees full."""
    for block in rand_blocks(300, M, 11 + N + M, kind):
        kept, _ = orc.block_cover(block, N, M)
        assert np.array_equal(kept, closed_form_cover(block, N, M))
        assert ((1 - kept).sum(axis=0) >= M - N).all() and ((1 - kept).sum(axis=1) >= M - N).all()


# ----------------------------------------------------------------------------------------------
# Exact optimum (Eq. 1): brute force, enumeration, min-cost flow
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("N,M,count", [(1, 2, 2), (1, 4, 24), (3, 4, 24), (2, 4, 90), (1, 3, 6), (2, 3, 6)])
def test_valid_pattern_counts(N, M, count):
    block = rand_blocks(1, M, 5)[0]
    assert len(valid_patterns(N, M)) == count
    assert orc.block_exact_enum(block, N, M)[1] == count
    assert orc.block_exact_bruteforce(block, N, M)[1] == count


def test_valid_pattern_count_3_6():
    assert orc.block_exact_enum(rand_blocks(1, 6, 5)[0], 3, 6)[1] == 297200


@pytest.mark.parametrize("N,M", [(2, 4), (1, 4), (3, 4), (1, 2), (2, 3)])
def test_exact_bruteforce_enum_mcf_python_agree(N, M):
    pats = valid_patterns(N, M)
    blocks = list(rand_blocks(120, M, 21, "normal")) + list(rand_blocks(120, M, 22, "ties"))
    if M == 4:
        blocks += list(workloads.adversarial_blocks_f32(4))
    for block in blocks:
        bf, _ = orc.block_exact_bruteforce(block, N, M)
        en, _ = orc.block_exact_enum(block, N, M)
        mc, info = orc.block_exact_mcf(block, N, M)
        py, _ = py_exact(block, N, M, pats)
        assert np.array_equal(bf, py), block
        assert np.array_equal(en, py), block
        assert np.array_equal(mc, py), block
        assert info == dict(nodes=2 * M + 2, edges=M * M + 2 * M, units=M * (M - N))


def test_exact_2_4_against_numpy_int_bruteforce_bulk():
    """10^5 blocks of integer weights (sums exact in int64), argmax over the 90 patterns in numpy."""
    pats = valid_patterns(2, 4)
    codes = np.array([c for c, _ in pats], np.int64)
    P = np.array([a.reshape(-1) for _, a in pats], np.int64)          # [90, 16]
    rng = np.random.Generator(np.random.PCG64(31))
    n = 100_000
    wi = rng.integers(0, 1 << 12, size=(n, 16))
    wi[: n // 4] = rng.integers(0, 4, size=(n // 4, 16))               # many ties
    W = (wi.astype(np.float32) * np.float32(2.0 ** -14)).reshape(n * 4 // 4, 4, 4)
    sums = wi @ P.T                                                    # [n, 90]
    best = sums.max(axis=1, keepdims=True)
    pick = np.where(sums == best, codes[None, :], -1).max(axis=1)      # ties -> largest code
    # oracle, whole-matrix entry point: lay the blocks side by side
    mat = np.ascontiguousarray(W.transpose(1, 0, 2).reshape(4, n * 4))
    res = orc.find_mask(mat, 2, 4, orc.EXACT)
    bits = orc.unpack_mask(res["mask"], n * 4).reshape(4, n, 4).transpose(1, 0, 2).reshape(n, 16).astype(np.int64)
    got = (bits << np.arange(16)).sum(axis=1)
    assert np.array_equal(got, pick)


def _lp_optimum(block, N, M):
    from scipy.optimize import linprog
    c = -np.abs(block.astype(np.float64)).reshape(-1)
    A = np.zeros((2 * M, M * M))
    for i in range(M):
        A[i, i * M:(i + 1) * M] = 1
        A[M + i, i::M] = 1
    r = linprog(c, A_eq=A, b_eq=np.full(2 * M, N), bounds=(0, 1), method="highs")
    assert r.status == 0
    return -r.fun, r.x


@pytest.mark.parametrize("N,M", [(4, 8), (2, 8), (3, 6), (2, 4)])
def test_mcf_matches_lp_relaxation(N, M):
    """The constraint matrix is totally unimodular, so the LP optimum equals the integer optimum."""
    rng = np.random.Generator(np.random.PCG64(41))
    for _ in range(40):
        block = rng.integers(1, 1 << 16, size=(M, M)).astype(np.float32)   # exact in fp64, ties unlikely
        kept, _ = orc.block_exact_mcf(block, N, M)
        assert (kept.sum(axis=0) == N).all() and (kept.sum(axis=1) == N).all()
        lp, _ = _lp_optimum(block, N, M)
        assert float(block[kept == 1].astype(np.float64).sum()) == pytest.approx(lp, rel=0, abs=1e-6)


def _has_improving_cycle(block, kept, M):
    """Bellman-Ford on the residual graph of the pruned-edge flow, exact integer costs (scaled by the
    tie term).  Residual arcs: row i -> col j (cost +c_ij) if (i,j) kept (can still be pruned),
    col j -> row i (cost -c_ij) if pruned.  An optimum of the perturbed problem has no negative cycle."""
    cost = {}
    for i in range(M):
        for j in range(M):
            q = exact_abs(block[i, j])
            cost[(i, j)] = q
    den = 1
    for v in cost.values():
        den = max(den, v.denominator)
    arcs = []
    for (i, j), q in cost.items():
        c = int(q * den) * (1 << (M * M)) + (1 << (i * M + j))
        if kept[i, j]:
            arcs.append((i, M + j, c))
        else:
            arcs.append((M + j, i, -c))
    dist = [0] * (2 * M)
    for it in range(2 * M + 1):
        changed = False
        for a, b, c in arcs:
            if dist[a] + c < dist[b]:
                dist[b] = dist[a] + c; changed = True
        if not changed:
            return False
    return True


@pytest.mark.parametrize("kind", ["normal", "ties", "laplace"])
def test_exact_4_8_has_no_improving_cycle(kind):
    """Optimality certificate for the 4:8 min-cost flow: no negative cycle in the residual graph.
    (A feasible mask with a negative residual cycle could be improved, e.g. the approximate one.)"""
    n_improvable = 0
    for block in rand_blocks(60, 8, 51, kind):
        kept, _ = orc.block_exact_mcf(block, 4, 8)
        assert (kept.sum(axis=0) == 4).all() and (kept.sum(axis=1) == 4).all()
        assert not _has_improving_cycle(block, kept, 8)
        ap = orc.block_approx(block, 4, 8)["kept"]
        n_improvable += _has_improving_cycle(block, ap, 8)
        assert kept_sum(block, kept) >= kept_sum(block, ap)
    assert n_improvable > 0        # the certificate is not vacuous


def test_exact_extreme_exponent_spread():
    """Blocks whose entries span ~240 binades: sums must still be compared exactly."""
    pats = valid_patterns(2, 4)
    rng = np.random.Generator(np.random.PCG64(61))
    for _ in range(60):
        block = np.ldexp(rng.standard_normal((4, 4)), rng.integers(-125, 120, size=(4, 4))).astype(np.float32)
        block[rng.integers(0, 4), rng.integers(0, 4)] = np.float32(rng.integers(1, 100) * 2.0 ** -149)
        py, _ = py_exact(block, 2, 4, pats)
        assert np.array_equal(orc.block_exact_enum(block, 2, 4)[0], py)
        assert np.array_equal(orc.block_exact_mcf(block, 2, 4)[0], py)


def test_exact_near_tie_needs_exact_sums():
    """Valid patterns whose sums differ by 2^-23 at a total of about 2^42: fp32 and fp64 sums see a tie
    (and the code rule would then pick another mask); exact sums do not."""
    B, u = np.float32(2.0 ** 40), np.float32(2.0 ** -23)
    block = np.array([[B, 0, 0, 0],
                      [0, B, 0, 0],
                      [B, 0, np.float32(1.0) + u, 1],
                      [0, B, 1, 1]], np.float32)
    pats = valid_patterns(2, 4)
    py, s = py_exact(block, 2, 4, pats)
    assert py[2, 2] == 1 and s == 4 * Fraction(2) ** 40 + 2 + Fraction(1, 2 ** 23)
    # what a floating-point sum would have chosen: all six completions tie, the largest code wins
    f64 = [(float(np.abs(block.astype(np.float64))[a == 1].sum()), code, a) for code, a in pats]
    naive = max(f64, key=lambda t: t[:2])[2]
    assert naive[2, 2] == 0
    for fn in (orc.block_exact_enum, orc.block_exact_mcf, orc.block_exact_bruteforce):
        assert np.array_equal(fn(block, 2, 4)[0], py)


# ----------------------------------------------------------------------------------------------
# Lemma: W(P) <= 2 W*, and the "factor of 1.2" remark
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("N,M,kind,n", [(2, 4, "normal", 1500), (2, 4, "ties", 500), (4, 8, "laplace", 150), (4, 8, "ties", 60)])
def test_lemma_two_approximation(N, M, kind, n):
    ratios = []
    for block in rand_blocks(n, M, 71, kind):
        cover, _ = orc.block_cover(block, N, M)
        exact = orc.block_exact_mcf(block, N, M)[0]
        wp = kept_sum(block, 1 - cover)          # weight pruned by Algorithm 1
        wstar = kept_sum(block, 1 - exact)       # minimal prunable weight
        assert wp <= 2 * wstar
        if wstar > 0:
            ratios.append(float(wp / wstar))
    if kind in ("normal", "laplace"):
        # Section 4.1, from-scratch paragraph: "on average within a factor of 1.2" (soft check)
        assert 1.1 < float(np.mean(ratios)) < 1.3


def test_lemma_on_all_zero_block():
    z = np.zeros((4, 4), np.float32)
    cover, _ = orc.block_cover(z, 2, 4)
    assert kept_sum(z, 1 - cover) == 0          # 0 <= 2 * 0: the bound is "<=", not "<"


# ----------------------------------------------------------------------------------------------
# Completion steps B and C (this build's definition): invariants only -- "parity unpinned"
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("N,M,kind", [(2, 4, "normal"), (2, 4, "ties"), (4, 8, "normal"), (4, 8, "ties"),
                                      (4, 8, "laplace"), (1, 4, "normal"), (3, 4, "ties"), (3, 6, "normal"), (2, 8, "ties")])
def test_completion_invariants(N, M, kind):
    saw_swap = False
    for block in rand_blocks(400, M, 81 + N, kind):
        r = orc.block_approx(block, N, M)
        a, b, k = r["after_a"], r["after_b"], r["kept"]
        assert (k.sum(axis=0) == N).all() and (k.sum(axis=1) == N).all()
        assert (a <= b).all()                                   # B only adds
        assert kept_sum(block, b) >= kept_sum(block, a)
        short_r = b.sum(axis=1) < N; short_c = b.sum(axis=0) < N
        assert b[np.ix_(short_r, short_c)].all()                # no free (short row, short column) entry left
        assert short_r.sum() <= max(N - 1, 0)
        shortfall = int(N * M - b.sum())
        assert shortfall <= (N * N) // 4 and r["n_swap"] == shortfall
        assert r["n_fill"] == int(b.sum() - a.sum())
        saw_swap |= r["n_swap"] > 0
    if (N, M) in ((2, 4), (4, 8)):
        assert saw_swap


@pytest.mark.parametrize("N,M,kind", [(2, 4, "normal"), (2, 4, "ties"), (4, 8, "laplace"), (4, 8, "ties"), (3, 6, "ties"), (1, 4, "ties")])
def test_step_b_is_the_heavy_to_light_greedy_fill(N, M, kind):
    """Step B checked as a certificate, without running it again: an entry outside Algorithm 1's kept set is taken by the
    fill exactly when, counting that kept set and the taken entries heavier than it, its row and its column both still hold
    fewer than N.  By induction from the heaviest entry down, only one set satisfies this for every entry."""
    for block in rand_blocks(300, M, 95 + M, kind):
        r = orc.block_approx(block, N, M)
        A, B = r["after_a"].astype(bool), r["after_b"].astype(bool)
        mag = np.abs(block.astype(np.float64))
        filled = B & ~A
        for i in range(M):
            for j in range(M):
                if A[i, j]:
                    continue
                p = i * M + j
                heavier = np.zeros((M, M), bool)
                for q in np.flatnonzero(filled):
                    qi, qj = divmod(int(q), M)
                    if (mag[qi, qj], q) > (mag[i, j], p):
                        heavier[qi, qj] = True
                H = A | heavier
                takes = H[i, :].sum() < N and H[:, j].sum() < N
                assert bool(filled[i, j]) == bool(takes), (i, j)


@pytest.mark.parametrize("N,M,kind", [(2, 4, "normal"), (2, 4, "ties"), (4, 8, "laplace"), (4, 8, "ties"), (3, 6, "ties")])
def test_step_c_single_swap_takes_the_lightest_eligible_entry(N, M, kind):
    """Blocks that need exactly one swap, checked against the rule itself: the entry that leaves is the lightest kept entry
    (r', c') for which some short row is free in column c' and some short column is free in row r'; the two that enter are
    the heaviest such free entries of column c' and of row r'."""
    seen = 0
    for block in rand_blocks(600, M, 97 + M, kind):
        r = orc.block_approx(block, N, M)
        if r["n_swap"] != 1:
            continue
        seen += 1
        B, K = r["after_b"].astype(bool), r["kept"].astype(bool)
        mag = np.abs(block.astype(np.float64))
        key = lambda i, j: (mag[i, j], i * M + j)
        DR = [i for i in range(M) if B[i].sum() < N]; DC = [j for j in range(M) if B[:, j].sum() < N]
        elig = [(i, j) for i in range(M) for j in range(M) if B[i, j]
                and any(not B[rr, j] for rr in DR) and any(not B[i, cc] for cc in DC)]
        x = min(elig, key=lambda e: key(*e))
        a = max(((rr, x[1]) for rr in DR if not B[rr, x[1]]), key=lambda e: key(*e))
        b = max(((x[0], cc) for cc in DC if not B[x[0], cc]), key=lambda e: key(*e))
        want = B.copy(); want[x] = False; want[a] = True; want[b] = True
        assert np.array_equal(K, want)
    assert seen > 20


def _swap_rule(S, block, N, M):
    """One application of step C's rule to the kept set S (bool [M, M]) with a short row: the set it must produce."""
    mag = np.abs(block.astype(np.float64))
    key = lambda i, j: (mag[i, j], i * M + j)
    DR = [i for i in range(M) if S[i].sum() < N]; DC = [j for j in range(M) if S[:, j].sum() < N]
    elig = [(i, j) for i in range(M) for j in range(M) if S[i, j]
            and any(not S[rr, j] for rr in DR) and any(not S[i, cc] for cc in DC)]
    x = min(elig, key=lambda e: key(*e))
    a = max(((rr, x[1]) for rr in DR if not S[rr, x[1]]), key=lambda e: key(*e))
    b = max(((x[0], cc) for cc in DC if not S[x[0], cc]), key=lambda e: key(*e))
    want = S.copy(); want[x] = False; want[a] = True; want[b] = True
    return want


@pytest.mark.parametrize("N,M,kind", [(4, 8, "laplace"), (4, 8, "ties"), (4, 8, "normal"), (3, 6, "ties"), (2, 4, "ties")])
def test_step_c_every_swap_of_a_sequence_follows_the_rule(N, M, kind):
    """Blocks that need several swaps: the kept set after every single swap (handed out by the oracle's trace entry) must
    be what one application of the rule makes of the set before it, and the last one is the result.  The rule is applied
    here to the oracle's intermediate states, so a wrong second or third swap cannot hide behind a right first one."""
    multi = swaps_seen = 0
    for block in rand_blocks(3000 if M == 8 else 800, M, 131 + M, kind):
        after_b, states = orc.block_approx_trace(block, N, M)
        assert len(states) == int(N * M - after_b.sum())                     # one swap per missing entry
        S = after_b.astype(bool)
        for nxt in states:
            assert np.array_equal(_swap_rule(S, block, N, M), nxt.astype(bool))
            S = nxt.astype(bool)
            swaps_seen += 1
        assert (S.sum(axis=0) == N).all() and (S.sum(axis=1) == N).all()
        assert np.array_equal(S, orc.block_approx(block, N, M)["kept"].astype(bool))
        multi += len(states) >= 2
    assert swaps_seen > 20
    if M == 8:
        assert multi > 10                                                    # sequences of two or more swaps were really seen


def _py_approx(block, N, M):
    """Steps A, B, C re-stated with Python sets (independent of the C code)."""
    mag = np.abs(block.astype(np.float64))
    key = lambda p: (mag[p // M, p % M], p)
    order = sorted(range(M * M), key=key)
    rd = [0] * M; cd = [0] * M; K = set(range(M * M))
    for p in order:
        if rd[p // M] < M - N or cd[p % M] < M - N:
            K.discard(p); rd[p // M] += 1; cd[p % M] += 1
    rk = [sum(1 for p in K if p // M == i) for i in range(M)]
    ck = [sum(1 for p in K if p % M == j) for j in range(M)]
    for p in reversed(order):
        if p not in K and rk[p // M] < N and ck[p % M] < N:
            K.add(p); rk[p // M] += 1; ck[p % M] += 1
    while any(r < N for r in rk):
        DR = [i for i in range(M) if rk[i] < N]; DC = [j for j in range(M) if ck[j] < N]
        for x in order:
            if x not in K:
                continue
            r2, c2 = divmod(x, M)
            ca = [r * M + c2 for r in DR if r * M + c2 not in K]
            cb = [r2 * M + c for c in DC if r2 * M + c not in K]
            if ca and cb:
                a = max(ca, key=key); b = max(cb, key=key)
                K.remove(x); K.add(a); K.add(b); rk[a // M] += 1; ck[b % M] += 1
                break
        else:
            raise AssertionError("no eligible entry")
    out = np.zeros((M, M), np.uint8)
    for p in K:
        out[p // M, p % M] = 1
    return out


@pytest.mark.parametrize("N,M,kind", [(2, 4, "normal"), (2, 4, "ties"), (4, 8, "laplace"), (4, 8, "ties"), (3, 6, "ties")])
def test_completion_matches_python_restatement(N, M, kind):
    for block in rand_blocks(250, M, 91, kind):
        assert np.array_equal(orc.block_approx(block, N, M)["kept"], _py_approx(block, N, M))


# ----------------------------------------------------------------------------------------------
# Metamorphic relations
# ----------------------------------------------------------------------------------------------
def _all_methods(block, N, M):
    return [orc.block_cover(block, N, M)[0], orc.block_approx(block, N, M)["kept"], orc.block_exact_mcf(block, N, M)[0]]


@pytest.mark.parametrize("N,M", [(2, 4), (4, 8)])
def test_scale_and_sign_invariance(N, M):
    rng = np.random.Generator(np.random.PCG64(101))
    for block in rand_blocks(40, M, 102, "normal"):
        ref = _all_methods(block, N, M)
        flipped = block * rng.choice(np.array([-1.0, 1.0], np.float32), size=block.shape)
        for k in (-20, 3, 40):
            scaled = np.ldexp(flipped, k).astype(np.float32)
            for a, b in zip(ref, _all_methods(scaled, N, M)):
                assert np.array_equal(a, b)


@pytest.mark.parametrize("N,M", [(2, 4), (4, 8)])
def test_transpose_and_permutation_on_tie_free_blocks(N, M):
    rng = np.random.Generator(np.random.PCG64(111))
    for block in rand_blocks(40, M, 112, "laplace"):
        assert len(set(np.abs(block).reshape(-1).tolist())) == M * M
        ref = _all_methods(block, N, M)
        for a, b in zip(ref, _all_methods(np.ascontiguousarray(block.T), N, M)):
            assert np.array_equal(a.T, b)                     # mask(W^T) = mask(W)^T
        pr, pc = rng.permutation(M), rng.permutation(M)
        perm = np.ascontiguousarray(block[pr][:, pc])
        for a, b in zip(ref, _all_methods(perm, N, M)):
            assert np.array_equal(a[pr][:, pc], b)


def test_transpose_with_ties_preserves_exact_objective():
    for block in rand_blocks(80, 4, 121, "ties"):
        a = orc.block_exact_mcf(block, 2, 4)[0]
        b = orc.block_exact_mcf(np.ascontiguousarray(block.T), 2, 4)[0]
        assert kept_sum(block, a) == kept_sum(block.T, b)


# ----------------------------------------------------------------------------------------------
# Whole-matrix entry point: tiling, packing, masked weights, objective, dtypes
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("N,M,method", [(2, 4, orc.APPROX), (2, 4, orc.EXACT), (2, 4, orc.APPROX_COVER),
                                        (4, 8, orc.APPROX), (4, 8, orc.EXACT)])
def test_matrix_layout_and_outputs(N, M, method):
    rows, cols = 3 * M * 2, 5 * 8 + 8 * (M // 8) + 4 * (M == 4)         # cols not a multiple of 32
    cols -= cols % M
    W = workloads.normal_f32(rows, cols, 0.02, 131)
    res = orc.find_mask(W, N, M, method)
    bits = orc.unpack_mask(res["mask"], cols)
    wpr = (cols + 31) // 32
    assert res["mask"].shape == (rows, wpr)
    full = np.unpackbits(res["mask"].view(np.uint8), axis=1, bitorder="little")
    assert not full[:, cols:].any()                                      # padding bits are zero
    for bi in range(rows // M):
        for bj in range(cols // M):
            blk = W[bi * M:(bi + 1) * M, bj * M:(bj + 1) * M]
            if method == orc.APPROX: want = orc.block_approx(blk, N, M)["kept"]
            elif method == orc.APPROX_COVER: want = orc.block_cover(blk, N, M)[0]
            else: want = orc.block_exact_mcf(blk, N, M)[0]
            assert np.array_equal(bits[bi * M:(bi + 1) * M, bj * M:(bj + 1) * M], want)
    assert np.array_equal(res["masked"].view(np.uint32), np.where(bits == 1, W.view(np.uint32), 0))
    assert res["objective"] == pytest.approx(float(np.abs(W.astype(np.float64))[bits == 1].sum()), rel=1e-12)
    assert res["nonfinite"] == 0


def test_block_independence():
    W = workloads.normal_f32(16, 32, 0.02, 141)
    base = orc.unpack_mask(orc.find_mask(W, 2, 4, orc.APPROX)["mask"], 32)
    W2 = W.copy(); W2[4:8, 12:16] = workloads.normal_f32(4, 4, 1.0, 142)
    other = orc.unpack_mask(orc.find_mask(W2, 2, 4, orc.APPROX)["mask"], 32)
    diff = base != other
    diff[4:8, 12:16] = False
    assert not diff.any()


@pytest.mark.parametrize("N,M,method", [(2, 4, orc.APPROX), (2, 4, orc.EXACT), (4, 8, orc.APPROX), (4, 8, orc.EXACT)])
def test_bf16_agrees_with_fp32_on_representable_values(N, M, method):
    b = workloads.normal_bf16(32, 64, 0.02, 151)
    f = workloads.bf16_bits_to_f32(b)
    rb = orc.find_mask(b, N, M, method); rf = orc.find_mask(f, N, M, method)
    assert np.array_equal(rb["mask"], rf["mask"])
    assert np.array_equal(workloads.bf16_bits_to_f32(rb["masked"]).view(np.uint32), rf["masked"].view(np.uint32))
    assert rb["objective"] == rf["objective"]


def test_nonfinite_count_and_negative_zero():
    W = workloads.normal_f32(8, 8, 0.02, 161)
    W[0, 0] = np.inf; W[3, 5] = np.nan; W[1, 1] = -0.0
    res = orc.find_mask(W, 2, 4, orc.APPROX)
    assert res["nonfinite"] == 2
    bits = orc.unpack_mask(res["mask"], 8)
    assert (bits.reshape(2, 4, 2, 4).sum(axis=1) == 2).all() and (bits.reshape(2, 4, 2, 4).sum(axis=3) == 2).all()


def test_zero_padded_columns_are_never_preferred():
    """The 64 x 147 stem layer is padded to 148 columns with zeros: a zero is kept only when forced."""
    W = workloads.config2()[0]
    assert W.shape == (64, 148) and not W[:, 147].any()
    for method in (orc.APPROX, orc.EXACT):
        bits = orc.unpack_mask(orc.find_mask(W, 2, 4, method)["mask"], 148)
        assert (bits.reshape(16, 4, 37, 4).sum(axis=1) == 2).all()
        assert (bits.reshape(16, 4, 37, 4).sum(axis=3) == 2).all()


def test_threads_do_not_change_results():
    W = workloads.normal_f32(64, 64, 0.02, 171)
    a = orc.find_mask(W, 2, 4, orc.APPROX, threads=1); b = orc.find_mask(W, 2, 4, orc.APPROX, threads=4)
    assert np.array_equal(a["mask"], b["mask"]) and a["objective"] == b["objective"]


def test_config1_quality_numbers():
    """256 x 256, N(0, 0.02): exact >= approx >= cover objective; gap of the completed mask is small."""
    W = workloads.config1()[0]
    ex = orc.find_mask(W, 2, 4, orc.EXACT)["objective"]
    ap = orc.find_mask(W, 2, 4, orc.APPROX)["objective"]
    cv = orc.find_mask(W, 2, 4, orc.APPROX_COVER)["objective"]
    assert ex >= ap >= cv > 0
    assert 1 - ap / ex < 0.03
