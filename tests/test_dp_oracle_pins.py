"""Pins for the oracle of the two dynamic programmes (Sec. 4.3, Algorithm 1, Algorithm 2): the
recurrences against the definitions they solve (Eq. 5, Eq. 6a) by enumeration, and the closed
cases the mathematics fixes."""
import math
import random

import pytest

from oracle import dp_oracle as P
from paper_2301_12187_b200 import inputs as I_


def random_tables(rng, L, unmergeable=0.2, neg_inf=0.0):
    return I_.random_dp_tables(rng, L, P.INF, unmergeable, neg_inf)


@pytest.mark.parametrize("seed", range(6))
def test_alg1_equals_enumeration_of_eq_6a(seed):
    rng = random.Random(seed)
    L = rng.randint(2, 9)
    T, _ = random_tables(rng, L)
    T_opt, S_opt = P.alg1(T, L)
    for k in range(L + 1):
        assert T_opt[k][k] == 0 and S_opt[k][k] == []
        for l in range(k + 1, L + 1):
            assert T_opt[k][l] == P.brute_topt(T, k, l)
            assert T_opt[k][l] <= T[k][l]
            # the set that is returned attains the optimum and lies strictly inside (k, l)
            assert all(k < s < l for s in S_opt[k][l]) and S_opt[k][l] == sorted(set(S_opt[k][l]))
            assert P.pieces_latency(T, [k] + S_opt[k][l] + [l]) == T_opt[k][l]


def test_alg1_closed_cases():
    L = 6
    # additive latencies: merging never helps or hurts -> T_opt is the span length times the unit
    T = [[3 * (j - i) if j > i else 0 for j in range(L + 1)] for i in range(L + 1)]
    T_opt, _ = P.alg1(T, L)
    assert all(T_opt[k][l] == 3 * (l - k) for k in range(L + 1) for l in range(k, L + 1))
    # every merged span costs 1: the whole network as one layer
    T = [[1 if j > i else 0 for j in range(L + 1)] for i in range(L + 1)]
    T_opt, S_opt = P.alg1(T, L)
    assert T_opt[0][L] == 1 and S_opt[0][L] == []
    # nothing longer than one layer can be merged: every boundary stays
    T = [[(2 if j == i + 1 else P.INF) if j > i else 0 for j in range(L + 1)] for i in range(L + 1)]
    T_opt, S_opt = P.alg1(T, L)
    assert T_opt[0][L] == 2 * L and S_opt[0][L] == list(range(1, L))
    # a planted mistake (argmax instead of argmin) would fail the first case above; so would T[k][m]
    # in place of T[m][l]: check the asymmetric table below
    T = [[0] * 4 for _ in range(4)]
    T[0][1], T[1][2], T[2][3], T[0][2], T[1][3], T[0][3] = 5, 1, 5, 2, 9, 20
    T_opt, S_opt = P.alg1(T, 3)
    assert T_opt[0][3] == 7 and S_opt[0][3] == [2]


@pytest.mark.parametrize("seed", range(8))
def test_alg2_equals_enumeration_of_eq_5(seed):
    rng = random.Random(100 + seed)
    L = rng.randint(2, 7)
    T, I = random_tables(rng, L, neg_inf=0.15 if seed % 2 else 0.0)
    T_opt, _ = P.alg1(T, L)
    for T0 in sorted({T_opt[0][L], T_opt[0][L] + 1, T_opt[0][L] + 4, sum(T[i][i + 1] for i in range(L)) + 1}):
        A, S, D, ok = P.alg2(T0, L, T, I)
        want = P.brute_select(T0, L, T, I)
        if want is None:
            assert (not ok) or D == -math.inf
            continue
        assert ok and D == pytest.approx(want, abs=1e-12)
        # the returned sets are a feasible point of Eq. 5 that attains it
        assert set(A) <= set(S) and all(0 < s < L for s in S)
        assert P.pieces_latency(T, [0] + S + [L]) < T0
        b = [0] + A + [L]
        assert sum(I[a][c] for a, c in zip(b[:-1], b[1:])) == pytest.approx(want, abs=1e-12)


def test_alg2_budget_properties():
    rng = random.Random(7)
    L = 6
    T, I = random_tables(rng, L, unmergeable=0.0)
    T_opt, _ = P.alg1(T, L)
    # strict constraint: a budget equal to the optimal latency is infeasible, one more is feasible
    assert not P.alg2(T_opt[0][L], L, T, I)[3]
    assert P.alg2(T_opt[0][L] + 1, L, T, I)[3]
    # the objective never decreases with the budget, and a budget above the unmerged network's
    # latency keeps every activation (objective 0: single layers cost nothing)
    prev = -math.inf
    for T0 in range(T_opt[0][L] + 1, sum(T[i][i + 1] for i in range(L)) + 3):
        D = P.alg2(T0, L, T, I)[2]
        assert D >= prev - 1e-12
        prev = D
    A, S, D, ok = P.alg2(sum(T[i][i + 1] for i in range(L)) + 1, L, T, I)
    assert ok and D == 0.0 and A == list(range(1, L)) and S == list(range(1, L))


# ---- the extended programmes (App. B: Algorithm 3, Algorithm 4) -----------------------------------
def brute_chain(J, k, l, a, b):
    """max over subsets of inner boundaries (all with d = 0) of the summed block importance."""
    import itertools
    best = -math.inf
    inner = list(range(k + 1, l))
    for r in range(len(inner) + 1):
        for Bs in itertools.combinations(inner, r):
            bs = [k] + list(Bs) + [l]
            d = {x: 0 for x in Bs}
            d[k], d[l] = a, b
            best = max(best, sum(J[x][y][d[x]][d[y]] for x, y in zip(bs[:-1], bs[1:])))
    return best


@pytest.mark.parametrize("seed", range(6))
def test_alg3_equals_enumeration_of_block_chains(seed):
    rng = random.Random(300 + seed)
    L = rng.randint(2, 7)
    _, I, sig = I_.random_dp_tables_ext(rng, L, P.INF)
    J = P.apply_exclusions(I, L, sig)
    I_opt, B_opt = P.alg3(I, L, sig)
    for k in range(L + 1):
        for l in range(k + 1, L + 1):
            for a in range(2):
                for b in range(2):
                    want = brute_chain(J, k, l, a, b)
                    assert I_opt[k][l][a][b] == pytest.approx(want, abs=1e-12) or (want == -math.inf and I_opt[k][l][a][b] == -math.inf)
                    if want > -math.inf:
                        Bs = B_opt[k][l][a][b]
                        assert all(k < x < l for x in Bs) and Bs == sorted(set(Bs))
                        bs = [k] + Bs + [l]
                        d = {x: 0 for x in Bs}
                        d[k], d[l] = a, b
                        assert sum(J[x][y][d[x]][d[y]] for x, y in zip(bs[:-1], bs[1:])) == pytest.approx(want, abs=1e-12)


def test_alg3_exclusions_and_single_block_term():
    L = 2
    I = [[[[0.0, 0.0], [0.0, 0.0]] for _ in range(L + 1)] for _ in range(L + 1)]
    # one block over both layers, distinguishable by its end indicators
    for a in range(2):
        for b in range(2):
            I[0][2][a][b] = -1.0 - a - 10 * b
            I[0][1][a][b] = I[1][2][a][b] = -100.0
    sig = [True, True, False]                      # input and boundary 1 identities, last activation not
    I_opt, B_opt = P.alg3(I, L, sig)
    # d_2 = 0 is excluded (sigma_2 is no identity); the single block keeps d_0 = a: the listing's
    # literal m' = k term, I[0][2][0][1], would give -11 for a = 1 too
    assert I_opt[0][2][0][1] == -11.0 and I_opt[0][2][1][1] == -12.0 and B_opt[0][2][1][1] == []
    assert I_opt[0][2][0][0] == -math.inf and I_opt[0][2][1][0] == -math.inf
    # identities on both edges with d_l = 0 are excluded (App. B.2): block (0, 1] with b = 0
    assert I_opt[0][1][0][0] == -math.inf and I_opt[0][1][1][0] == -math.inf and I_opt[0][1][1][1] == -100.0


@pytest.mark.parametrize("seed", range(8))
def test_alg4_equals_enumeration_of_the_extended_problem(seed):
    rng = random.Random(400 + seed)
    L = rng.randint(2, 6)
    T, I, sig = I_.random_dp_tables_ext(rng, L, P.INF, p_identity=0.3 + 0.1 * (seed % 4))
    J = P.apply_exclusions(I, L, sig)
    T_opt, _ = P.alg1(T, L)
    for T0 in sorted({T_opt[0][L], T_opt[0][L] + 1, T_opt[0][L] + 3, sum(T[i][i + 1] for i in range(L)) + 1}):
        A, S, B, d0, dL, obj, ok = P.alg4(T0, L, T, I, sig)
        want = P.brute_select_ext(T0, L, T, I, sig)
        if want is None:
            assert not ok
            continue
        assert ok and obj == pytest.approx(want, abs=1e-12)
        # the returned point is feasible and attains the optimum
        assert set(A) <= set(B) and set(A) <= set(S) and all(0 < x < L for x in S + B)
        assert P.pieces_latency(T, [0] + S + [L]) < T0
        d = {x: (1 if x in A else 0) for x in B}
        d[0], d[L] = d0, dL
        bs = [0] + B + [L]
        assert sum(J[x][y][d[x]][d[y]] for x, y in zip(bs[:-1], bs[1:])) == pytest.approx(want, abs=1e-12)


@pytest.mark.parametrize("seed", range(4))
def test_alg4_reduces_to_alg2_when_every_activation_is_nonlinear(seed):
    """With no identity in the original network every end indicator is forced to 1, B = A, and the
    extended problem is Eq. 5 with I[i][j] = I[i][j][1][1]."""
    rng = random.Random(500 + seed)
    L = rng.randint(3, 8)
    T, I, _ = I_.random_dp_tables_ext(rng, L, P.INF)
    sig = [False] * (L + 1)
    I2 = [[I[i][j][1][1] if j > i else 0.0 for j in range(L + 1)] for i in range(L + 1)]
    T_opt, _ = P.alg1(T, L)
    for T0 in (T_opt[0][L] + 1, T_opt[0][L] + 5, sum(T[i][i + 1] for i in range(L)) + 1):
        A, S, B, d0, dL, obj, ok = P.alg4(T0, L, T, I, sig)
        A2, S2, obj2, ok2 = P.alg2(T0, L, T, I2)
        assert ok == ok2
        if ok:
            assert obj == pytest.approx(obj2, abs=1e-12) and A == A2 and S == S2 and B == A and (d0, dL) == (1, 1)


def test_alg4_budget_properties_and_normalisation():
    rng = random.Random(11)
    L = 6
    T, I, sig = I_.random_dp_tables_ext(rng, L, P.INF, unmergeable=0.0)
    T_opt, _ = P.alg1(T, L)
    assert not P.alg4(T_opt[0][L], L, T, I, sig)[6]          # strict budget
    prev = -math.inf
    for T0 in range(T_opt[0][L] + 1, sum(T[i][i + 1] for i in range(L)) + 3):
        obj, ok = P.alg4(T0, L, T, I, sig)[5:7]
        if ok:
            assert obj >= prev - 1e-12
            prev = obj
    # App. B.3: every block moves by alpha times the mean accuracy change of the size-one blocks
    deltas = [-0.5, -1.5, -1.0]
    N = P.normalize_importance(I, L, deltas, alpha=2.0)
    assert N[1][4][1][0] == pytest.approx(I[1][4][1][0] + 2.0) and N[0][1][0][0] == pytest.approx(I[0][1][0][0] + 2.0)
    # a uniform shift s per block changes a pattern of n blocks by n * s: with a large positive shift
    # the optimum uses as many blocks as the exclusions allow, never fewer than before
    nb = lambda r: len(r[2]) + 1
    T0 = sum(T[i][i + 1] for i in range(L)) + 1
    assert nb(P.alg4(T0, L, T, P.normalize_importance(I, L, [-50.0], 1.0), sig)) >= nb(P.alg4(T0, L, T, I, sig))
