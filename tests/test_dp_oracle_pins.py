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
