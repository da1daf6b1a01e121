"""The library's host implementation of Algorithm 1 and Algorithm 2 against the oracle and against
enumeration of the definitions (Eq. 5, Eq. 6a).  Host-only calls through the C ABI: no GPU needed."""
import math
import random

import pytest

from oracle import dp_oracle as P
from paper_2301_12187_b200 import inputs as I_


def random_tables(rng, L, unmergeable=0.2, neg_inf=0.0):
    return I_.random_dp_tables(rng, L, P.INF, unmergeable, neg_inf)


@pytest.fixture(scope="module")
def dc():
    from paper_2301_12187_b200 import dc as _dc
    _dc.lib()
    return _dc


@pytest.mark.parametrize("seed", range(8))
def test_optimal_latency_matches_oracle_and_enumeration(dc, seed):
    rng = random.Random(seed)
    L = rng.randint(1, 10)
    T, _ = random_tables(rng, L)
    t_opt, split = dc.dp_optimal_latency(T, L)
    o_opt, o_s = P.alg1(T, L)
    for k in range(L + 1):
        for l in range(k, L + 1):
            assert t_opt[k][l] == o_opt[k][l]
            assert dc.dp_pattern(split, L, k, l) == o_s[k][l]
            if L <= 8:
                assert t_opt[k][l] == P.brute_topt(T, k, l)


def test_optimal_latency_on_a_52_layer_table(dc):
    """MobileNetV2-sized problem: agreement with the oracle on every (k, l), unmergeable spans
    (a k > 1 layer after a stride-2 layer, spans longer than 6) marked infinite."""
    rng = random.Random(3)
    L = 52
    T, _ = random_tables(rng, L, unmergeable=0.3)
    for i in range(L + 1):
        for j in range(i + 7, L + 1):
            T[i][j] = P.INF
    t_opt, split = dc.dp_optimal_latency(T, L)
    o_opt, o_s = P.alg1(T, L)
    assert t_opt == o_opt
    assert dc.dp_pattern(split, L, 0, L) == o_s[0][L]
    assert dc.DP_INF == P.INF


@pytest.mark.parametrize("seed", range(8))
def test_select_matches_oracle_and_enumeration(dc, seed):
    rng = random.Random(200 + seed)
    L = rng.randint(1, 7)
    T, I = random_tables(rng, L, neg_inf=0.15 if seed % 2 else 0.0)
    o_opt, _ = P.alg1(T, L)
    budgets = {0, o_opt[0][L], o_opt[0][L] + 1, o_opt[0][L] + 3, sum(T[i][i + 1] for i in range(L)) + 1}
    for T0 in sorted(b for b in budgets if b < P.INF):
        A, S, obj, ok = dc.dp_select(T, I, L, T0)
        oA, oS, oD, ook = P.alg2(T0, L, T, I)
        want = P.brute_select(T0, L, T, I)
        assert ok == (ook and oD > -math.inf) == (want is not None)
        if not ok:
            assert A == [] and S == []
            continue
        assert obj == oD and A == oA and S == oS
        assert obj == pytest.approx(want, abs=1e-12)
        assert set(A) <= set(S) and P.pieces_latency(T, [0] + S + [L]) < T0


def test_select_rejects_bad_arguments(dc):
    T = [[0, 1], [0, 0]]
    I = [[0, 0.0], [0, 0]]
    with pytest.raises(RuntimeError):
        dc.dp_select(T, I, 0, 5)
    with pytest.raises(RuntimeError):
        dc.dp_select([[0, -1], [0, 0]], I, 1, 5)
    assert dc.dp_select(T, I, 1, 2) == ([], [], 0.0, True)
    assert dc.dp_select(T, I, 1, 1)[3] is False
