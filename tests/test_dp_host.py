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


# ---- the extended programmes (App. B: Algorithm 3, Algorithm 4) -----------------------------------
@pytest.mark.parametrize("seed", range(8))
def test_optimal_importance_matches_oracle(dc, seed):
    rng = random.Random(600 + seed)
    L = rng.randint(1, 10)
    _, I, sig = I_.random_dp_tables_ext(rng, L, P.INF)
    i_opt, split = dc.dp_optimal_importance(I, sig, L)
    o_opt, o_b = P.alg3(I, L, sig)
    for k in range(L + 1):
        for l in range(k + 1, L + 1):
            for a in range(2):
                for b in range(2):
                    assert i_opt[k][l][a][b] == o_opt[k][l][a][b]        # the same sums in the same order
                    if o_opt[k][l][a][b] > -math.inf:
                        assert dc.dp_importance_pattern(split, L, k, l, a, b) == o_b[k][l][a][b]


@pytest.mark.parametrize("seed", range(10))
def test_select_ext_matches_oracle_and_enumeration(dc, seed):
    rng = random.Random(700 + seed)
    L = rng.randint(2, 7)
    T, I, sig = I_.random_dp_tables_ext(rng, L, P.INF, p_identity=0.3 + 0.1 * (seed % 4))
    J = P.apply_exclusions(I, L, sig)
    T_opt, _ = P.alg1(T, L)
    for T0 in sorted({0, T_opt[0][L], T_opt[0][L] + 1, T_opt[0][L] + 3, sum(T[i][i + 1] for i in range(L)) + 1}):
        got = dc.dp_select_ext(T, I, sig, L, T0)
        want = P.alg4(T0, L, T, I, sig)
        assert got[6] == want[6]
        if not want[6]:
            assert got[0] == [] and got[1] == [] and got[2] == []
            continue
        assert got[:5] == want[:5] and got[5] == pytest.approx(want[5], abs=1e-12)
        if L <= 6:
            assert got[5] == pytest.approx(P.brute_select_ext(T0, L, T, I, sig), abs=1e-12)
        A, S, B, d0, dL = got[:5]
        assert set(A) <= set(B) and set(A) <= set(S)
        assert P.pieces_latency(T, [0] + S + [L]) < T0
        d = {x: (1 if x in A else 0) for x in B}
        d[0], d[L] = d0, dL
        bs = [0] + B + [L]
        assert sum(J[x][y][d[x]][d[y]] for x, y in zip(bs[:-1], bs[1:])) == pytest.approx(got[5], abs=1e-12)


def test_select_ext_reduces_to_select_and_normalises(dc):
    rng = random.Random(800)
    L = 9
    T, I, _ = I_.random_dp_tables_ext(rng, L, P.INF)
    sig = [False] * (L + 1)                      # no identity anywhere: every indicator is forced to 1
    I2 = [[I[i][j][1][1] if j > i else 0.0 for j in range(L + 1)] for i in range(L + 1)]
    T_opt, _ = P.alg1(T, L)
    for T0 in (T_opt[0][L] + 1, T_opt[0][L] + 6, sum(T[i][i + 1] for i in range(L)) + 1):
        A, S, B, d0, dL, obj, ok = dc.dp_select_ext(T, I, sig, L, T0)
        A2, S2, obj2, ok2 = dc.dp_select(T, I2, L, T0)
        assert ok and ok2 and A == A2 and S == S2 and B == A and (d0, dL) == (1, 1)
        assert obj == pytest.approx(obj2, abs=1e-12)
    N = dc.dp_normalize_importance(I, L, [-0.5, -1.5, -1.0], 2.0)
    O = P.normalize_importance(I, L, [-0.5, -1.5, -1.0], 2.0)
    assert all(N[i][j][a][b] == pytest.approx(O[i][j][a][b], abs=1e-15)
               for i in range(L + 1) for j in range(i + 1, L + 1) for a in range(2) for b in range(2))


def test_select_ext_on_a_52_layer_table(dc):
    """MobileNetV2-sized problem (project outputs are identities in the original network)."""
    rng = random.Random(52)
    L = 52
    T, I, _ = I_.random_dp_tables_ext(rng, L, P.INF, unmergeable=0.0)
    for i in range(L + 1):
        for j in range(i + 1, L + 1):
            if j - i > 6:
                T[i][j] = P.INF
    sig = [True] + [(p % 3 == 0) for p in range(1, L)] + [False]
    T_opt, _ = P.alg1(T, L)
    T0 = T_opt[0][L] + (sum(T[i][i + 1] for i in range(L)) - T_opt[0][L]) // 2
    got = dc.dp_select_ext(T, I, sig, L, T0)
    want = P.alg4(T0, L, T, I, sig)
    assert got[6] and want[6] and got[:5] == want[:5] and got[5] == pytest.approx(want[5], abs=1e-9)


def test_extended_dp_argument_errors(dc):
    import ctypes as C
    L = 2
    T = [[0, 1, 2], [0, 0, 1], [0, 0, 0]]
    I = [[[[0.0, 0.0], [0.0, 0.0]] for _ in range(3)] for _ in range(3)]
    lib = dc.lib()
    bad = (C.c_ubyte * 3)(1, 2, 0)
    out = (C.c_double * 36)()
    sp = (C.c_int * 36)()
    assert lib.dc_dp_optimal_importance(dc._imp4(I, L), bad, L, out, sp) == dc.ERR_INVALID_ARG
    assert lib.dc_dp_optimal_importance(None, bad, L, out, sp) == dc.ERR_INVALID_ARG
    with pytest.raises(dc.DcError):
        dc.dp_select_ext(T, I, [True, True, False], L, -1)
