"""Test infrastructure: plain CPU statement of the paper's two dynamic programmes.

Only tests, the smoke check and the CPU-baseline leg of the benchmark may import this module; the
library's own implementation (csrc/dp.cu) shares no code with it.

Notation (Sec. 4): layers 1..L, boundaries 0..L.  T[i][j] (i < j) is the latency of the single
convolution that layers i+1..j merge into, an integer (Sec. 4.3 needs integer budgets); INF marks a
span that cannot be merged.  I[i][j] is the importance of replacing the activations strictly inside
(i, j) by identities; -inf excludes a block.

  alg1  -- Algorithm 1: T_opt[k][l] = min over S of the summed latency of the pieces of (k, l],
           S_opt[k][l] the minimising boundaries (Eq. 6a, 6b); base case T_opt[k][k] = 0.
  alg2  -- Algorithm 2: D[l][t], A[l][t], S[l][t] for integer budgets t <= T0 with the strict
           constraint "total latency < t" (Eq. 5, Eq. 7, Eq. 8).

Readings where the listings leave a choice: argmin / argmax take the first index that attains the
optimum; a candidate whose sub-problem would have budget t - T_opt[k'][l] below 0 cannot satisfy
the constraint and is skipped by it; sums with INF stay INF.
"""
from __future__ import annotations

import itertools
import math

INF = 1 << 60


def _add(a, b):
    return INF if a >= INF or b >= INF else a + b


def alg1(T, L):
    """Algorithm 1.  Returns (T_opt, S_opt): (L+1) x (L+1) lists; S_opt[k][l] is a sorted list."""
    T_opt = [[0] * (L + 1) for _ in range(L + 1)]
    S_opt = [[[] for _ in range(L + 1)] for _ in range(L + 1)]
    for l in range(1, L + 1):
        for k in range(0, l):
            best_m, best = None, None
            for m in range(k, l):
                cand = _add(T_opt[k][m], T[m][l])
                if best is None or cand < best:
                    best_m, best = m, cand
            T_opt[k][l] = best
            if best_m != k:
                S_opt[k][l] = S_opt[k][best_m] + [best_m]
            else:
                S_opt[k][l] = []
    return T_opt, S_opt


def alg2(T0, L, T, I):
    """Algorithm 2.  Returns (A, S, D[L][T0], feasible).  A, S sorted lists of boundaries."""
    T_opt, S_opt = alg1(T, L)
    D = [[0.0] * (T0 + 1) for _ in range(L + 1)]
    A = [[[] for _ in range(T0 + 1)] for _ in range(L + 1)]
    S = [[[] for _ in range(T0 + 1)] for _ in range(L + 1)]
    done = [[False] * (T0 + 1) for _ in range(L + 1)]
    for t in range(T0 + 1):
        done[0][t] = True
    for l in range(1, L + 1):
        if T_opt[0][l] >= INF:
            continue
        for t in range(T_opt[0][l] + 1, T0 + 1):
            best_k, best = None, None
            for k in range(0, l):
                if not _add(T_opt[0][k], T_opt[k][l]) < t:
                    continue
                val = D[k][t - T_opt[k][l]] + I[k][l]
                if best is None or val > best:
                    best_k, best = k, val
            if best_k is None:
                continue
            k = best_k
            t_last = T_opt[k][l]
            D[l][t] = D[k][t - t_last] + I[k][l]
            A[l][t] = A[k][t - t_last] + ([k] if k > 0 else [])
            S[l][t] = sorted(set(S[k][t - t_last] + ([k] if k > 0 else []) + S_opt[k][l]))
            done[l][t] = True
    ok = T0 >= 0 and done[L][T0]
    return A[L][T0], S[L][T0], D[L][T0], ok


# ---- the definitions, by enumeration (pins for the two recurrences) --------------------------------
def pieces_latency(T, bounds):
    tot = 0
    for a, b in zip(bounds[:-1], bounds[1:]):
        tot = _add(tot, T[a][b])
    return tot


def brute_topt(T, k, l):
    """min over S subset of {k+1..l-1} of the summed latency (Eq. 6a), by enumeration."""
    if k == l:
        return 0
    inner = list(range(k + 1, l))
    best = INF
    for r in range(len(inner) + 1):
        for Sset in itertools.combinations(inner, r):
            best = min(best, pieces_latency(T, [k] + list(Sset) + [l]))
    return best


def brute_select(T0, L, T, I):
    """max over A subset S subset [L-1] of sum I over the pieces of A, subject to the summed latency
    of the pieces of S being < T0 (Eq. 5), by enumeration.  Returns the best objective or None."""
    inner = list(range(1, L))
    best = None
    for r in range(len(inner) + 1):
        for Sset in itertools.combinations(inner, r):
            if not pieces_latency(T, [0] + list(Sset) + [L]) < T0:
                continue
            for q in range(len(Sset) + 1):
                for Aset in itertools.combinations(Sset, q):
                    b = [0] + list(Aset) + [L]
                    val = sum(I[a][c] for a, c in zip(b[:-1], b[1:]))
                    if val == -math.inf:
                        continue
                    if best is None or val > best:
                        best = val
    return best
