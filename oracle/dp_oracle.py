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

  alg3  -- Algorithm 3 (App. B): I_opt[k][l][a][b], the best summed importance of a chain of blocks
           from boundary k to boundary l whose end indicators are d_k = a, d_l = b and whose inner
           boundaries all carry an identity (d = 0), with the exclusions of App. B.2 applied first.
  alg4  -- Algorithm 4 (App. B): the extended surrogate problem (Eq. "opt-ext"): D[l][t][a].
  normalize_importance -- App. B.3: I <- I - alpha * mean(D).

Readings of the two garbled listings (App. B): in Algorithm 3 the update uses the maximiser m (the
listing prints m'), its m' = k term is the single block I[k][l][a][b] (as printed,
I_opt[k][k][a][0] + I[k][l][0][b] would drop d_k = a), and B_opt carries the indices (a, b) like
I_opt, since the maximiser depends on them; in Algorithm 4 S and B carry the index a like A, the
last line takes a_last = argmax_a D[L][T0][a] (the listing prints A), and the indicators of the
two ends of the network (d_0, d_L) are returned with the sets.

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


def apply_exclusions(I, L, sigma_id):
    """Copy of I[i][j][a][b] with the blocks that App. B excludes set to -inf.  sigma_id[p] says
    whether the activation at boundary p of the original network is an identity (p = 0..L)."""
    ninf = -math.inf
    J = [[[[I[i][j][a][b] if j > i else 0.0 for b in range(2)] for a in range(2)] for j in range(L + 1)]
         for i in range(L + 1)]
    for k in range(L + 1):
        for l in range(k + 1, L + 1):
            for x in range(2):
                if not sigma_id[k]:
                    J[k][l][0][x] = ninf          # a non-linear activation stays: d_k = 1
                if not sigma_id[l]:
                    J[k][l][x][0] = ninf          # likewise d_l = 1
                if sigma_id[k] and sigma_id[l]:
                    J[k][l][x][0] = ninf          # identities on both edges, d_l = 0 (App. B.2)
    return J


def alg3(I, L, sigma_id):
    """Algorithm 3.  Returns (I_opt, B_opt): I_opt[k][l][a][b]; B_opt[k][l][a][b] a sorted list."""
    J = apply_exclusions(I, L, sigma_id)
    I_opt = [[[[0.0, 0.0], [0.0, 0.0]] for _ in range(L + 1)] for _ in range(L + 1)]
    B_opt = [[[[[], []], [[], []]] for _ in range(L + 1)] for _ in range(L + 1)]
    for l in range(1, L + 1):
        for k in range(0, l):
            for a, b in ((0, 0), (0, 1), (1, 0), (1, 1)):
                best_m, best = k, J[k][l][a][b]
                for m in range(k + 1, l):
                    cand = I_opt[k][m][a][0] + J[m][l][0][b]
                    if cand > best:
                        best_m, best = m, cand
                I_opt[k][l][a][b] = best
                B_opt[k][l][a][b] = [] if best_m == k else B_opt[k][best_m][a][0] + [best_m]
    return I_opt, B_opt


def alg4(T0, L, T, I, sigma_id):
    """Algorithm 4.  Returns (A, S, B, d0, dL, objective, feasible)."""
    T_opt, S_opt = alg1(T, L)
    I_opt, B_opt = alg3(I, L, sigma_id)
    ninf = -math.inf
    D = [[[0.0, 0.0] for _ in range(T0 + 1)] for _ in range(L + 1)]
    done = [[[False, False] for _ in range(T0 + 1)] for _ in range(L + 1)]
    sets = [[[None, None] for _ in range(T0 + 1)] for _ in range(L + 1)]      # (A, S, B, d0)
    for l in range(1, L + 1):
        if T_opt[0][l] >= INF:
            continue
        for t in range(T_opt[0][l] + 1, T0 + 1):
            for a in range(2):
                best, arg = None, None
                for k in range(0, l):
                    if not _add(T_opt[0][k], T_opt[k][l]) < t:
                        continue
                    tk = t - T_opt[k][l]
                    for al in range(2):
                        if k > 0 and not done[k][tk][al]:
                            continue
                        val = (D[k][tk][al] if k > 0 else 0.0) + I_opt[k][l][al][a]
                        if best is None or val > best:
                            best, arg = val, (k, al)
                if arg is None:
                    continue
                k, al = arg
                tk = t - T_opt[k][l]
                pA, pS, pB, pd0 = sets[k][tk][al] if k > 0 else ([], [], [], al)
                D[l][t][a] = best
                done[l][t][a] = True
                sets[l][t][a] = (pA + ([k] if k > 0 and al == 1 else []),
                                 sorted(set(pS + ([k] if k > 0 else []) + S_opt[k][l])),
                                 sorted(set(pB + ([k] if k > 0 else []) + B_opt[k][l][al][a])),
                                 pd0)
    if T0 < 0 or not (done[L][T0][0] or done[L][T0][1]):
        return [], [], [], 0, 0, 0.0, False
    cands = [a for a in range(2) if done[L][T0][a]]
    a_last = max(cands, key=lambda a: (D[L][T0][a], -a))
    obj = D[L][T0][a_last]
    if obj == ninf:
        return [], [], [], 0, 0, obj, False
    A, S, B, d0 = sets[L][T0][a_last]
    return A, S, B, d0, a_last, obj, True


def normalize_importance(I, L, deltas, alpha):
    """App. B.3: subtract alpha times the mean of the size-one accuracy changes from every block."""
    shift = alpha * sum(deltas) / len(deltas)
    return [[[[I[i][j][a][b] - shift if j > i else 0.0 for b in range(2)] for a in range(2)]
             for j in range(L + 1)] for i in range(L + 1)]


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


def brute_select_ext(T0, L, T, I, sigma_id):
    """The extended problem by enumeration: max over A subset B subset [L-1], S superset of A, and
    the end indicators d_0, d_L, of sum over the blocks of B of I[b', b, d_b', d_b] (d = 1 on A,
    0 on B minus A; excluded blocks count -inf), subject to the pieces of S summing to < T0.
    Returns the best objective or None."""
    J = apply_exclusions(I, L, sigma_id)
    inner = list(range(1, L))
    # cheapest pattern that keeps every boundary of A
    best = None
    for r in range(len(inner) + 1):
        for Bset in itertools.combinations(inner, r):
            for mask in range(1 << len(Bset)):
                Aset = [b for i, b in enumerate(Bset) if (mask >> i) & 1]
                free = [p for p in inner if p not in Aset]
                lat = INF
                for q in range(len(free) + 1):
                    for extra in itertools.combinations(free, q):
                        lat = min(lat, pieces_latency(T, [0] + sorted(Aset + list(extra)) + [L]))
                if not lat < T0:
                    continue
                for d0 in range(2):
                    for dL in range(2):
                        d = {0: d0, L: dL}
                        for b in Bset:
                            d[b] = 1 if b in Aset else 0
                        bs = [0] + list(Bset) + [L]
                        val = sum(J[x][y][d[x]][d[y]] for x, y in zip(bs[:-1], bs[1:]))
                        if val == -math.inf:
                            continue
                        if best is None or val > best:
                            best = val
    return best
