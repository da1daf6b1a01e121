// The selector's dynamic programmes: latency-optimal merge pattern of every span
// (Algorithm 1) and the budgeted choice of activations and merge boundaries (Algorithm 2).
// Serial host code: O(L^3) and O(L^2 T0) table updates for L of a few dozen layers; nothing here
// touches the device.
#include <cmath>
#include <limits>
#include <new>
#include <vector>

#include "common.cuh"

namespace {

inline long long sat_add(long long a, long long b) { return (a >= DC_DP_INF || b >= DC_DP_INF) ? DC_DP_INF : a + b; }

// T_opt and the last boundary of every optimal pattern, filled column by column: T_opt[k][l] needs
// T_opt[k][m] for m < l only.
dc_status optimal_latency(const long long *T, int L, long long *T_opt, int *split) {
  const int W = L + 1;
  for (int i = 0; i < W; ++i)
    for (int j = i + 1; j < W; ++j)
      if (T[i * W + j] < 0) return DC_ERR_INVALID_ARG;
  for (int k = 0; k < W; ++k)
    for (int l = 0; l < W; ++l) { T_opt[k * W + l] = 0; split[k * W + l] = k; }
  for (int l = 1; l <= L; ++l)
    for (int k = 0; k < l; ++k) {
      int arg = k;
      long long best = sat_add(T_opt[k * W + k], T[k * W + l]);
      for (int m = k + 1; m < l; ++m) {
        const long long cand = sat_add(T_opt[k * W + m], T[m * W + l]);
        if (cand < best) { best = cand; arg = m; }
      }
      T_opt[k * W + l] = best;
      split[k * W + l] = arg;
    }
  return DC_OK;
}

// Appends S_opt[k][l] in increasing order.
void pattern(const int *split, int W, int k, int l, std::vector<int> &out) {
  if (l <= k) return;
  const int m = split[k * W + l];
  if (m <= k) return;
  pattern(split, W, k, m, out);
  out.push_back(m);
}

}  // namespace

extern "C" dc_status dc_dp_optimal_latency(const long long *T, int L, long long *T_opt, int *split) {
  if (!T || !T_opt || !split || L <= 0) return DC_ERR_INVALID_ARG;
  return optimal_latency(T, L, T_opt, split);
}

extern "C" dc_status dc_dp_pattern(const int *split, int L, int k, int l, int *S, int *n_S) {
  if (!split || !S || !n_S || L <= 0 || k < 0 || l > L || k > l) return DC_ERR_INVALID_ARG;
  const int W = L + 1;
  for (int a = 0; a < W; ++a)
    for (int b = a + 1; b < W; ++b)
      if (split[a * W + b] < a || split[a * W + b] >= b) return DC_ERR_INVALID_ARG;
  std::vector<int> out;
  pattern(split, W, k, l, out);
  *n_S = (int)out.size();
  for (size_t i = 0; i < out.size(); ++i) S[i] = out[i];
  return DC_OK;
}

extern "C" dc_status dc_dp_select(const long long *T, const double *I, int L, long long T0, int *A, int *n_A,
                                  int *S, int *n_S, double *objective, int *feasible) {
  if (!T || !I || !A || !n_A || !S || !n_S || !objective || !feasible || L <= 0 || T0 < 0) return DC_ERR_INVALID_ARG;
  if (T0 >= (1ll << 31) / (L + 1)) return DC_ERR_WORKSPACE;
  const int W = L + 1;
  const long long B = T0 + 1;
  std::vector<long long> T_opt;
  std::vector<int> split, choice;
  std::vector<double> D;
  std::vector<unsigned char> done;
  try {
    T_opt.resize((size_t)W * W);
    split.resize((size_t)W * W);
    D.assign((size_t)W * B, 0.0);
    choice.assign((size_t)W * B, -1);
    done.assign((size_t)W * B, 0);
  } catch (const std::bad_alloc &) {
    return DC_ERR_WORKSPACE;
  }
  dc_status st = optimal_latency(T, L, T_opt.data(), split.data());
  if (st != DC_OK) return st;
  for (long long t = 0; t < B; ++t) done[t] = 1;       // l = 0: nothing kept, nothing spent
  for (int l = 1; l <= L; ++l) {
    const long long t_min = T_opt[l];                    // T_opt[0][l]
    if (t_min >= DC_DP_INF) continue;
    for (long long t = t_min + 1; t < B; ++t) {
      int arg = -1;
      double best = 0.0;
      for (int k = 0; k < l; ++k) {
        const long long t_kl = T_opt[(size_t)k * W + l];
        if (!(sat_add(T_opt[k], t_kl) < t)) continue;    // T_opt[0][k] + T_opt[k][l] < t
        const double val = D[(size_t)k * B + (t - t_kl)] + I[(size_t)k * W + l];
        if (arg < 0 || val > best) { arg = k; best = val; }
      }
      if (arg < 0) continue;
      D[(size_t)l * B + t] = best;
      choice[(size_t)l * B + t] = arg;
      done[(size_t)l * B + t] = 1;
    }
  }
  *n_A = 0;
  *n_S = 0;
  *objective = D[(size_t)L * B + T0];
  *feasible = done[(size_t)L * B + T0] && *objective > -std::numeric_limits<double>::infinity() ? 1 : 0;
  if (!*feasible) return DC_OK;
  // walk the choices back from (L, T0): each step closes the block (k, l] with its optimal pattern
  std::vector<int> a_rev;
  std::vector<int> s_all;
  int l = L;
  long long t = T0;
  while (l > 0) {
    const int k = choice[(size_t)l * B + t];
    if (k < 0) return DC_ERR_INVALID_ARG;                // cannot happen for a finished state
    std::vector<int> inner;
    pattern(split.data(), W, k, l, inner);
    for (size_t i = inner.size(); i-- > 0;) s_all.push_back(inner[i]);
    if (k > 0) { a_rev.push_back(k); s_all.push_back(k); }
    t -= T_opt[(size_t)k * W + l];
    l = k;
  }
  for (size_t i = a_rev.size(); i-- > 0;) A[(*n_A)++] = a_rev[i];
  for (size_t i = s_all.size(); i-- > 0;) S[(*n_S)++] = s_all[i];
  return DC_OK;
}

// ------------------------------------------------------------------ extended programmes (App. B)
namespace {

constexpr double kNegInf = -std::numeric_limits<double>::infinity();

inline size_t i4(int W, int i, int j, int a, int b) { return (((size_t)i * W + j) * 2 + a) * 2 + b; }

// Algorithm 3 on a copy J of the importances with the excluded blocks at -infinity.  split[k][l][a][b]
// = m is the last inner boundary of the best chain (m == k: the single block).
void optimal_importance(const double *I, const unsigned char *sigma_id, int L, std::vector<double> &J, double *I_opt,
                        int *split) {
  const int W = L + 1;
  J.assign((size_t)W * W * 4, 0.0);
  for (int k = 0; k < W; ++k)
    for (int l = k + 1; l < W; ++l)
      for (int a = 0; a < 2; ++a)
        for (int b = 0; b < 2; ++b) {
          double v = I[i4(W, k, l, a, b)];
          if (a == 0 && !sigma_id[k]) v = kNegInf;                 // a non-linear activation stays
          if (b == 0 && !sigma_id[l]) v = kNegInf;
          if (b == 0 && sigma_id[k] && sigma_id[l]) v = kNegInf;   // identities on both edges
          J[i4(W, k, l, a, b)] = v;
        }
  for (size_t i = 0; i < (size_t)W * W * 4; ++i) { I_opt[i] = 0.0; split[i] = 0; }
  for (int k = 0; k < W; ++k)
    for (int l = 0; l < W; ++l)
      for (int ab = 0; ab < 4; ++ab) split[i4(W, k, l, 0, 0) + ab] = k;
  for (int l = 1; l <= L; ++l)
    for (int k = 0; k < l; ++k)
      for (int a = 0; a < 2; ++a)
        for (int b = 0; b < 2; ++b) {
          int arg = k;
          double best = J[i4(W, k, l, a, b)];
          for (int m = k + 1; m < l; ++m) {
            const double cand = I_opt[i4(W, k, m, a, 0)] + J[i4(W, m, l, 0, b)];
            if (cand > best) { best = cand; arg = m; }
          }
          I_opt[i4(W, k, l, a, b)] = best;
          split[i4(W, k, l, a, b)] = arg;
        }
}

// Appends B_opt[k][l][a][b] in increasing order.
void chain(const int *split, int W, int k, int l, int a, int b, std::vector<int> &out) {
  if (l <= k) return;
  const int m = split[i4(W, k, l, a, b)];
  if (m <= k) return;
  chain(split, W, k, m, a, 0, out);
  out.push_back(m);
}

bool bad_flags(const unsigned char *sigma_id, int L) {
  for (int p = 0; p <= L; ++p)
    if (sigma_id[p] > 1) return true;
  return false;
}

}  // namespace

extern "C" dc_status dc_dp_optimal_importance(const double *I, const unsigned char *sigma_id, int L, double *I_opt,
                                              int *split) {
  if (!I || !sigma_id || !I_opt || !split || L <= 0 || bad_flags(sigma_id, L)) return DC_ERR_INVALID_ARG;
  std::vector<double> J;
  try {
    optimal_importance(I, sigma_id, L, J, I_opt, split);
  } catch (const std::bad_alloc &) {
    return DC_ERR_WORKSPACE;
  }
  return DC_OK;
}

extern "C" dc_status dc_dp_importance_pattern(const int *split, int L, int k, int l, int a, int b, int *B, int *n_B) {
  if (!split || !B || !n_B || L <= 0 || k < 0 || l > L || k > l || (a | b) < 0 || a > 1 || b > 1) return DC_ERR_INVALID_ARG;
  const int W = L + 1;
  for (int x = 0; x < W; ++x)
    for (int y = x + 1; y < W; ++y)
      for (int ab = 0; ab < 4; ++ab) {
        const int m = split[i4(W, x, y, 0, 0) + ab];
        if (m < x || m >= y) return DC_ERR_INVALID_ARG;
      }
  std::vector<int> out;
  chain(split, W, k, l, a, b, out);
  *n_B = (int)out.size();
  for (size_t i = 0; i < out.size(); ++i) B[i] = out[i];
  return DC_OK;
}

extern "C" dc_status dc_dp_normalize_importance(double *I, int L, const double *deltas, int n_deltas, double alpha) {
  if (!I || !deltas || L <= 0 || n_deltas <= 0) return DC_ERR_INVALID_ARG;
  double sum = 0.0;
  for (int i = 0; i < n_deltas; ++i) sum += deltas[i];
  const double shift = alpha * sum / n_deltas;
  const int W = L + 1;
  for (int i = 0; i < W; ++i)
    for (int j = i + 1; j < W; ++j)
      for (int ab = 0; ab < 4; ++ab) I[i4(W, i, j, 0, 0) + ab] -= shift;
  return DC_OK;
}

extern "C" dc_status dc_dp_select_ext(const long long *T, const double *I, const unsigned char *sigma_id, int L,
                                      long long T0, int *A, int *n_A, int *S, int *n_S, int *B, int *n_B, int *d_first,
                                      int *d_last, double *objective, int *feasible) {
  if (!T || !I || !sigma_id || !A || !n_A || !S || !n_S || !B || !n_B || !d_first || !d_last || !objective ||
      !feasible || L <= 0 || T0 < 0 || bad_flags(sigma_id, L))
    return DC_ERR_INVALID_ARG;
  if (T0 >= (1ll << 30) / (L + 1)) return DC_ERR_WORKSPACE;
  const int W = L + 1;
  const long long NB = T0 + 1;
  std::vector<long long> T_opt;
  std::vector<int> split, isplit, choice;
  std::vector<double> J, I_opt, D;
  try {
    T_opt.resize((size_t)W * W);
    split.resize((size_t)W * W);
    I_opt.resize((size_t)W * W * 4);
    isplit.resize((size_t)W * W * 4);
    D.assign((size_t)W * NB * 2, 0.0);
    choice.assign((size_t)W * NB * 2, -1);               // 2 * k + alpha of the state's last block, -1: not reached
    optimal_importance(I, sigma_id, L, J, I_opt.data(), isplit.data());
  } catch (const std::bad_alloc &) {
    return DC_ERR_WORKSPACE;
  }
  dc_status st = optimal_latency(T, L, T_opt.data(), split.data());
  if (st != DC_OK) return st;
  auto at = [&](int l, long long t, int a) { return ((size_t)l * NB + t) * 2 + a; };
  for (int l = 1; l <= L; ++l) {
    const long long t_min = T_opt[l];                    // T_opt[0][l]
    if (t_min >= DC_DP_INF) continue;
    for (long long t = t_min + 1; t < NB; ++t)
      for (int a = 0; a < 2; ++a) {
        int arg = -1;
        double best = 0.0;
        for (int k = 0; k < l; ++k) {
          const long long t_kl = T_opt[(size_t)k * W + l];
          if (!(sat_add(T_opt[k], t_kl) < t)) continue;  // T_opt[0][k] + T_opt[k][l] < t
          for (int al = 0; al < 2; ++al) {
            double prev = 0.0;                           // k = 0: nothing kept, nothing spent
            if (k > 0) {
              if (choice[at(k, t - t_kl, al)] < 0) continue;
              prev = D[at(k, t - t_kl, al)];
            }
            const double val = prev + I_opt[i4(W, k, l, al, a)];
            if (arg < 0 || val > best) { arg = 2 * k + al; best = val; }
          }
        }
        if (arg < 0) continue;
        D[at(l, t, a)] = best;
        choice[at(l, t, a)] = arg;
      }
  }
  *n_A = *n_S = *n_B = 0;
  *d_first = *d_last = 0;
  *objective = 0.0;
  *feasible = 0;
  int a_last = -1;
  for (int a = 0; a < 2; ++a)
    if (choice[at(L, T0, a)] >= 0 && (a_last < 0 || D[at(L, T0, a)] > D[at(L, T0, a_last)])) a_last = a;
  if (a_last < 0) return DC_OK;
  *objective = D[at(L, T0, a_last)];
  if (!(*objective > kNegInf)) return DC_OK;
  *feasible = 1;
  *d_last = a_last;
  // walk the choices back from (L, T0, a_last): each step closes the stretch (k, l] with its
  // latency-optimal pattern and its importance-optimal chain of blocks
  std::vector<int> a_rev, s_rev, b_rev, inner;
  int l = L, a = a_last;
  long long t = T0;
  while (l > 0) {
    const int c = choice[at(l, t, a)];
    if (c < 0) return DC_ERR_INVALID_ARG;                // cannot happen for a reached state
    const int k = c >> 1, al = c & 1;
    inner.clear();
    pattern(split.data(), W, k, l, inner);
    for (size_t i = inner.size(); i-- > 0;) s_rev.push_back(inner[i]);
    inner.clear();
    chain(isplit.data(), W, k, l, al, a, inner);
    for (size_t i = inner.size(); i-- > 0;) b_rev.push_back(inner[i]);
    if (k > 0) {
      s_rev.push_back(k);
      b_rev.push_back(k);
      if (al) a_rev.push_back(k);
    } else {
      *d_first = al;
    }
    t -= T_opt[(size_t)k * W + l];
    l = k;
    a = al;
  }
  for (size_t i = a_rev.size(); i-- > 0;) A[(*n_A)++] = a_rev[i];
  for (size_t i = s_rev.size(); i-- > 0;) S[(*n_S)++] = s_rev[i];
  for (size_t i = b_rev.size(); i-- > 0;) B[(*n_B)++] = b_rev[i];
  return DC_OK;
}
