// The selector's two dynamic programmes (Sec. 4.3): latency-optimal merge pattern of every span
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
