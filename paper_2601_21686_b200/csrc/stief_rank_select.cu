// stief_select_ranks: the sequential budgeted rank selector (Algorithm 2; Eq. 15-17 with the cost of Eq. 23).
// Host code only: L is a few dozen and the candidate grid a few dozen pairs, so the work is the caller's surface
// evaluation, not this loop.  What matters here is that the feasibility test is EXACT: a pair whose cost equals the
// per-layer budget must be accepted on every machine, so budgets are kept as integers.
//
// rho is a double, i.e. m / 2^k with integers m < 2^53 and k.  In units of 1 / (2 d_h 2^k) the remaining budget is
//   W_l = L * 2 d_h * m  -  2^k * (sum of r_K + r_V chosen so far)
// and the constraint c <= tau_l = B_l / (L - l) reads  (r_K + r_V) * (L - l) * 2^k <= W_l : integers below 2^100.
#include <cmath>
#include <cstdint>
#include <vector>

#include "stief.h"

namespace {
using wide = __int128;
constexpr int kMaxLayers = 4096;
constexpr int kMaxCandidates = 64;
}  // namespace

extern "C" int stief_select_ranks(int32_t L, int32_t d_h, const int32_t* cand_k, int32_t n_k, const int32_t* cand_v,
                                  int32_t n_v, double rho, const double* surfaces, stief_surface_fn surface, void* ctx,
                                  int32_t* r_k, int32_t* r_v, double* spent, int32_t* failed_layer) {
  if (failed_layer) *failed_layer = -1;
  if (L <= 0 || L > kMaxLayers || d_h <= 0 || d_h > 1024 || !cand_k || !cand_v || n_k <= 0 || n_v <= 0 ||
      n_k > kMaxCandidates || n_v > kMaxCandidates || !r_k || !r_v)
    return STIEF_ERR_INVALID_ARG;
  if ((surfaces == nullptr) == (surface == nullptr)) return STIEF_ERR_INVALID_ARG;   // exactly one source of tables
  if (!(rho >= 1.0 / 1024.0) || !(rho <= 1.0)) return STIEF_ERR_INVALID_ARG;        // also rejects NaN
  for (int i = 0; i < n_k; ++i) if (cand_k[i] <= 0 || cand_k[i] > d_h) return STIEF_ERR_INVALID_ARG;
  for (int j = 0; j < n_v; ++j) if (cand_v[j] <= 0 || cand_v[j] > d_h) return STIEF_ERR_INVALID_ARG;

  int e = 0;
  const double f = std::frexp(rho, &e);                       // rho = f 2^e, f in [0.5, 1), e in [-9, 1]
  const wide m = (wide)std::ldexp(f, 53);                     // exact: f has at most 53 significant bits
  const int k = 53 - e;                                       // rho = m / 2^k, 52 <= k <= 62
  const wide unit = (wide)1 << k;
  wide left = (wide)L * (2 * d_h) * m;                        // B_1 = L rho

  std::vector<double> table;
  if (surface) table.resize((size_t)n_k * n_v);
  int64_t rank_sum = 0;
  for (int l = 0; l < L; ++l) {
    const double* delta = surfaces ? surfaces + (size_t)l * n_k * n_v : table.data();
    if (surface && surface(ctx, l, r_k, r_v, table.data()) != 0) {
      if (failed_layer) *failed_layer = l;
      return STIEF_ERR_INVALID_ARG;
    }
    const wide layers_left = L - l;
    int bi = -1, bj = -1;
    for (int i = 0; i < n_k; ++i)
      for (int j = 0; j < n_v; ++j) {
        const double d = delta[(size_t)i * n_v + j];
        if (d != d) { if (failed_layer) *failed_layer = l; return STIEF_ERR_INVALID_ARG; }   // NaN in a table
        const int s = cand_k[i] + cand_v[j];
        if ((wide)s * layers_left * unit > left) continue;   // c(r_K, r_V) > tau_l
        bool take = bi < 0;
        if (!take) {
          const double bd = delta[(size_t)bi * n_v + bj];
          const int bs = cand_k[bi] + cand_v[bj];
          take = d < bd || (d == bd && (s < bs || (s == bs && cand_k[i] < cand_k[bi])));
        }
        if (take) { bi = i; bj = j; }
      }
    if (bi < 0) {
      if (failed_layer) *failed_layer = l;
      return STIEF_ERR_INFEASIBLE;
    }
    r_k[l] = cand_k[bi];
    r_v[l] = cand_v[bj];
    left -= (wide)(r_k[l] + r_v[l]) * unit;                   // Eq. 17
    rank_sum += r_k[l] + r_v[l];
  }
  if (spent) *spent = (double)rank_sum / (2.0 * d_h);
  return STIEF_OK;
}
