// Host-side tensor selector: the dynamic program of Section 6 of the paper, on integer
// (quantised) times.  Tensors are counted from the OUTPUT side inside this file, as the
// paper's P[k, t] does; the public arrays are in forward order.
#include <cmath>
#include <cstdint>
#include <limits>
#include <vector>

#include "et.h"

namespace {

const double kNegInf = -std::numeric_limits<double>::infinity();

// Backward time of a mask in forward order (Section 2.2 / Eq. 3).
template <typename C>
double time_of(const uint8_t* mask, const C* t_dw, const C* t_dy, int n, int variant) {
  int deepest = -1;
  for (int t = 0; t < n; ++t)
    if (mask[t]) { deepest = t; break; }
  if (deepest < 0) return 0.0;
  double total = 0.0;
  for (int t = deepest; t < n; ++t) {
    if (mask[t]) total += (double)t_dw[t];
    if (t > deepest || variant == ET_COST_INCLUSIVE) total += (double)t_dy[t];
  }
  return total;
}

}  // namespace

extern "C" {

et_status et_time_selective(const uint8_t* mask, const double* t_dw, const double* t_dy, int32_t n,
                            int32_t variant, double* t_out) {
  if (mask == nullptr || t_dw == nullptr || t_dy == nullptr || t_out == nullptr || n < 0) return ET_ERR_INVALID_ARG;
  if (variant != ET_COST_STRICT && variant != ET_COST_INCLUSIVE) return ET_ERR_INVALID_ARG;
  *t_out = time_of(mask, t_dw, t_dy, n, variant);
  return ET_OK;
}

// Q[k][t]: best importance of a selection in which tensor k (counted from the output, 0 =
// last) is selected and is the deepest selected one, with backward time <= t.  Selecting k on
// top of a solution whose deepest tensor is kc < k adds t_dw(k) plus the error-gradient
// times between them (Eq. 7); k alone pays every error-gradient time above it.
// P[k][t] = max(P[k-1][t], Q[k][t]) is the paper's subproblem (Case 1 / Case 2); the answer
// is P[n-1][budget], with the empty selection (value 0) as the floor.
et_status et_select_dp_int(const double* importance, const int64_t* t_dw, const int64_t* t_dy, int32_t n,
                           int64_t budget, int32_t variant, uint8_t* mask_out, double* value_out) {
  if (importance == nullptr || t_dw == nullptr || t_dy == nullptr || mask_out == nullptr || n < 0)
    return ET_ERR_INVALID_ARG;
  if (variant != ET_COST_STRICT && variant != ET_COST_INCLUSIVE) return ET_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    if (t_dw[i] < 0 || t_dy[i] < 0 || !std::isfinite(importance[i])) return ET_ERR_INVALID_ARG;
    mask_out[i] = 0;
  }
  if (value_out != nullptr) *value_out = 0.0;
  if (n == 0 || budget < 0) return ET_OK;
  if ((double)n * (double)(budget + 1) > 4e8) return ET_ERR_UNSUPPORTED;
  const int64_t B = budget;
  const bool incl = variant == ET_COST_INCLUSIVE;

  // output-side order
  std::vector<double> I(n);
  std::vector<int64_t> w(n), y(n), ypre(n + 1, 0);      // ypre[k] = sum_{j<k} y[j]
  for (int k = 0; k < n; ++k) {
    I[k] = importance[n - 1 - k];
    w[k] = t_dw[n - 1 - k];
    y[k] = t_dy[n - 1 - k];
    ypre[k + 1] = ypre[k] + y[k];
  }
  const size_t row = (size_t)B + 1;
  std::vector<double> Q((size_t)n * row, kNegInf);
  std::vector<int32_t> from((size_t)n * row, -2);        // -1: k alone; kc >= 0: extends Q[kc]
  double best = 0.0;                                     // P[-1][.] = 0: nothing selected
  int best_k = -1;
  for (int k = 0; k < n; ++k) {
    double* Qk = &Q[(size_t)k * row];
    int32_t* Fk = &from[(size_t)k * row];
    const int64_t alone = w[k] + ypre[k] + (incl ? y[k] : 0);
    for (int64_t t = alone; t <= B; ++t) { Qk[t] = I[k]; Fk[t] = -1; }
    for (int kc = 0; kc < k; ++kc) {
      // strict: sum_{j=kc}^{k-1} y[j];  inclusive: sum_{j=kc+1}^{k} y[j]
      const int64_t dt = w[k] + (incl ? ypre[k + 1] - ypre[kc + 1] : ypre[k] - ypre[kc]);
      const double* Qc = &Q[(size_t)kc * row];
      for (int64_t t = dt; t <= B; ++t) {
        const double cand = I[k] + Qc[t - dt];
        if (cand > Qk[t]) { Qk[t] = cand; Fk[t] = kc; }
      }
    }
    if (Qk[B] > best) { best = Qk[B]; best_k = k; }       // Case 2 beats Case 1 only if strictly better
  }
  // back-trace
  int k = best_k;
  int64_t t = B;
  while (k >= 0) {
    mask_out[n - 1 - k] = 1;
    const int32_t kc = from[(size_t)k * row + t];
    if (kc < 0) break;
    t -= w[k] + (incl ? ypre[k + 1] - ypre[kc + 1] : ypre[k] - ypre[kc]);
    k = kc;
  }
  if (value_out != nullptr) *value_out = best;
  return ET_OK;
}

et_status et_select_dp(const double* importance, const double* t_dw, const double* t_dy, int32_t n, double t_fwd,
                       double rho, int32_t Tq, int32_t variant, uint8_t* mask_out, double* value_out,
                       double* est_time_out) {
  if (importance == nullptr || t_dw == nullptr || t_dy == nullptr || mask_out == nullptr || n < 0 || Tq < 1 ||
      !(rho >= 0.0) || !(t_fwd >= 0.0))
    return ET_ERR_INVALID_ARG;
  double T = 0.0;
  for (int i = 0; i < n; ++i) {
    if (!(t_dw[i] >= 0.0) || !(t_dy[i] >= 0.0)) return ET_ERR_INVALID_ARG;
    T += t_dw[i];
  }
  for (int i = 0; i < n; ++i) T += t_dy[i];
  std::vector<int64_t> qw(n), qy(n);
  int64_t budget;
  if (T > 0.0) {
    // Eq. 8: every time is scaled by Z = Tq / T and floored; so is the backward budget
    // rho * T_full - T_forward with T_full = T_forward + T.
    const double Z = (double)Tq / T;
    for (int i = 0; i < n; ++i) {
      qw[i] = (int64_t)std::floor(t_dw[i] * Z);
      qy[i] = (int64_t)std::floor(t_dy[i] * Z);
    }
    budget = (int64_t)std::floor((rho * (t_fwd + T) - t_fwd) * Z);
  } else {
    budget = (rho * t_fwd - t_fwd) >= 0.0 ? 0 : -1;
  }
  et_status st = et_select_dp_int(importance, qw.data(), qy.data(), n, budget, variant, mask_out, value_out);
  if (st != ET_OK) return st;
  if (est_time_out != nullptr) *est_time_out = time_of(mask_out, t_dw, t_dy, n, variant);
  return ET_OK;
}

}  // extern "C"
