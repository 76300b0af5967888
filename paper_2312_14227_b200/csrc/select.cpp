// Host-side tensor selector: the dynamic program of Section 6 of the paper, on integer
// (quantised) times.  Tensors are counted from the OUTPUT side inside this file, as the
// paper's P[k, t] does; the public arrays are in forward order.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <limits>
#include <thread>
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
//
// Section 6.3's two prunings, in this form of the table:
//   invalid    subproblems are those with t beyond the budget: the table is only budget + 1 wide;
//   redundant  ones are (k, t) with t below the cheapest selection that has k as its deepest tensor,
//              low(k) = t_dw(k) + the error-gradient times above k: their value is "impossible".  Rows
//              whose low(k) exceeds the budget are dead as a whole, and a transition from kc is only
//              tried for t >= dt + low(kc).
// prune = 0 evaluates the full table instead (every k, every t up to `t_full`, every transition), as
// the reference the pruned run is tested against.
// threads > 1 (at most the host's hardware threads are used): the predecessors of each row are dealt
// out to the threads, whose partial maxima are then merged; rows are taken in order.
et_status et_select_dp_int_ex(const double* importance, const int64_t* t_dw, const int64_t* t_dy, int32_t n,
                              int64_t budget, int32_t variant, int32_t threads, int32_t prune, uint8_t* mask_out,
                              double* value_out, et_dp_stats* stats) {
  if (importance == nullptr || t_dw == nullptr || t_dy == nullptr || mask_out == nullptr || n < 0)
    return ET_ERR_INVALID_ARG;
  if (variant != ET_COST_STRICT && variant != ET_COST_INCLUSIVE) return ET_ERR_INVALID_ARG;
  if (threads < 1 || threads > 256) return ET_ERR_INVALID_ARG;
  int64_t t_full = 0;
  for (int i = 0; i < n; ++i) {
    if (t_dw[i] < 0 || t_dy[i] < 0 || !std::isfinite(importance[i])) return ET_ERR_INVALID_ARG;
    mask_out[i] = 0;
    t_full += t_dw[i] + t_dy[i];
  }
  if (value_out != nullptr) *value_out = 0.0;
  if (stats != nullptr) {
    *stats = et_dp_stats{};
    stats->table_full = (int64_t)n * (t_full + 1);
    stats->table_budget = budget >= 0 ? (int64_t)n * (std::min(budget, t_full) + 1) : 0;
    stats->threads = threads;
  }
  if (n == 0 || budget < 0) return ET_OK;
  // width of the table: the budget when pruning, the full backward time otherwise
  const int64_t B = prune ? std::min(budget, t_full) : std::max(budget, t_full);
  if ((double)n * (double)(B + 1) > 4e8) return ET_ERR_UNSUPPORTED;
  const int64_t ask = std::min(budget, B);                // where the answer is read
  const bool incl = variant == ET_COST_INCLUSIVE;

  // output-side order
  std::vector<double> I(n);
  std::vector<int64_t> w(n), y(n), ypre(n + 1, 0), low(n);   // ypre[k] = sum_{j<k} y[j]
  for (int k = 0; k < n; ++k) {
    I[k] = importance[n - 1 - k];
    w[k] = t_dw[n - 1 - k];
    y[k] = t_dy[n - 1 - k];
    ypre[k + 1] = ypre[k] + y[k];
    low[k] = w[k] + ypre[k] + (incl ? y[k] : 0);
  }
  const size_t row = (size_t)B + 1;
  std::vector<double> Q((size_t)n * row, kNegInf);
  std::vector<int32_t> from((size_t)n * row, -2);        // -1: k alone; kc >= 0: extends Q[kc]
  auto step = [&](int k, int kc) {                       // time added by selecting k below kc
    return w[k] + (incl ? ypre[k + 1] - ypre[kc + 1] : ypre[k] - ypre[kc]);
  };
  // Row k restricted to the predecessors kc = first, first + stride, ...: the best candidate per t goes
  // to (val, arg), which start as "k alone" (first == 0) or "impossible".
  auto scan = [&](int k, int first, int stride, double* val, int32_t* arg) {
    for (int64_t t = 0; t <= B; ++t) {
      const bool alone = first == 0 && t >= low[k];
      val[t] = alone ? I[k] : kNegInf;
      arg[t] = alone ? -1 : -2;
    }
    for (int kc = first; kc < k; kc += stride) {
      if (prune && low[kc] > B) continue;
      const int64_t dt = step(k, kc);
      const double* Qc = &Q[(size_t)kc * row];
      for (int64_t t = dt + (prune ? low[kc] : 0); t <= B; ++t) {
        const double cand = I[k] + Qc[t - dt];
        if (cand > val[t]) { val[t] = cand; arg[t] = kc; }
      }
    }
  };
  std::vector<int> rows;                                 // rows that are evaluated, in order
  for (int k = 0; k < n; ++k)
    if (!prune || low[k] <= B) rows.push_back(k);
  int64_t visited = 0, transitions = 0;
  for (int k : rows) {
    visited += prune ? B + 1 - low[k] : B + 1;
    for (int kc = 0; kc < k; ++kc) {
      if (prune && low[kc] > B) continue;
      const int64_t from_t = step(k, kc) + (prune ? low[kc] : 0);
      if (from_t <= B) transitions += B + 1 - from_t;
    }
  }
  if (stats != nullptr) {
    stats->rows_reached = (int32_t)rows.size();
    stats->visited = visited;
    stats->transitions = transitions;
  }
  // two barriers per row cost a few microseconds: threads pay only when a row holds far more work
  const int hw = (int)std::max(1u, std::thread::hardware_concurrency());
  const bool worth = !rows.empty() && transitions / (int64_t)rows.size() > 200000;
  const int nthreads = worth ? std::min(threads, hw) : 1;
  if (nthreads <= 1) {
    for (int k : rows) scan(k, 0, 1, &Q[(size_t)k * row], &from[(size_t)k * row]);
  } else {
    // Persistent workers.  Per row, thread i scans the predecessors kc = i, i + nthreads, ... into its own
    // buffer (the work of a row is (number of predecessors) x (width), so this divides all of it), then
    // the threads merge the buffers, each over its share of t; on equal values the smaller kc wins, as
    // in the one-thread scan.  A counting barrier with a generation number separates the phases.
    std::vector<double> pval((size_t)nthreads * row);
    std::vector<int32_t> parg((size_t)nthreads * row);
    std::atomic<int> arrived{0};
    std::atomic<int> generation{0};
    auto barrier = [&]() {
      const int gen = generation.load(std::memory_order_acquire);
      if (arrived.fetch_add(1, std::memory_order_acq_rel) + 1 == nthreads) {
        arrived.store(0, std::memory_order_relaxed);
        generation.fetch_add(1, std::memory_order_release);
      } else {
        int spins = 0;
        while (generation.load(std::memory_order_acquire) == gen)
          if (++spins > 256) std::this_thread::yield();
      }
    };
    auto work = [&](int tid) {
      const int64_t chunk = (B + 1 + nthreads - 1) / nthreads;
      const int64_t lo = std::min<int64_t>(B + 1, tid * chunk), hi = std::min<int64_t>(B + 1, lo + chunk);
      for (int k : rows) {
        scan(k, tid, nthreads, &pval[(size_t)tid * row], &parg[(size_t)tid * row]);
        barrier();
        double* Qk = &Q[(size_t)k * row];
        int32_t* Fk = &from[(size_t)k * row];
        for (int64_t t = lo; t < hi; ++t) {
          double v = pval[t];
          int32_t a = parg[t];
          for (int i = 1; i < nthreads; ++i) {
            const double vi = pval[(size_t)i * row + t];
            const int32_t ai = parg[(size_t)i * row + t];
            if (vi > v || (vi == v && ai >= 0 && (a < -1 || (a >= 0 && ai < a)))) { v = vi; a = ai; }
          }
          Qk[t] = v;
          Fk[t] = a;
        }
        barrier();
      }
    };
    std::vector<std::thread> pool;
    for (int tid = 1; tid < nthreads; ++tid) pool.emplace_back(work, tid);
    work(0);
    for (auto& th : pool) th.join();
  }
  if (stats != nullptr) stats->threads = nthreads;
  double best = 0.0;                                     // P[-1][.] = 0: nothing selected
  int best_k = -1;
  for (int k : rows) {
    const double v = Q[(size_t)k * row + ask];
    if (v > best) { best = v; best_k = k; }              // Case 2 beats Case 1 only if strictly better
  }
  // back-trace
  int k = best_k;
  int64_t t = ask;
  while (k >= 0) {
    mask_out[n - 1 - k] = 1;
    const int32_t kc = from[(size_t)k * row + t];
    if (kc < 0) break;
    t -= step(k, kc);
    k = kc;
  }
  if (value_out != nullptr) *value_out = best;
  return ET_OK;
}

et_status et_select_dp_int(const double* importance, const int64_t* t_dw, const int64_t* t_dy, int32_t n,
                           int64_t budget, int32_t variant, uint8_t* mask_out, double* value_out) {
  return et_select_dp_int_ex(importance, t_dw, t_dy, n, budget, variant, 1, 1, mask_out, value_out, nullptr);
}

et_status et_select_dp_ex(const double* importance, const double* t_dw, const double* t_dy, int32_t n, double t_fwd,
                          double rho, int32_t Tq, int32_t variant, int32_t threads, int32_t prune, uint8_t* mask_out,
                          double* value_out, double* est_time_out, et_dp_stats* stats) {
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
  et_status st = et_select_dp_int_ex(importance, qw.data(), qy.data(), n, budget, variant, threads, prune, mask_out,
                                     value_out, stats);
  if (st != ET_OK) return st;
  if (est_time_out != nullptr) *est_time_out = time_of(mask_out, t_dw, t_dy, n, variant);
  return ET_OK;
}

et_status et_select_dp(const double* importance, const double* t_dw, const double* t_dy, int32_t n, double t_fwd,
                       double rho, int32_t Tq, int32_t variant, uint8_t* mask_out, double* value_out,
                       double* est_time_out) {
  return et_select_dp_ex(importance, t_dw, t_dy, n, t_fwd, rho, Tq, variant, 1, 1, mask_out, value_out, est_time_out,
                         nullptr);
}

}  // extern "C"
