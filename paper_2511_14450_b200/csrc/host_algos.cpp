// Host-side algorithms of the paper: HypSplit-DP (Algorithm 1) and HypSched-RT (Algorithm 2).
// Pure C++, no GPU, thread-safe (no global state).
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <vector>

#include "hyperion.h"

namespace {

// Decision problem P_check(tau) of Section IV-A: boolean DP over (tier j, blocks 1..n) with the
// predecessor taken as the first feasible k while scanning upward.  Tables are (T+1) x (N+1).
struct CheckTables {
  int N, T;
  std::vector<uint8_t> dp;
  std::vector<int32_t> pred;
  CheckTables(int n, int t) : N(n), T(t), dp((size_t)(t + 1) * (n + 1)), pred((size_t)(t + 1) * (n + 1)) {}
  uint8_t& D(int j, int n) { return dp[(size_t)j * (N + 1) + n]; }
  int32_t& P(int j, int n) { return pred[(size_t)j * (N + 1) + n]; }
};

bool p_check(double tau, CheckTables& tb, const std::vector<double>& Sf, const std::vector<double>& Sm,
             const double* C, const double* Mcap) {
  const int N = tb.N, T = tb.T;
  std::fill(tb.dp.begin(), tb.dp.end(), 0);
  std::fill(tb.pred.begin(), tb.pred.end(), -1);
  tb.D(0, 0) = 1;
  for (int j = 1; j <= T; ++j) {
    for (int n = j; n <= N; ++n) {
      for (int k = j - 1; k < n; ++k) {
        if (!tb.D(j - 1, k)) continue;
        const double L = (Sf[n] - Sf[k]) / C[j - 1];
        const double U = Sm[n] - Sm[k];
        if (L <= tau && U <= Mcap[j - 1]) {
          tb.D(j, n) = 1;
          tb.P(j, n) = k;
          break;
        }
      }
    }
  }
  return tb.D(T, N) != 0;
}

void backtrack(CheckTables& tb, int32_t* p) {
  int n = tb.N;
  for (int j = tb.T; j >= 2; --j) {
    n = tb.P(j, n);
    p[j - 2] = n;
  }
}

double bottleneck(const int32_t* p, int N, int T, const std::vector<double>& Sf, const double* C) {
  double tau = 0.0;
  int prev = 0;
  for (int j = 0; j < T; ++j) {
    const int cut = (j == T - 1) ? N : p[j];
    const double L = (Sf[cut] - Sf[prev]) / C[j];
    if (L > tau) tau = L;
    prev = cut;
  }
  return tau;
}

}  // namespace

extern "C" int hyp_split_dp(int32_t N, int32_t T, const double* f, const double* m, const double* C,
                            const double* Mcap, double eps, int32_t* p_out, double* tau_out) {
  if (N < 1 || T < 1 || !f || !m || !C || !Mcap || !tau_out) return HYP_EINVAL;
  if (T > 1 && !p_out) return HYP_EINVAL;
  if (!(eps >= 0.0)) return HYP_EINVAL;
  for (int i = 0; i < N; ++i)
    if (!(f[i] >= 0.0) || !(m[i] >= 0.0) || std::isinf(f[i]) || std::isinf(m[i])) return HYP_EINVAL;
  for (int j = 0; j < T; ++j)
    if (!(C[j] > 0.0) || std::isinf(C[j]) || !(Mcap[j] >= 0.0)) return HYP_EINVAL;
  if (N < T) return HYP_EINFEASIBLE;

  std::vector<double> Sf(N + 1, 0.0), Sm(N + 1, 0.0);
  for (int i = 0; i < N; ++i) {
    Sf[i + 1] = Sf[i] + f[i];
    Sm[i + 1] = Sm[i] + m[i];
  }
  CheckTables tb(N, T);
  std::vector<int32_t> p(std::max(T - 1, 1), 0);

  if (eps > 0.0) {
    // Algorithm 1 as printed: bisection on tau.
    double c_min = C[0];
    for (int j = 1; j < T; ++j) c_min = std::min(c_min, C[j]);
    double lo = 0.0, hi = Sf[N] / c_min;
    if (!p_check(hi, tb, Sf, Sm, C, Mcap)) return HYP_EINFEASIBLE;
    backtrack(tb, p.data());
    while ((hi - lo) > eps) {
      const double mid = (lo + hi) / 2.0;
      if (p_check(mid, tb, Sf, Sm, C, Mcap)) {
        hi = mid;
        backtrack(tb, p.data());
      } else {
        lo = mid;
      }
    }
  } else {
    // Exact: the optimum is one of the finitely many values a tier load can take, and
    // feasibility is monotone in tau, so bisect over the sorted candidate set.
    std::vector<double> cand;
    cand.reserve((size_t)T * N * (N + 1) / 2);
    for (int j = 0; j < T; ++j)
      for (int n = 1; n <= N; ++n)
        for (int k = 0; k < n; ++k) cand.push_back((Sf[n] - Sf[k]) / C[j]);
    std::sort(cand.begin(), cand.end());
    cand.erase(std::unique(cand.begin(), cand.end()), cand.end());
    if (!p_check(cand.back(), tb, Sf, Sm, C, Mcap)) return HYP_EINFEASIBLE;
    size_t lo = 0, hi = cand.size() - 1;  // invariant: cand[hi] feasible
    while (lo < hi) {
      const size_t mid = lo + (hi - lo) / 2;
      if (p_check(cand[mid], tb, Sf, Sm, C, Mcap)) hi = mid; else lo = mid + 1;
    }
    p_check(cand[hi], tb, Sf, Sm, C, Mcap);
    backtrack(tb, p.data());
  }
  for (int j = 0; j + 1 < T; ++j) p_out[j] = p[j];
  *tau_out = bottleneck(p.data(), N, T, Sf, C);
  return HYP_OK;
}

extern "C" int hyp_sched_rt(double F_new, double m_act, const hyp_node_state* nodes, int32_t K,
                            int32_t* k_out) {
  if (!nodes || !k_out || K < 1 || !(F_new >= 0.0) || std::isnan(m_act)) return HYP_EINVAL;
  for (int k = 0; k < K; ++k)
    if (!(nodes[k].C > 0.0) || std::isnan(nodes[k].F_rem) || std::isnan(nodes[k].F_wait)) return HYP_EINVAL;
  double min_cost = INFINITY;
  int32_t k_star = -1;
  for (int k = 0; k < K; ++k) {
    if (nodes[k].available && nodes[k].M_avail >= m_act) {
      const double queued = nodes[k].F_rem + nodes[k].F_wait;
      const double cost = (queued + F_new) / nodes[k].C;
      if (cost < min_cost) {
        min_cost = cost;
        k_star = k;
      }
    }
  }
  if (k_star < 0) return HYP_EINFEASIBLE;
  *k_out = k_star;
  return HYP_OK;
}

// -------------------------------------------------------------------------------------------------
// The partitioning halves of the paper's two comparison systems (Section V names them, gives no algorithm;
// the readings are stated in hyperion.h).  They exist to show, on measured per-block costs, the bottleneck
// gap that HypSplit-DP closes.
// -------------------------------------------------------------------------------------------------
namespace {

int check_split_args(int32_t N, int32_t T, const double* f, const double* m, const double* C, const double* Mcap,
                     const int32_t* p_out, const double* tau_out) {
  if (N < 1 || T < 1 || !f || !m || !C || !Mcap || !tau_out) return HYP_EINVAL;
  if (T > 1 && !p_out) return HYP_EINVAL;
  for (int i = 0; i < N; ++i)
    if (!(f[i] >= 0.0) || !(m[i] >= 0.0) || std::isinf(f[i]) || std::isinf(m[i])) return HYP_EINVAL;
  for (int j = 0; j < T; ++j)
    if (!(C[j] > 0.0) || std::isinf(C[j]) || !(Mcap[j] >= 0.0)) return HYP_EINVAL;
  return N < T ? HYP_EINFEASIBLE : HYP_OK;
}

// max_j load and memory feasibility of a partition given as cut points (1-based last blocks of tiers 1..T-1)
bool evaluate_partition(const std::vector<int32_t>& p, int N, int T, const double* f, const double* m, const double* C,
                        const double* Mcap, double* tau) {
  bool fits = true;
  double worst = 0.0;
  int first = 0;
  for (int j = 0; j < T; ++j) {
    const int last = j == T - 1 ? N : p[j];
    double load = 0.0, mem = 0.0;
    for (int i = first; i < last; ++i) {
      load += f[i];
      mem += m[i];
    }
    if (mem > Mcap[j]) fits = false;
    if (load / C[j] > worst) worst = load / C[j];
    first = last;
  }
  *tau = worst;
  return fits;
}

}  // namespace

extern "C" int hyp_split_even(int32_t N, int32_t T, const double* f, const double* m, const double* C,
                              const double* Mcap, int32_t* p_out, double* tau_out) {
  int rc = check_split_args(N, T, f, m, C, Mcap, p_out, tau_out);
  if (rc) return rc;
  std::vector<int32_t> p(std::max(T - 1, 1), 0);
  const int base = N / T, extra = N % T;
  int cut = 0;
  for (int j = 0; j < T - 1; ++j) {
    cut += base + (j < extra ? 1 : 0);
    p[j] = cut;
  }
  double tau = 0.0;
  const bool fits = evaluate_partition(p, N, T, f, m, C, Mcap, &tau);
  for (int j = 0; j < T - 1; ++j) p_out[j] = p[j];
  *tau_out = tau;
  return fits ? HYP_OK : HYP_EINFEASIBLE;
}

extern "C" int hyp_split_greedy(int32_t N, int32_t T, const double* f, const double* m, const double* C,
                                const double* Mcap, int32_t* p_out, double* tau_out) {
  int rc = check_split_args(N, T, f, m, C, Mcap, p_out, tau_out);
  if (rc) return rc;
  double total = 0.0, csum = 0.0;
  for (int i = 0; i < N; ++i) total += f[i];
  for (int j = 0; j < T; ++j) csum += C[j];
  std::vector<int32_t> p(std::max(T - 1, 1), 0);
  int next = 0;  // first block not yet assigned
  for (int j = 0; j < T - 1; ++j) {
    const double share = total * C[j] / csum;  // what the tier would carry if load followed capacity
    double load = 0.0, mem = 0.0;
    int taken = 0;
    while (next < N - (T - 1 - j)) {  // every later tier keeps at least one block
      const double nl = load + f[next], nm = mem + m[next];
      if (nm > Mcap[j]) break;
      if (taken >= 1 && nl > share) break;
      load = nl;
      mem = nm;
      ++taken;
      ++next;
    }
    if (taken == 0) return HYP_EINFEASIBLE;  // the tier cannot even hold its first block
    p[j] = next;
  }
  double tau = 0.0;
  if (next >= N || !evaluate_partition(p, N, T, f, m, C, Mcap, &tau)) return HYP_EINFEASIBLE;
  for (int j = 0; j < T - 1; ++j) p_out[j] = p[j];
  *tau_out = tau;
  return HYP_OK;
}
