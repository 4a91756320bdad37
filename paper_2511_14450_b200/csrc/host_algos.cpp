// Host-side algorithms of the paper: HypSplit-DP (Algorithm 1) and HypSched-RT (Algorithm 2).
// Pure C++, no GPU, thread-safe (no global state).
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <vector>

#include "hyperion.h"

namespace {

// Feasibility of a latency budget tau for problem P1 (Section III-D), and the canonical partition that meets it.
//
// A tier's load (S_f[n] - S_f[k]) / C_j and memory S_m[n] - S_m[k] only shrink as the segment's left edge k moves
// right (prefix sums of non-negative numbers are monotone, also in floating point), and only grow with its right
// edge n.  So for tier j and right edge n the admissible left edges form a run [left_j(n), n-1] whose start never
// moves left as n grows: one two-pointer sweep per tier finds every left_j(n).  Tier j can end at n iff some
// prefix length in that run is reachable by tiers 1..j-1; `next_reachable` answers "smallest reachable prefix at
// or after k" in O(1), which is also the predecessor the tie rule of hyperion.h asks for (the smallest one).
// One probe costs O(T N).
class BudgetSweep {
 public:
  BudgetSweep(int N, int T, const std::vector<double>& Sf, const std::vector<double>& Sm, const double* C,
              const double* Mcap)
      : N_(N), T_(T), Sf_(Sf), Sm_(Sm), C_(C), Mcap_(Mcap), first_pred_((size_t)T * (N + 1)),
        next_reachable_(N + 2), reach_(N + 1) {}

  bool feasible(double tau) {
    std::fill(reach_.begin(), reach_.end(), 0);
    reach_[0] = 1;  // zero tiers cover the empty prefix
    for (int j = 0; j < T_; ++j) {
      // smallest reachable prefix length >= k (N_ + 1: none)
      next_reachable_[N_ + 1] = N_ + 1;
      for (int k = N_; k >= 0; --k) next_reachable_[k] = reach_[k] ? k : next_reachable_[k + 1];
      std::fill(reach_.begin(), reach_.end(), 0);
      int32_t* pred = &first_pred_[(size_t)j * (N_ + 1)];
      int left = 0;
      for (int n = 1; n <= N_; ++n) {
        while (left < n && !fits(j, left, n, tau)) ++left;
        const int k = left < n ? next_reachable_[left] : n;
        pred[n] = k < n ? k : -1;
        reach_[n] = k < n;
      }
    }
    return reach_[N_] != 0;
  }

  // cut points of the partition the last feasible() call found: walk the predecessors back from (T, N)
  void cuts(int32_t* p) const {
    int n = N_;
    for (int j = T_ - 1; j >= 1; --j) {
      n = first_pred_[(size_t)j * (N_ + 1) + n];
      p[j - 1] = n;
    }
  }

 private:
  bool fits(int j, int k, int n, double tau) const {
    return (Sf_[n] - Sf_[k]) / C_[j] <= tau && Sm_[n] - Sm_[k] <= Mcap_[j];
  }
  int N_, T_;
  const std::vector<double>&Sf_, &Sm_;
  const double *C_, *Mcap_;
  std::vector<int32_t> first_pred_;
  std::vector<int> next_reachable_;
  std::vector<uint8_t> reach_;
};

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
  // The optimum is one of the finitely many values a tier load can take, and feasibility is monotone in the
  // budget (Section IV-A), so the search runs over the sorted set of those values: exact, no tolerance needed.
  // With eps > 0 the search may stop as soon as the bracket [largest infeasible, smallest feasible seen] is
  // narrower than eps; the partition of the feasible end is then within eps of the optimum.
  std::vector<double> cand;
  cand.reserve((size_t)T * N * (N + 1) / 2);
  for (int j = 0; j < T; ++j)
    for (int n = 1; n <= N; ++n)
      for (int k = 0; k < n; ++k) cand.push_back((Sf[n] - Sf[k]) / C[j]);
  std::sort(cand.begin(), cand.end());
  cand.erase(std::unique(cand.begin(), cand.end()), cand.end());

  BudgetSweep sweep(N, T, Sf, Sm, C, Mcap);
  if (!sweep.feasible(cand.back())) return HYP_EINFEASIBLE;   // only memory can rule out the largest budget
  size_t lo = 0, hi = cand.size() - 1;  // cand[hi] is feasible; everything below cand[lo] is infeasible
  double below = 0.0;                    // a budget known to be <= the optimum
  while (lo < hi && !(eps > 0.0 && cand[hi] - below <= eps)) {
    const size_t mid = lo + (hi - lo) / 2;
    if (sweep.feasible(cand[mid])) {
      hi = mid;
    } else {
      lo = mid + 1;
      below = cand[mid];
    }
  }
  std::vector<int32_t> p(std::max(T - 1, 1), 0);
  sweep.feasible(cand[hi]);
  sweep.cuts(p.data());
  for (int j = 0; j + 1 < T; ++j) p_out[j] = p[j];
  *tau_out = bottleneck(p.data(), N, T, Sf, C);
  return HYP_OK;
}

extern "C" int hyp_sched_rt(double F_new, double m_act, const hyp_node_state* nodes, int32_t K,
                            int32_t* k_out) {
  if (!nodes || !k_out || K < 1 || !(F_new >= 0.0) || !std::isfinite(F_new) || std::isnan(m_act)) return HYP_EINVAL;
  for (int k = 0; k < K; ++k)
    if (!(nodes[k].C > 0.0) || !std::isfinite(nodes[k].F_rem) || !std::isfinite(nodes[k].F_wait)) return HYP_EINVAL;
  // the nodes that may take the task (Section IV-B: switched on, enough free memory) ...
  std::vector<int32_t> eligible;
  for (int k = 0; k < K; ++k)
    if (nodes[k].available && nodes[k].M_avail >= m_act) eligible.push_back(k);
  if (eligible.empty()) return HYP_EINFEASIBLE;
  // ... and among them the earliest estimated completion of the new task; min_element keeps the first of equal
  // minima, i.e. the lowest node index
  auto finish = [&](int32_t k) { return (nodes[k].F_rem + nodes[k].F_wait + F_new) / nodes[k].C; };
  *k_out = *std::min_element(eligible.begin(), eligible.end(),
                             [&](int32_t a, int32_t b) { return finish(a) < finish(b); });
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
