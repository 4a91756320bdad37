"""CPU oracle for the host-side algorithms.  TEST INFRASTRUCTURE ONLY.

* `enumerate_split`   - the plain definition of problem P1 (Section III-D): try every
  partition vector, keep the memory-feasible ones, take the smallest bottleneck.
* `hypsplit_dp_bisect` - Algorithm 1 (HypSplit-DP) taken step by step in the paper's notation:
  bisection on the target latency tau, each probe a boolean DP with predecessor table.
* `sched_rt_argmin`   - the definition of HypSched-RT's decision (the arg-min of Section IV-B
  over available nodes with enough memory).
* `hypsched_rt_scan`  - Algorithm 2 taken step by step.

Pure Python / float (IEEE double).  Shares no code with the library.

Readings where the paper is silent (each is restated in the library's header):
  - a segment's load is (S_f[n] - S_f[k]) / C_j with S_f the left-to-right prefix sum in double;
    the constant communication term of the objective is dropped, as Section IV-A does;
  - among partitions with equal bottleneck the result is the one that is smallest when read
    as (p_{T-1}, ..., p_1): Algorithm 1 takes the first feasible predecessor while scanning k
    upward, and backtracking starts at the last tier;
  - initial bounds: tau_low = 0, tau_high = S_f[N] / min_j C_j;
  - the returned tau* is max_j L_j(p*) of the returned partition, not the last probe value.

* `split_even`, `split_greedy` - the inter-tier partitioning halves of the paper's two comparison
  systems (Section V, baselines), which it only names: GPipe's static split of the chain into
  contiguous, equally long segments, and the greedy, memory-checking partitioning step that
  precedes HEFT.  Readings taken (the paper gives no algorithm for either):
  - even: contiguous segments of equal block count, the N mod T leading tiers one block longer;
    blind to costs, capacities and memory (a violated memory limit is reported, not repaired);
  - greedy: tiers are filled in order; tier j keeps taking the next block while its memory limit
    holds and its load stays within its capacity-proportional share S_f[N] * C_j / sum(C), takes at
    least one block, and always leaves one block for every later tier; the last tier takes the rest.

The block allocations printed in the paper's utilisation table: parity unpinned (the f_i, m_i
and capacities that produced them are not published).
"""
from __future__ import annotations

from itertools import combinations


def prefix_sums(a):
    """S[n] = sum_{i<=n} a_i, S[0] = 0, accumulated left to right (Section IV-A)."""
    S = [0.0]
    for v in a:
        S.append(S[-1] + float(v))
    return S


def tier_loads(p, f, C):
    """L_j(p) = (1/C_j) * sum_{i=p_{j-1}+1}^{p_j} f_i for j = 1..T with p_0 = 0, p_T = N."""
    Sf = prefix_sums(f)
    cuts = [0] + list(p) + [len(f)]
    return [(Sf[cuts[j + 1]] - Sf[cuts[j]]) / float(C[j]) for j in range(len(C))]


def enumerate_split(f, m, C, Mcap):
    """Exact optimum of P1 by exhaustive enumeration.

    Every strictly increasing vector 1 <= p_1 < ... < p_{T-1} < N is tried; those with a tier
    whose memory sum exceeds M_j are discarded; the objective is the largest tier load.
    Returns (p, tau) with p a tuple of 1-based last-block indices, or (None, inf) if no
    partition is memory-feasible (or N < T)."""
    N, T = len(f), len(C)
    Sf, Sm = prefix_sums(f), prefix_sums(m)
    best_p, best_tau, best_key = None, float("inf"), None
    if N < T:
        return None, float("inf")
    for p in combinations(range(1, N), T - 1):
        cuts = (0,) + p + (N,)
        ok = True
        tau = 0.0
        for j in range(T):
            if Sm[cuts[j + 1]] - Sm[cuts[j]] > float(Mcap[j]):
                ok = False
                break
            L = (Sf[cuts[j + 1]] - Sf[cuts[j]]) / float(C[j])
            if L > tau:
                tau = L
        if not ok:
            continue
        key = tuple(reversed(p))
        if tau < best_tau or (tau == best_tau and key < best_key):
            best_p, best_tau, best_key = p, tau, key
    return best_p, best_tau


def dp_check(tau, N, T, Sf, Sm, C, Mcap):
    """Decision problem P_check(tau): boolean table DP[j][n] and predecessor table P[j][n].

    DP[j][n] is true iff blocks 1..n can be placed on tiers 1..j with every tier load <= tau and
    every tier memory within its limit.  The predecessor scan runs k upward and stops at the
    first k that works."""
    DP = [[False] * (N + 1) for _ in range(T + 1)]
    P = [[-1] * (N + 1) for _ in range(T + 1)]
    DP[0][0] = True
    for j in range(1, T + 1):
        for n in range(j, N + 1):
            for k in range(j - 1, n):
                if DP[j - 1][k]:
                    L = (Sf[n] - Sf[k]) / float(C[j - 1])
                    U = Sm[n] - Sm[k]
                    if L <= tau and U <= float(Mcap[j - 1]):
                        DP[j][n] = True
                        P[j][n] = k
                        break
    return DP, P


def backtrack(P, N, T):
    """Read p_{T-1}, ..., p_1 off the predecessor table, starting from (T, N)."""
    p = [0] * (T - 1)
    n = N
    for j in range(T, 1, -1):
        n = P[j][n]
        p[j - 2] = n
    return tuple(p)


def hypsplit_dp_bisect(f, m, C, Mcap, eps):
    """Algorithm 1 (HypSplit-DP) step by step: bisection until tau_high - tau_low <= eps.

    Returns (p*, tau*, probes) where tau* = max_j L_j(p*) and probes is the number of DP
    checks made; (None, inf, probes) if even tau_high is infeasible."""
    N, T = len(f), len(C)
    if N < T:
        return None, float("inf"), 0
    Sf, Sm = prefix_sums(f), prefix_sums(m)
    tau_low, tau_high = 0.0, Sf[N] / min(float(c) for c in C)
    probes = 1
    DP, P = dp_check(tau_high, N, T, Sf, Sm, C, Mcap)
    if not DP[T][N]:
        return None, float("inf"), probes
    p_star = backtrack(P, N, T)
    while (tau_high - tau_low) > eps:
        tau_mid = (tau_low + tau_high) / 2.0
        DP, P = dp_check(tau_mid, N, T, Sf, Sm, C, Mcap)
        probes += 1
        if DP[T][N]:
            tau_high = tau_mid
            p_star = backtrack(P, N, T)
        else:
            tau_low = tau_mid
    return p_star, max(tier_loads(p_star, f, C)), probes


def sched_rt_argmin(F_new, m_act, nodes):
    """Definition of the HypSched-RT decision (Section IV-B).

    nodes: list of dicts {C, M_avail, F_rem, F_wait (list), available}.  Among nodes that are
    available and have M_avail >= m_act, pick the one minimising
    (F_rem + sum(F_wait) + F_new) / C; the lowest index wins ties.  Returns -1 if none."""
    cands = []
    for k, nd in enumerate(nodes):
        if nd["available"] and nd["M_avail"] >= m_act:
            queued = float(nd["F_rem"])
            for w in nd["F_wait"]:
                queued += float(w)
            cands.append(((queued + F_new) / float(nd["C"]), k))
    if not cands:
        return -1
    return min(cands)[1]


def hypsched_rt_scan(F_new, m_act, nodes):
    """Algorithm 2 (HypSched-RT): one linear scan keeping the strictly smaller cost."""
    min_cost, k_star = float("inf"), -1
    for k, nd in enumerate(nodes):
        if nd["available"] and nd["M_avail"] >= m_act:
            F_queued = float(nd["F_rem"])
            for w in nd["F_wait"]:
                F_queued += float(w)
            cost = (F_queued + F_new) / float(nd["C"])
            if cost < min_cost:
                min_cost, k_star = cost, k
    return k_star


def split_even(N, T):
    """GPipe-style static partition (Section V, second baseline): contiguous segments of equal
    block count; the first N mod T tiers get one block more.  Returns p (1-based last block of
    tiers 1..T-1)."""
    base, extra = divmod(N, T)
    p, cut = [], 0
    for j in range(T - 1):
        cut += base + (1 if j < extra else 0)
        p.append(cut)
    return tuple(p)


def split_greedy(f, m, C, Mcap):
    """Memory-aware greedy contiguous partition (Section V, first baseline, its partitioning step).
    Returns p, or None if some tier's first block, or the remainder left to the last tier, breaks
    a memory limit."""
    N, T = len(f), len(C)
    total = 0.0
    for x in f:
        total += float(x)
    csum = 0.0
    for c in C:
        csum += float(c)
    p, nxt = [], 0                      # nxt = 0-based index of the next unassigned block
    for j in range(T - 1):
        share = total * float(C[j]) / csum
        load, mem, taken = 0.0, 0.0, 0
        while nxt < N - (T - 1 - j):    # leave one block for every later tier
            nl, nm = load + float(f[nxt]), mem + float(m[nxt])
            if nm > Mcap[j]:
                break
            if taken >= 1 and nl > share:
                break
            load, mem, taken, nxt = nl, nm, taken + 1, nxt + 1
        if taken == 0:
            return None
        p.append(nxt)
    rest = 0.0
    for i in range(nxt, N):
        rest += float(m[i])
    if nxt >= N or rest > Mcap[T - 1]:
        return None
    return tuple(p)


def memory_feasible(p, m, Mcap):
    """Does every tier's segment of the partition p fit its memory limit?"""
    cuts = [0] + list(p) + [len(m)]
    for j in range(len(Mcap)):
        u = 0.0
        for i in range(cuts[j], cuts[j + 1]):
            u += float(m[i])
        if u > Mcap[j]:
            return False
    return True
