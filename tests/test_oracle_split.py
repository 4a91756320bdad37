"""Pins for the split / scheduling oracle: textbook special cases, closed forms, invariants and a
second, independently written solver.  CPU only."""
import math
from functools import lru_cache

import numpy as np
import pytest

from oracle import split as osp
from paper_2511_14450_b200 import inputs


def painters_partition(f, T):
    """Textbook linear-partition DP (min over last cut of max(prefix, last segment)); cost only."""
    N = len(f)
    S = [0.0]
    for v in f:
        S.append(S[-1] + v)

    @lru_cache(None)
    def best(n, t):
        if t == 1:
            return S[n]
        return min(max(best(k, t - 1), S[n] - S[k]) for k in range(t - 1, n))
    return best(N, T)


def test_equal_capacity_no_memory_limit_is_the_painters_partition_problem():
    r = np.random.default_rng(0)
    for N, T in [(6, 2), (9, 3), (12, 4), (12, 5), (7, 7)]:
        f = list(np.floor(r.uniform(1, 20, N)))
        p, tau = osp.enumerate_split(f, [1.0] * N, [1.0] * T, [1e9] * T)
        assert tau == painters_partition(tuple(f), T)
        assert max(osp.tier_loads(p, f, [1.0] * T)) == tau


def test_uniform_costs_closed_form():
    for N, T in [(8, 3), (12, 5), (10, 2), (5, 5)]:
        p, tau = osp.enumerate_split([2.0] * N, [1.0] * N, [4.0] * T, [1e9] * T)
        assert tau == math.ceil(N / T) * 2.0 / 4.0


def test_uniform_40_blocks_3_tiers_tie_break_gives_12_14_14():
    # 40 equal blocks on 3 equal tiers: bottleneck 14 blocks; the first-feasible-predecessor rule
    # pushes split points as low as possible from the last tier backwards.  Checked with the DP
    # (enumeration of C(39,2)=741 vectors is also cheap).
    f, m, C, M = [1.0] * 40, [1.0] * 40, [1.0] * 3, [1e9] * 3
    p, tau = osp.enumerate_split(f, m, C, M)
    assert tau == 14.0 and p == (12, 26)
    p2, tau2, _ = osp.hypsplit_dp_bisect(f, m, C, M, 1e-3)
    assert p2 == (12, 26) and tau2 == 14.0


def test_one_block_per_tier_and_single_tier():
    f, C = [3.0, 8.0, 2.0, 9.0], [1.0, 4.0, 0.5, 3.0]
    p, tau = osp.enumerate_split(f, [1] * 4, C, [10] * 4)
    assert p == (1, 2, 3) and tau == max(a / b for a, b in zip(f, C))
    p, tau = osp.enumerate_split(f, [1] * 4, [2.0], [10])
    assert p == () and tau == sum(f) / 2.0


def test_infeasible_cases():
    assert osp.enumerate_split([1, 1], [1, 1], [1, 1, 1], [9, 9, 9]) == (None, float("inf"))   # N < T
    assert osp.enumerate_split([1] * 4, [5] * 4, [1, 1], [9, 9])[0] is None                      # memory
    assert osp.hypsplit_dp_bisect([1] * 4, [5] * 4, [1, 1], [9, 9], 1e-3)[0] is None


def test_memory_limit_overrides_the_compute_optimal_split():
    # compute-optimal is 2|2 (tau 2) but tier 1 holds one block only -> 1|3 (tau 3)
    p, tau = osp.enumerate_split([1.0] * 4, [1.0] * 4, [1.0, 1.0], [1.0, 10.0])
    assert p == (1,) and tau == 3.0
    # the memory constraint is per tier j against M_j (not shifted or transposed)
    p, tau = osp.enumerate_split([1.0] * 4, [1.0] * 4, [1.0, 1.0], [10.0, 1.0])
    assert p == (3,) and tau == 3.0


def test_heterogeneous_capacity_hand_example():
    # f = 1..6, C = (1, 2): cut after block k gives max(S_k, (21 - S_k)/2); S = 1,3,6,10,15
    # -> k=3: max(6, 7.5)=7.5 ; k=4: max(10, 5.5)=10 ; optimum k=3
    p, tau = osp.enumerate_split([1, 2, 3, 4, 5, 6], [0] * 6, [1.0, 2.0], [1, 1])
    assert p == (3,) and tau == 7.5


def test_monotone_feasibility_of_the_decision_problem():
    f, m, C, M = inputs.split_instance(10, 3, stream=5)
    Sf, Sm = osp.prefix_sums(f), osp.prefix_sums(m)
    taus = np.linspace(0, Sf[-1] / min(C), 200)
    feas = [osp.dp_check(t, 10, 3, Sf, Sm, C, M)[0][3][10] for t in taus]
    assert feas == sorted(feas) and feas[-1] and not feas[0]
    _, tau_star = osp.enumerate_split(f, m, C, M)
    for t, ok in zip(taus, feas):
        assert ok == (t >= tau_star)


def test_dp_table_equals_recurrence_evaluated_naively():
    f, m, C, M = inputs.split_instance(7, 3, stream=6, integer=True)
    Sf, Sm = osp.prefix_sums(f), osp.prefix_sums(m)
    tau = 0.12
    DP, P = osp.dp_check(tau, 7, 3, Sf, Sm, C, M)

    def rec(j, n):           # the recurrence and base case as stated, no table
        if j == 1:
            return n >= 1 and sum(f[:n]) / C[0] <= tau and sum(m[:n]) <= M[0]
        return any(rec(j - 1, k) and sum(f[k:n]) / C[j - 1] <= tau and sum(m[k:n]) <= M[j - 1]
                   for k in range(j - 1, n))
    for j in range(1, 4):
        for n in range(j, 8):
            assert DP[j][n] == rec(j, n)
            if DP[j][n] and j > 1:
                assert rec(j - 1, P[j][n]) and all(
                    not (rec(j - 1, k) and sum(f[k:n]) / C[j - 1] <= tau and sum(m[k:n]) <= M[j - 1])
                    for k in range(j - 1, P[j][n]))


@pytest.mark.parametrize("N", range(1, 13))
def test_bisection_is_within_eps_of_enumeration(N):
    for T in range(1, min(N, 5) + 1):
        for s in range(3):
            f, m, C, M = inputs.split_instance(N, T, stream=100 * N + 10 * T + s, tight_memory=(s == 2))
            p_e, tau_e = osp.enumerate_split(f, m, C, M)
            eps = 1e-3 * (sum(f) / min(C))
            p_b, tau_b, probes = osp.hypsplit_dp_bisect(f, m, C, M, eps)
            if p_e is None:
                assert p_b is None
                continue
            assert tau_e <= tau_b <= tau_e + eps
            assert probes <= 12


def test_bisection_with_tiny_eps_recovers_the_exact_partition():
    for s in range(20):
        f, m, C, M = inputs.split_instance(11, 4, stream=900 + s, integer=True, tight_memory=(s % 3 == 0))
        p_e, tau_e = osp.enumerate_split(f, m, C, M)
        p_b, tau_b, _ = osp.hypsplit_dp_bisect(f, m, C, M, 1e-12)
        assert p_b == p_e and tau_b == tau_e


def test_sched_rt_scan_equals_argmin_definition_and_hand_cases():
    nodes = [
        {"C": 10.0, "M_avail": 4.0, "F_rem": 5.0, "F_wait": [10.0, 5.0], "available": True},   # (20+10)/10 = 3
        {"C": 20.0, "M_avail": 4.0, "F_rem": 0.0, "F_wait": [50.0], "available": True},         # 60/20 = 3 (tie)
        {"C": 40.0, "M_avail": 1.0, "F_rem": 0.0, "F_wait": [], "available": True},             # memory too small
        {"C": 40.0, "M_avail": 9.0, "F_rem": 0.0, "F_wait": [], "available": False},            # down
        {"C": 5.0, "M_avail": 9.0, "F_rem": 0.0, "F_wait": [], "available": True},              # 10/5 = 2
    ]
    assert osp.hypsched_rt_scan(10.0, 2.0, nodes) == 4 == osp.sched_rt_argmin(10.0, 2.0, nodes)
    assert osp.hypsched_rt_scan(10.0, 2.0, nodes[:4]) == 0          # strict '<' keeps the first minimum
    assert osp.hypsched_rt_scan(10.0, 20.0, nodes) == -1            # nobody has the memory
    assert osp.hypsched_rt_scan(10.0, 0.5, nodes[2:3]) == 0
    r = np.random.default_rng(7)
    for _ in range(200):
        K = int(r.integers(1, 9))
        nd = [{"C": float(r.integers(1, 5)), "M_avail": float(r.integers(0, 4)), "F_rem": float(r.integers(0, 4)),
               "F_wait": [float(v) for v in r.integers(0, 6, int(r.integers(0, 4)))],
               "available": bool(r.integers(0, 4))} for _ in range(K)]
        assert osp.hypsched_rt_scan(3.0, 2.0, nd) == osp.sched_rt_argmin(3.0, 2.0, nd)


def test_baseline_partitioners_hand_worked_and_dominated_by_the_optimum():
    """The two comparison partitioners (Section V names them; the readings are in the oracle's header).
    Hand-worked cases, structural properties, and: neither can beat the exact optimum."""
    # even: sizes differ by at most one, longer segments first
    assert osp.split_even(40, 3) == (14, 27) and osp.split_even(8, 3) == (3, 6) and osp.split_even(6, 3) == (2, 4)
    assert osp.split_even(5, 1) == () and osp.split_even(4, 4) == (1, 2, 3)
    # greedy by hand: f = 4,1,1,4,1,1; C = (1,1,1): share 4 each.  Tier 1 takes block 1 (load 4; a second
    # block would exceed 4).  Tier 2 takes 1,1 (load 2; the next block, 4, would exceed).  p = (1, 3).
    assert osp.split_greedy([4, 1, 1, 4, 1, 1], [1] * 6, [1, 1, 1], [9, 9, 9]) == (1, 3)
    # capacities 1:3 -> shares 3 and 9 of a total of 12: tier 1 stops after 3 unit blocks
    assert osp.split_greedy([1] * 12, [1] * 12, [1, 3], [99, 99]) == (3,)
    # memory binds before the share does: tier 1 may hold only 2 blocks
    assert osp.split_greedy([1] * 12, [1] * 12, [3, 1], [2, 99]) == (2,)
    # the last tier cannot hold what is left -> no partition; a first block that does not fit -> none
    assert osp.split_greedy([1] * 12, [1] * 12, [1, 1], [6, 3]) is None
    assert osp.split_greedy([1, 1, 1], [5, 1, 1], [1, 1], [4, 9]) is None
    # every later tier keeps a block even when the shares would starve it
    assert osp.split_greedy([1, 1, 1], [1, 1, 1], [100, 1, 1], [9, 9, 9]) == (1, 2)
    # uniform blocks, equal tiers, N divisible by T: greedy = even = optimal
    for N, T in [(6, 3), (12, 4), (10, 5)]:
        f, m, C, M = [2.0] * N, [1.0] * N, [1.0] * T, [1e9] * T
        assert osp.split_greedy(f, m, C, M) == osp.split_even(N, T) == osp.enumerate_split(f, m, C, M)[0]
    r = np.random.default_rng(5)
    for trial in range(200):
        N, T = int(r.integers(3, 11)), int(r.integers(2, 4))
        f = list(np.floor(r.uniform(1, 9, N)))
        m = list(np.floor(r.uniform(1, 4, N)))
        C = list(np.floor(r.uniform(1, 4, T)))
        M = list(np.floor(r.uniform(4, 20, T)))
        opt = osp.enumerate_split(f, m, C, M)
        for p in (osp.split_greedy(f, m, C, M), osp.split_even(N, T)):
            if p is None or not osp.memory_feasible(p, m, M):
                continue
            assert list(p) == sorted(set(p)) and 1 <= p[0] and p[-1] < N     # a valid partition vector
            assert opt is not None and max(osp.tier_loads(p, f, C)) >= opt[1]
        g = osp.split_greedy(f, m, C, M)
        assert g is None or osp.memory_feasible(g, m, M)                      # greedy never breaks a limit
