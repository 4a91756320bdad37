"""Library host algorithms (through the C ABI, no GPU needed) against the oracle: bit-exact
boundaries and tau for hyp_split_dp, identical node for hyp_sched_rt; error codes; ABI exports."""
import os
import re

import numpy as np
import pytest

from oracle import split as osp
from paper_2511_14450_b200 import hyperion as hyp
from paper_2511_14450_b200 import inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    declared = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        declared |= set(re.findall(r"\b(hyp_[a-z0-9_]+)\s*\(", text))
    assert declared, "no declarations parsed"
    L = hyp.lib()
    for name in sorted(declared):
        assert hasattr(L, name), f"{name} declared in include/ but not exported"
    assert declared == set(hyp.SIGNATURES), (declared ^ set(hyp.SIGNATURES))


@pytest.mark.parametrize("N", range(1, 13))
def test_split_dp_exact_equals_enumeration_bit_exact(N):
    for T in range(1, min(N, 5) + 1):
        for s in range(6):
            f, m, C, M = inputs.split_instance(N, T, stream=1000 * N + 10 * T + s, integer=(s % 2 == 1),
                                               tight_memory=(s >= 4))
            p_e, tau_e = osp.enumerate_split(f, m, C, M)
            if p_e is None:
                with pytest.raises(hyp.HyperionError) as ei:
                    hyp.hyp_split_dp(f, m, C, M)
                assert ei.value.code == hyp.HYP_EINFEASIBLE
                continue
            p, tau = hyp.hyp_split_dp(f, m, C, M)
            assert p == p_e and tau == tau_e          # bit-exact, including the tie-break


def test_split_dp_ties_with_integer_costs():
    # many equal-bottleneck partitions: the canonical one must come back
    r = np.random.default_rng(5)
    for _ in range(60):
        N, T = int(r.integers(3, 12)), int(r.integers(2, 5))
        if N < T:
            continue
        f = r.integers(1, 3, N).astype(float)
        m = np.ones(N)
        C = np.ones(T)
        M = np.full(T, float(r.integers(2, N + 1)))
        p_e, tau_e = osp.enumerate_split(f, m, C, M)
        if p_e is None:
            continue
        assert hyp.hyp_split_dp(f, m, C, M) == (p_e, tau_e)


def test_split_dp_tolerance_mode_is_within_eps_of_the_enumerated_optimum():
    """eps > 0 lets the search stop early: the partition returned must be memory-feasible, its reported tau must be
    its own bottleneck, and that bottleneck must lie within eps of the exhaustive optimum; a tiny eps gives the
    exact answer.  (The oracle's step-by-step Algorithm 1 is held to the same bound in test_oracle_split.py.)"""
    hit_inexact = 0
    for s in range(60):
        N, T = 5 + s % 8, 2 + s % 3
        f, m, C, M = inputs.split_instance(N, T, stream=5000 + s, tight_memory=(s % 4 == 0))
        p_e, tau_e = osp.enumerate_split(f, m, C, M)
        for eps in (0.3 * tau_e if p_e else 1.0, 1e-3, 1e-12):
            if p_e is None:
                with pytest.raises(hyp.HyperionError) as ei:
                    hyp.hyp_split_dp(f, m, C, M, eps)
                assert ei.value.code == hyp.HYP_EINFEASIBLE
                continue
            p, tau = hyp.hyp_split_dp(f, m, C, M, eps)
            assert list(p) == sorted(set(p)) and all(1 <= c < N for c in p)
            assert osp.memory_feasible(p, m, M) and tau == max(osp.tier_loads(p, f, C))
            assert tau_e <= tau <= tau_e + eps
            hit_inexact += tau > tau_e
            if eps == 1e-12:
                assert (p, tau) == (p_e, tau_e)
    assert hit_inexact > 0          # the loose tolerance really stops early somewhere


def test_split_dp_config0_instance_and_40_layer_uniform():
    u = inputs.uniform_f64(inputs.SEED_SPLIT, 0, 8)
    f, m, C, M = 1.0 + u, np.ones(8), [67.0, 157.0, 200.0], [2.0, 4.0, 8.0]
    assert hyp.hyp_split_dp(f, m, C, M) == osp.enumerate_split(f, m, C, M)
    assert hyp.hyp_split_dp([1.0] * 40, [1.0] * 40, [1.0] * 3, [1e9] * 3) == ((12, 26), 14.0)


def test_split_dp_errors():
    ok = ([1.0, 2.0], [1.0, 1.0], [1.0, 1.0], [5.0, 5.0])
    assert hyp.hyp_split_dp(*ok)[0] == (1,)
    bad = [
        ([1.0, -2.0], ok[1], ok[2], ok[3]), (ok[0], [1.0, float("nan")], ok[2], ok[3]),
        (ok[0], ok[1], [1.0, 0.0], ok[3]), (ok[0], ok[1], ok[2], [5.0, -1.0]),
    ]
    for args in bad:
        with pytest.raises(hyp.HyperionError) as ei:
            hyp.hyp_split_dp(*args)
        assert ei.value.code == hyp.HYP_EINVAL
    with pytest.raises(hyp.HyperionError) as ei:
        hyp.hyp_split_dp([1.0], [1.0], [1.0, 1.0], [5.0, 5.0])      # N < T
    assert ei.value.code == hyp.HYP_EINFEASIBLE
    with pytest.raises(hyp.HyperionError) as ei:
        hyp.hyp_split_dp(ok[0], ok[1], ok[2], ok[3], eps=-1.0)
    assert ei.value.code == hyp.HYP_EINVAL


def test_sched_rt_matches_oracle():
    r = np.random.default_rng(11)
    for _ in range(300):
        K = int(r.integers(1, 10))
        nodes_o, nodes_l = [], []
        for _k in range(K):
            nd = {"C": float(r.integers(1, 6)), "M_avail": float(r.integers(0, 5)), "F_rem": float(r.integers(0, 5)),
                  "F_wait": [float(v) for v in r.integers(0, 7, int(r.integers(0, 4)))],
                  "available": bool(r.integers(0, 4))}
            nodes_o.append(nd)
            nodes_l.append((nd["C"], nd["M_avail"], nd["F_rem"], sum(nd["F_wait"]), int(nd["available"])))
        want = osp.sched_rt_argmin(4.0, 2.0, nodes_o)        # the definition, not the scan of Algorithm 2
        if want < 0:
            with pytest.raises(hyp.HyperionError) as ei:
                hyp.hyp_sched_rt(4.0, 2.0, nodes_l)
            assert ei.value.code == hyp.HYP_EINFEASIBLE
        else:
            assert hyp.hyp_sched_rt(4.0, 2.0, nodes_l) == want


def test_strerror_covers_all_codes():
    L = hyp.lib()
    seen = {L.hyp_strerror(c).decode() for c in range(0, -8, -1)}
    assert len(seen) == 8 and "unknown status" not in seen
    assert L.hyp_strerror(-99).decode() == "unknown status"


def test_packed_weight_size_and_tuning_switch_ranges():
    """Host-only parts of the single-kernel API: the packed size is whole 2 KB tiles with an even number of 16-row
    strips and 64-k blocks per half, and the tuning switches refuse values outside their range."""
    L = hyp.lib()
    for N, K, sw in [(5120, 5120, 0), (17920, 5120, 1), (256, 688, 0), (272, 328, 1), (1, 8, 0)]:
        strips = -(-N // 16)
        strips += strips & 1
        kblocks = -(-K // 64)
        kblocks += kblocks & 1
        assert L.hyp_op_weight_packed_bytes(N, K, sw) == (2 if sw else 1) * strips * kblocks * 2048
    assert L.hyp_op_weight_packed_bytes(0, 64, 0) == 0 and L.hyp_op_weight_packed_bytes(16, 12, 0) == 0
    assert L.hyp_tune(hyp.HYP_TUNE_PDL, 4) == hyp.HYP_EINVAL and L.hyp_tune(hyp.HYP_TUNE_STREAM_SLOTS, 9) == hyp.HYP_EINVAL
    assert L.hyp_tune(hyp.HYP_TUNE_ATTN_SPLITS, 9) == hyp.HYP_EINVAL and L.hyp_tune(99, 0) == hyp.HYP_EINVAL
    assert L.hyp_tune(hyp.HYP_TUNE_STREAM_SLOTS, 0) == hyp.HYP_OK


def test_baseline_partitioners_equal_the_oracle():
    """hyp_split_even / hyp_split_greedy against the oracle's versions on seeded instances (bit-exact boundaries),
    infeasible cases included, and never better than hyp_split_dp."""
    r = np.random.default_rng(11)
    n_inf = 0
    for trial in range(400):
        N, T = int(r.integers(1, 13)), int(r.integers(1, 5))
        if N < T:
            continue
        f = [float(x) for x in np.floor(r.uniform(1, 9, N))]
        m = [float(x) for x in np.floor(r.uniform(1, 4, N))]
        Cp = [float(x) for x in np.floor(r.uniform(1, 4, T))]
        M = [float(x) for x in np.floor(r.uniform(3, 20, T))]
        p, tau, fits = hyp.hyp_split_even(f, m, Cp, M)
        assert p == osp.split_even(N, T) and fits == osp.memory_feasible(p, m, M)
        assert tau == max(osp.tier_loads(p, f, Cp))
        want = osp.split_greedy(f, m, Cp, M)
        if want is None:
            n_inf += 1
            with pytest.raises(hyp.HyperionError) as ei:
                hyp.hyp_split_greedy(f, m, Cp, M)
            assert ei.value.code == hyp.HYP_EINFEASIBLE
        else:
            pg, tg = hyp.hyp_split_greedy(f, m, Cp, M)
            assert pg == want and tg == max(osp.tier_loads(pg, f, Cp))
            assert tg >= hyp.hyp_split_dp(f, m, Cp, M)[1]
    assert n_inf > 10
    with pytest.raises(hyp.HyperionError):
        hyp.hyp_split_greedy([1.0, 2.0], [1.0, 1.0], [1.0, 0.0], [9.0, 9.0])      # zero capacity


def test_compare_splits_report_on_uneven_costs():
    """The serving tool's comparison of the three partitioners (host logic only): HypSplit-DP is never worse, the
    ratios are reported against it, and a first block heavier than the small tier's share shows the greedy gap."""
    from paper_2511_14450_b200 import serving
    f = [9.0, 1.0, 1.0, 1.0, 5.0, 1.0, 1.0, 1.0, 1.0, 3.0, 1.0, 1.0]
    m = [1.0] * 12
    for tiers in (2, 3, 4):
        rep = serving.compare_splits(f, m, tiers)
        meth = rep["methods"]
        assert meth["hypsplit_dp"]["vs_hypsplit_dp"] == 1.0 and len(meth["hypsplit_dp"]["boundaries"]) == tiers + 1
        for name in ("greedy_memory_aware", "even_count"):
            if meth[name]["bottleneck"] is not None and meth[name]["fits_memory"]:
                assert meth[name]["vs_hypsplit_dp"] >= 1.0
        assert abs(sum(rep["memory_limits_bytes"]) - 1.25 * 12) < 1e-9
    assert serving.compare_splits(f, m, 3)["methods"]["even_count"]["vs_hypsplit_dp"] > 1.0


def test_stage_create_rejects_shapes_before_touching_the_gpu():
    """Shape checks come first in hyp_stage_create, so they answer without a GPU: a vocabulary that is not a
    multiple of 8 (rows of the logits matrix would not start on 16-byte boundaries), an odd hidden size, a group
    size the attention kernels do not have."""
    def code(**kw):
        sh = inputs.tiny_shape()
        for k, v in kw.items():
            setattr(sh, k, v)
        with pytest.raises(hyp.HyperionError) as ei:
            hyp.hyp_stage_create(0, 1, hyp.make_cfg(sh, 1, 32, 32))
        return ei.value.code
    assert code(vocab=1001) == hyp.HYP_EINVAL and code(vocab=4) == hyp.HYP_EINVAL
    assert code(hidden=100) == hyp.HYP_EINVAL and code(n_q_heads=6) == hyp.HYP_EINVAL
    assert code(head_dim=96) == hyp.HYP_EINVAL and code(kv_block_size=32) == hyp.HYP_EINVAL
