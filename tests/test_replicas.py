"""HypSched-RT routing over stage replicas: host logic on a deterministic service-time model (no GPU)."""
import copy

import pytest

from oracle import split as osplit
from paper_2511_14450_b200 import hyperion as hyp
from paper_2511_14450_b200 import inputs, replicas


class ModelRunner:
    """Service times of a node at capacity 1: prefill a_p seconds per prompt token, a decode step a_d seconds
    whatever the batch (weight streaming dominates a step)."""

    def __init__(self, a_p=2e-5, a_d=2e-3):
        self.a_p, self.a_d = a_p, a_d
        self.calls = []
        self.released = []

    def prefill(self, k, tasks):
        self.calls.append(("p", k, tuple(t.rid for t in tasks)))
        assert len({t.slot for t in tasks}) == len(tasks) and all(t.slot >= 0 for t in tasks)
        return self.a_p * sum(t.prompt_len for t in tasks)

    def decode(self, k, tasks):
        self.calls.append(("d", k, tuple(t.rid for t in tasks)))
        return self.a_d

    def release(self, k, task):
        self.released.append((k, task.rid))


def make_router(caps, max_seqs=8, mem_tasks=8.0, runner=None):
    sh = inputs.tiny_shape()
    runner = runner or ModelRunner()
    kvpt, fpt = 1024.0, 1.0e6
    mem = mem_tasks * 1200 * kvpt   # room for about mem_tasks of the largest requests
    return replicas.ReplicaRouter(runner, caps, [mem] * len(caps), max_seqs, fpt, kvpt), runner, sh


def tasks_for(sh, n=40, rate=20.0):
    return replicas.poisson_tasks(sh, n, rate, 128, 1024, 48, with_tokens=False)


def test_every_decision_is_the_arg_min_of_the_paper():
    router, _, sh = make_router([1.0, 0.5, 0.25])
    res = router.run(tasks_for(sh), "hypsched")
    assert res["served"] == 40 and res["rejected"] == 0
    assert len(router.decisions) == 40
    for rid, F_new, m_act, states, k in router.decisions:
        nodes = [{"C": s[0], "M_avail": s[1], "F_rem": s[2], "F_wait": [s[3]], "available": s[4]} for s in states]
        assert k == osplit.sched_rt_argmin(F_new, m_act, nodes) == osplit.hypsched_rt_scan(F_new, m_act, nodes), rid


def test_all_tasks_finish_memory_and_slots_are_returned():
    router, runner, sh = make_router([1.0, 0.5])
    tasks = tasks_for(sh)
    res = router.run(tasks, "hypsched")
    assert res["served"] == len(tasks)
    assert sorted(r for _, r in runner.released) == list(range(len(tasks)))
    for nd in router.nodes:
        assert abs(nd.reserved) < 1e-6 and sorted(nd.free_slots) == list(range(nd.max_seqs))
        assert not nd.running and not nd.waiting
    for t in tasks:
        assert t.generated == t.n_out and t.arrival <= t.t_first <= t.t_done
    # a node never serves more sequences at once than it has slots
    for kind, k, rids in runner.calls:
        assert len(rids) <= router.nodes[k].max_seqs


def test_memory_limit_rejects_or_diverts():
    # node 0 is the fastest but holds one request at a time: the second arrival must go elsewhere or be refused
    router, _, sh = make_router([1.0, 0.1], mem_tasks=1.0)
    tasks = tasks_for(sh, n=6, rate=200.0)
    res = router.run(tasks, "hypsched")
    for rid, F_new, m_act, states, k in router.decisions:
        if k >= 0:
            assert states[k][1] >= m_act and states[k][4]
        else:
            assert all((not s[4]) or s[1] < m_act for s in states)
    assert res["served"] + res["rejected"] == 6


def test_hypsched_beats_blind_policies_on_unequal_nodes():
    sh = inputs.tiny_shape()
    base = tasks_for(sh, n=60, rate=30.0)
    out = {}
    for pol in ("hypsched", "round_robin", "random"):
        router, _, _ = make_router([1.0, 0.25], max_seqs=64, mem_tasks=64.0)   # room for everything: nobody is refused
        out[pol] = router.run([copy.copy(t) for t in base], pol, seed=1)
        assert out[pol]["served"] == 60
    assert out["hypsched"]["latency_s"]["mean"] < out["round_robin"]["latency_s"]["mean"]
    assert out["hypsched"]["latency_s"]["mean"] < out["random"]["latency_s"]["mean"]
    # the faster node takes the larger share
    per = out["hypsched"]["per_node"]
    assert per[0]["tasks"] > per[1]["tasks"]


def test_equal_nodes_split_evenly_and_replay_is_deterministic():
    sh = inputs.tiny_shape()
    base = tasks_for(sh, n=30, rate=10.0)
    runs = []
    for _ in range(2):
        router, _, _ = make_router([1.0, 1.0])
        runs.append(router.run([copy.copy(t) for t in base], "hypsched"))
    assert runs[0] == runs[1]
    a, b = (n["tasks"] for n in runs[0]["per_node"])
    assert abs(a - b) <= 6


def test_unknown_policy():
    router, _, sh = make_router([1.0])
    with pytest.raises(ValueError):
        router.run(tasks_for(sh, n=2), "fastest")


@pytest.mark.gpu
def test_replicas_of_a_real_stage_serve_every_request():
    """Two replicas of a small stage on the GPU, routed by hyp_sched_rt on measured call times."""
    sh = inputs.tiny_shape()
    runner = replicas.StageRunner(sh, 0, sh.n_layers_total, 2, max_seqs=4, max_ctx=160, max_tokens=512)
    try:
        kvpt = sh.n_layers_total * 2 * sh.n_kv_heads * sh.head_dim * 2
        fpt = 2.0 * sh.n_layers_total * sh.layer_linear_params
        mem = 4 * 160 * kvpt
        tasks = replicas.poisson_tasks(sh, 10, 2000.0, 16, 96, 12)
        router = replicas.ReplicaRouter(runner, [1.0, 0.5], [mem, mem], 4, fpt, kvpt, max_prefill_tokens=512)
        res = router.run(tasks, "hypsched")
        assert res["served"] + res["rejected"] == 10 and res["served"] >= 8
        assert sum(n["tasks"] for n in res["per_node"]) == res["served"]
        assert res["per_node"][0]["busy_s"] > 0     # which node serves how many depends on the measured times
        for rid, F_new, m_act, states, k in router.decisions:
            assert k < 0 or (states[k][4] and states[k][1] >= m_act)
        assert all(t.t_done is None or t.t_done >= t.t_first >= t.arrival for t in tasks)
        for st in runner.stages:
            assert all(hyp.hyp_stage_seq_len(st.handle, s) == 0 for s in range(4))
    finally:
        runner.close()
