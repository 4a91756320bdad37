"""HypSched-RT routing requests over replicas of one pipeline stage (the paper's intra-tier parallelism).

A tier holds K_j nodes with the same blocks I_j(p*); an arriving task goes to the node that minimises
(F_rem + sum F_wait + F_new) / C among the available nodes with enough memory (Section IV-B, Algorithm 2).
Here every node is one `hyp_stage` replica with its own KV pool; all replicas live on one GPU and are
executed one call at a time, so each replica keeps a clock of its own that advances by the measured GPU time of
its calls divided by its relative capacity C_k (C_k < 1 emulates a slower node of the tier).  The routing
decision is `hyp_sched_rt` on the node states at the arrival's time; round-robin and seeded random routing
run on the same arrivals for comparison.

Work is counted as the paper does, in floating-point operations: a request of p prompt tokens and n output
tokens carries F = (p + n) * flops_per_token of the stage; its memory need is the KV pages of p + n tokens.

    python -m paper_2511_14450_b200.replicas --replicas 2 --capacity 1.0,0.5 --policy all

The data path of every call is the library's; this module only decides where a request runs.
"""
from __future__ import annotations

import argparse
import json
import os
import random
import sys
from dataclasses import dataclass, field
from typing import Callable, List, Optional, Sequence

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
from paper_2511_14450_b200 import hyperion as hyp  # noqa: E402


@dataclass
class Task:
    rid: int
    arrival: float            # seconds
    prompt_len: int
    n_out: int
    prompt: object = None     # int32 token ids (runner-specific container)
    forced: object = None
    node: int = -1
    slot: int = -1
    generated: int = 0
    t_first: Optional[float] = None
    t_done: Optional[float] = None


@dataclass
class Node:
    C: float                                  # relative capacity
    mem_cap: float                            # bytes of KV cache
    max_seqs: int
    clock: float = 0.0                        # this node's own time, seconds
    reserved: float = 0.0                     # bytes promised to routed tasks
    waiting: List[Task] = field(default_factory=list)
    running: List[Task] = field(default_factory=list)
    free_slots: List[int] = field(default_factory=list)
    busy_s: float = 0.0


class ReplicaRouter:
    """Discrete-event replay of arrivals over nodes whose service times come from `runner`.

    runner.prefill(k, tasks) and runner.decode(k, tasks) run the calls of node k and return their duration in
    seconds at capacity 1; runner.release(k, task) frees the task's cache.  flops_per_token and
    kv_bytes_per_token describe the stage."""

    def __init__(self, runner, capacities: Sequence[float], mem_caps: Sequence[float], max_seqs: int,
                 flops_per_token: float, kv_bytes_per_token: float, page_tokens: int = 16,
                 max_prefill_tokens: int = 4096):
        self.runner = runner
        self.nodes = [Node(C=float(c), mem_cap=float(m), max_seqs=max_seqs,
                           free_slots=list(range(max_seqs - 1, -1, -1))) for c, m in zip(capacities, mem_caps)]
        self.fpt, self.kvpt, self.page = float(flops_per_token), float(kv_bytes_per_token), page_tokens
        self.max_prefill_tokens = max_prefill_tokens
        self.decisions = []   # (rid, F_new, m_act, node states, chosen) per routed task

    # --- the paper's quantities -------------------------------------------------------------------
    def work(self, t: Task) -> float:
        return (t.prompt_len + t.n_out) * self.fpt

    def mem_need(self, t: Task) -> float:
        pages = -(-(t.prompt_len + t.n_out) // self.page)
        return pages * self.page * self.kvpt

    def node_state(self, nd: Node):
        """(C, M_avail, F_rem, sum F_wait, available): F_rem = work left in the tasks being served."""
        f_rem = sum((t.n_out - t.generated) * self.fpt for t in nd.running)
        f_wait = sum(self.work(t) for t in nd.waiting)
        available = len(nd.running) + len(nd.waiting) < nd.max_seqs
        return (nd.C, nd.mem_cap - nd.reserved, f_rem, f_wait, available)

    # --- one scheduling quantum of a node ---------------------------------------------------------------
    def _step(self, k: int) -> bool:
        nd = self.nodes[k]
        admit, rows = [], 0
        while nd.waiting and nd.waiting[0].arrival <= nd.clock and nd.free_slots:
            t = nd.waiting[0]
            if admit and rows + t.prompt_len > self.max_prefill_tokens:
                break
            nd.waiting.pop(0)
            t.slot = nd.free_slots.pop()
            admit.append(t)
            rows += t.prompt_len
        if admit:
            dt = self.runner.prefill(k, admit) / nd.C
            nd.clock += dt
            nd.busy_s += dt
            for t in admit:
                t.generated, t.t_first = 1, nd.clock
                if t.generated >= t.n_out:
                    self._finish(k, t)
                else:
                    nd.running.append(t)
            return True
        if nd.running:
            dt = self.runner.decode(k, nd.running) / nd.C
            nd.clock += dt
            nd.busy_s += dt
            for t in list(nd.running):
                t.generated += 1
                if t.generated >= t.n_out:
                    nd.running.remove(t)
                    self._finish(k, t)
            return True
        if nd.waiting:   # idle until the next routed task arrives
            nd.clock = max(nd.clock, nd.waiting[0].arrival)
            return True
        return False

    def _finish(self, k: int, t: Task):
        nd = self.nodes[k]
        t.t_done = nd.clock
        nd.reserved -= self.mem_need(t)
        nd.free_slots.append(t.slot)
        self.runner.release(k, t)
        t.slot = -1

    def _advance(self, k: int, until: float):
        nd = self.nodes[k]
        while nd.clock < until and (nd.running or (nd.waiting and nd.waiting[0].arrival <= until)):
            self._step(k)
        if not nd.running and not nd.waiting:
            nd.clock = max(nd.clock, until)

    # --- the replay -----------------------------------------------------------------------------------
    def run(self, tasks: Sequence[Task], policy: str = "hypsched", seed: int = 0,
            choose: Optional[Callable] = None):
        """policy: 'hypsched' (hyp_sched_rt), 'round_robin', 'random'; `choose(F_new, m_act, states)` overrides."""
        rng = random.Random(seed)
        rr = 0
        rejected = 0
        for t in sorted(tasks, key=lambda x: x.arrival):
            for k in range(len(self.nodes)):
                self._advance(k, t.arrival)
            states = [self.node_state(nd) for nd in self.nodes]
            F_new, m_act = self.work(t), self.mem_need(t)
            feasible = [k for k, s in enumerate(states) if s[4] and s[1] >= m_act]
            if choose is not None:
                k = choose(F_new, m_act, states)
            elif policy == "hypsched":
                try:
                    k = hyp.hyp_sched_rt(F_new, m_act, states)
                except hyp.HyperionError as e:
                    if e.code != hyp.HYP_EINFEASIBLE:
                        raise
                    k = -1
            elif policy == "round_robin":
                k = -1
                for i in range(len(self.nodes)):
                    if (rr + i) % len(self.nodes) in feasible:
                        k = (rr + i) % len(self.nodes)
                        rr = k + 1
                        break
            elif policy == "random":
                k = rng.choice(feasible) if feasible else -1
            else:
                raise ValueError(policy)
            self.decisions.append((t.rid, F_new, m_act, states, k))
            if k < 0:
                rejected += 1
                continue
            t.node = k
            nd = self.nodes[k]
            nd.reserved += m_act
            nd.waiting.append(t)
        for k in range(len(self.nodes)):
            while self._step(k):
                pass
        done = [t for t in tasks if t.t_done is not None]
        lat = sorted(t.t_done - t.arrival for t in done)
        ttft = sorted(t.t_first - t.arrival for t in done)
        makespan = max((nd.clock for nd in self.nodes), default=0.0)
        pct = lambda v, p: v[min(len(v) - 1, int(p * len(v)))] if v else None  # noqa: E731
        return {"policy": policy, "served": len(done), "rejected": rejected, "makespan_s": makespan,
                "output_tokens_per_s": sum(t.n_out for t in done) / makespan if makespan > 0 else 0.0,
                "latency_s": {"mean": sum(lat) / len(lat) if lat else None, "p50": pct(lat, 0.5), "p95": pct(lat, 0.95),
                              "max": lat[-1] if lat else None},
                "ttft_s": {"mean": sum(ttft) / len(ttft) if ttft else None, "max": ttft[-1] if ttft else None},
                "per_node": [{"C": nd.C, "tasks": sum(1 for t in done if t.node == k), "busy_s": nd.busy_s}
                             for k, nd in enumerate(self.nodes)]}


class StageRunner:
    """Replicas of one stage on the current GPU; durations from CUDA events around the library calls."""

    def __init__(self, shape, layer_lo: int, layer_hi: int, n_replicas: int, max_seqs: int, max_ctx: int,
                 max_tokens: int):
        import torch
        from paper_2511_14450_b200 import inputs
        self.torch = torch
        self.stages = []
        for _ in range(n_replicas):
            st = hyp.Stage(shape, layer_lo, layer_hi, max_seqs, max_ctx, max_tokens)
            for layer in range(layer_lo, layer_hi):
                st.load_layer(layer, inputs.layer_weights(shape, layer, device="cuda"))
            if st.first:
                st.load_embed(inputs.embed_weights(shape, device="cuda"))
            if st.last:
                st.load_head(*inputs.head_weights(shape, device="cuda"))
            self.stages.append(st)
        torch.cuda.synchronize()
        self.first = self.stages[0].first
        width = shape.vocab if self.stages[0].last else shape.hidden
        self.out = torch.empty(max(max_tokens, hyp.HYP_MAX_DECODE_BATCH), width, dtype=torch.float32, device="cuda")
        self.hidden_in = None if self.first else torch.zeros(max(max_tokens, hyp.HYP_MAX_DECODE_BATCH), shape.hidden,
                                                             dtype=torch.float32, device="cuda")
        self.e0, self.e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def _timed(self, fn) -> float:
        self.e0.record()
        fn()
        self.e1.record()
        self.e1.synchronize()
        return self.e0.elapsed_time(self.e1) * 1e-3

    def _rows(self, ids):
        return ids.cuda() if self.first else self.hidden_in[:ids.numel()]

    def prefill(self, k: int, tasks) -> float:
        torch = self.torch
        x = self._rows(torch.cat([t.prompt for t in tasks]))
        return self._timed(lambda: self.stages[k].prefill([t.slot for t in tasks], [t.prompt_len for t in tasks],
                                                          [0] * len(tasks), x, self.out))

    def decode(self, k: int, tasks) -> float:
        torch = self.torch
        total = 0.0
        for g0 in range(0, len(tasks), hyp.HYP_MAX_DECODE_BATCH):
            grp = tasks[g0:g0 + hyp.HYP_MAX_DECODE_BATCH]
            x = self._rows(torch.stack([t.forced[t.generated - 1] for t in grp]))
            ctx = [t.prompt_len + t.generated - 1 for t in grp]
            total += self._timed(lambda: self.stages[k].decode([t.slot for t in grp], ctx, x, self.out))
        return total

    def release(self, k: int, task):
        self.stages[k].free_seq(task.slot)

    def close(self):
        for st in self.stages:
            st.close()


def poisson_tasks(shape, n: int, rate: float, len_lo: int, len_hi: int, n_out: int, with_tokens: bool = True):
    """Seeded arrivals (exponential gaps of mean 1 / rate) with prompt lengths uniform in [len_lo, len_hi]."""
    from paper_2511_14450_b200 import inputs
    arr = inputs.poisson_arrivals(n, rate)
    lens = inputs.uniform_lengths(n, len_lo, len_hi)
    tasks = []
    for i in range(n):
        p = int(lens[i])
        t = Task(rid=i, arrival=float(arr[i]), prompt_len=p, n_out=n_out)
        if with_tokens:
            t.prompt = inputs.token_ids(inputs.SEED_PROMPTS, 1000 + i, p, shape.vocab)
            t.forced = inputs.token_ids(inputs.SEED_FORCED, 1000 + i, n_out, shape.vocab)
        tasks.append(t)
    return tasks


def main():
    import copy
    import torch
    from paper_2511_14450_b200 import inputs
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--replicas", type=int, default=2)
    ap.add_argument("--capacity", default="1.0,0.5", help="relative capacity C_k of every replica")
    ap.add_argument("--layers", type=int, default=14)
    ap.add_argument("--requests", type=int, default=32)
    ap.add_argument("--rate", type=float, default=8.0)
    ap.add_argument("--len-lo", type=int, default=128)
    ap.add_argument("--len-hi", type=int, default=1024)
    ap.add_argument("--n-out", type=int, default=64)
    ap.add_argument("--max-seqs", type=int, default=16)
    ap.add_argument("--policy", default="all", choices=["all", "hypsched", "round_robin", "random"])
    a = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("replicas: needs a CUDA device")
    caps = [float(c) for c in a.capacity.split(",")]
    if len(caps) != a.replicas:
        raise SystemExit("--capacity needs one value per replica")
    sh = inputs.phi3_medium_shape()
    max_ctx = a.len_hi + a.n_out + 16
    runner = StageRunner(sh, 0, a.layers, a.replicas, a.max_seqs, max_ctx, max_tokens=4096)
    kvpt = a.layers * 2 * sh.n_kv_heads * sh.head_dim * 2
    fpt = 2.0 * a.layers * sh.layer_linear_params
    mem = a.max_seqs * (-(-max_ctx // 16)) * 16 * kvpt
    base = poisson_tasks(sh, a.requests, a.rate, a.len_lo, a.len_hi, a.n_out)
    for pol in (["hypsched", "round_robin", "random"] if a.policy == "all" else [a.policy]):
        tasks = [copy.copy(t) for t in base]
        router = ReplicaRouter(runner, caps, [mem] * a.replicas, a.max_seqs, fpt, kvpt)
        res = router.run(tasks, pol)
        res["workload"] = (f"{a.replicas} replicas of a {a.layers}-block Phi-3-medium-shaped stage, capacities {caps}, "
                           f"{a.requests} requests, Poisson {a.rate}/s, prompts U[{a.len_lo},{a.len_hi}], {a.n_out} output tokens")
        print(json.dumps(res))
    runner.close()


if __name__ == "__main__":
    main()
