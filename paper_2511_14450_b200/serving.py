"""Run a whole model as a chain of pipeline stages on one GPU with continuous batching.

The paper deploys tier j with blocks I_j(p*) and hands activations from tier to tier (Section IV); the
partition p* comes from HypSplit-DP fed with per-block cost vectors (Algorithm 1).  Here every stage is one
`hyp_stage` on the same GPU; a request's prompt is prefilled through all stages, then every decode step
sends the running batch's rows through stage 1 .. T in order (each generated token crosses every stage).
Each stage has its own CUDA stream; an event chains stage j+1 behind stage j.

Host-side scheduling only - every step of the data path is a library call.

    python -m paper_2511_14450_b200.serving --mode closed      # all requests at t = 0: throughput
    python -m paper_2511_14450_b200.serving --mode replay      # Poisson arrivals in real time: latency
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import time
from dataclasses import dataclass, field
from typing import List, Optional

import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
from paper_2511_14450_b200 import hyperion as hyp  # noqa: E402
from paper_2511_14450_b200 import inputs  # noqa: E402


@dataclass
class Request:
    rid: int
    arrival: float                      # seconds after the start of the run
    prompt: torch.Tensor                # int32 [prompt_len] (CPU)
    forced: torch.Tensor                # int32 [n_out]: teacher-forced output tokens (CPU)
    slot: int = -1
    generated: int = 0                  # logits rows produced so far (the prefill produces the first)
    t_first: Optional[float] = None
    t_done: Optional[float] = None
    last_logits: Optional[torch.Tensor] = None
    keep_logits: bool = False
    logits: List[torch.Tensor] = field(default_factory=list)


def plan_stages(shape, n_tiers: int, batch: int = 8, ctx: int = 1024, capacity=None, mem_cap=None, iters: int = 3):
    """Measure per-block cost on this GPU and split with HypSplit-DP.

    f_i = decode-step milliseconds of block i (batch, ctx) and m_i = its bytes, both from hyp_stage_profile on a
    stage that holds all blocks; C_j = relative speed of tier j (default all 1), M_j = memory limit of tier j
    (default: device memory / tiers).  Returns (boundaries [0, p_1, .., N], tau, f, m)."""
    N = shape.n_layers_total
    st = hyp.Stage(shape, 0, N, max_seqs=batch, max_ctx=ctx + 16, max_tokens=max(batch, 64))
    for layer in range(N):
        st.load_layer(layer, inputs.layer_weights(shape, layer, device="cuda"))
    st.load_embed(inputs.embed_weights(shape, device="cuda"))
    st.load_head(*inputs.head_weights(shape, device="cuda"))
    torch.cuda.synchronize()
    ms, nbytes = st.profile(1, batch, ctx, iters=iters)
    st.close()
    torch.cuda.empty_cache()
    C = list(capacity) if capacity is not None else [1.0] * n_tiers
    if mem_cap is None:
        total = torch.cuda.get_device_properties(0).total_memory
        mem_cap = [total / n_tiers] * n_tiers
    p, tau = hyp.hyp_split_dp(ms, [float(b) for b in nbytes], C, [float(v) for v in mem_cap])
    return [0] + list(p) + [N], tau, ms, nbytes


# Relative compute capacity and memory of the paper's three device tiers (its hardware table: 67 / 157 / 200 TOPS,
# 8 / 16 / 32 GB); the two- and four-tier rows extend the ladder the same way.
TIER_LADDERS = {2: ([67.0, 200.0], [8.0, 32.0]), 3: ([67.0, 157.0, 200.0], [8.0, 16.0, 32.0]),
                4: ([67.0, 157.0, 200.0, 275.0], [8.0, 16.0, 32.0, 64.0])}


def compare_splits(f, m, n_tiers: int, slack: float = 1.25):
    """HypSplit-DP beside the two comparison partitioners on the same per-block costs f (ms) and bytes m.

    Tiers follow TIER_LADDERS; the memory limits keep the ladder's ratios and sum to `slack` x the model's bytes,
    so that the small tier's limit can bind.  Returns one record per method: boundaries, bottleneck
    max_j L_j(p) (in units of f / capacity) and the bottleneck relative to HypSplit-DP's."""
    cap, mem = TIER_LADDERS[n_tiers]
    total = float(sum(m))
    limits = [slack * total * g / sum(mem) for g in mem]
    mb = [float(v) for v in m]
    N = len(f)
    out = {}
    p, tau = hyp.hyp_split_dp(f, mb, cap, limits)
    out["hypsplit_dp"] = {"boundaries": [0] + list(p) + [N], "bottleneck": tau, "fits_memory": True}
    try:
        pg, tg = hyp.hyp_split_greedy(f, mb, cap, limits)
        out["greedy_memory_aware"] = {"boundaries": [0] + list(pg) + [N], "bottleneck": tg, "fits_memory": True}
    except hyp.HyperionError:
        out["greedy_memory_aware"] = {"boundaries": None, "bottleneck": None, "fits_memory": False}
    pe, te, fits = hyp.hyp_split_even(f, mb, cap, limits)
    out["even_count"] = {"boundaries": [0] + list(pe) + [N], "bottleneck": te, "fits_memory": fits}
    for rec in out.values():
        rec["vs_hypsplit_dp"] = rec["bottleneck"] / tau if rec["bottleneck"] is not None else None
    return {"tiers": n_tiers, "capacity": cap, "memory_limits_bytes": limits, "methods": out}


class PipelineEngine:
    def __init__(self, shape, boundaries, max_seqs: int, max_ctx: int, max_tokens: int, random_gains: bool = False):
        assert boundaries[0] == 0 and boundaries[-1] == shape.n_layers_total
        self.shape = shape
        self.boundaries = list(boundaries)
        self.max_seqs, self.max_tokens = max_seqs, max_tokens
        self.stages: List[hyp.Stage] = []
        for lo, hi in zip(boundaries[:-1], boundaries[1:]):
            st = hyp.Stage(shape, lo, hi, max_seqs, max_ctx, max_tokens)
            for layer in range(lo, hi):
                st.load_layer(layer, inputs.layer_weights(shape, layer, device="cuda", random_gains=random_gains))
            if st.first:
                st.load_embed(inputs.embed_weights(shape, device="cuda"))
            if st.last:
                st.load_head(*inputs.head_weights(shape, device="cuda", random_gains=random_gains))
            self.stages.append(st)
        torch.cuda.synchronize()
        T = len(self.stages)
        self.streams = [torch.cuda.Stream() for _ in range(T)]
        self.events = [torch.cuda.Event() for _ in range(T)]
        rows = max(max_tokens, hyp.HYP_MAX_DECODE_BATCH)
        self.act = [torch.empty(rows, shape.hidden, dtype=torch.float32, device="cuda") for _ in range(T - 1)]
        self.logits = torch.empty(max(max_seqs, hyp.HYP_MAX_DECODE_BATCH), shape.vocab, dtype=torch.float32, device="cuda")
        self.free_slots = list(range(max_seqs - 1, -1, -1))

    def close(self):
        for st in self.stages:
            st.close()

    # one call through all stages; `ids` int32 device tensor with sum(q_lens) rows
    def _chain(self, decode: bool, slots, q_lens, ctx_lens, ids):
        x = ids
        self.streams[0].wait_event(self.events[-1])   # the previous pass has left the hand-off buffers
        for j, st in enumerate(self.stages):
            out = self.logits if st.last else self.act[j]
            with torch.cuda.stream(self.streams[j]):
                if j > 0:
                    self.streams[j].wait_event(self.events[j - 1])
                if decode:
                    st.decode(slots, ctx_lens, x, out, stream=self.streams[j])
                else:
                    st.prefill(slots, q_lens, ctx_lens, x, out, stream=self.streams[j])
                self.events[j].record(self.streams[j])
            x = out
        return self.logits

    def _prefill(self, reqs: List[Request]):
        """Prompts of `reqs` through all stages, in calls of at most max_tokens rows (whole prompts per call;
        a prompt longer than max_tokens is chunked on its own)."""
        group, rows = [], 0
        for r in reqs + [None]:
            plen = int(r.prompt.numel()) if r is not None else 0
            if r is None or (group and rows + plen > self.max_tokens):
                if group:
                    ids = torch.cat([g.prompt for g in group]).cuda(non_blocking=True)
                    self.streams[0].wait_stream(torch.cuda.current_stream())
                    lg = self._chain(False, [g.slot for g in group], [int(g.prompt.numel()) for g in group],
                                     [0] * len(group), ids)
                    self.streams[-1].synchronize()
                    for i, g in enumerate(group):
                        g.generated = 1
                        self._take_logits(g, lg[i])
                group, rows = [], 0
            if r is None:
                break
            if plen > self.max_tokens:          # a single long prompt: chunked prefill
                done = 0
                while done < plen:
                    n = min(self.max_tokens, plen - done)
                    ids = r.prompt[done:done + n].cuda(non_blocking=True)
                    self.streams[0].wait_stream(torch.cuda.current_stream())
                    lg = self._chain(False, [r.slot], [n], [done], ids)
                    done += n
                self.streams[-1].synchronize()
                r.generated = 1
                self._take_logits(r, lg[0])
            else:
                group.append(r)
                rows += plen

    def _take_logits(self, r: Request, row: torch.Tensor):
        if r.keep_logits:
            r.logits.append(row.detach().cpu().clone())

    def run(self, requests: List[Request], realtime: bool):
        """Serve `requests`.  realtime: honour arrival times (sleeping while idle); otherwise everything is
        admitted as soon as a slot is free (closed loop).  Returns a dict of statistics."""
        waiting = sorted(requests, key=lambda r: r.arrival)
        running: List[Request] = []
        t0 = time.perf_counter()
        steps = decode_rows = 0
        prefill_tokens = 0
        while waiting or running:
            now = time.perf_counter() - t0
            admit = []
            while waiting and self.free_slots and (not realtime or waiting[0].arrival <= now):
                r = waiting.pop(0)
                r.slot = self.free_slots.pop()
                admit.append(r)
            if admit:
                self._prefill(admit)
                t = time.perf_counter() - t0
                for r in admit:
                    r.t_first = t
                    prefill_tokens += int(r.prompt.numel())
                    if r.generated >= int(r.forced.numel()):
                        self._finish(r, t)
                    else:
                        running.append(r)
            if not running:
                if waiting and realtime:
                    time.sleep(max(0.0, waiting[0].arrival - (time.perf_counter() - t0)))
                continue
            # one decode step for the whole running batch (in groups of at most 32 rows)
            finishing = False
            for g0 in range(0, len(running), hyp.HYP_MAX_DECODE_BATCH):
                grp = running[g0:g0 + hyp.HYP_MAX_DECODE_BATCH]
                tok = torch.stack([r.forced[r.generated - 1] for r in grp]).cuda(non_blocking=True)
                self.streams[0].wait_stream(torch.cuda.current_stream())
                ctx = [int(r.prompt.numel()) + r.generated - 1 for r in grp]
                lg = self._chain(True, [r.slot for r in grp], None, ctx, tok)
                for i, r in enumerate(grp):
                    r.generated += 1
                    if r.keep_logits:
                        self.streams[-1].synchronize()
                        self._take_logits(r, lg[i])
                    finishing |= r.generated >= int(r.forced.numel())
                decode_rows += len(grp)
            steps += 1
            if finishing or (realtime and waiting):
                self.streams[-1].synchronize()      # completion / admission times need the GPU's clock
                t = time.perf_counter() - t0
                for r in [r for r in running if r.generated >= int(r.forced.numel())]:
                    running.remove(r)
                    self._finish(r, t)
        torch.cuda.synchronize()
        makespan = time.perf_counter() - t0
        out_tokens = sum(int(r.forced.numel()) for r in requests)
        ttft = sorted(r.t_first - (r.arrival if realtime else 0.0) for r in requests)
        lat = sorted(r.t_done - (r.arrival if realtime else 0.0) for r in requests)
        return {"requests": len(requests), "output_tokens": out_tokens, "prefill_tokens": prefill_tokens,
                "makespan_s": makespan, "output_tokens_per_s": out_tokens / makespan, "decode_steps": steps,
                "mean_decode_batch": decode_rows / max(steps, 1),
                "ttft_s": {"mean": sum(ttft) / len(ttft), "p50": ttft[len(ttft) // 2], "max": ttft[-1]},
                "latency_s": {"mean": sum(lat) / len(lat), "p50": lat[len(lat) // 2], "max": lat[-1]}}

    def _finish(self, r: Request, t: float):
        r.t_done = t
        for st in self.stages:
            st.free_seq(r.slot)
        self.free_slots.append(r.slot)
        r.slot = -1


def synthetic_requests(shape, n: int, rate: float, len_lo: int, len_hi: int, n_out: int, keep_logits=False):
    """Seeded workload: Poisson arrivals at `rate` per second, prompt lengths uniform in [len_lo, len_hi],
    `n_out` teacher-forced output tokens each."""
    arr = inputs.poisson_arrivals(n, rate)
    lens = inputs.uniform_lengths(n, len_lo, len_hi)
    return [Request(i, float(arr[i]), inputs.token_ids(inputs.SEED_PROMPTS, 1000 + i, int(lens[i]), shape.vocab),
                    inputs.token_ids(inputs.SEED_FORCED, 1000 + i, n_out, shape.vocab), keep_logits=keep_logits)
            for i in range(n)]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--mode", choices=["closed", "replay", "compare-splits"], default="closed")
    ap.add_argument("--shape", choices=["phi3", "llama3"], default="phi3")
    ap.add_argument("--requests", type=int, default=32)
    ap.add_argument("--rate", type=float, default=4.0)
    ap.add_argument("--len-lo", type=int, default=128)
    ap.add_argument("--len-hi", type=int, default=1024)
    ap.add_argument("--n-out", type=int, default=256)
    ap.add_argument("--tiers", type=int, default=3)
    ap.add_argument("--layers", type=int, default=40)
    a = ap.parse_args()
    if a.mode == "compare-splits":
        # measured per-block decode cost of the whole model, then the three partitioners on 2, 3 and 4 tiers
        shape = inputs.llama3_8b_shape() if a.shape == "llama3" else inputs.phi3_medium_shape()
        _, _, ms, nbytes = plan_stages(shape, 1)
        print(json.dumps({"shape": a.shape, "blocks": shape.n_layers_total, "block_ms_min_max": [min(ms), max(ms)],
                          "splits": [compare_splits(ms, nbytes, t) for t in (2, 3, 4)]}))
        return
    print(json.dumps(run_workload(a.mode == "replay", a.requests, a.rate, a.len_lo, a.len_hi, a.n_out, a.tiers, a.layers)))


def run_workload(realtime: bool, requests: int = 32, rate: float = 4.0, len_lo: int = 128, len_hi: int = 1024,
                 n_out: int = 256, tiers: int = 3, layers: int = 40) -> dict:
    """The serving configuration end to end: profile the blocks, split them with HypSplit-DP, build one stage per
    tier and serve the seeded request set (in real time, or closed-loop with everything admitted at once)."""
    shape = inputs.phi3_medium_shape(layers)
    bounds, tau, ms, nbytes = plan_stages(shape, tiers)
    eng = PipelineEngine(shape, bounds, max_seqs=requests, max_ctx=len_hi + n_out + 16, max_tokens=2048)
    reqs = synthetic_requests(shape, requests, rate, len_lo, len_hi, n_out)
    stats = eng.run(reqs, realtime=realtime)
    eng.close()
    stats.update({"mode": "replay" if realtime else "closed", "stage_boundaries": bounds, "split_bottleneck_ms": tau,
                  "block_ms_min_max": [min(ms), max(ms)], "offered_tokens_per_s": rate * n_out,
                  "workload": f"configs[3]: {layers} Phi-3-medium-shaped blocks as {tiers} stages, {requests} requests, "
                              f"Poisson {rate}/s, prompts U[{len_lo},{len_hi}], {n_out} forced output tokens"})
    return stats


def run_closed_loop() -> dict:
    """configs[3] with all 32 requests admitted at t = 0: output tokens per second of the three-stage engine."""
    return run_workload(False)


if __name__ == "__main__":
    main()
