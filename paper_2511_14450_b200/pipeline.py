"""One pipeline stage per process: tier j holds the blocks I_j(p*) and hands its activations to tier j + 1.

The paper's inter-tier split (Section III-C, Section IV-A): the model's blocks are cut into T contiguous
segments, tier j computes its segment and sends the [rows, hidden] activations on; the cost of that hand-off is
the communication term S_act / R of the per-tier latency, which the partitioning objective treats as a
constant.  Here a tier is one rank of a `torch.distributed` group (one process per GPU, backend nccl; gloo on
CPU for the tests), the hand-off is one point-to-point send / recv of a small int64 header and the fp32
payload into the receiver's own memory, and there is no collective on the data path.

Work is pushed through the pipe in calls ("micro-batches"): a prefill of some prompts or one decode step of
some sequences.  Output tokens are teacher-forced, so rank 0 knows every call in advance and can keep several
calls in flight; rank j works on call c while rank j - 1 works on call c + 1.

    torchrun --nproc-per-node 3 -m paper_2511_14450_b200.pipeline --requests 8 --n-out 32

Every step of the data path runs in the library (`hyp_stage_prefill` / `hyp_stage_decode`); this module moves
buffers between ranks and keeps the books.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import time
from dataclasses import dataclass
from typing import List, Optional, Sequence

import torch
import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

PREFILL, DECODE, STOP = 0, 1, 2
HEADER_FIXED = 4          # kind, n_seqs, rows, call id


@dataclass
class Call:
    kind: int                       # PREFILL or DECODE
    slots: List[int]
    q_lens: List[int]
    ctx_lens: List[int]
    ids: Optional[torch.Tensor] = None   # int32 token ids (rank 0 only)
    cid: int = 0

    @property
    def rows(self) -> int:
        return sum(self.q_lens)


def encode_header(c: Call, max_seqs: int) -> torch.Tensor:
    """Fixed-size int64 header: [kind, n_seqs, rows, call id, then (slot, q_len, ctx_len) per sequence]."""
    h = torch.zeros(HEADER_FIXED + 3 * max_seqs, dtype=torch.int64)
    n = len(c.slots)
    if n > max_seqs or not (len(c.q_lens) == len(c.ctx_lens) == n):
        raise ValueError("call does not fit the header")
    h[0], h[1], h[2], h[3] = c.kind, n, c.rows, c.cid
    for i in range(n):
        h[HEADER_FIXED + 3 * i: HEADER_FIXED + 3 * i + 3] = torch.tensor([c.slots[i], c.q_lens[i], c.ctx_lens[i]])
    return h


def decode_header(h: torch.Tensor) -> Call:
    kind, n, rows, cid = (int(v) for v in h[:HEADER_FIXED])
    body = h[HEADER_FIXED: HEADER_FIXED + 3 * n].view(n, 3).tolist() if n else []
    c = Call(kind, [b[0] for b in body], [b[1] for b in body], [b[2] for b in body], cid=cid)
    if kind != STOP and c.rows != rows:
        raise ValueError("corrupt hand-off header")
    return c


class LibraryStage:
    """The stage of this rank: blocks [lo, hi) of the model on the current CUDA device."""

    def __init__(self, shape, lo: int, hi: int, max_seqs: int, max_ctx: int, max_tokens: int):
        from paper_2511_14450_b200 import hyperion as hyp, inputs
        self.hyp = hyp
        self.st = hyp.Stage(shape, lo, hi, max_seqs, max_ctx, max_tokens)
        for layer in range(lo, hi):
            self.st.load_layer(layer, inputs.layer_weights(shape, layer, device="cuda"))
        if self.st.first:
            self.st.load_embed(inputs.embed_weights(shape, device="cuda"))
        if self.st.last:
            self.st.load_head(*inputs.head_weights(shape, device="cuda"))
        torch.cuda.synchronize()
        self.in_width = shape.hidden
        self.out_width = shape.vocab if self.st.last else shape.hidden
        self.device = torch.device("cuda")

    def out_rows(self, c: Call) -> int:
        # the last stage returns one logits row per sequence for a prefill, one per row for a decode step
        return len(c.slots) if (self.st.last and c.kind == PREFILL) else c.rows

    def run(self, c: Call, x: torch.Tensor, out: torch.Tensor):
        if c.kind == PREFILL:
            self.st.prefill(c.slots, c.q_lens, c.ctx_lens, x, out)
        else:
            self.st.decode(c.slots, c.ctx_lens, x, out)
        torch.cuda.synchronize()   # the payload is handed to the communication library next

    def release(self, slot: int):
        self.st.free_seq(slot)

    def close(self):
        self.st.close()


class PipelineRank:
    """Rank j of a T-rank pipe.  `stage` offers in_width, out_width, device, out_rows(call), run(call, x, out)."""

    def __init__(self, stage, rank: int, world: int, max_seqs: int, max_rows: int, group=None):
        self.stage, self.rank, self.world, self.group = stage, rank, world, group
        self.max_seqs = max_seqs
        dev = stage.device
        self.x = None if rank == 0 else torch.empty(max_rows, stage.in_width, dtype=torch.float32, device=dev)
        self.y = torch.empty(max_rows, stage.out_width, dtype=torch.float32, device=dev)
        self.header_dev = dev if dev.type == "cuda" else torch.device("cpu")
        self.sent_bytes = 0
        self.send_s = 0.0
        self.compute_s = 0.0
        self.calls = 0

    # --- hand-off -------------------------------------------------------------------------------------
    def _send(self, c: Call, payload: Optional[torch.Tensor]):
        t0 = time.perf_counter()
        dist.send(encode_header(c, self.max_seqs).to(self.header_dev), self.rank + 1, group=self.group)
        if payload is not None:
            dist.send(payload, self.rank + 1, group=self.group)
            self.sent_bytes += payload.numel() * payload.element_size()
        self.send_s += time.perf_counter() - t0

    def _recv(self):
        h = torch.empty(HEADER_FIXED + 3 * self.max_seqs, dtype=torch.int64, device=self.header_dev)
        dist.recv(h, self.rank - 1, group=self.group)
        c = decode_header(h.cpu())
        if c.kind == STOP:
            return c, None
        x = self.x[:c.rows]
        dist.recv(x, self.rank - 1, group=self.group)
        return c, x

    # --- one call on this rank -----------------------------------------------------------------------------
    def _work(self, c: Call, x: torch.Tensor):
        out = self.y[:self.stage.out_rows(c)]
        t0 = time.perf_counter()
        self.stage.run(c, x, out)
        self.compute_s += time.perf_counter() - t0
        self.calls += 1
        return out

    def feed(self, calls: Sequence[Call], on_result=None):
        """Rank 0: push the calls through the pipe, then the stop marker.  A one-rank pipe returns the results
        through on_result(call, out) directly."""
        assert self.rank == 0
        for c in calls:
            out = self._work(c, c.ids.to(self.stage.device))
            if self.world == 1:
                if on_result:
                    on_result(c, out)
            else:
                self._send(c, out)
        if self.world > 1:
            self._send(Call(STOP, [], [], []), None)

    def serve(self, on_result=None):
        """Ranks 1 .. T-1: receive, compute, pass on (the last rank hands results to on_result) until the stop
        marker arrives."""
        assert self.rank > 0
        last = self.rank == self.world - 1
        while True:
            c, x = self._recv()
            if c.kind == STOP:
                if not last:
                    self._send(c, None)
                return
            out = self._work(c, x)
            if last:
                if on_result:
                    on_result(c, out)
            else:
                self._send(c, out)

    def stats(self):
        return {"rank": self.rank, "calls": self.calls, "compute_s": self.compute_s, "send_s": self.send_s,
                "sent_bytes": self.sent_bytes,
                "send_gbs": self.sent_bytes / self.send_s / 1e9 if self.send_s > 0 else None}


def tier_latency_with_comm(f, boundaries, C, act_bytes: float, R: float):
    """Per-tier latency of a partition including the hand-off: sum of block costs / C_j + S_act / R for every
    tier that sends (Section III-C's latency with its communication term); returns (bottleneck, list)."""
    lat = []
    T = len(boundaries) - 1
    for j in range(T):
        t = sum(f[boundaries[j]:boundaries[j + 1]]) / C[j]
        if j < T - 1:
            t += act_bytes / R
        lat.append(t)
    return max(lat), lat


def schedule_calls(prompts: Sequence[torch.Tensor], forced: Sequence[torch.Tensor], group_size: int) -> List[Call]:
    """Calls for a set of teacher-forced requests: the requests are cut into groups of `group_size` sequences;
    every group is prefilled, then the groups' decode steps are interleaved round-robin, so that up to
    n_groups calls are in flight at once."""
    n = len(prompts)
    groups = [list(range(g, min(g + group_size, n))) for g in range(0, n, group_size)]
    calls, cid = [], 0
    for grp in groups:
        calls.append(Call(PREFILL, grp, [int(prompts[i].numel()) for i in grp], [0] * len(grp),
                          torch.cat([prompts[i] for i in grp]), cid))
        cid += 1
    steps = max(int(f.numel()) for f in forced) if n else 0
    for s in range(steps - 1):          # the prefill produced output 1; step s consumes forced token s
        for grp in groups:
            live = [i for i in grp if s < int(forced[i].numel()) - 1]
            if not live:
                continue
            calls.append(Call(DECODE, live, [1] * len(live), [int(prompts[i].numel()) + s for i in live],
                              torch.stack([forced[i][s] for i in live]), cid))
            cid += 1
    return calls


def main():
    from paper_2511_14450_b200 import hyperion as hyp, inputs
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--layers", type=int, default=40)
    ap.add_argument("--requests", type=int, default=8)
    ap.add_argument("--group", type=int, default=4, help="sequences per call")
    ap.add_argument("--prompt", type=int, default=512)
    ap.add_argument("--n-out", type=int, default=32)
    a = ap.parse_args()
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("pipeline: needs one CUDA device per rank")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    if world > 1:
        dist.init_process_group("nccl")
    sh = inputs.phi3_medium_shape(a.layers)
    f = [1.0] * a.layers                      # equal blocks: the profile of one GPU type (hyp_stage_profile) is flat
    m = [float(2 * sh.layer_linear_params)] * a.layers
    if world > 1:
        p, _ = hyp.hyp_split_dp(f, m, [1.0] * world, [150e9] * world)
        bounds = [0] + list(p) + [a.layers]
    else:
        bounds = [0, a.layers]
    max_ctx = a.prompt + a.n_out + 16
    stage = LibraryStage(sh, bounds[rank], bounds[rank + 1], a.requests, max_ctx, a.group * a.prompt)
    pr = PipelineRank(stage, rank, world, a.requests, a.group * a.prompt)
    done = {"rows": 0}

    def on_result(c, out):
        done["rows"] += out.shape[0]
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    if rank == 0:
        prompts = [inputs.token_ids(inputs.SEED_PROMPTS, 1000 + i, a.prompt, sh.vocab) for i in range(a.requests)]
        forced = [inputs.token_ids(inputs.SEED_FORCED, 1000 + i, a.n_out, sh.vocab) for i in range(a.requests)]
        pr.feed(schedule_calls(prompts, forced, a.group), on_result)
    else:
        pr.serve(on_result)
    if world > 1:
        dist.barrier()
    wall = time.perf_counter() - t0
    st = pr.stats()
    st.update({"blocks": [bounds[rank], bounds[rank + 1]], "wall_s": wall, "result_rows": done["rows"]})
    print(json.dumps(st), flush=True)
    stage.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
