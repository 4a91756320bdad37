"""Pipeline of stages across ranks: headers, call schedule and the hand-off on CPU (gloo, 2 and 3 ranks)."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
from paper_2511_14450_b200 import pipeline as pl  # noqa: E402

H = 24


class ToyStage:
    """Stands in for a stage: keeps one running vector per sequence slot (as a KV cache keeps the past), so the
    result depends on every earlier call having reached this stage, in order.  Rank 0 maps token ids to rows."""

    def __init__(self, rank, world, n_slots=8):
        self.rank, self.first, self.last = rank, rank == 0, rank == world - 1
        self.in_width, self.out_width = H, (H + 3 if self.last else H)
        self.device = torch.device("cpu")
        self.state = torch.zeros(n_slots, H, dtype=torch.float64)
        self.log = []

    def out_rows(self, c):
        return len(c.slots) if (self.last and c.kind == pl.PREFILL) else c.rows

    def run(self, c, x, out):
        self.log.append((c.cid, c.kind, tuple(c.slots), tuple(c.q_lens), tuple(c.ctx_lens)))
        if self.first:
            x = (x.to(torch.float64).unsqueeze(1) * 0.001 + torch.arange(H, dtype=torch.float64) * 0.01)
        x = x.to(torch.float64)
        rows, r0 = [], 0
        for s, q in zip(c.slots, c.q_lens):
            seg = x[r0:r0 + q]
            self.state[s] += seg.sum(0)
            y = seg * (self.rank + 2) + self.state[s]
            rows.append(y[-1:] if (self.last and c.kind == pl.PREFILL) else y)
            r0 += q
        y = torch.cat(rows)
        if self.last:
            y = torch.cat([y, y[:, :3] * 0.5], dim=1)
        out.copy_(y.to(torch.float32))


def requests(n=5, n_out=4):
    g = torch.Generator().manual_seed(7)
    prompts = [torch.randint(0, 500, (int(torch.randint(3, 9, (1,), generator=g)),), generator=g, dtype=torch.int32)
               for _ in range(n)]
    forced = [torch.randint(0, 500, (n_out - (i % 2),), generator=g, dtype=torch.int32) for i in range(n)]
    return prompts, forced


def sequential(world, calls):
    stages = [ToyStage(r, world) for r in range(world)]
    results = {}
    for c in calls:
        x = c.ids
        for st in stages:
            out = torch.empty(st.out_rows(c), st.out_width, dtype=torch.float32)
            st.run(c, x, out)
            x = out
        results[c.cid] = x.clone()
    return results


def _worker(rank, world, port, path):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    stage = ToyStage(rank, world)
    pr = pl.PipelineRank(stage, rank, world, max_seqs=8, max_rows=64)
    got = {}
    if rank == 0:
        prompts, forced = requests()
        pr.feed(pl.schedule_calls(prompts, forced, group_size=2), lambda c, o: got.__setitem__(c.cid, o.clone()))
    else:
        pr.serve(lambda c, o: got.__setitem__(c.cid, o.clone()))
    torch.save({"got": got, "log": stage.log, "stats": pr.stats()}, f"{path}.{rank}")
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_pipeline_over_gloo_matches_sequential_composition(world, tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    path = str(tmp_path / "out")
    procs = [ctx.Process(target=_worker, args=(r, world, port, path)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=180)
        assert p.exitcode == 0
    prompts, forced = requests()
    calls = pl.schedule_calls(prompts, forced, group_size=2)
    want = sequential(world, calls)
    outs = [torch.load(f"{path}.{r}") for r in range(world)]
    got = outs[-1]["got"]
    assert sorted(got) == sorted(want) == list(range(len(calls)))
    for cid in want:
        assert torch.equal(got[cid], want[cid]), cid
    # every rank saw every call, in the order rank 0 issued them
    for r in range(world):
        assert [e[0] for e in outs[r]["log"]] == list(range(len(calls)))
        assert outs[r]["stats"]["calls"] == len(calls)
    # bytes handed on = rows x hidden x 4 for every call, from every rank but the last
    rows = sum(c.rows for c in calls)
    for r in range(world - 1):
        assert outs[r]["stats"]["sent_bytes"] == rows * H * 4
    assert outs[-1]["stats"]["sent_bytes"] == 0


def test_single_rank_pipe_returns_results_directly():
    prompts, forced = requests(3, 3)
    calls = pl.schedule_calls(prompts, forced, group_size=2)
    pr = pl.PipelineRank(ToyStage(0, 1), 0, 1, max_seqs=8, max_rows=64)
    got = {}
    pr.feed(calls, lambda c, o: got.__setitem__(c.cid, o.clone()))
    want = sequential(1, calls)
    assert all(torch.equal(got[k], want[k]) for k in want) and len(got) == len(calls)


def test_schedule_covers_every_token_once_and_in_order():
    prompts, forced = requests(5, 4)
    calls = pl.schedule_calls(prompts, forced, group_size=2)
    assert [c.cid for c in calls] == list(range(len(calls)))
    seen = {i: 0 for i in range(5)}          # tokens of the sequence that have been through the pipe
    for c in calls:
        for s, q, ctx in zip(c.slots, c.q_lens, c.ctx_lens):
            assert ctx == seen[s]
            seen[s] += q
        assert c.ids.numel() == c.rows and (c.kind == pl.PREFILL or all(q == 1 for q in c.q_lens))
    for i in range(5):
        assert seen[i] == prompts[i].numel() + forced[i].numel() - 1
    # decode calls carry the forced tokens in order
    for i in range(5):
        toks = [int(c.ids[c.slots.index(i)]) for c in calls if c.kind == pl.DECODE and i in c.slots]
        assert toks == forced[i][:-1].tolist()


def test_header_round_trip_and_limits():
    c = pl.Call(pl.DECODE, [3, 0, 5], [1, 1, 1], [17, 4, 99], cid=12)
    d = pl.decode_header(pl.encode_header(c, 8))
    assert (d.kind, d.slots, d.q_lens, d.ctx_lens, d.cid) == (c.kind, c.slots, c.q_lens, c.ctx_lens, 12)
    with pytest.raises(ValueError):
        pl.encode_header(pl.Call(pl.DECODE, list(range(9)), [1] * 9, [0] * 9), 8)
    h = pl.encode_header(c, 8)
    h[2] = 7
    with pytest.raises(ValueError):
        pl.decode_header(h)
    assert pl.decode_header(pl.encode_header(pl.Call(pl.STOP, [], [], []), 8)).kind == pl.STOP


def test_tier_latency_with_comm_term():
    f = [1.0, 2.0, 3.0, 4.0]
    worst, lat = pl.tier_latency_with_comm(f, [0, 2, 3, 4], [1.0, 2.0, 4.0], act_bytes=8e6, R=4e9)
    assert lat == [3.0 + 0.002, 1.5 + 0.002, 1.0] and worst == lat[0]


@pytest.mark.gpu
def test_one_rank_pipe_runs_the_library_stage():
    """The same calls through PipelineRank + LibraryStage and through a stage driven directly."""
    from paper_2511_14450_b200 import inputs
    from tests import helpers as Hh
    sh = inputs.tiny_shape()
    prompts = [inputs.token_ids(inputs.SEED_PROMPTS, 70 + i, 5 + i, sh.vocab) for i in range(3)]
    forced = [inputs.token_ids(inputs.SEED_FORCED, 70 + i, 4, sh.vocab) for i in range(3)]
    calls = pl.schedule_calls(prompts, forced, group_size=2)
    stage = pl.LibraryStage(sh, 0, sh.n_layers_total, 4, 64, 64)
    pr = pl.PipelineRank(stage, 0, 1, max_seqs=4, max_rows=64)
    got = {}
    pr.feed(calls, lambda c, o: got.__setitem__(c.cid, o.clone()))
    ref = Hh.gpu_stage(sh, 0, sh.n_layers_total, 4, 64, 64)
    try:
        for c in calls:
            out = torch.empty(stage.out_rows(c), sh.vocab, dtype=torch.float32, device="cuda")
            if c.kind == pl.PREFILL:
                ref.prefill(c.slots, c.q_lens, c.ctx_lens, c.ids.cuda(), out)
            else:
                ref.decode(c.slots, c.ctx_lens, c.ids.cuda(), out)
            torch.cuda.synchronize()
            assert got[c.cid].shape == out.shape
            assert torch.allclose(got[c.cid], out, rtol=0, atol=5e-3), c.cid
        assert pr.stats()["calls"] == len(calls)
    finally:
        ref.close()
        stage.close()
