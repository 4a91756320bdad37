"""The benchmark's multi-rank bookkeeping on CPU: two gloo ranks, slowest rank's time, summed units."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, units = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 64.0 * (rank + 1), dist, "cpu")
    q.put((rank, ms, units))
    dist.barrier()
    dist.destroy_process_group()


def test_aggregate_takes_max_time_and_sums_units_over_two_ranks():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [(0, 15.0, 192.0), (1, 15.0, 192.0)]


def test_aggregate_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(3.5, 8.0) == (3.5, 8.0)


def test_bench_starts_its_own_ranks_when_no_launcher_is_around():
    """`python bench.py --gpus 2` outside any launcher: the script re-launches itself as two ranks (here gloo ranks
    with the GPU work replaced by the stand-in) and rank 0 prints one line for the whole job."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env["HYP_BENCH_STAND_IN"] = "1"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "6", "--warmup", "1"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["stand_in"] is True and d["steps"] == 6
    # rank 1 sleeps twice as long per step as rank 0: the job's time is rank 1's, the tokens are both ranks'
    assert d["ms_per_step"] >= 2.0 and abs(d["value"] - 2 * 8 * 6 / (d["ms_per_step"] * 6 / 1e3)) < 1e-6 * d["value"]


def test_traffic_figure_is_dropped_when_the_kernel_source_changed(tmp_path, monkeypatch):
    sys.path.insert(0, ROOT)
    import bench
    import hashlib
    src = os.path.join(ROOT, "paper_2511_14450_b200", "csrc", "gemm_stream.cu")
    sha = hashlib.sha256(open(src, "rb").read()).hexdigest()[:16]
    prof = tmp_path / "profiles"
    prof.mkdir()
    (prof / "a.md").write_text(f"traffic_bytes_per_launch: 371200000\nkernel_source: gemm_stream.cu sha256/16 {sha}\n")
    (prof / "b.md").write_text("traffic_bytes_per_launch: 1\nkernel_source: gemm_stream.cu sha256/16 0123456789abcdef\n")
    real_join = os.path.join
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    os.makedirs(real_join(str(tmp_path), "paper_2511_14450_b200", "csrc"))
    with open(real_join(str(tmp_path), "paper_2511_14450_b200", "csrc", "gemm_stream.cu"), "wb") as fh:
        fh.write(open(src, "rb").read())
    assert bench.measured_traffic("a.md") == 371200000.0
    assert bench.measured_traffic("b.md") is None and bench.measured_traffic("missing.md") is None
