"""N > 1 host logic on CPU: two gloo ranks shard a token batch, agree on coverage, and combine
their timings with a max-reduction (what `bench.py --gpus N` does over NCCL)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2310_08041_b200.shard import max_over_ranks, token_shard


def test_token_shard_partitions_rows():
    for M in (0, 1, 7, 64, 2048, 4097):
        for world in (1, 2, 3, 8):
            cover = []
            for r in range(world):
                s, n = token_shard(M, r, world)
                cover.extend(range(s, s + n))
            assert cover == list(range(M))
            sizes = [token_shard(M, r, world)[1] for r in range(world)]
            assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, M, out_q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    start, count = token_shard(M, rank, world)
    # each rank "processes" its rows: here, marks them
    mine = torch.zeros(M, dtype=torch.int32)
    mine[start:start + count] = rank + 1
    dist.all_reduce(mine, op=dist.ReduceOp.SUM)
    t = max_over_ranks(10.0 + rank)           # rank-dependent step time
    total = torch.tensor([count], dtype=torch.int64)
    dist.all_reduce(total)
    out_q.put((rank, mine.numpy().copy(), t, int(total.item())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_and_reduce():
    world, M = 2, 101
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, M, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, marks, t, total in res:
        assert t == 11.0                      # max over ranks, identical on every rank
        assert total == M
        s0, n0 = token_shard(M, 0, world)
        assert np.all(marks[:n0] == 1) and np.all(marks[n0:] == 2)   # every row owned exactly once


def test_bench_gpus_flag_starts_that_many_ranks():
    """`bench.py --gpus 2` with no rendezvous in the environment starts two ranks itself; rank 0 prints one line
    whose n_gpus is the world size and whose time is the slowest rank's.  (--stub: gloo and a stand-in step.)"""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--steps", "3", "--warmup", "1", "--stub"],
                       capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["config"]["parallelism"] == "tokens x2"
    assert d["ms_per_step"] >= 1.9                 # rank 1 sleeps 2 ms per step: the max, not rank 0's 1 ms
    # a world size that contradicts --gpus prints no line
    env2 = dict(env, WORLD_SIZE="1", RANK="0")
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "4", "--steps", "1", "--warmup", "1", "--stub"],
                       capture_output=True, text=True, timeout=120, env=env2)
    assert r.returncode != 0 and not [l for l in r.stdout.splitlines() if l.startswith("{")]


def test_traffic_record_is_tied_to_the_kernel_sources(tmp_path, monkeypatch):
    """bench.py takes roofline.traffic from a `traffic-record:` line of a profile summary only while the kernel's
    sources still hash to what the line recorded; a changed source, another workload or another M give None."""
    import hashlib
    import bench
    src_dir = tmp_path / "paper_2310_08041_b200" / "csrc"
    src_dir.mkdir(parents=True)
    (tmp_path / "profiles").mkdir()
    (src_dir / "k.cu").write_text("kernel v1\n")
    (src_dir / "h.cuh").write_text("header\n")
    sha = hashlib.sha256(b"kernel v1\n" + b"header\n").hexdigest()[:16]
    (tmp_path / "profiles" / "k.md").write_text(
        "# some kernel\n\ntraffic-record: kernel=k_kernel workload=w1 M=64 bytes=123456 sources=k.cu,h.cuh sha256=%s\n" % sha)
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    assert bench._traffic("k_kernel", "w1", 64) == 123456.0
    assert bench._traffic("k_kernel", "w1", 65) is None
    assert bench._traffic("k_kernel", "w2", 64) is None
    assert bench._traffic("other", "w1", 64) is None
    (src_dir / "k.cu").write_text("kernel v2\n")
    assert bench._traffic("k_kernel", "w1", 64) is None
    (src_dir / "k.cu").unlink()
    assert bench._traffic("k_kernel", "w1", 64) is None
