"""Several GPUs = independent replicas: the bookkeeping the ranks share (stream ownership, barrier,
slowest-rank time, whole-job rate), run as two gloo ranks on CPU; and the reference arm of
bench.py under a two-rank launch (rank 0 alone works and prints)."""
import json
import os
import socket
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2505_15380_b200 import replicas

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_every_stream_has_exactly_one_owner():
    for n, world in [(1, 1), (16, 2), (16, 8), (5, 4), (3, 8), (64, 3)]:
        shards = [replicas.shard_streams(n, world, r) for r in range(world)]
        assert sorted(sum(shards, [])) == list(range(n))
        assert max(map(len, shards)) - min(map(len, shards)) <= 1
    with pytest.raises(ValueError):
        replicas.shard_streams(4, 2, 2)


def test_single_rank_needs_no_process_group():
    cpu = torch.device("cpu")
    assert replicas.slowest([1.5, 2.5], 1, cpu) == [1.5, 2.5]
    assert replicas.total(7, 1, cpu) == 7
    assert replicas.job_rate(10, 500.0, 1, cpu) == pytest.approx(20.0)
    replicas.barrier(1)


def _rank_main(rank: int, world: int, port: int, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cpu = torch.device("cpu")
        assert replicas.env_world() == (world, rank, rank)
        replicas.barrier(world)
        mine = replicas.shard_streams(5, world, rank)
        # rank 1 is the slow one on the first timer, rank 0 on the second
        worst = replicas.slowest([10.0 + 5.0 * rank, 7.0 - rank], world, cpu)
        n_all = replicas.total(len(mine), world, cpu)
        rate = replicas.job_rate(100 * len(mine), 250.0 * (rank + 1), world, cpu)
        q.put((rank, mine, worst, n_all, rate))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_time_and_the_job_total():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, w0, n0, j0), (r1, s1, w1, n1, j1) = got
    assert (r0, r1) == (0, 1)
    assert s0 == [0, 2, 4] and s1 == [1, 3]
    assert w0 == w1 == [15.0, 7.0]                      # element-wise max over the ranks
    assert n0 == n1 == 5
    assert j0 == j1 == pytest.approx(500 / 0.5)         # all units over the slowest rank's 500 ms


def test_reference_arm_under_a_two_rank_launch_prints_one_line():
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()),
           os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "0", "--config", "0"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                               # rank 0 alone prints
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["n_gpus"] == 2 and out["value"] > 0
    assert out["cpu_baseline"]["kind"] == "oracle" and out["e2e"]["h2d_bytes_per_step"] == 0
