"""Host-side logic of `bench.py --gpus N` on CPU with two gloo ranks.

The path shards with no exchange: every rank generates and processes its own synthetic shard, the
only communication is the barrier and the MAX of the per-rank times, and rank 0 alone reports.
"""
import hashlib
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2603_15619_b200 import synthetic
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = synthetic.WORKLOADS["c1"]
        x = synthetic.tensor(w, "Q", bench.shard_seed(rank), 0, "cpu")
        digest = hashlib.sha1(x.view(torch.int16).numpy().tobytes()).hexdigest()
        digests = [None] * world
        dist.all_gather_object(digests, digest)
        dist.barrier()
        my_ms = 2.0 + 3.0 * rank                       # rank 1 is the slow shard
        ms = bench.max_over_ranks(my_ms, world, torch.device("cpu"))
        value = bench.job_value(world, 1e12, ms)
        q.put((rank, digests, ms, value))
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_distinct_shards_and_the_slowest_time():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, digests, ms, value in got:
        assert len(set(digests)) == world, "ranks must generate different shards"
        assert ms == 5.0, "every rank must see the slowest rank's time"
        assert abs(value - world * 1e12 / 5e-3 / 1e12) < 1e-9   # whole-job throughput = all ranks' work / that time
    assert got[0][1] == got[1][1]


def test_reference_arm_prints_on_rank_zero_only():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1", "--gpus", "2",
           "--steps", "1", "--warmup", "0"]
    outs = []
    for rank in (0, 1):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1")
        r = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300, cwd=ROOT)
        assert r.returncode == 0, r.stderr[-400:]
        outs.append(r.stdout.strip())
    line = json.loads(outs[0].splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["gpu_launches"] == 0
    assert outs[1] == "", "ranks other than 0 print nothing"


def test_gpus_flag_outside_a_launcher_spawns_the_ranks_itself():
    # `python bench.py --gpus 2` with no WORLD_SIZE in the environment must mean two ranks, not one: the script
    # starts them on 127.0.0.1 and rank 0 alone prints the line (the oracle arm runs without a GPU).
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1", "--gpus", "2",
           "--steps", "1", "--warmup", "0"]
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_PORT")}
    r = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-400:]
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1, lines
    assert json.loads(lines[0])["n_gpus"] == 2
