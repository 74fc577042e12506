"""world_size-2 gloo test of the rank plumbing used by bench.py (CPU only)."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2604_17397_b200 import dist_util


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist_util.barrier(world)
    m = dist_util.max_over_ranks(10.0 + 5.0 * rank, world)
    heads = list(dist_util.shard_heads(40, world, rank))
    q.put((rank, m, heads))
    dist_util.barrier(world)
    dist.destroy_process_group()


def test_two_rank_max_and_head_shards():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1] == res[1][1] == 15.0
    assert res[0][2] == list(range(0, 20)) and res[1][2] == list(range(20, 40))
    assert dist_util.aggregate_throughput(3.0, 1.5, 2) == pytest.approx(4000.0)


def test_single_rank_passthrough():
    assert dist_util.max_over_ranks(3.5, 1) == 3.5
    dist_util.barrier(1)
    with pytest.raises(ValueError):
        dist_util.shard_heads(12, 8, 0)


def test_bench_gpus_flag_spawns_that_many_ranks():
    # `bench.py --gpus 2` run without a launcher's environment must start two ranks itself; --plumbing-only makes
    # the ranks meet over gloo and report their places instead of touching a GPU
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--plumbing-only"],
                       capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                    # rank 0 alone prints
    line = lines[0]
    assert line["n_gpus"] == 2 and line["gpus_requested"] == 2
    assert [p["rank"] for p in line["places"]] == [0, 1]
    assert [p["local_rank"] for p in line["places"]] == [0, 1]
    assert line["places"][0]["pid"] != line["places"][1]["pid"]
    assert line["max_over_ranks"] == 2.0


def test_spawner_refuses_zero_ranks():
    with pytest.raises(ValueError):
        dist_util.spawn_ranks(0, ["x.py"])
