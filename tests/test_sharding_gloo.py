"""World-size-2 CPU (gloo) test of the multi-GPU host logic: env partition and max-over-ranks timing,
and that oracle actions do not depend on the partition."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import hts_workloads as wl
from paper_2012_09849_b200 import sharding


def test_env_ranges_tile_the_pool():
    for total in (0, 1, 7, 8192, 1000):
        for world in (1, 2, 3, 8):
            spans = [sharding.env_range(r, world, total) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == total
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import hts_oracle as orc
    cfg = wl.CONFIGS[1]
    pool = 6
    lo, hi = sharding.env_range(rank, world, pool)
    obs = wl.make_obs(cfg, pool)                               # same seeded pool on every rank
    wt = orc.Weights(wl.make_weights(cfg))
    ids = np.arange(lo, hi, dtype=np.int32)
    mine = orc.policy_step(wt, obs[lo:hi], ids, 5, seed=31)["actions"]
    gathered = [None] * world
    dist.all_gather_object(gathered, (lo, hi, mine.tolist()))
    slow = sharding.reduce_step_time_ms(10.0 + 5.0 * rank, dist)
    if rank == 0:
        full = orc.policy_step(wt, obs, np.arange(pool, dtype=np.int32), 5, seed=31)["actions"]
        merged = np.empty(pool, np.int32)
        for a, b, acts in gathered:
            merged[a:b] = acts
        out.put((bool(np.array_equal(merged, full)), slow))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_partition_actions_and_timing():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    same, slow = out.get(timeout=180)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert same, "actions changed with the partition"
    assert slow == 15.0


def test_bench_starts_its_own_ranks_with_disjoint_env_ranges():
    """`python bench.py --gpus 2` without a launcher starts two ranks itself; each takes its own range of global
    environment ids (checked with the dry-run switch, which stops before any GPU work)."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    env["MASTER_PORT"] = str(port)
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--dry-run-ranks"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    rows = [json.loads(line) for line in out.stdout.splitlines() if line.startswith("{")]
    assert sorted(r["rank"] for r in rows) == [0, 1] and all(r["world"] == 2 for r in rows)
    n = wl.CONFIGS[3].N
    spans = sorted((r["env_lo"], r["env_hi"]) for r in rows)
    assert spans == [(0, n), (n, 2 * n)]
