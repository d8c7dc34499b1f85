"""The N > 1 path of the benchmark on CPU: two gloo ranks, no GPU.

With several GPUs every rank aggregates its own replica (the method's target is one GPU; there is no
data-path collective), so the only cross-rank logic is the timing reduction (max over ranks) and the
whole-job sum, plus the reference arm's rule that rank 0 alone works.  Also checked: sharding the
partitions of one tensor across ranks with `first_partition` / `partition_base` reproduces the
unsharded verification, which is what a partition-sharded deployment would rely on.
"""
import json
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import bench
    import oracle
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, "cpu")
    value = bench.whole_job_value(1e9, ms, world)
    # partition-sharded verification: rank r owns partitions r, r + world, ...
    rng = np.random.default_rng(0)                       # same tensor on every rank
    P, n, L = 4, 3, 40
    g = rng.standard_normal((P, n, L)).astype(np.float32)
    v = rng.standard_normal((P, L)).astype(np.float32)
    mine = list(range(rank, P, world))
    dots = np.zeros((P, n, 2))
    for p in mine:
        o = oracle.verify(g[p:p + 1], v[p:p + 1], 1.0, seed=9, K=2, first_partition=p)
        dots[p] = o["dot"][0]
    t = torch.from_numpy(dots)
    dist.all_reduce(t)                                   # gathering the scalars, as peers would broadcast them
    full = oracle.verify(g, v, 1.0, seed=9, K=2)["dot"]
    with open(os.path.join(out_dir, "rank%d.json" % rank), "w") as f:
        json.dump({"ms": ms, "value": value, "shard_ok": bool(np.array_equal(t.numpy(), full))}, f)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_time_as_max_and_sum_as_job(tmp_path):
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    res = [json.load(open(tmp_path / ("rank%d.json" % r))) for r in range(2)]
    for r in res:
        assert r["ms"] == 15.0                            # the slower rank decides
        assert abs(r["value"] - 2 * 1e9 / 15e-3 / 1e9) < 1e-9
        assert r["shard_ok"]


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--config", "1", "--steps", "1", "--warmup", "0"],
                         env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env["RANK"] = "0"
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--config", "1", "--steps", "2", "--warmup", "1"],
                         env=env, capture_output=True, text=True, timeout=120)
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0
