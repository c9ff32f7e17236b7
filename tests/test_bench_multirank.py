"""The N > 1 path of the benchmark on CPU: two `gloo` ranks reduce their timings the way bench.py
does (max over ranks of the elapsed time, sum over ranks of the units processed).  The path itself
does not shard ("replicas only"), so this reduction is all there is to the multi-rank logic."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms, units = bench.reduce_over_ranks(10.0 + 5.0 * rank, 100.0 * (rank + 1), dist)
    dist.barrier()
    out.put((rank, ms, units))
    dist.destroy_process_group()


def test_reduce_over_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = [out.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for _, ms, units in results:
        assert ms == pytest.approx(15.0)       # the slower rank
        assert units == pytest.approx(300.0)   # both ranks' work


def test_single_rank_is_identity():
    import bench
    assert bench.reduce_over_ranks(3.0, 7.0, None) == (3.0, 7.0)


def test_reference_arm_runs_only_on_rank_zero(tmp_path):
    import subprocess
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
