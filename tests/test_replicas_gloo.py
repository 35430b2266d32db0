"""Multi-rank bookkeeping of the benchmark, on CPU with the gloo backend (world size 2).

The path shards with no exchange: every rank runs its own replica of the workload on its own seeds, and
the only collectives are the two reductions that turn per-rank figures into whole-job figures (time =
max over ranks, work = sum over ranks). Checked here: those reductions, and that two ranks derive
different, reproducible inputs from the same workload description.
"""
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
    try:
        import bench
        from paper_2504_14051_b200 import workloads as wl

        # rank r took (10 + 5 r) ms for (1000 + r) units of work
        ms, units = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 1000.0 + rank, world, torch.device("cpu"))
        w = wl.scaled(wl.WORKLOADS["c1"], seed=wl.WORKLOADS["c1"].seed + 7919 * rank)
        q, _, _ = wl.step_inputs(w, "cpu", 0)
        q_again, _, _ = wl.step_inputs(w, "cpu", 0)
        gathered = [torch.zeros_like(q) for _ in range(world)]
        dist.all_gather(gathered, q)
        out[rank] = (ms, units, bool(torch.equal(q, q_again)), bool(torch.equal(gathered[0], gathered[1])))
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(300)
def test_two_replicas_aggregate_max_time_and_summed_work():
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in range(world):
        ms, units, reproducible, same_inputs = res[rank]
        assert ms == 15.0 and units == 2001.0  # max of (10, 15), sum of (1000, 1001), on every rank
        assert reproducible and not same_inputs


def test_single_rank_needs_no_process_group():
    import bench

    assert bench.aggregate_over_ranks(3.5, 7.0, 1, torch.device("cpu")) == (3.5, 7.0)


@pytest.mark.timeout(300)
def test_bench_gpus_flag_launches_that_many_ranks():
    """`bench.py --gpus 2` started as a plain process must become two ranks by itself (never print an N = 1 line
    for an N = 2 request). --dry-run keeps it on CPU: launcher, rendezvous and the two reductions are real, the
    per-rank figures are made up (rank r: 10 + 5 r ms, 1000 + r units)."""
    import json
    import subprocess

    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run"], env=env,
                         capture_output=True, text=True, timeout=280)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, res.stdout
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2 and out["ms_per_step"] == 15.0 and out["units"] == 2001.0
    # a world size that does not match the request is an error, not a silently smaller run
    env2 = dict(env, WORLD_SIZE="1", RANK="0", LOCAL_RANK="0")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run"], env=env2,
                         capture_output=True, text=True, timeout=120)
    assert res.returncode != 0 and "does not match" in res.stderr
