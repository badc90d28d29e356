"""The N > 1 bench path on CPU: two gloo ranks stand in for two GPUs.  The local update step has no
exchange between replicas, so what N > 1 adds is only: per-rank seeds, a max over ranks of the timed
region, and the whole-job rate; the reference arm runs on rank 0 alone."""
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
import lp_synth  # noqa: E402


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = [10.0 + 5.0 * rank, 30.0 - 7.0 * rank]           # rank 1 is slower on the first, faster on the second
        got = bench.max_over_ranks(mine, dist, torch.device("cpu"))
        cfg = bench.replica_config(lp_synth.config("c1"), rank)
        x, _ = lp_synth.minibatch(cfg, 0)
        sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(sums, torch.tensor([float(np.abs(x).sum())], dtype=torch.float64))
        out.put((rank, got, cfg["seed"], [float(s) for s in sums]))
    finally:
        dist.destroy_process_group()


def test_two_ranks_max_and_seeds():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, seed, sums in res:
        assert got == [15.0, 30.0]                               # both ranks hold the max over ranks
        assert seed == lp_synth.config("c1")["seed"] + rank
        assert sums[0] != sums[1]                                # the replicas really drew different minibatches


def test_whole_job_rate_is_aggregate():
    assert bench.whole_job_rate(1, 8192, 100.0) == 81920.0
    assert bench.whole_job_rate(8, 8192, 100.0) == 8 * 81920.0   # weak scaling: N replicas, same step time
    assert bench.max_over_ranks([1.5, 2.5], None, None) == [1.5, 2.5]


def test_reference_arm_other_ranks_exit_without_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1",
                        "--gpus", "2", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
