"""The N > 1 path of the benchmark on CPU: two gloo ranks.  Every rank holds the same centroids, draws its own
query batch, and the whole-job throughput divides by the slowest rank's time."""
import os
import sys

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import argparse

    import bench
    args = argparse.Namespace(rows=2048, queries=64)
    w = bench.workload(args, rank, 1)
    digest = (int(w.centroids.astype(np.uint64).sum()), int(w.queries.astype(np.uint64).sum()))
    gathered = [None] * world
    dist.all_gather_object(gathered, digest)
    local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    slow = bench.max_over_ranks(local_ms, world)
    out[rank] = (gathered, slow, bench.whole_job_value(args.queries, world, slow))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_share_centroids_draw_own_queries_and_time_by_the_slowest():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.get_context("spawn").Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        gathered, slow, value = res[rank]
        assert gathered[0][0] == gathered[1][0]       # same centroid replica on every rank
        assert gathered[0][1] != gathered[1][1]       # different query batches
        assert slow == 15.0                           # max over ranks
        assert abs(value - 2 * 64 / 15e-3) < 1e-6     # whole-job queries per second


def test_reference_arm_runs_on_rank_zero_only(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import argparse

    import bench
    args = argparse.Namespace(rows=512, queries=16, steps=1, warmup=0, gpus=2)
    monkeypatch.setenv("RANK", "1")
    assert bench.run_reference(args) == 0 and capsys.readouterr().out == ""
    monkeypatch.setenv("RANK", "0")
    assert bench.run_reference(args) == 0
    line = capsys.readouterr().out.strip()
    import json
    d = json.loads(line)
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["n_gpus"] == 2
