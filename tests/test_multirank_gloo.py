"""World-size-2 check (gloo, CPU) of the multi-rank plumbing of bench.py: ranks draw different
batches, the reported time is the maximum over ranks, and the value is the whole job's rate.
The hot path itself has no collective; this is all the communication there is."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2506_07366_b200 import workloads as wl
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = wl.WORKLOADS["tiny"]
        x = wl.activations(bench.rank_workload(w, rank), "cpu")
        # pretend rank r needed (r + 1) * 10 ms
        mine = 10.0 * (rank + 1)
        slowest = bench.max_over_ranks(mine, dist, "cpu")
        value = bench.whole_job_rate(world, w.T, 5, slowest)
        gathered = [torch.zeros_like(x, dtype=torch.float32) for _ in range(world)]
        dist.all_gather(gathered, x.float())
        distinct = not torch.equal(gathered[0], gathered[1])
        torch.save(dict(slowest=slowest, value=value, distinct=distinct), os.path.join(out_dir, f"r{rank}.pt"))
    finally:
        dist.destroy_process_group()


def test_two_ranks_report_the_slowest_rank_and_the_whole_job(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    res = [torch.load(tmp_path / f"r{r}.pt") for r in range(world)]
    for r in res:
        assert r["slowest"] == 20.0                         # max over ranks, on every rank
        assert r["value"] == pytest.approx(2 * 256 * 5 / 0.020)
        assert r["distinct"]                                # each rank has its own batch


def test_single_process_path_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None, "cpu") == 3.5
    assert bench.whole_job_rate(1, 4096, 20, 46.8) == pytest.approx(4096 * 20 / 0.0468)
