"""World-size-2 check (gloo, CPU) of the benchmark's multi-rank plumbing: ranks get different
sequences of the same shape, the step time is the maximum over ranks on every rank, and the job
rate counts every rank's work."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2506_11498_b200 import replicas, workloads


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert replicas.env_rank_world() == (rank, world, rank)
        base = workloads.Workload("r", 1, 2, 1, 64, 64, 16, 4, 2, seed=7)
        w = replicas.rank_workload(base, rank)
        k = workloads.generate(w, ("K",))["K"]
        mine = 10.0 + 5.0 * rank                    # rank 1 is the slow one
        slowest = replicas.max_over_ranks(mine, dist)
        gathered = [torch.zeros_like(k, dtype=torch.float32) for _ in range(world)]
        dist.all_gather(gathered, k.float())
        out[rank] = (w.seed, slowest, bool(torch.equal(gathered[0], gathered[1])), w.N, w.d)
    finally:
        dist.destroy_process_group()


def test_two_ranks_are_independent_replicas_timed_by_the_slowest():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == 7 and res[1][0] == 1007
    assert res[0][1] == res[1][1] == 15.0
    assert res[0][2] is False and res[1][2] is False      # different data on the two ranks
    assert res[0][3:] == res[1][3:]                        # same shape
    assert replicas.job_rate(3.0, world, 15.0) == 2 * 3.0 / 15.0


def test_single_process_defaults():
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    assert replicas.env_rank_world() == (0, 1, 0)
    assert replicas.max_over_ranks(2.5) == 2.5
    w = workloads.CFG1
    assert replicas.rank_workload(w, 0) == w
