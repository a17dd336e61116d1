"""Multi-rank bookkeeping of the benchmark (replicas, max-over-ranks timing) with two gloo ranks on
CPU."""
import os

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2602_02071_b200 import replicas


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert replicas.dist_env() == (rank, world, rank)
        ms = 1.0 + rank                      # rank 1 is the slow one
        dist.barrier()
        mx = replicas.max_over_ranks(ms)
        rate = replicas.whole_job_rate(10.0, mx, world)
        out[rank] = (mx, rate)
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank():
    mgr = mp.Manager()
    out = mgr.dict()
    port = 29500 + (os.getpid() % 2000)
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    assert out[0] == out[1]
    mx, rate = out[0]
    assert mx == 2.0
    assert rate == pytest.approx(2 * 10.0 / 2.0e-3)


def test_single_process_is_identity():
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.whole_job_rate(4.0, 2.0, 1) == pytest.approx(2000.0)
