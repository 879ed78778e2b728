"""The only cross-rank logic of a multi-GPU run (replicas only: no data-path
collective) is the timing reduction of bench.py: every rank must end up with
the slowest rank's device time, and the reported value is the work of all
replicas over that time.  Checked here with two gloo ranks on CPU."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = 10.0 + 5.0 * rank                 # rank 1 is the slow one
        got = bench.max_over_ranks(mine, world, torch.device("cpu"))
        dist.barrier()
        out[rank] = got
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_every_rank_gets_the_slowest_ranks_time():
    world = 2
    port = _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        assert dict(out) == {0: 15.0, 1: 15.0}


def test_single_rank_needs_no_process_group():
    assert bench.max_over_ranks(3.25, 1, torch.device("cpu")) == 3.25


def test_whole_job_value_counts_every_replica():
    # 2 replicas x 4 steps x 1e12 flops in 8 ms -> 1000 TFLOP/s
    assert bench.whole_job_value(1e12, 4, 2, 8.0) == pytest.approx(1000.0)
    assert bench.whole_job_value(1e12, 4, 1, 8.0) == pytest.approx(500.0)
