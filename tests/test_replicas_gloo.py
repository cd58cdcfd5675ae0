"""The multi-GPU path is N independent replicas; what crosses ranks is the timing aggregation.  Exercised here
with two CPU processes over gloo."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2604_10103_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms_local = 10.0 + 5.0 * rank          # rank 1 is the slow one
        units_local = 3.0 * (rank + 1)        # 3 and 6 latent frames
        dist.barrier()
        ms, units = replicas.aggregate(ms_local, units_local)
        out[rank] = (ms, units, replicas.throughput(units, ms), replicas.replica_seed(1234, rank))
    finally:
        dist.destroy_process_group()


def test_two_replicas_aggregate_max_time_and_sum_units():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for r in range(world):
        ms, units, thr, seed = res[r]
        assert ms == 15.0 and units == 9.0
        assert thr == pytest.approx(9.0 / 0.015)
    assert res[0][3] != res[1][3]


def test_single_process_is_identity():
    assert replicas.aggregate(2.5, 3.0) == (2.5, 3.0)
    assert replicas.throughput(6.0, 2000.0) == 3.0
