"""The N > 1 path is replicas only (no collective on the data path); what the ranks share -- the
slowest rank's time and the aggregate -- is checked here with two gloo ranks on the CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2601_13143_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 2.0 + rank            # rank 1 is the slow one
    slowest = replicas.max_over_ranks(ms, dist)
    dist.barrier()
    out[rank] = (slowest, replicas.aggregate_throughput(1000.0, slowest, world), list(replicas.split_sequences(5, world, rank)))
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_slowest_time_and_aggregate():
    world, port = 2, _free_port()
    with mp.Manager() as manager:
        out = manager.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        results = dict(out)
    assert results[0][0] == results[1][0] == 3.0
    assert abs(results[0][1] - 2 * 1000.0 / 3e-3) < 1e-6 and results[0][1] == results[1][1]
    assert results[0][2] + results[1][2] == [0, 1, 2, 3, 4]            # every sequence goes to exactly one replica


def test_single_process_is_identity():
    assert replicas.max_over_ranks(1.5) == 1.5
    assert list(replicas.split_sequences(3, 1, 0)) == [0, 1, 2]
