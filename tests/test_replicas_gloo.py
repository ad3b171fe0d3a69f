"""The N>1 path of the benchmark (independent replicas, max time over ranks, summed work) with two gloo ranks on CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2506_05096_b200 import replicas


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 + 5.0 * rank            # rank 1 is the slow one
    local_work = 100.0 * (rank + 1)
    ms, work = replicas.aggregate(local_ms, local_work)
    out[rank] = (ms, work, replicas.rank_seed(7, rank))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_summed_work():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][:2] == (15.0, 300.0) and res[1][:2] == (15.0, 300.0)
    assert res[0][2] != res[1][2]
    assert replicas.throughput(300.0, 15.0) == 300.0 / 0.015


def test_without_a_process_group_aggregate_is_the_identity():
    assert replicas.aggregate(3.0, 4.0) == (3.0, 4.0)
