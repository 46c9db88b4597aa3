"""The N>1 benchmark path on CPU: two gloo ranks, each a replica with its own time; the aggregate uses
the slowest rank's time and the sum of the work."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_36800_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        my_ms = 10.0 + 5.0 * rank            # rank 1 is slower
        dist.barrier()
        total, ms, per_s = replicas.aggregate_throughput(1000.0, my_ms, dist)
        out[rank] = (total, ms, per_s)
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_two_replicas_report_sum_of_work_over_slowest_time():
    world = 2
    port = _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    for rank in range(world):
        total, ms, per_s = out[rank]
        assert total == 2000.0
        assert ms == 15.0
        assert per_s == pytest.approx(2000.0 / 0.015)
