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


def test_tenant_shards_are_an_even_contiguous_cut():
    for B, world in ((8, 2), (7, 3), (2, 4), (0, 3), (33, 8)):
        cuts = [replicas.shard_tenants(B, world, r) for r in range(world)]
        assert cuts[0][0] == 0 and sum(c for _, c in cuts) == B
        for (s0, c0), (s1, _) in zip(cuts, cuts[1:]):
            assert s0 + c0 == s1
        assert max(c for _, c in cuts) - min(c for _, c in cuts) <= 1
    with pytest.raises(ValueError):
        replicas.shard_tenants(4, 2, 2)


def _shard_worker(rank, world, port, out):
    import numpy as np
    import oracle
    from paper_2609_36800_b200 import synth
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = synth.Workload("t", B=5, m=2, K=96, N=12, seed=3)
        X, W, bits, alpha = synth.make_inputs(wl)                    # every rank draws the same inputs
        Xs, bs, als, start = replicas.tenant_shard(X, bits, alpha, world, rank)
        Ys = oracle.gemm(np.ascontiguousarray(Xs), W, np.ascontiguousarray(bs), np.ascontiguousarray(als))
        # gather only to check: the path itself needs no exchange
        parts = [None] * world
        dist.all_gather_object(parts, (start, Ys))
        if rank == 0:
            full = np.concatenate([y for _, y in sorted(parts, key=lambda p: p[0])], axis=0)
            out["equal"] = bool(np.array_equal(full, oracle.gemm(X, W, bits, alpha)))
            out["rows"] = [int(y.shape[0]) for _, y in sorted(parts, key=lambda p: p[0])]
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_products_of_tenant_shards_are_the_rows_of_the_full_product():
    world = 2
    port = _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_shard_worker, args=(world, port, out), nprocs=world, join=True)
    assert out["equal"] is True
    assert out["rows"] == [3, 2]
