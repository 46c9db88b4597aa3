"""Tenant sharding on a GPU: the shards of a workload's tenants (what each rank of a multi-GPU deployment runs, with
W_base replicated and nothing exchanged) are run one after the other on the one GPU through the C ABI, and their
outputs, put back in tenant order, are the full product of the fp64 oracle."""
import numpy as np
import pytest

import oracle
from paper_2609_36800_b200 import replicas, synth

from gpu_util import assert_parity, run_gemm

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape,world", [((8, 1, 512, 1024), 2), ((5, 4, 384, 512), 2), ((7, 40, 256, 384), 4), ((3, 2, 256, 256), 4)],
                         ids=["B8_m1_2ranks", "B5_m4_2ranks", "B7_m40_4ranks", "B3_m2_4ranks_one_empty"])
def test_shard_products_concatenate_to_the_full_product(shape, world):
    B, m, N, K = shape
    wl = synth.Workload("t", B=B, m=m, N=N, K=K, seed=B + m + world)
    X, W, bits, alpha = synth.make_inputs(wl)
    Yref = oracle.gemm(X, W, bits, alpha)
    Y = np.full_like(Yref, np.nan)
    covered = 0
    for rank in range(world):
        Xs, bs, als, start = replicas.tenant_shard(X, bits, alpha, world, rank)
        if Xs.shape[0] == 0:          # more ranks than tenants: this rank has nothing to serve
            continue
        Y[start:start + Xs.shape[0]] = run_gemm(np.ascontiguousarray(Xs), W, np.ascontiguousarray(bs), np.ascontiguousarray(als))
        covered += Xs.shape[0]
    assert covered == B and not np.isnan(Y).any()
    assert_parity(Y, Yref, f"{shape} over {world} ranks")
    # a shard's product is exactly the corresponding rows of the one-GPU product when both take the same schedule
    if m > 16:
        assert np.array_equal(Y, run_gemm(X, W, bits, alpha))
