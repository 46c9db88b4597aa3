"""GPU parity tests of the streaming decode kernel (csrc/gemm_stream.cu), which the library plans only when
BITDELTA_STREAM=1 is set: both of its forms (flat work list; clusters of blocks whose partial sums meet in
distributed shared memory), against the fp64 CPU oracle at the gates of test_gpu_parity.py."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_36800_b200 as bd
from paper_2609_36800_b200 import synth

from gpu_util import assert_parity, errors, run_gemm, to_device, y_to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def stream_kernel(monkeypatch):
    monkeypatch.setenv("BITDELTA_STREAM", "1")


SHAPES = [
    # B, m, N, K                 expected schedule (5 flat, 6 clusters)
    ((1, 1, 128, 128), 5),       # one step: nothing to split across a cluster
    ((1, 16, 512, 512), 6),      # the tiny workload: 4 tiles x 4 steps, one step per block
    ((2, 1, 200, 256), 6),       # ragged N, clusters of two
    ((3, 2, 384, 640), 6),       # odd tenant count, five steps over clusters of four (2 + 1 + 1 + 1)
    ((5, 3, 130, 384), 5),       # two tiles x three steps: too few blocks in clusters -> flat list
    ((8, 1, 1024, 1024), 6),     # eight tenants, eight tiles x eight steps, clusters of eight
    ((8, 2, 1024, 512), 6),      # 16 token rows per unit
    ((7, 1, 2048, 2048), 6),     # 16 tiles x 16 steps, clusters of eight
    ((4, 4, 4096, 1024), 6),     # 32 tiles, clusters of four (128 blocks)
    ((1, 8, 2176, 512), 6),      # 17 tiles x four steps, clusters of four, ragged last tile
    ((2, 5, 11008, 256), 5),     # 86 tiles x 2 steps: clusters fill too little of the device -> flat list
    ((16, 1, 512, 1024), 5),     # two tenant groups: flat list by teams
    ((33, 2, 1920, 384), 5),     # five groups, last one with a single tenant
    ((3, 5, 512, 384), 5),
    ((1, 16, 128, 4096), 5),     # one tile, 32 steps: the flat list uses 32 blocks, a cluster only eight
]


@pytest.mark.parametrize("shape,schedule", SHAPES, ids=[f"B{s[0]}_m{s[1]}_N{s[2]}_K{s[3]}" for s, _ in SHAPES])
def test_stream_kernel_matches_oracle(shape, schedule):
    B, m, N, K = shape
    assert bd.gemm_plan(B, m, N, K)["schedule"] == schedule
    wl = synth.Workload("t", B=B, m=m, K=K, N=N, seed=B * 1000 + m * 100 + N + K)
    X, W, bits, alpha = synth.make_inputs(wl)
    Y = run_gemm(X, W, bits, alpha)
    max_abs, rel_fro = assert_parity(Y, oracle.gemm(X, W, bits, alpha), str(shape))
    assert rel_fro > 1e-5 or max_abs == 0.0   # (a bf16 result cannot sit closer to the fp64 one: guards against comparing a thing with itself)


def test_stream_kernel_one_hot_probe_is_exact():
    # X = e_k per token, W = 0, alpha = 1  =>  Y[b,t,n] = s[b,n,k_t]: exact in bf16, pins bit, word and tenant order
    B, m, N, K = 8, 1, 256, 1024
    rng = np.random.default_rng(5)
    bits = rng.integers(0, 2**32, size=(B, N, K // 32), dtype=np.uint32)
    ks = rng.integers(0, K, size=(B, m))
    ks[:4, 0] = [0, 31, 32, K - 1]
    x = np.zeros((B, m, K), dtype=np.float32)
    for b in range(B):
        x[b, 0, ks[b, 0]] = 1.0
    X = synth.f32_to_bf16_bits(x)
    W = np.zeros((N, K), dtype=np.uint16)
    alpha = np.ones(B, dtype=np.float32)
    assert np.array_equal(run_gemm(X, W, bits, alpha), oracle.gemm(X, W, bits, alpha))


def test_stream_kernel_headline_shape_and_determinism():
    wl = synth.WORKLOADS_BY_NAME["decode_attn"]
    assert bd.gemm_plan(wl.B, wl.m, wl.N, wl.K)["schedule"] == 6
    X, W, bits, alpha = synth.make_inputs(wl)
    Y1 = run_gemm(X, W, bits, alpha)
    assert_parity(Y1, oracle.gemm(X, W, bits, alpha), "decode_attn")
    # back-to-back launches (the second becomes resident next to the first) give bit-identical results
    dX, dW, dbits, dalpha = to_device(X, W, bits, alpha)
    outs = [bd.gemm(dX, dW, dbits, dalpha) for _ in range(4)]
    torch.cuda.synchronize()
    st, site = bd.last_device_status()
    assert st == 0, (st, site)
    for Y in outs:
        assert np.array_equal(y_to_f64(Y), Y1)


def test_stream_kernel_general_form_fp16_bias_silu():
    B, m, N, K = 8, 1, 1024, 1024
    wl = synth.Workload("t", B=B, m=m, K=K, N=N, seed=21)
    X, W, bits, alpha, bias = synth.make_inputs_f16(wl)
    f16 = lambda a: torch.from_numpy(a.view(np.int16)).cuda().view(torch.float16)
    Y = bd.gemm(f16(X), f16(W), torch.from_numpy(bits.view(np.int32)).cuda(), torch.from_numpy(alpha).cuda(),
                bias=f16(bias), act="silu")
    st, site = bd.last_device_status()
    assert st == 0, (st, site)
    got = Y.cpu().numpy().astype(np.float64)
    ref = oracle.gemm_ex(X, W, bits, alpha, bias=bias, dtype="f16", act="silu")
    max_abs, rel_fro = errors(got, ref)
    assert max_abs <= 2e-2 and rel_fro <= 5e-3, (max_abs, rel_fro)


WIDE_SHAPES = [
    # units of 17..32 token rows: taken by the streaming kernel only with BITDELTA_STREAM=2 (a whole multiprocessor per
    # block, whole 32-k groups per splitter thread)
    ((8, 4, 512, 512), 6), ((16, 4, 1024, 1024), 5), ((4, 8, 512, 1024), 6), ((32, 8, 256, 1024), 5),
    ((8, 3, 640, 384), 5), ((5, 6, 384, 512), 5), ((3, 8, 256, 256), 6), ((2, 16, 384, 512), 6),
]


@pytest.mark.parametrize("shape,schedule", WIDE_SHAPES, ids=[f"B{s[0]}_m{s[1]}_N{s[2]}_K{s[3]}" for s, _ in WIDE_SHAPES])
def test_stream_kernel_up_to_32_token_rows_per_unit(shape, schedule, monkeypatch):
    monkeypatch.setenv("BITDELTA_STREAM", "2")
    B, m, N, K = shape
    assert bd.gemm_plan(B, m, N, K)["schedule"] == schedule
    wl = synth.Workload("t", B=B, m=m, K=K, N=N, seed=B * 1000 + m * 100 + N + K)
    X, W, bits, alpha = synth.make_inputs(wl)
    assert_parity(run_gemm(X, W, bits, alpha), oracle.gemm(X, W, bits, alpha), str(shape))
