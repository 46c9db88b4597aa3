"""GPU parity of the compress step (signs and per-tenant scale from fine-tuned weights) against the oracle."""
import numpy as np
import pytest

import oracle
from paper_2609_36800_b200 import synth

pytestmark = pytest.mark.gpu

# alpha: the kernel forms |delta| in fp32 (<= 2^-24 relative each), adds four of them in fp32 (<= 3 * 2^-24) and
# everything else in double in a fixed order; the oracle sums in double.  Worst case ~2.4e-7 relative.
ALPHA_RTOL = 1e-6

SHAPES = [
    (1, 8, 32),          # one word per row
    (2, 16, 1024),       # exactly one warp tile per row
    (3, 33, 1056),       # ragged: a second, mostly empty tile per row; rows not a multiple of the block
    (5, 130, 4096),      # several tiles per row
    (40, 9, 2048),       # more tenants than one shared-memory chunk
]


def _run(B, N, K, seed):
    import torch
    import paper_2609_36800_b200 as bd
    fine, W = synth.make_fine_weights(B, N, K, seed=seed)
    d_fine = torch.from_numpy(fine.view(np.int16)).cuda().view(torch.bfloat16)
    d_W = torch.from_numpy(W.view(np.int16)).cuda().view(torch.bfloat16)
    bits, alpha = bd.compress(d_fine, d_W)
    torch.cuda.synchronize()
    return fine, W, bits.cpu().numpy().view(np.uint32), alpha.cpu().numpy()


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "B%d_N%d_K%d" % s)
def test_compress_matches_oracle(shape):
    B, N, K = shape
    fine, W, bits, alpha = _run(B, N, K, seed=B * 1000 + N)
    ref_bits, ref_alpha = oracle.compress(fine, W)
    assert np.array_equal(bits, ref_bits)                     # integer work: bit-exact
    assert np.allclose(alpha, ref_alpha, rtol=ALPHA_RTOL, atol=0)


def test_compress_equal_weights_and_signed_zeros_give_a_zero_bit():
    # bit = (fine > base) in IEEE terms: equal values, and +0 against -0 either way round, are NOT greater
    import torch
    import paper_2609_36800_b200 as bd
    B, N, K = 2, 16, 1024
    fine, W = synth.make_fine_weights(B, N, K, seed=11)
    fine = fine.copy(); W = W.copy()
    fine[:, :, 0::7] = W[None, :, 0::7]                 # equal
    W[:, 1::7] = 0x8000; fine[:, :, 1::7] = 0x0000      # base -0, fine +0
    W[:, 2::7] = 0x0000; fine[:, :, 2::7] = 0x8000      # base +0, fine -0
    W[:, 3::7] = 0x8000; fine[:, :, 3::7] = 0x8000      # both -0
    W[:, 4::7] = 0x8000; fine[0, :, 4::7] = 0x0001      # base -0, fine the smallest positive subnormal: greater
    fine[1, :, 4::7] = 0x8001                           # ... the smallest negative one: not greater
    d_fine = torch.from_numpy(fine.view(np.int16)).cuda().view(torch.bfloat16)
    d_W = torch.from_numpy(W.view(np.int16)).cuda().view(torch.bfloat16)
    bits, alpha = bd.compress(d_fine, d_W)
    torch.cuda.synchronize()
    got = bits.cpu().numpy().view(np.uint32)
    ref_bits, ref_alpha = oracle.compress(fine, W)
    assert np.array_equal(got, ref_bits)
    unpacked = oracle.unpack(ref_bits)                  # (pins the expectation itself: +-1 signs, -1 where not greater)
    for c in (0, 1, 2, 3):
        assert (unpacked[:, :, c::7] == -1).all()
    assert (unpacked[0, :, 4::7] == 1).all() and (unpacked[1, :, 4::7] == -1).all()
    assert np.allclose(alpha.cpu().numpy(), ref_alpha, rtol=ALPHA_RTOL, atol=0)


def test_compress_is_deterministic_and_feeds_the_gemm():
    import torch
    import paper_2609_36800_b200 as bd
    B, N, K, m = 4, 256, 512, 2
    fine, W, bits, alpha = _run(B, N, K, seed=3)
    _, _, bits2, alpha2 = _run(B, N, K, seed=3)
    assert np.array_equal(bits, bits2) and np.array_equal(alpha, alpha2)
    # compress -> gemm on the GPU equals the oracle's compress -> gemm
    rng = np.random.default_rng(9)
    X = synth.f32_to_bf16_bits(rng.standard_normal((B, m, K), dtype=np.float32))
    dX = torch.from_numpy(X.view(np.int16)).cuda().view(torch.bfloat16)
    dW = torch.from_numpy(W.view(np.int16)).cuda().view(torch.bfloat16)
    dbits, dalpha = bd.compress(torch.from_numpy(fine.view(np.int16)).cuda().view(torch.bfloat16), dW)
    Y = bd.gemm(dX, dW, dbits, dalpha)
    torch.cuda.synchronize()
    ref_bits, ref_alpha = oracle.compress(fine, W)
    Yref = oracle.gemm(X, W, ref_bits, ref_alpha)
    Yg = synth.bf16_bits_to_f32(Y.view(torch.int16).cpu().numpy().view(np.uint16)).astype(np.float64)
    assert np.max(np.abs(Yg - Yref)) <= 2e-2
    assert np.linalg.norm(Yg - Yref) / np.linalg.norm(Yref) <= 5e-3


def test_gemm_queued_directly_behind_compress_reads_the_new_signs():
    # compress and gemm back to back on one stream, workspace made beforehand, nothing in between: the GEMM's early
    # weight prefetch must not run ahead of the compress kernels that are still writing the sign words and alpha.
    # Three rounds into the SAME device buffers with different fine-tuned weights: stale signs would be the
    # previous round's and miss the gate by far.
    import torch
    import paper_2609_36800_b200 as bd
    B, N, K, m = 8, 1024, 2048, 1
    rng = np.random.default_rng(4)
    X = synth.f32_to_bf16_bits(rng.standard_normal((B, m, K), dtype=np.float32))
    dX = torch.from_numpy(X.view(np.int16)).cuda().view(torch.bfloat16)
    ws = bd.make_workspace(B, m, N, K)
    d_fine = torch.empty((B, N, K), dtype=torch.bfloat16, device="cuda")
    d_W = torch.empty((N, K), dtype=torch.bfloat16, device="cuda")
    d_bits = torch.empty((B, N, K // 32), dtype=torch.int32, device="cuda")
    d_alpha = torch.empty((B,), dtype=torch.float32, device="cuda")
    Y = torch.empty((B, m, N), dtype=torch.bfloat16, device="cuda")
    for rnd in range(3):
        fine, W = synth.make_fine_weights(B, N, K, seed=100 + rnd)
        d_fine.copy_(torch.from_numpy(fine.view(np.int16)).view(torch.bfloat16))
        d_W.copy_(torch.from_numpy(W.view(np.int16)).view(torch.bfloat16))
        torch.cuda.synchronize()
        bd.compress(d_fine, d_W, bits=d_bits, alpha=d_alpha)
        bd.gemm(dX, d_W, d_bits, d_alpha, out=Y, workspace=ws)
        torch.cuda.synchronize()
        ref_bits, ref_alpha = oracle.compress(fine, W)
        assert np.array_equal(d_bits.cpu().numpy().view(np.uint32), ref_bits)
        Yref = oracle.gemm(X, W, ref_bits, ref_alpha)
        Yg = synth.bf16_bits_to_f32(Y.view(torch.int16).cpu().numpy().view(np.uint16)).astype(np.float64)
        assert np.max(np.abs(Yg - Yref)) <= 2e-2, rnd
        assert np.linalg.norm(Yg - Yref) / np.linalg.norm(Yref) <= 5e-3, rnd
