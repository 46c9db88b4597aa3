"""Pins for the CPU oracle: every check here is fixed by something other than
the oracle itself (hand-computed values, one-hot probes, numpy's fp64 matmul on
a dense S built by independent Python code, pure-Python brute force, algebraic
invariants of the formula)."""
import itertools
import json
import os

import numpy as np
import pytest

import oracle
from paper_2609_36800_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------
# independent helpers (no oracle code involved)
# ----------------------------------------------------------------------------
def bf16(a):
    return synth.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def widen(h):
    return synth.bf16_bits_to_f32(h).astype(np.float64)


def dense_signs_py(bits):
    """Dense +1/-1 from packed words with explicit Python integer arithmetic."""
    B, N, Wn = bits.shape
    S = np.empty((B, N, Wn * 32), dtype=np.float64)
    for b, n, w in itertools.product(range(B), range(N), range(Wn)):
        word = int(bits[b, n, w])
        for j in range(32):
            S[b, n, 32 * w + j] = 1.0 if (word >> j) & 1 else -1.0
    return S


def dense_signs_np(bits):
    """Dense +1/-1 via numpy's unpackbits on the little-endian byte view."""
    B, N, Wn = bits.shape
    by = bits.astype("<u4").view(np.uint8).reshape(B, N, Wn * 4)
    b01 = np.unpackbits(by, axis=-1, bitorder="little")
    return b01.astype(np.float64) * 2.0 - 1.0


def reference_np(X, W, bits, alpha, dense=dense_signs_np):
    x, w, S = widen(X), widen(W), dense(bits)
    base = np.einsum("btk,nk->btn", x, w)
    delta = np.einsum("btk,bnk->btn", x, S)
    return base + alpha.astype(np.float64)[:, None, None] * delta


def small_case(B, m, N, K, seed, w_std=0.02):
    wl = synth.Workload("t", B=B, m=m, K=K, N=N, w_std=w_std, seed=seed)
    return synth.make_inputs(wl)


# ----------------------------------------------------------------------------
# packing
# ----------------------------------------------------------------------------
def test_pack_single_positive_element_sets_one_bit():
    B, N, K = 2, 3, 96
    for (b, n, k) in [(0, 0, 0), (0, 1, 1), (1, 2, 31), (1, 0, 32), (0, 2, 33), (1, 1, 63), (0, 0, 64), (1, 2, 95)]:
        S = -np.ones((B, N, K), dtype=np.int8)
        S[b, n, k] = 1
        bits = oracle.pack(S)
        expect = np.zeros((B, N, K // 32), dtype=np.uint32)
        expect[b, n, k // 32] = np.uint32(1) << np.uint32(k % 32)
        assert np.array_equal(bits, expect), (b, n, k)


def test_pack_hand_word():
    # first 16 weights +1, last 16 weights -1  ->  0x0000FFFF
    S = np.concatenate([np.ones(16), -np.ones(16)]).astype(np.int8).reshape(1, 1, 32)
    assert oracle.pack(S)[0, 0, 0] == 0x0000FFFF
    # alternating starting with +1 at k=0 -> 0x55555555
    S = np.tile(np.array([1, -1], dtype=np.int8), 16).reshape(1, 1, 32)
    assert oracle.pack(S)[0, 0, 0] == 0x55555555


def test_pack_zero_and_negative_map_to_clear_bit():
    S = np.array([0, -1, -128, 1, 127, 2] + [0] * 26, dtype=np.int8).reshape(1, 1, 32)
    assert oracle.pack(S)[0, 0, 0] == (1 << 3) | (1 << 4) | (1 << 5)


def test_pack_matches_numpy_packbits():
    S = synth.make_signs(3, 17, 160, seed=5)
    got = oracle.pack(S)
    by = np.packbits((S > 0).astype(np.uint8), axis=-1, bitorder="little")
    expect = by.reshape(3, 17, 5, 4).copy().view("<u4").reshape(3, 17, 5)
    assert np.array_equal(got, expect)


def test_pack_unpack_round_trip():
    S = synth.make_signs(2, 9, 128, seed=11)
    assert np.array_equal(oracle.unpack(oracle.pack(S)), S)
    words = np.random.default_rng(3).integers(0, 2**32, size=(2, 5, 7), dtype=np.uint32)
    assert np.array_equal(oracle.pack(oracle.unpack(words)), words)


def test_unpack_matches_independent_decoders():
    words = np.random.default_rng(4).integers(0, 2**32, size=(2, 3, 2), dtype=np.uint32)
    S = oracle.unpack(words).astype(np.float64)
    assert np.array_equal(S, dense_signs_py(words))
    assert np.array_equal(S, dense_signs_np(words))


# ----------------------------------------------------------------------------
# the fused product
# ----------------------------------------------------------------------------
def test_hand_computed_known_answer():
    # K=32, x_k = k+1, word 0x0000FFFF: (1+..+16) - (17+..+32) = 136 - 392 = -256
    X = bf16(np.arange(1, 33, dtype=np.float32)).reshape(1, 1, 32)
    W = np.zeros((1, 32), dtype=np.uint16)
    bits = np.array([[[0x0000FFFF]]], dtype=np.uint32)
    Y = oracle.gemm(X, W, bits, np.array([1.0], dtype=np.float32))
    assert Y[0, 0, 0] == -256.0
    # with alpha = 0.5 and w = 2 everywhere: 2*528 + 0.5*(-256) = 928
    W2 = bf16(np.full((1, 32), 2.0))
    Y = oracle.gemm(X, W2, bits, np.array([0.5], dtype=np.float32))
    assert Y[0, 0, 0] == 928.0


@pytest.mark.parametrize("k", [0, 1, 31, 32, 33, 63, 64, 95])
def test_one_hot_probe_reads_the_right_bit(k):
    # X = e_k, W = 0, alpha = 1  =>  Y[n] = s[n,k]
    B, N, K = 2, 4, 96
    rng = np.random.default_rng(100 + k)
    bits = rng.integers(0, 2**32, size=(B, N, K // 32), dtype=np.uint32)
    x = np.zeros((B, 1, K), dtype=np.float32)
    x[:, 0, k] = 1.0
    Y = oracle.gemm(bf16(x), np.zeros((N, K), dtype=np.uint16), bits, np.ones(B, dtype=np.float32))
    expect = np.where((bits[:, :, k // 32] >> np.uint32(k % 32)) & np.uint32(1), 1.0, -1.0)
    assert np.array_equal(Y[:, 0, :], expect)


@pytest.mark.parametrize("j", [0, 1, 15, 16, 30, 31])
def test_single_bit_words(j):
    # word = 1<<j, x = 1 everywhere: sum = (+1) + 31*(-1) = -30; x = e_j: +1
    K = 32
    bits = np.array([[[1 << j]]], dtype=np.uint32)
    ones = bf16(np.ones((1, 1, K)))
    Wz = np.zeros((1, K), dtype=np.uint16)
    a1 = np.ones(1, dtype=np.float32)
    assert oracle.gemm(ones, Wz, bits, a1)[0, 0, 0] == -30.0
    e = np.zeros((1, 1, K), dtype=np.float32)
    e[0, 0, j] = 1.0
    assert oracle.gemm(bf16(e), Wz, bits, a1)[0, 0, 0] == 1.0


@pytest.mark.parametrize("shape", [(2, 3, 5, 64), (1, 1, 7, 96), (3, 2, 4, 32)])
def test_brute_force_python_loops(shape):
    B, m, N, K = shape
    X, W, bits, alpha = small_case(B, m, N, K, seed=sum(shape))
    got = oracle.gemm(X, W, bits, alpha)
    x, w = widen(X), widen(W)
    for b, t, n in itertools.product(range(B), range(m), range(N)):
        base = 0.0
        delta = 0.0
        for k in range(K):
            s = 1.0 if (int(bits[b, n, k // 32]) >> (k % 32)) & 1 else -1.0
            base += float(x[b, t, k]) * float(w[n, k])
            delta += float(x[b, t, k]) * s
        expect = base + float(np.float64(alpha[b])) * delta
        assert got[b, t, n] == pytest.approx(expect, rel=1e-13, abs=1e-13)


@pytest.mark.parametrize("shape", [(2, 3, 5, 64), (2, 5, 33, 96), (4, 16, 64, 512)])
def test_matches_numpy_fp64_matmul_on_dense_signs(shape):
    B, m, N, K = shape
    X, W, bits, alpha = small_case(B, m, N, K, seed=7 + K)
    got = oracle.gemm(X, W, bits, alpha)
    expect = reference_np(X, W, bits, alpha)
    assert np.max(np.abs(got - expect)) <= 1e-12 * max(1.0, np.max(np.abs(expect)))


def test_alpha_zero_is_plain_gemm():
    X, W, bits, alpha = small_case(2, 4, 24, 128, seed=21)
    got = oracle.gemm(X, W, bits, np.zeros_like(alpha))
    expect = np.einsum("btk,nk->btn", widen(X), widen(W))
    assert np.allclose(got, expect, rtol=1e-13, atol=1e-13)


def test_all_bits_set_adds_alpha_times_rowsum():
    X, W, bits, alpha = small_case(2, 4, 24, 128, seed=22)
    ones = np.full_like(bits, 0xFFFFFFFF)
    zeros = np.zeros_like(bits)
    x, w, a = widen(X), widen(W), alpha.astype(np.float64)
    expect_p = np.einsum("btk,bnk->btn", x, w[None] + a[:, None, None])
    expect_m = np.einsum("btk,bnk->btn", x, w[None] - a[:, None, None])
    assert np.allclose(oracle.gemm(X, W, ones, alpha), expect_p, rtol=1e-12, atol=1e-12)
    assert np.allclose(oracle.gemm(X, W, zeros, alpha), expect_m, rtol=1e-12, atol=1e-12)


def test_flipping_every_bit_negates_the_delta_term():
    X, W, bits, alpha = small_case(3, 2, 16, 160, seed=23)
    y1 = oracle.gemm(X, W, bits, alpha)
    y2 = oracle.gemm(X, W, ~bits, alpha)
    base = np.einsum("btk,nk->btn", widen(X), widen(W))
    assert np.allclose(y1 + y2, 2.0 * base, rtol=1e-12, atol=1e-12)
    assert not np.allclose(y1, y2)


def test_delta_is_linear_in_alpha():
    X, W, bits, alpha = small_case(2, 3, 8, 64, seed=24)
    y0 = oracle.gemm(X, W, bits, np.zeros_like(alpha))
    ya = oracle.gemm(X, W, bits, alpha)
    y2a = oracle.gemm(X, W, bits, (2 * alpha).astype(np.float32))
    assert np.allclose(y2a - y0, 2.0 * (ya - y0), rtol=1e-11, atol=1e-13)


def test_tenants_are_isolated_and_permute():
    X, W, bits, alpha = small_case(3, 2, 8, 64, seed=25)
    y = oracle.gemm(X, W, bits, alpha)
    X2, bits2, alpha2 = X.copy(), bits.copy(), alpha.copy()
    X2[1] = bf16(np.random.default_rng(1).standard_normal((2, 64)))
    bits2[1] ^= np.uint32(0xDEADBEEF)
    alpha2[1] = 0.5
    y2 = oracle.gemm(X2, W, bits2, alpha2)
    assert np.array_equal(y[0], y2[0]) and np.array_equal(y[2], y2[2])
    assert not np.array_equal(y[1], y2[1])
    perm = [2, 0, 1]
    yp = oracle.gemm(X[perm], W, bits[perm], alpha[perm])
    assert np.array_equal(yp, y[perm])


def test_transposed_operands_would_be_caught():
    # N != m and W != W^T: a transposed or mis-strided operand changes the result.
    X, W, bits, alpha = small_case(1, 3, 5, 64, seed=26)
    got = oracle.gemm(X, W, bits, alpha)
    assert got.shape == (1, 3, 5)
    expect = reference_np(X, W, bits, alpha, dense=dense_signs_py)
    assert np.allclose(got, expect, rtol=1e-13, atol=1e-13)


def test_gemm_at_equals_full_result_and_numpy():
    X, W, bits, alpha = small_case(3, 4, 40, 256, seed=27)
    full = oracle.gemm(X, W, bits, alpha)
    rng = np.random.default_rng(0)
    idx = np.stack([rng.integers(0, 3, 50), rng.integers(0, 4, 50), rng.integers(0, 40, 50)], axis=1).astype(np.int32)
    got = oracle.gemm_at(X, W, bits, alpha, idx)
    assert np.array_equal(got, full[idx[:, 0], idx[:, 1], idx[:, 2]])
    ref = reference_np(X, W, bits, alpha)
    assert np.allclose(got, ref[idx[:, 0], idx[:, 1], idx[:, 2]], rtol=1e-12, atol=1e-12)


def test_extreme_magnitudes_and_cancellation():
    # all-equal x with a balanced word: the delta term cancels exactly
    K = 64
    X = bf16(np.full((1, 1, K), 3.0))
    bits = np.array([[[0x0F0F0F0F, 0xF0F0F0F0]]], dtype=np.uint32)
    W = np.zeros((1, K), dtype=np.uint16)
    assert oracle.gemm(X, W, bits, np.array([123.0], dtype=np.float32))[0, 0, 0] == 0.0
    # large and tiny magnitudes stay exact in fp64
    x = np.zeros((1, 1, K), dtype=np.float32)
    x[0, 0, 0], x[0, 0, 1] = 2.0**15, 2.0**-20
    w = np.zeros((1, K), dtype=np.float32)
    w[0, 0], w[0, 1] = 2.0**-10, 2.0**10
    y = oracle.gemm(bf16(x), bf16(w), np.zeros((1, 1, 2), dtype=np.uint32), np.array([0.0], dtype=np.float32))
    assert y[0, 0, 0] == 2.0**5 + 2.0**-10


# ----------------------------------------------------------------------------
# generator determinism + stored seed-0 statistics
# ----------------------------------------------------------------------------
def test_bf16_rounding_is_nearest_even():
    # 1 + 2^-8 is a tie between 1.0 (even) and 1 + 2^-7 -> 1.0; 1 + 3*2^-8 ties up to 1 + 2^-6
    vals = np.array([1.0, 1.0 + 2.0**-8, 1.0 + 3 * 2.0**-8, 1.0 + 2.0**-8 + 2.0**-20, -2.5], dtype=np.float32)
    got = synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(vals))
    assert list(got) == [1.0, 1.0, 1.0 + 2.0**-6, 1.0 + 2.0**-7, -2.5]
    import ml_dtypes
    r = np.random.default_rng(0).standard_normal(10000).astype(np.float32)
    assert np.array_equal(synth.f32_to_bf16_bits(r), r.astype(ml_dtypes.bfloat16).view(np.uint16))


@pytest.mark.parametrize("name", ["tiny", "decode_attn"])
def test_seed0_statistics_match_stored_values(name):
    with open(os.path.join(GOLDEN, "seed0_stats.json")) as f:
        stats = json.load(f)[name]
    wl = synth.WORKLOADS_BY_NAME[name]
    X, W, bits, alpha = synth.make_inputs(wl)
    assert int(X[0, 0, 0]) == stats["x000_bits"]
    assert int(W[0, 0]) == stats["w00_bits"]
    assert int(bits[0, 0, 0]) == stats["bits_first"]
    assert int(bits[-1, -1, -1]) == stats["bits_last"]
    Y = oracle.gemm(X, W, bits, alpha)
    assert Y[0, 0, 0] == pytest.approx(stats["y_first"], rel=1e-10)
    assert Y[-1, -1, -1] == pytest.approx(stats["y_last"], rel=1e-10)
    assert np.abs(Y).max() == pytest.approx(stats["y_absmax"], rel=1e-10)
    assert np.linalg.norm(Y) == pytest.approx(stats["y_fro"], rel=1e-10)
    assert Y.sum() == pytest.approx(stats["y_sum"], rel=1e-8)


# ----------------------------------------------------------------------------------------------------
# compress: bits = [W_fine - W_base > 0], alpha = mean |W_fine - W_base| (the BitDelta method the paper
# cites in its BitDelta paragraph).  Pins that do not reuse the oracle's code.

def _bf16(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def test_compress_hand_example():
    # one tenant, one row of 32 weights; deltas chosen by hand (all exactly representable in bf16)
    base = np.zeros(32, dtype=np.float32)
    fine = np.zeros(32, dtype=np.float32)
    base[:4] = [1.0, 2.0, -1.0, 0.5]
    fine[:4] = [1.5, 1.0, -1.0, 0.75]          # deltas +0.5, -1.0, 0 (packs as 0), +0.25
    fine[31] = -2.0                            # delta -2.0 at the word's top bit
    bits, alpha = oracle.compress(_bf16(fine).reshape(1, 1, 32), _bf16(base).reshape(1, 32))
    assert bits.shape == (1, 1, 1) and bits[0, 0, 0] == (1 << 0) | (1 << 3)
    assert alpha[0] == np.float32((0.5 + 1.0 + 0.0 + 0.25 + 2.0) / 32)


def test_compress_bit_order_and_row_indexing():
    # a single positive delta at (b, n, k) must set exactly bit k%32 of word k//32 of row (b, n)
    B, N, K = 2, 3, 96
    base = np.zeros((N, K), dtype=np.float32)
    for (b, n, k) in [(0, 0, 0), (1, 2, 95), (0, 1, 37), (1, 0, 64)]:
        fine = np.zeros((B, N, K), dtype=np.float32)
        fine[b, n, k] = 3.0
        bits, alpha = oracle.compress(_bf16(fine), _bf16(base))
        expect = np.zeros((B, N, K // 32), dtype=np.uint32)
        expect[b, n, k // 32] = np.uint32(1) << np.uint32(k % 32)
        assert np.array_equal(bits, expect)
        expect_alpha = np.zeros(B, dtype=np.float32)
        expect_alpha[b] = np.float32(3.0 / (N * K))
        assert np.array_equal(alpha, expect_alpha)


@pytest.mark.parametrize("shape", [(1, 4, 32), (3, 5, 64), (2, 16, 256)])
def test_compress_matches_numpy(shape):
    # independent statement with numpy: sign through np.packbits, mean through np.mean in float64
    B, N, K = shape
    fine, W = synth.make_fine_weights(B, N, K, seed=11)
    bits, alpha = oracle.compress(fine, W)
    d = synth.bf16_bits_to_f32(fine).astype(np.float64) - synth.bf16_bits_to_f32(W).astype(np.float64)[None]
    assert (d == 0).any() and (d > 0).any() and (d < 0).any()
    packed = np.packbits((d > 0).astype(np.uint8), axis=-1, bitorder="little").view(np.uint32)
    assert np.array_equal(bits, packed.reshape(B, N, K // 32))
    ref = np.abs(d).mean(axis=(1, 2))
    assert np.allclose(alpha.astype(np.float64), ref, rtol=1e-7, atol=0)   # fp32 rounding of an fp64 mean


def test_compress_invariants():
    B, N, K = 2, 8, 64
    fine, W = synth.make_fine_weights(B, N, K, seed=5)
    bits, alpha = oracle.compress(fine, W)
    wf = synth.bf16_bits_to_f32(fine)
    wb = synth.bf16_bits_to_f32(W)
    # the pair (W_base = 0, W_fine = delta) has the same signs and the same alpha whenever delta is a bf16 value
    d = wf - wb[None]
    d_bits = _bf16(d)
    exact = synth.bf16_bits_to_f32(d_bits) == d
    if exact.all():
        b2, a2 = oracle.compress(d_bits, _bf16(np.zeros((N, K))))
        assert np.array_equal(b2, bits) and np.array_equal(a2, alpha)
    # doubling the delta around a zero base doubles alpha and keeps the bits
    z = _bf16(np.zeros((N, K)))
    b1, a1 = oracle.compress(_bf16(d), z)
    b2, a2 = oracle.compress(_bf16(2.0 * synth.bf16_bits_to_f32(_bf16(d))), z)
    assert np.array_equal(b1, b2) and np.allclose(a2, 2.0 * a1, rtol=1e-7)
    # negating the delta flips exactly the bits of the non-zero deltas
    dn = synth.bf16_bits_to_f32(_bf16(d))
    b3, a3 = oracle.compress(_bf16(-dn), z)
    nz = np.packbits((dn != 0).astype(np.uint8), axis=-1, bitorder="little").view(np.uint32).reshape(b1.shape)
    assert np.array_equal(b1 ^ b3, nz) and np.array_equal(a1, a3)
    # compress followed by unpack gives +1 exactly where the delta is positive
    S = oracle.unpack(bits)
    assert np.array_equal(S > 0, d > 0)
    # tenants are independent
    b4, a4 = oracle.compress(fine[1:], W)
    assert np.array_equal(b4[0], bits[1]) and a4[0] == alpha[1]


# ----------------------------------------------------------------------------
# extended product: fp16 operands, bias, SiLU
# ----------------------------------------------------------------------------
def f16(a):
    return np.asarray(a, dtype=np.float32).astype(np.float16).view(np.uint16)


def test_half_decode_matches_numpy_on_every_finite_pattern():
    h = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    finite = ((h >> 10) & 0x1F) != 31
    got = oracle.half_to_double(h[finite])
    expect = h[finite].view(np.float16).astype(np.float64)
    assert np.array_equal(got, expect)
    assert np.array_equal(np.signbit(got), np.signbit(expect))          # -0.0 keeps its sign
    assert oracle.half_to_double(np.array([0x3C00, 0xC000, 0x0001, 0x7BFF], dtype=np.uint16)).tolist() == \
        [1.0, -2.0, 2.0 ** -24, 65504.0]                                 # format constants


def test_ex_without_options_is_the_plain_product_bit_for_bit():
    X, W, bits, alpha = small_case(3, 4, 20, 160, seed=3)
    assert np.array_equal(oracle.gemm_ex(X, W, bits, alpha), oracle.gemm(X, W, bits, alpha))


@pytest.mark.parametrize("shape", [(2, 3, 5, 64), (3, 5, 33, 96)])
def test_f16_product_matches_numpy_fp64_matmul(shape):
    B, m, N, K = shape
    wl = synth.Workload("t", B=B, m=m, K=K, N=N, seed=11 + K)
    X, W, bits, alpha, _ = synth.make_inputs_f16(wl)
    x = X.view(np.float16).astype(np.float64)
    w = W.view(np.float16).astype(np.float64)
    S = dense_signs_py(bits)
    expect = np.einsum("btk,nk->btn", x, w) + alpha.astype(np.float64)[:, None, None] * np.einsum("btk,bnk->btn", x, S)
    got = oracle.gemm_ex(X, W, bits, alpha, dtype="f16")
    assert np.max(np.abs(got - expect)) <= 1e-12 * max(1.0, np.max(np.abs(expect)))
    # reading the same patterns as bf16 gives something else entirely
    assert np.max(np.abs(oracle.gemm_ex(X, W, bits, alpha, dtype="bf16") - expect)) > 1e-3


def test_bias_is_added_per_output_feature():
    wl = synth.Workload("t", B=2, m=3, K=64, N=7, seed=5)
    X, W, bits, alpha, bias = synth.make_inputs_f16(wl)
    y0 = oracle.gemm_ex(X, W, bits, alpha, dtype="f16")
    y1 = oracle.gemm_ex(X, W, bits, alpha, bias=bias, dtype="f16")
    b = bias.view(np.float16).astype(np.float64)
    assert np.max(np.abs((y1 - y0) - b[None, None, :])) <= 1e-13
    # bf16 bias patterns are read as bf16
    Xb, Wb, bitsb, alphab = small_case(2, 3, 7, 64, seed=5)
    bb = synth.make_bias_bf16(7, seed=1)
    d = oracle.gemm_ex(Xb, Wb, bitsb, alphab, bias=bb) - oracle.gemm(Xb, Wb, bitsb, alphab)
    assert np.max(np.abs(d - widen(bb)[None, None, :])) <= 1e-13


def _probe(y, bias=None, act="none"):
    """One output whose pre-activation value is exactly y: x = e_0, w[0,0] = y, alpha = 0."""
    X = np.zeros((1, 1, 32), dtype=np.float32); X[0, 0, 0] = 1.0
    W = np.zeros((1, 32), dtype=np.float32); W[0, 0] = y
    bits = np.zeros((1, 1, 1), dtype=np.uint32)
    alpha = np.zeros(1, dtype=np.float32)
    b = None if bias is None else f16([bias])
    return float(oracle.gemm_ex(f16(X), f16(W), bits, alpha, bias=b, dtype="f16", act=act)[0, 0, 0])


def test_silu_closed_forms():
    assert _probe(0.0, act="silu") == 0.0
    assert _probe(1.0, act="silu") == pytest.approx(0.7310585786300049, rel=1e-15)      # sigmoid(1), textbook value
    assert _probe(-1.0, act="silu") == pytest.approx(-0.2689414213699951, rel=1e-15)    # -sigmoid(-1)
    for y in (0.5, 2.0, 7.25):
        assert _probe(y, act="silu") - _probe(-y, act="silu") == pytest.approx(y, rel=1e-14)   # y (s(y) + s(-y)) = y
    assert _probe(40.0, act="silu") == pytest.approx(40.0, rel=1e-15)
    assert abs(_probe(-40.0, act="silu")) < 1e-15
    assert _probe(3.0, act="none") == 3.0


def test_activation_is_applied_after_the_bias():
    # y = -1, bias = +2: silu(-1 + 2) = sigmoid(1); silu(-1) + 2 would be 1.731...
    assert _probe(-1.0, bias=2.0, act="silu") == pytest.approx(0.7310585786300049, rel=1e-15)


def test_ex_at_listed_outputs_equals_full_result():
    wl = synth.Workload("t", B=3, m=4, K=96, N=10, seed=9)
    X, W, bits, alpha, bias = synth.make_inputs_f16(wl)
    full = oracle.gemm_ex(X, W, bits, alpha, bias=bias, dtype="f16", act="silu")
    idx = np.array([[0, 0, 0], [2, 3, 9], [1, 2, 5], [2, 0, 7]], dtype=np.int32)
    at = oracle.gemm_ex(X, W, bits, alpha, bias=bias, dtype="f16", act="silu", idx=idx)
    assert np.array_equal(at, np.array([full[b, t, n] for b, t, n in idx]))


# ----------------------------------------------------------------------------
# SiLU gate over interleaved gate / up rows
# ----------------------------------------------------------------------------
def _gate_probe(gate, up, bias=None):
    """Two weight rows with pre-activation values `gate` (row 0) and `up` (row 1): x = e_0, alpha = 0."""
    X = np.zeros((1, 1, 32), dtype=np.float32); X[0, 0, 0] = 1.0
    W = np.zeros((2, 32), dtype=np.float32); W[0, 0] = gate; W[1, 0] = up
    bits = np.zeros((1, 2, 1), dtype=np.uint32)
    alpha = np.zeros(1, dtype=np.float32)
    b = None if bias is None else f16(bias)
    y = oracle.gemm_ex(f16(X), f16(W), bits, alpha, bias=b, dtype="f16", act="silu_gate")
    assert y.shape == (1, 1, 1)
    return float(y[0, 0, 0])


def test_silu_gate_closed_forms_and_row_roles():
    assert _gate_probe(1.0, 3.0) == pytest.approx(3.0 * 0.7310585786300049, rel=1e-15)   # sigmoid(1) * 1 * 3
    assert _gate_probe(3.0, 1.0) == pytest.approx(3.0 / (1.0 + np.exp(-3.0)), rel=1e-15)  # roles are not symmetric
    assert _gate_probe(0.0, 5.0) == 0.0 and _gate_probe(5.0, 0.0) == 0.0
    assert _gate_probe(40.0, -2.0) == pytest.approx(-80.0, rel=1e-15)                       # silu(y) -> y for large y
    # the bias enters both rows before the gate: (-1 + 2, 3 + 0.5)
    assert _gate_probe(-1.0, 3.0, bias=[2.0, 0.5]) == pytest.approx(3.5 * 0.7310585786300049, rel=1e-15)


def test_silu_gate_equals_recombined_plain_outputs():
    wl = synth.Workload("t", B=2, m=3, K=96, N=12, seed=13)
    X, W, bits, alpha, bias = synth.make_inputs_f16(wl)
    z = oracle.gemm_ex(X, W, bits, alpha, bias=bias, dtype="f16")               # pinned above
    expect = (z[:, :, 0::2] / (1.0 + np.exp(-z[:, :, 0::2]))) * z[:, :, 1::2]
    got = oracle.gemm_ex(X, W, bits, alpha, bias=bias, dtype="f16", act="silu_gate")
    assert got.shape == (2, 3, 6)
    assert np.max(np.abs(got - expect)) <= 1e-13
    idx = np.array([[0, 0, 0], [1, 2, 5], [1, 1, 3]], dtype=np.int32)
    at = oracle.gemm_ex(X, W, bits, alpha, bias=bias, dtype="f16", act="silu_gate", idx=idx)
    assert np.array_equal(at, np.array([got[b, t, i] for b, t, i in idx]))
