"""GPU parity of the extended product (fp16 operands, bias, SiLU) against the CPU oracle, through the C ABI."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2609_36800_b200 as bd
from paper_2609_36800_b200 import synth
from gpu_util import assert_parity, MAX_ABS_TOL, REL_FRO_TOL

pytestmark = pytest.mark.gpu


def dev16(a, dtype):
    return torch.from_numpy(a.view(np.int16)).cuda().view(dtype)


def run_ex(X, W, bits, alpha, bias, dtype, act):
    td = torch.float16 if dtype == "f16" else torch.bfloat16
    Y = bd.gemm(dev16(X, td), dev16(W, td), torch.from_numpy(bits.view(np.int32)).cuda(),
                torch.from_numpy(alpha).cuda(), bias=None if bias is None else dev16(bias, td), act=act)
    st, site = bd.last_device_status()
    assert st == 0, f"device status {st} at wait site {site}"
    h = Y.view(torch.int16).cpu().numpy().view(np.uint16)
    if dtype == "f16":
        return h.view(np.float16).astype(np.float64)
    return synth.bf16_bits_to_f32(h).astype(np.float64)


# every schedule: in-kernel split (m small), pre-pass split, tiled, cut tiles (split-K fix-up), teams,
# ragged N, CUDA-core fallback (K not a multiple of 128)
SHAPES = [
    (1, 1, 128, 128),
    (8, 1, 1024, 1024),
    (3, 2, 384, 640),
    (9, 4, 520, 512),
    (16, 8, 384, 768),
    (7, 9, 256, 256),
    (2, 17, 256, 384),
    (2, 100, 300, 640),
    (2, 130, 256, 512),     # token tiles of 128 and two W_base tiles: the schedule on CTA pairs
    (2, 90, 256, 384),      # CTA pairs, token tile of 96
    (5, 20, 384, 512),
    (3, 33, 264, 384),
    (1, 200, 520, 384),
    (12, 8, 6400, 256),
    (33, 2, 1920, 384),
    (2, 3, 96, 96),
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "B%d_m%d_N%d_K%d" % s)
def test_f16_with_bias_and_silu_matches_oracle(shape):
    B, m, N, K = shape
    wl = synth.Workload("t", B=B, m=m, K=K, N=N, seed=B * 100 + m)
    X, W, bits, alpha, bias = synth.make_inputs_f16(wl)
    Yref = oracle.gemm_ex(X, W, bits, alpha, bias=bias, dtype="f16", act="silu")
    assert_parity(run_ex(X, W, bits, alpha, bias, "f16", "silu"), Yref, str(shape))


@pytest.mark.parametrize("shape", [(8, 1, 1024, 1024), (9, 4, 520, 512), (2, 100, 300, 640), (12, 8, 6400, 256)],
                         ids=lambda s: "B%d_m%d_N%d_K%d" % s)
def test_f16_plain_matches_oracle(shape):
    B, m, N, K = shape
    wl = synth.Workload("t", B=B, m=m, K=K, N=N, seed=17)
    X, W, bits, alpha, _ = synth.make_inputs_f16(wl, with_bias=False)
    assert_parity(run_ex(X, W, bits, alpha, None, "f16", "none"), oracle.gemm_ex(X, W, bits, alpha, dtype="f16"), str(shape))


@pytest.mark.parametrize("opts", [("bias", "none"), (None, "silu"), ("bias", "silu")], ids=lambda o: f"{o[0]}_{o[1]}")
@pytest.mark.parametrize("shape", [(8, 1, 1024, 1024), (16, 8, 384, 768), (2, 100, 300, 640), (2, 3, 96, 96)],
                         ids=lambda s: "B%d_m%d_N%d_K%d" % s)
def test_bf16_epilogues_match_oracle(shape, opts):
    B, m, N, K = shape
    wl = synth.Workload("t", B=B, m=m, K=K, N=N, seed=23)
    X, W, bits, alpha = synth.make_inputs(wl)
    bias = synth.make_bias_bf16(N, seed=4) if opts[0] else None
    Yref = oracle.gemm_ex(X, W, bits, alpha, bias=bias, dtype="bf16", act=opts[1])
    assert_parity(run_ex(X, W, bits, alpha, bias, "bf16", opts[1]), Yref, f"{shape} {opts}")


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "B%d_m%d_N%d_K%d" % s)
def test_silu_gate_over_interleaved_rows_matches_oracle(shape, dtype):
    B, m, N, K = shape
    wl = synth.Workload("t", B=B, m=m, K=K, N=N, seed=B * 7 + m)
    if dtype == "f16":
        X, W, bits, alpha, bias = synth.make_inputs_f16(wl)
    else:
        X, W, bits, alpha = synth.make_inputs(wl)
        bias = synth.make_bias_bf16(N, seed=2)
    Yref = oracle.gemm_ex(X, W, bits, alpha, bias=bias, dtype=dtype, act="silu_gate")
    Y = run_ex(X, W, bits, alpha, bias, dtype, "silu_gate")
    assert Y.shape == (B, m, N // 2)
    assert_parity(Y, Yref, f"{shape} {dtype}")


def test_silu_gate_needs_an_even_feature_count():
    lib = bd.load_library()
    t = torch.zeros(256 * 128, dtype=torch.bfloat16, device="cuda")
    bits = torch.zeros(129 * 4, dtype=torch.int32, device="cuda")
    al = torch.zeros(1, dtype=torch.float32, device="cuda")
    ws = bd.make_workspace(1, 1, 129, 128)
    p = lambda x: ctypes.c_void_p(x.data_ptr())
    assert lib.bitdelta_gemm_ex(p(t), p(t), p(bits), p(al), None, p(t), 1, 1, 129, 128, 0, 2, p(ws), ws.numel(), None) == 2


def test_f16_delta_term_is_exact_for_full_precision_activations():
    # alpha = 1, W_base = 0, activations with all eleven significant bits set: Y is the exact sum of +-x,
    # and any piece of x lost by the e5m2 split would show at the 2^-10 level.
    B, m, N, K = 2, 1, 128, 128
    rng = np.random.default_rng(3)
    x = (1.0 + 1023.0 / 1024.0) * np.exp2(rng.integers(-3, 4, size=(B, m, K))).astype(np.float32)
    X = x.astype(np.float16).view(np.uint16)
    assert np.array_equal(X.view(np.float16).astype(np.float32), x)
    W = np.zeros((N, K), dtype=np.uint16)
    bits = rng.integers(0, 2**32, size=(B, N, K // 32), dtype=np.uint32)
    alpha = np.ones(B, dtype=np.float32)
    Yref = oracle.gemm_ex(X, W, bits, alpha, dtype="f16")
    Y = run_ex(X, W, bits, alpha, None, "f16", "none")
    # fp32 accumulation of exact products, one rounding to fp16 at the end
    assert np.max(np.abs(Y - Yref) / np.maximum(np.abs(Yref), 1.0)) <= 2.0 ** -10


def test_headline_shape_f16_bias_silu_sampled():
    wl = synth.WORKLOADS_BY_NAME["decode_attn"]
    X, W, bits, alpha, bias = synth.make_inputs_f16(wl)
    Y = run_ex(X, W, bits, alpha, bias, "f16", "silu")
    rng = np.random.default_rng(1)
    idx = np.stack([rng.integers(0, wl.B, 4096), rng.integers(0, wl.m, 4096), rng.integers(0, wl.N, 4096)], axis=1).astype(np.int32)
    ref = oracle.gemm_ex(X, W, bits, alpha, bias=bias, dtype="f16", act="silu", idx=idx)
    got = Y[idx[:, 0], idx[:, 1], idx[:, 2]]
    assert np.max(np.abs(got - ref)) <= MAX_ABS_TOL
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= REL_FRO_TOL


def test_unknown_option_codes_are_refused():
    lib = bd.load_library()
    t = torch.zeros(128 * 128, dtype=torch.bfloat16, device="cuda")
    bits = torch.zeros(128 * 4, dtype=torch.int32, device="cuda")
    al = torch.zeros(1, dtype=torch.float32, device="cuda")
    ws = bd.make_workspace(1, 1, 128, 128)
    p = lambda x: ctypes.c_void_p(x.data_ptr())
    for dtype, act in ((2, 0), (0, 3), (-1, 0)):
        st = lib.bitdelta_gemm_ex(p(t), p(t), p(bits), p(al), None, p(t), 1, 1, 128, 128, dtype, act, p(ws), ws.numel(), None)
        assert st == 8
