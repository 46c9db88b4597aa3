"""GPU tests of the activation range of the decode schedules (m <= 16), whose delta term runs on e5m2 operands.

Finite bf16 activations below 2^16 must give the oracle's result in every schedule: in-kernel split (few token
rows per unit), pre-pass split (many) and, for reference, the tiled schedule (m > 16).  Beyond that the decode schedules clamp the delta term and report BITDELTA_ERR_RANGE; the wide-range option
routes such inputs to the tiled schedule, which is exact.  Per-element gate as in the stress test of
test_gpu_parity.py: max(2e-2, |Y_ref| 2^-8) (bf16 spacing exceeds 2e-2 once |Y| reaches 8)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_36800_b200 as bd
from paper_2609_36800_b200 import synth

from gpu_util import to_device, y_to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def eight_bit_decode_kernels(monkeypatch):
    # (the 4-bit decode kernel, which takes some of these shapes by default, has no range limit: test_gpu_fp4.py)
    monkeypatch.setenv("BITDELTA_FP4", "0")

# (B, m, N, K): in-kernel split; pre-pass split (B >= 3 tenants of 8 tokens: 32 rows per unit); tiled schedule
SCHEDULES = {"in_kernel_m1": ((4, 1, 256, 512), 2), "prepass_m8": ((5, 8, 256, 512), 1), "tiled_m40": ((2, 40, 256, 512), 0)}


def _inputs(shape, big):
    B, m, N, K = shape
    rng = np.random.default_rng(int(big) % 1000 + B + m)
    x = rng.standard_normal((B, m, K)).astype(np.float32)
    x[:, 0, ::7] = big                       # large magnitudes, both signs, scattered over every 32-k group
    x[:, 0, 3::11] = -big
    x[0, m - 1, :] = big                     # a whole row of them (the delta sum reaches big * K)
    sub = np.float32(2.0**-130)              # a bf16 subnormal
    x[B - 1, m - 1, ::2] = sub
    x[B - 1, m - 1, 1::2] = -sub
    w = (0.02 * rng.standard_normal((N, K))).astype(np.float32)
    bits = rng.integers(0, 2**32, size=(B, N, K // 32), dtype=np.uint32)
    alpha = rng.uniform(0.001, 0.01, B).astype(np.float32)
    return synth.f32_to_bf16_bits(x), synth.f32_to_bf16_bits(w), bits, alpha


def _run(X, W, bits, alpha, **kw):
    dX, dW, dbits, dalpha = to_device(X, W, bits, alpha)
    Y = bd.gemm(dX, dW, dbits, dalpha, **kw)
    st, site = bd.last_device_status()
    return y_to_f64(Y), st


def _gate(Y, Yref):
    tol = np.maximum(2e-2, np.abs(Yref) * 2.0**-8)
    bad = np.abs(Y - Yref) > tol
    assert not bad.any(), f"{int(bad.sum())} outputs off, worst {np.max(np.abs(Y - Yref) / tol):.2f} x the gate"


@pytest.mark.parametrize("big", [2.0**15, 57344.0, 65280.0], ids=["2^15", "57344", "65280"])   # 65280: the largest bf16 below 65504
@pytest.mark.parametrize("name", list(SCHEDULES))
def test_large_and_subnormal_activations_match_the_oracle(name, big):
    shape, schedule = SCHEDULES[name]
    assert bd.gemm_plan(*shape)["schedule"] == schedule
    X, W, bits, alpha = _inputs(shape, big)
    Y, st = _run(X, W, bits, alpha)
    assert st == 0, f"device status {st}"
    assert np.isfinite(Y).all()
    _gate(Y, oracle.gemm(X, W, bits, alpha))


@pytest.mark.parametrize("name", ["in_kernel_m1", "prepass_m8"])
def test_out_of_range_activations_are_clamped_flagged_and_routable(name):
    shape, _ = SCHEDULES[name]
    X, W, bits, alpha = _inputs(shape, 2.0**17)
    Yref = oracle.gemm(X, W, bits, alpha)
    # decode schedule: finite output (no infinity or NaN from the e5m2 pieces), status says what happened, once
    Y, st = _run(X, W, bits, alpha)
    assert st == bd.STATUS_RANGE and np.isfinite(Y).all()
    assert bd.last_device_status()[0] == 0
    # both decode splits clamp alike: the delta term is that of the activations clamped to +-65504
    Xc = synth.f32_to_bf16_bits(np.clip(synth.bf16_bits_to_f32(X), -65280.0, 65280.0))   # (bf16 neighbours of 65504)
    # rows without an out-of-range value are unaffected
    rows_ok = ~(np.abs(synth.bf16_bits_to_f32(X)) >= 2.0**16).any(axis=2)
    _gate(Y[rows_ok], Yref[rows_ok])
    assert Xc.shape == X.shape
    # the wide-range option runs the same call on the tiled schedule: exact, no flag
    Yw, stw = _run(X, W, bits, alpha, wide_range=True)
    assert stw == 0
    _gate(Yw, Yref)
    # a following in-range call is clean again
    X2, W2, bits2, alpha2 = _inputs(shape, 4.0)
    Y2, st2 = _run(X2, W2, bits2, alpha2)
    assert st2 == 0
    _gate(Y2, oracle.gemm(X2, W2, bits2, alpha2))


def test_wide_range_option_small_m_plain_inputs():
    # the tiled schedule at m <= 16 (only reachable through the option): several tenants per unit and one tenant
    for shape in [(8, 1, 384, 512), (1, 3, 256, 256), (3, 16, 200, 384)]:
        wl = synth.Workload("t", B=shape[0], m=shape[1], N=shape[2], K=shape[3], seed=sum(shape))
        X, W, bits, alpha = synth.make_inputs(wl)
        Y, st = _run(X, W, bits, alpha, wide_range=True)
        assert st == 0
        d = Y - oracle.gemm(X, W, bits, alpha)
        assert np.max(np.abs(d)) <= 2e-2
