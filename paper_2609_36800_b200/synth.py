"""Seeded synthetic inputs for the BitDelta fused GEMM.

This module only draws numbers: it holds none of the method's arithmetic and
imports neither the CUDA binding nor the CPU oracle, so both sides can be fed
from it.  bf16 tensors are returned as uint16 bit patterns (numpy has no bf16).

Recipe (one generator per workload, draw order X, W_base, sign words, alpha):
  X      ~ N(0, 1)            float32 -> bf16, round to nearest even
  W_base ~ N(0, w_std)        float32 -> bf16, round to nearest even
  bits   ~ uniform uint32     (i.i.d. signs at 50 % density, 1 bit per weight)
  alpha  ~ U(alpha_lo, alpha_hi) float64 -> float32
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    B: int          # tenants
    m: int          # tokens per tenant
    K: int          # reduction length
    N: int          # output features
    w_std: float = 0.02
    alpha_lo: float = 0.001
    alpha_hi: float = 0.01
    seed: int = 0

    @property
    def flops(self) -> int:
        """Two contractions of 2*B*m*N*K flops each."""
        return 4 * self.B * self.m * self.N * self.K

    @property
    def bytes(self) -> int:
        """Algorithmic bytes: X + W_base + sign words + alpha + Y."""
        B, m, K, N = self.B, self.m, self.K, self.N
        return 2 * B * m * K + 2 * N * K + B * N * K // 8 + 4 * B + 2 * B * m * N


# The five workloads the build is measured on (Llama-shaped projections).
WORKLOADS = (
    Workload("tiny", B=1, m=16, K=512, N=512),
    Workload("decode_attn", B=8, m=1, K=4096, N=4096),
    Workload("decode_mlp_up", B=16, m=4, K=4096, N=11008),
    Workload("prefill", B=4, m=512, K=4096, N=4096),
    Workload("many_tenant_down", B=32, m=8, K=14336, N=4096,
             w_std=0.01, alpha_lo=0.0005, alpha_hi=0.005),
)
WORKLOADS_BY_NAME = {w.name: w for w in WORKLOADS}


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern with round-to-nearest-even (finite inputs)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    """bf16 bit pattern -> the float32 with the same value (exact)."""
    return (np.ascontiguousarray(h, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def make_inputs(wl: Workload, seed: int | None = None):
    """Return (X[B,m,K] u16, W[N,K] u16, bits[B,N,K/32] u32, alpha[B] f32)."""
    rng = np.random.default_rng(wl.seed if seed is None else seed)
    X = f32_to_bf16_bits(rng.standard_normal((wl.B, wl.m, wl.K), dtype=np.float32))
    W = f32_to_bf16_bits(np.float32(wl.w_std) * rng.standard_normal((wl.N, wl.K), dtype=np.float32))
    bits = rng.integers(0, 2**32, size=(wl.B, wl.N, wl.K // 32), dtype=np.uint32)
    alpha = rng.uniform(wl.alpha_lo, wl.alpha_hi, wl.B).astype(np.float32)
    return X, W, bits, alpha


def make_inputs_f16(wl: Workload, seed: int | None = None, with_bias: bool = True):
    """The same recipe in IEEE binary16: (X u16, W u16, bits u32, alpha f32, bias[N] u16 or None), the 16-bit
    arrays being float16 bit patterns (numpy rounds float32 -> float16 to nearest even).  bias ~ N(0, 0.5)."""
    rng = np.random.default_rng(wl.seed if seed is None else seed)
    X = rng.standard_normal((wl.B, wl.m, wl.K), dtype=np.float32).astype(np.float16).view(np.uint16)
    W = (np.float32(wl.w_std) * rng.standard_normal((wl.N, wl.K), dtype=np.float32)).astype(np.float16).view(np.uint16)
    bits = rng.integers(0, 2**32, size=(wl.B, wl.N, wl.K // 32), dtype=np.uint32)
    alpha = rng.uniform(wl.alpha_lo, wl.alpha_hi, wl.B).astype(np.float32)
    bias = (np.float32(0.5) * rng.standard_normal(wl.N, dtype=np.float32)).astype(np.float16).view(np.uint16) if with_bias else None
    return X, W, bits, alpha, bias


def make_bias_bf16(N: int, seed: int = 0) -> np.ndarray:
    """bias[N] ~ N(0, 0.5) as bf16 bit patterns."""
    rng = np.random.default_rng(seed)
    return f32_to_bf16_bits(np.float32(0.5) * rng.standard_normal(N, dtype=np.float32))


def make_signs(B: int, N: int, K: int, seed: int = 0) -> np.ndarray:
    """Dense S int8 [B,N,K] of +1/-1 (input of the packing step)."""
    rng = np.random.default_rng(seed)
    return (rng.integers(0, 2, size=(B, N, K), dtype=np.int8) * 2 - 1).astype(np.int8)


def make_fine_weights(B: int, N: int, K: int, seed: int = 0, w_std: float = 0.02, delta_std: float = 0.004,
                      zero_frac: float = 0.01):
    """Inputs of the compress step: (W_fine[B,N,K] u16, W_base[N,K] u16), bf16 bit patterns.
    W_fine = bf16(W_base + delta) with delta ~ N(0, delta_std) drawn per tenant (a fine-tune moves every
    weight a little, either way); a fraction `zero_frac` of the positions keeps the base value exactly,
    so that zero deltas (which must pack as -1) occur.  No arithmetic of the method lives here."""
    rng = np.random.default_rng(seed)
    Wf32 = np.float32(w_std) * rng.standard_normal((N, K), dtype=np.float32)
    W = f32_to_bf16_bits(Wf32)
    Wb = bf16_bits_to_f32(W)
    fine = np.empty((B, N, K), dtype=np.uint16)
    for b in range(B):
        d = np.float32(delta_std) * rng.standard_normal((N, K), dtype=np.float32)
        keep = rng.random((N, K)) < zero_frac
        fb = f32_to_bf16_bits(Wb + d)
        fb[keep] = W[keep]
        fine[b] = fb
    return fine, W

