"""CPU oracle for the BitDelta fused GEMM.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may
import this package.  It wraps ``bitdelta_oracle.c`` (plain C, fp64) through
ctypes and shares nothing with the CUDA library: no source, no header, no
helper.  Arrays are numpy host arrays; bf16 values travel as uint16 bit
patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bitdelta_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP, strict IEEE arithmetic)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
               "-fno-fast-math", "-ffp-contract=off", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        c_int = ctypes.c_int
        p = ctypes.c_void_p
        lib.oracle_num_threads.restype = c_int
        lib.oracle_set_num_threads.argtypes = [c_int]
        lib.oracle_pack.argtypes = [p, p, c_int, c_int, c_int]
        lib.oracle_unpack.argtypes = [p, p, c_int, c_int, c_int]
        lib.oracle_gemm.argtypes = [p, p, p, p, p, c_int, c_int, c_int, c_int]
        lib.oracle_gemm_at.argtypes = [p, p, p, p, p, c_int, p, c_int, c_int, c_int, c_int]
        lib.oracle_compress.argtypes = [p, p, p, p, c_int, c_int, c_int]
        lib.oracle_half_to_double.argtypes = [p, p, ctypes.c_longlong]
        lib.oracle_gemm_ex.argtypes = [p, p, p, p, p, p, c_int, p, c_int, c_int, c_int, c_int, c_int, c_int]
        _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def _as(a, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.dtype(dtype):
        raise TypeError(f"expected {np.dtype(dtype)}, got {a.dtype}")
    return a


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    _load().oracle_set_num_threads(int(n))


def pack(S: np.ndarray) -> np.ndarray:
    """S int8 [B,N,K] -> words uint32 [B,N,K/32]; bit j of word w is (S[...,32w+j] > 0)."""
    S = _as(S, np.int8)
    B, N, K = S.shape
    if K % 32:
        raise ValueError("K must be a multiple of 32")
    out = np.empty((B, N, K // 32), dtype=np.uint32)
    _load().oracle_pack(_ptr(S), _ptr(out), B, N, K)
    return out


def unpack(bits: np.ndarray) -> np.ndarray:
    """words uint32 [B,N,K/32] -> S int8 [B,N,K] of +1/-1."""
    bits = _as(bits, np.uint32)
    B, N, Wn = bits.shape
    out = np.empty((B, N, Wn * 32), dtype=np.int8)
    _load().oracle_unpack(_ptr(bits), _ptr(out), B, N, Wn * 32)
    return out


def compress(W_fine: np.ndarray, W_base: np.ndarray):
    """W_fine uint16 [B,N,K] and W_base uint16 [N,K] (bf16 bit patterns) -> (bits uint32 [B,N,K/32],
    alpha float32 [B]): bit = (W_fine - W_base > 0), alpha = mean |W_fine - W_base| per tenant."""
    wf = _as(W_fine, np.uint16)
    wb = _as(W_base, np.uint16)
    B, N, K = wf.shape
    if wb.shape != (N, K) or K % 32:
        raise ValueError("inconsistent shapes, or K not a multiple of 32")
    bits = np.empty((B, N, K // 32), dtype=np.uint32)
    alpha = np.empty((B,), dtype=np.float32)
    _load().oracle_compress(_ptr(wf), _ptr(wb), _ptr(bits), _ptr(alpha), B, N, K)
    return bits, alpha


def _check(X, W, bits, alpha):
    X = _as(X, np.uint16)
    W = _as(W, np.uint16)
    bits = _as(bits, np.uint32)
    alpha = _as(alpha, np.float32)
    B, m, K = X.shape
    N, K2 = W.shape
    if K2 != K or K % 32 or bits.shape != (B, N, K // 32) or alpha.shape != (B,):
        raise ValueError("inconsistent shapes")
    return X, W, bits, alpha, B, m, N, K


def gemm(X, W, bits, alpha) -> np.ndarray:
    """Y[b,t,n] = sum_k x w + alpha[b] sum_k x s, in fp64.  X/W are bf16 bit patterns (uint16)."""
    X, W, bits, alpha, B, m, N, K = _check(X, W, bits, alpha)
    Y = np.empty((B, m, N), dtype=np.float64)
    _load().oracle_gemm(_ptr(X), _ptr(W), _ptr(bits), _ptr(alpha), _ptr(Y), B, m, N, K)
    return Y


def gemm_at(X, W, bits, alpha, idx) -> np.ndarray:
    """The same definition at listed outputs only; idx is int32 [count,3] of (b,t,n)."""
    X, W, bits, alpha, B, m, N, K = _check(X, W, bits, alpha)
    idx = _as(idx, np.int32)
    if idx.ndim != 2 or idx.shape[1] != 3:
        raise ValueError("idx must be [count,3]")
    out = np.empty((idx.shape[0],), dtype=np.float64)
    _load().oracle_gemm_at(_ptr(X), _ptr(W), _ptr(bits), _ptr(alpha), _ptr(idx),
                           idx.shape[0], _ptr(out), B, m, N, K)
    return out


DTYPES = {"bf16": 0, "f16": 1}
ACTS = {"none": 0, "silu": 1, "silu_gate": 2}


def half_to_double(h: np.ndarray) -> np.ndarray:
    """IEEE binary16 bit patterns (uint16) -> float64, by the format's definition."""
    h = _as(h, np.uint16)
    out = np.empty(h.shape, dtype=np.float64)
    _load().oracle_half_to_double(_ptr(h), _ptr(out), h.size)
    return out


def gemm_ex(X, W, bits, alpha, bias=None, dtype="bf16", act="none", idx=None) -> np.ndarray:
    """Y = act(sum_k x w + alpha[b] sum_k x s + bias[n]) in fp64.  X, W, bias are 16-bit patterns of
    `dtype` ("bf16" or "f16"); act is "none", "silu", or "silu_gate" (rows 2i / 2i+1 of W are the gate / up
    projections of feature i: Y[b,t,i] = silu(z[2i]) * z[2i+1], N/2 features per token).  With idx (int32
    [count,3] of (b,t,output feature)) only the listed outputs are computed and returned as a vector."""
    X, W, bits, alpha, B, m, N, K = _check(X, W, bits, alpha)
    bp = None
    if bias is not None:
        bias = _as(bias, np.uint16)
        if bias.shape != (N,):
            raise ValueError("bias must have N entries")
        bp = _ptr(bias)
    if idx is not None:
        idx = _as(idx, np.int32)
        if idx.ndim != 2 or idx.shape[1] != 3:
            raise ValueError("idx must be [count,3]")
        out = np.empty((idx.shape[0],), dtype=np.float64)
        ip, cnt = _ptr(idx), idx.shape[0]
    else:
        if act == "silu_gate" and N % 2:
            raise ValueError("silu_gate needs an even N")
        out = np.empty((B, m, N // 2 if act == "silu_gate" else N), dtype=np.float64)
        ip, cnt = None, 0
    _load().oracle_gemm_ex(_ptr(X), _ptr(W), _ptr(bits), _ptr(alpha), bp, ip, cnt, _ptr(out),
                           B, m, N, K, DTYPES[dtype], ACTS[act])
    return out
