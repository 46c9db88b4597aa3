"""ctypes binding of libbitdelta.so (see include/bitdelta.h).

Argument marshalling only: torch supplies device memory and streams, every
step of the computation runs in the library's CUDA kernels.  Nothing here falls
back to the CPU: a missing library or a non-sm_100 device raises.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
# BITDELTA_LIB points at another build of the same library (the trace build made by `build.py --trace`).
_LIB_PATH = os.environ.get("BITDELTA_LIB") or os.path.join(_HERE, "libbitdelta.so")
_lib = None

STATUS_OK = 0
STATUS_TIMEOUT = 7
STATUS_RANGE = 9
DTYPE_WIDE_RANGE = 0x100

EXPORTS = (
    "bitdelta_pack", "bitdelta_unpack", "bitdelta_compress_workspace_bytes", "bitdelta_compress",
    "bitdelta_gemm_workspace_bytes", "bitdelta_workspace_init",
    "bitdelta_gemm", "bitdelta_gemm_ex", "bitdelta_gemm_noalloc", "bitdelta_gemm_simt", "bitdelta_gemm_host_arena_bytes", "bitdelta_gemm_host",
    "bitdelta_gemm_plan", "bitdelta_gemm_plan_cta_items", "bitdelta_gemm_plan_item_cta",
    "bitdelta_last_device_status", "bitdelta_kernel_launch_count", "bitdelta_status_string", "bitdelta_selftest_timeout",
)


class BitDeltaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Load libbitdelta.so (built in-tree by paper_2609_36800_b200.build); raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2609_36800_b200.build` "
            "(there is no CPU fallback)")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, ci, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    lib.bitdelta_pack.argtypes = [vp, vp, ci, ci, ci, vp]
    lib.bitdelta_unpack.argtypes = [vp, vp, ci, ci, ci, vp]
    lib.bitdelta_compress_workspace_bytes.argtypes = [ci, ci, ci]
    lib.bitdelta_compress_workspace_bytes.restype = sz
    lib.bitdelta_compress.argtypes = [vp, vp, vp, vp, ci, ci, ci, vp, sz, vp]
    lib.bitdelta_gemm_workspace_bytes.argtypes = [ci, ci, ci, ci]
    lib.bitdelta_gemm_workspace_bytes.restype = sz
    lib.bitdelta_workspace_init.argtypes = [vp, sz, vp]
    lib.bitdelta_gemm.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, vp, sz, vp]
    lib.bitdelta_gemm_ex.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, vp, sz, vp]
    lib.bitdelta_gemm_simt.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, vp]
    lib.bitdelta_gemm_noalloc.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, vp]
    lib.bitdelta_gemm_host_arena_bytes.argtypes = [ci, ci, ci, ci]
    lib.bitdelta_gemm_host_arena_bytes.restype = sz
    lib.bitdelta_gemm_host.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, vp, sz, vp]
    lib.bitdelta_gemm_plan.argtypes = [ci, ci, ci, ci, ci, ctypes.POINTER(ci)]
    lib.bitdelta_gemm_plan_cta_items.argtypes = [ci, ci, ci, ci, ci, ci, ctypes.POINTER(ci), ctypes.POINTER(ci)]
    lib.bitdelta_gemm_plan_item_cta.argtypes = [ci, ci, ci, ci, ci, ci]
    lib.bitdelta_last_device_status.argtypes = [vp, ctypes.POINTER(ci)]
    lib.bitdelta_kernel_launch_count.restype = ctypes.c_ulonglong
    lib.bitdelta_selftest_timeout.argtypes = [ctypes.c_longlong, ci, vp]
    lib.bitdelta_status_string.argtypes = [ci]
    lib.bitdelta_status_string.restype = ctypes.c_char_p
    for fn in ("bitdelta_pack", "bitdelta_unpack", "bitdelta_compress", "bitdelta_workspace_init", "bitdelta_gemm",
               "bitdelta_gemm_simt", "bitdelta_gemm_noalloc", "bitdelta_gemm_host", "bitdelta_last_device_status"):
        getattr(lib, fn).restype = ci
    _lib = lib
    return lib


def selftest_timeout(limit_cycles: int = 1_000_000, site: int = 99, stream=None) -> None:
    """Queues the one-warp kernel whose bounded wait expires after `limit_cycles`; last_device_status() then
    reports (STATUS_TIMEOUT, site) once."""
    _check(load_library().bitdelta_selftest_timeout(int(limit_cycles), int(site), _stream_ptr(stream)), "bitdelta_selftest_timeout")


def status_string(status: int) -> str:
    return load_library().bitdelta_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != STATUS_OK:
        raise BitDeltaError(status, where)


def _stream_ptr(stream=None):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _dev(t, dtype, name):
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name} must be a contiguous CUDA tensor of dtype {dtype}")
    return ctypes.c_void_p(t.data_ptr())


def pack(S, stream=None):
    """S int8 [B,N,K] (device) -> packed sign words, int32 storage [B,N,K/32] (bit j of word w <-> k = 32w+j)."""
    import torch
    B, N, K = S.shape
    bits = torch.empty((B, N, K // 32), dtype=torch.int32, device=S.device)
    _check(load_library().bitdelta_pack(_dev(S, torch.int8, "S"), ctypes.c_void_p(bits.data_ptr()),
                                        B, N, K, _stream_ptr(stream)), "bitdelta_pack")
    return bits


def unpack(bits, stream=None):
    """Packed sign words [B,N,K/32] (int32 storage, device) -> S int8 [B,N,K] of +1/-1."""
    import torch
    B, N, Wn = bits.shape
    S = torch.empty((B, N, Wn * 32), dtype=torch.int8, device=bits.device)
    _check(load_library().bitdelta_unpack(_dev(bits, torch.int32, "bits"), ctypes.c_void_p(S.data_ptr()),
                                          B, N, Wn * 32, _stream_ptr(stream)), "bitdelta_unpack")
    return S


def compress(W_fine, W_base, stream=None, bits=None, alpha=None):
    """Fine-tuned weights bf16 [B,N,K] and base weights bf16 [N,K] (device) -> (bits int32 storage
    [B,N,K/32], alpha fp32 [B]): bit = (W_fine - W_base > 0), alpha = mean |W_fine - W_base| per tenant.
    `bits` / `alpha`: caller's output tensors (allocated here if omitted)."""
    import torch
    lib = load_library()
    B, N, K = W_fine.shape
    if tuple(W_base.shape) != (N, K) or K % 32:
        raise ValueError("inconsistent shapes, or K not a multiple of 32")
    if bits is None:
        bits = torch.empty((B, N, K // 32), dtype=torch.int32, device=W_fine.device)
    if alpha is None:
        alpha = torch.empty((B,), dtype=torch.float32, device=W_fine.device)
    if tuple(bits.shape) != (B, N, K // 32) or tuple(alpha.shape) != (B,):
        raise ValueError("inconsistent output shapes")
    nbytes = int(lib.bitdelta_compress_workspace_bytes(B, N, K))
    ws = torch.empty(max(nbytes, 8), dtype=torch.uint8, device=W_fine.device)
    _check(lib.bitdelta_compress(_dev(W_fine, torch.bfloat16, "W_fine"), _dev(W_base, torch.bfloat16, "W_base"),
                                 _dev(bits, torch.int32, "bits"), _dev(alpha, torch.float32, "alpha"), B, N, K,
                                 ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream_ptr(stream)), "bitdelta_compress")
    return bits, alpha


def gemm_workspace_bytes(B: int, m: int, N: int, K: int) -> int:
    return int(load_library().bitdelta_gemm_workspace_bytes(B, m, N, K))


def make_workspace(B: int, m: int, N: int, K: int, device="cuda", stream=None):
    """Allocate and prepare a workspace for bitdelta_gemm on this shape."""
    import torch
    nbytes = gemm_workspace_bytes(B, m, N, K)
    if nbytes == 0:
        raise BitDeltaError(2, "bitdelta_gemm_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    _check(load_library().bitdelta_workspace_init(ctypes.c_void_p(ws.data_ptr()), nbytes, _stream_ptr(stream)),
           "bitdelta_workspace_init")
    return ws


ACTS = {"none": 0, "silu": 1, "silu_gate": 2}


def gemm(X, W_base, bits, alpha, out=None, workspace=None, stream=None, simt: bool = False, bias=None,
         act: str = "none", wide_range: bool = False):
    """Y[b,t,n] = act(sum_k X W_base + alpha[b] sum_k X S + bias[n]).  X [B,m,K] and W_base [N,K] in bf16 or
    (both) fp16, bits int32 storage [B,N,K/32], alpha fp32 [B], optional bias [N] of X's type, act "none", "silu"
    or "silu_gate" (rows 2i / 2i+1 are gate / up projections: Y[b,t,i] = silu(z[2i]) * z[2i+1], Y is [B,m,N/2]);
    returns Y [B,m,N] of X's type.  wide_range=True plans every m on the tiled schedule (for activations of
    magnitude 2^16 or more, which the decode schedules clamp and flag).  (simt=True runs the diagnostic
    CUDA-core kernel: bf16, no epilogue.)"""
    import torch
    lib = load_library()
    B, m, K = X.shape
    N = W_base.shape[0]
    if W_base.shape != (N, K) or tuple(bits.shape) != (B, N, K // 32) or tuple(alpha.shape) != (B,):
        raise ValueError("inconsistent shapes")
    io = X.dtype
    if io not in (torch.bfloat16, torch.float16):
        raise TypeError("X must be bfloat16 or float16")
    if act not in ACTS:
        raise ValueError(f"unknown activation {act!r}")
    if bias is not None and tuple(bias.shape) != (N,):
        raise ValueError("bias must have N entries")
    if act == "silu_gate" and N % 2:
        raise ValueError("silu_gate needs an even N (interleaved gate / up rows)")
    if out is None:
        out = torch.empty((B, m, N // 2 if act == "silu_gate" else N), dtype=io, device=X.device)
    args = [_dev(X, io, "X"), _dev(W_base, io, "W_base"), _dev(bits, torch.int32, "bits"),
            _dev(alpha, torch.float32, "alpha")]
    shape = [B, m, N, K]
    if simt:
        if io != torch.bfloat16 or bias is not None or act != "none":
            raise ValueError("the diagnostic kernel takes bf16 and has no epilogue")
        _check(lib.bitdelta_gemm_simt(*args, _dev(out, io, "out"), *shape, _stream_ptr(stream)), "bitdelta_gemm_simt")
        return out
    if workspace is None:
        workspace = make_workspace(B, m, N, K, device=X.device, stream=stream)
    ws = (ctypes.c_void_p(workspace.data_ptr()), workspace.numel(), _stream_ptr(stream))
    if io == torch.bfloat16 and bias is None and act == "none" and not wide_range:
        _check(lib.bitdelta_gemm(*args, _dev(out, io, "out"), *shape, *ws), "bitdelta_gemm")
    else:
        bp = _dev(bias, io, "bias") if bias is not None else ctypes.c_void_p(0)
        _check(lib.bitdelta_gemm_ex(*args, bp, _dev(out, io, "out"), *shape,
                                    (1 if io == torch.float16 else 0) | (DTYPE_WIDE_RANGE if wide_range else 0),
                                    ACTS[act], *ws), "bitdelta_gemm_ex")
    return out


PLAN_FIELDS = ("schedule", "blocks", "tenants_per_unit", "units", "k_steps", "order", "teams", "smem_bytes",
               "w_ring", "x_ring", "piece_ring", "operand_buffers", "handovers_per_k_step", "token_tile", "groups",
               "w_tiles")


def gemm_plan(B: int, m: int, N: int, K: int, num_sms: int = 148) -> dict:
    """How bitdelta_gemm would run this shape (host-only query): schedule, blocks, work order, ring depths."""
    info = (ctypes.c_int * 16)()
    _check(load_library().bitdelta_gemm_plan(B, m, N, K, num_sms, info), "bitdelta_gemm_plan")
    return dict(zip(PLAN_FIELDS, list(info)))


def gemm_plan_cta_items(B: int, m: int, N: int, K: int, cta: int, num_sms: int = 148):
    """Items [first, end) of the flat (unit, k-step) work list that thread block `cta` takes."""
    first, end = ctypes.c_int(0), ctypes.c_int(0)
    _check(load_library().bitdelta_gemm_plan_cta_items(B, m, N, K, num_sms, cta, ctypes.byref(first), ctypes.byref(end)),
           "bitdelta_gemm_plan_cta_items")
    return first.value, end.value


def gemm_plan_item_cta(B: int, m: int, N: int, K: int, item: int, num_sms: int = 148) -> int:
    return int(load_library().bitdelta_gemm_plan_item_cta(B, m, N, K, num_sms, item))


NOALLOC_SCRATCH_BYTES = 16 * 1024 * 1024


def gemm_noalloc(X, W_base, bits, alpha, out, stream=None):
    """bitdelta_gemm for callers that may not allocate device memory: same arguments as `gemm` with a
    caller-provided `out`, no workspace.  The scratch is a fixed array inside the library (16 MiB per GPU);
    shapes needing more raise BitDeltaError(status 4).  Calls that may overlap on the device race on it."""
    import torch
    B, m, K = X.shape
    N = W_base.shape[0]
    if W_base.shape != (N, K) or tuple(bits.shape) != (B, N, K // 32) or tuple(alpha.shape) != (B,) \
            or tuple(out.shape) != (B, m, N):
        raise ValueError("inconsistent shapes")
    _check(load_library().bitdelta_gemm_noalloc(
        _dev(X, torch.bfloat16, "X"), _dev(W_base, torch.bfloat16, "W_base"), _dev(bits, torch.int32, "bits"),
        _dev(alpha, torch.float32, "alpha"), _dev(out, torch.bfloat16, "out"), B, m, N, K, _stream_ptr(stream)),
        "bitdelta_gemm_noalloc")
    return out


def gemm_host_arena_bytes(B: int, m: int, N: int, K: int) -> int:
    return int(load_library().bitdelta_gemm_host_arena_bytes(B, m, N, K))


def gemm_host(X, W_base, bits, alpha, out, arena, stream=None):
    """Host-buffer form: all tensors are CPU tensors (pinned for asynchronous copies), `arena` is a
    CUDA uint8 tensor of gemm_host_arena_bytes.  Returns `out` (complete on return)."""
    import torch
    B, m, K = X.shape
    N = W_base.shape[0]
    for t, dt, nm in ((X, torch.bfloat16, "X"), (W_base, torch.bfloat16, "W_base"), (bits, torch.int32, "bits"),
                      (alpha, torch.float32, "alpha"), (out, torch.bfloat16, "out")):
        if t.is_cuda or t.dtype != dt or not t.is_contiguous():
            raise TypeError(f"{nm} must be a contiguous CPU tensor of dtype {dt}")
    _check(load_library().bitdelta_gemm_host(
        ctypes.c_void_p(X.data_ptr()), ctypes.c_void_p(W_base.data_ptr()), ctypes.c_void_p(bits.data_ptr()),
        ctypes.c_void_p(alpha.data_ptr()), ctypes.c_void_p(out.data_ptr()), B, m, N, K,
        ctypes.c_void_p(arena.data_ptr()), arena.numel(), _stream_ptr(stream)), "bitdelta_gemm_host")
    return out


def last_device_status(stream=None):
    """Synchronise and return (status, site) of the device-side bounded waits."""
    site = ctypes.c_int(0)
    st = load_library().bitdelta_last_device_status(_stream_ptr(stream), ctypes.byref(site))
    return int(st), int(site.value)


def kernel_launch_count() -> int:
    return int(load_library().bitdelta_kernel_launch_count())
