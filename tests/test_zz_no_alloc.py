"""bitdelta_gemm_noalloc: the entry point for hosts that may not allocate device memory (a serving
engine after start-up, a plug-in inside a process that owns its whole memory pool).  Its scratch is a
fixed array inside the library, so the caller passes only inputs and the output.

Collected last on purpose: a run that stops at the first failure has then already run every other test.
Each check goes through the C ABI and compares with the existing entry point (bitdelta_gemm with a
caller-owned workspace) on two calls in a row, which also shows that the shared scratch is left usable."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2609_36800_b200 as bd
from paper_2609_36800_b200 import synth

from gpu_util import MAX_ABS_TOL, REL_FRO_TOL, errors, to_device, y_to_f64

pytestmark = pytest.mark.gpu


def _both(wl):
    X, W, bits, alpha = synth.make_inputs(wl)
    dX, dW, dbits, dalpha = to_device(X, W, bits, alpha)
    ref = bd.gemm(dX, dW, dbits, dalpha)                       # existing entry point, own workspace
    out = torch.full((wl.B, wl.m, wl.N), float("nan"), dtype=torch.bfloat16, device="cuda")
    bd.gemm_noalloc(dX, dW, dbits, dalpha, out)                # new entry point, library-held scratch
    st, site = bd.last_device_status()
    assert st == 0, (st, site)
    return y_to_f64(out), y_to_f64(ref), oracle.gemm(X, W, bits, alpha)


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    # two different problems back to back: a cut-across-CTAs decode shape, then a tiled one
    for wl in (synth.Workload("a", B=8, m=1, K=2048, N=1024, seed=31),
               synth.Workload("b", B=2, m=40, K=512, N=384, seed=32),
               synth.Workload("a2", B=8, m=1, K=2048, N=1024, seed=33)):
        got, ref, exact = _both(wl)
        assert not np.isnan(got).any()
        max_abs, rel_fro = errors(got, ref)
        assert max_abs <= MAX_ABS_TOL and rel_fro <= REL_FRO_TOL, (wl.name, max_abs, rel_fro)
        # same kernels, same schedule: in fact identical
        assert np.array_equal(got, ref), wl.name
        # ... and both are the product itself: the fp64 CPU oracle at the parity gates
        max_abs, rel_fro = errors(got, exact)
        assert max_abs <= MAX_ABS_TOL and rel_fro <= REL_FRO_TOL, (wl.name, max_abs, rel_fro)


def test_a_warm_call_allocates_no_device_memory():
    # the entry point's defining property: once the first call on the device has been made, a call leaves the
    # device's free memory exactly as it found it (inputs and output are the caller's, made beforehand)
    wl = synth.Workload("c", B=8, m=1, K=2048, N=1024, seed=34)
    X, W, bits, alpha = synth.make_inputs(wl)
    dX, dW, dbits, dalpha = to_device(X, W, bits, alpha)
    out = torch.empty((wl.B, wl.m, wl.N), dtype=torch.bfloat16, device="cuda")
    bd.gemm_noalloc(dX, dW, dbits, dalpha, out)                # first call on this device (if no test ran before)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        bd.gemm_noalloc(dX, dW, dbits, dalpha, out)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before


def test_shapes_beyond_the_fixed_scratch_are_refused_without_a_launch():
    wl = synth.WORKLOADS_BY_NAME["prefill"]
    assert bd.gemm_workspace_bytes(wl.B, wl.m, wl.N, wl.K) > bd.binding.NOALLOC_SCRATCH_BYTES
    lib = bd.load_library()
    buf = torch.zeros(4096, dtype=torch.uint8, device="cuda")   # never dereferenced: the size check comes first
    p = ctypes.c_void_p(buf.data_ptr())
    before = bd.kernel_launch_count()
    status = lib.bitdelta_gemm_noalloc(p, p, p, p, p, wl.B, wl.m, wl.N, wl.K, None)
    assert status == 4 and "workspace" in bd.status_string(status)
    assert bd.kernel_launch_count() == before
