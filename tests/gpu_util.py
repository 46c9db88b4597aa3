"""Helpers shared by the GPU tests: host<->device marshalling and the parity gate."""
import numpy as np
import torch

import paper_2609_36800_b200 as bd
from paper_2609_36800_b200 import synth

MAX_ABS_TOL = 2e-2      # max |Y - Y_ref|
REL_FRO_TOL = 5e-3      # ||Y - Y_ref||_F / ||Y_ref||_F


def to_device(X, W, bits, alpha):
    """numpy (uint16 bf16 bits, uint16, uint32, float32) -> CUDA tensors (bf16, bf16, int32, fp32)."""
    dX = torch.from_numpy(X.view(np.int16)).cuda().view(torch.bfloat16)
    dW = torch.from_numpy(W.view(np.int16)).cuda().view(torch.bfloat16)
    dbits = torch.from_numpy(bits.view(np.int32)).cuda()
    dalpha = torch.from_numpy(alpha).cuda()
    return dX, dW, dbits, dalpha


def y_to_f64(Y):
    """bf16 CUDA tensor -> float64 numpy (exact widening)."""
    h = Y.view(torch.int16).cpu().numpy().view(np.uint16)
    return synth.bf16_bits_to_f32(h).astype(np.float64)


def run_gemm(X, W, bits, alpha, simt=False):
    dX, dW, dbits, dalpha = to_device(X, W, bits, alpha)
    Y = bd.gemm(dX, dW, dbits, dalpha, simt=simt)
    st, site = bd.last_device_status()
    assert st == 0, f"device status {st} ({bd.status_string(st)}) at wait site {site}"
    return y_to_f64(Y)


def errors(Y, Yref):
    d = Y - Yref
    return float(np.max(np.abs(d))), float(np.linalg.norm(d) / max(np.linalg.norm(Yref), 1e-300))


def assert_parity(Y, Yref, what=""):
    max_abs, rel_fro = errors(Y, Yref)
    if not (max_abs <= MAX_ABS_TOL and rel_fro <= REL_FRO_TOL):
        # where the outputs beyond the gate sit ([B, m, N]: tenant, token, weight row): points at the tile / role at fault
        d = np.argwhere(np.abs(Y - Yref) > MAX_ABS_TOL)
        where = ""
        if len(d):
            where = (f"; {len(d)} outputs off: tenants {sorted(set(d[:, 0].tolist()))[:8]}, tokens {sorted(set(d[:, 1].tolist()))[:8]}, "
                     f"128-row tiles {sorted(set((d[:, 2] // 128).tolist()))[:12]}, rows in tile {sorted(set((d[:, 2] % 128).tolist()))[:12]}")
        raise AssertionError(f"{what}: max_abs={max_abs:.3e} (tol {MAX_ABS_TOL}), rel_fro={rel_fro:.3e} (tol {REL_FRO_TOL}){where}")
    return max_abs, rel_fro
