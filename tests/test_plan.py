"""Host logic of the work decomposition, through the plan queries of the C ABI (no GPU needed): whatever the
shape, every (unit, k-step) item must be taken by exactly one thread block, the inverse map must agree, and
the properties the kernel relies on (at most two cut tiles per block, teams aligned with tenant groups) hold."""
import numpy as np
import pytest

import paper_2609_36800_b200 as bd
from paper_2609_36800_b200 import synth

SHAPES = [(w.B, w.m, w.N, w.K) for w in synth.WORKLOADS] + [
    (1, 1, 128, 128), (2, 1, 200, 256), (20, 1, 128, 256), (12, 8, 6400, 256), (33, 2, 1920, 384),
    (80, 1, 3712, 256), (3, 16, 264, 384), (2, 17, 256, 384), (2, 300, 136, 512), (16, 4, 4096, 8192),
    (5, 3, 130, 384), (64, 2, 512, 1024), (24, 2, 1280, 1024), (7, 9, 256, 256),
    (5, 20, 384, 512), (9, 24, 1280, 1024), (8, 32, 4096, 4096), (8, 64, 4096, 4096),
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "B%d_m%d_N%d_K%d" % s)
@pytest.mark.parametrize("sms", [148, 132, 7])
def test_every_item_is_taken_exactly_once(shape, sms):
    B, m, N, K = shape
    info = bd.gemm_plan(B, m, N, K, num_sms=sms)
    blocks, units, P, order, teams = info["blocks"], info["units"], info["k_steps"], info["order"], info["teams"]
    T = units * P
    assert 1 <= blocks <= sms
    pair = info["schedule"] == 4     # a unit is two W_base tiles, two thread blocks share every share of the list
    assert P == K // 128 and units == info["w_tiles"] * info["groups"] // (2 if pair else 1)
    if pair:
        assert blocks % 2 == 0 and info["w_tiles"] % 2 == 0 and order == 0
        for b in range(0, blocks, 2):
            assert bd.gemm_plan_cta_items(B, m, N, K, b, num_sms=sms) == bd.gemm_plan_cta_items(B, m, N, K, b + 1, num_sms=sms)
    step = 2 if pair else 1
    if order == 1:
        # whole units round-robin: block b starts at unit b; all units are reached when blocks <= units
        assert blocks <= units
        for b in (0, blocks - 1):
            assert bd.gemm_plan_cta_items(B, m, N, K, b, num_sms=sms) == (b * P, b * P + P)
        for item in (0, T - 1, T // 2):
            assert bd.gemm_plan_item_cta(B, m, N, K, item, num_sms=sms) == (item // P) % blocks
        return
    ranges = [bd.gemm_plan_cta_items(B, m, N, K, b, num_sms=sms) for b in range(0, blocks, step)]
    # contiguous, in order, covering [0, T)
    assert ranges[0][0] == 0 and ranges[-1][1] == T
    for (lo, hi), (lo2, _) in zip(ranges, ranges[1:]):
        assert hi == lo2
    sizes = [hi - lo for lo, hi in ranges]
    assert min(sizes) >= 1
    if order == 3:
        # clusters: every unit belongs to one cluster of blocks / units blocks, no block's share crosses a unit
        assert blocks % units == 0 and blocks // units in (2, 4, 8)
        for b, (lo, hi) in enumerate(ranges):
            assert lo // P == (hi - 1) // P == b // (blocks // units)
    if order == 2:
        assert teams == info["groups"] and blocks % teams == 0
        cpt, Tg = blocks // teams, T // teams
        assert Tg == info["w_tiles"] * P
        for t in range(teams):
            team = ranges[t * cpt:(t + 1) * cpt]
            assert team[0][0] == t * Tg and team[-1][1] == (t + 1) * Tg        # a team owns exactly its group's items
            s = [hi - lo for lo, hi in team]
            assert max(s) - min(s) <= 1
            # the same cut in every team: block i of each team is at the same (tile, k-step)
            assert [lo - t * Tg for lo, _ in team] == [lo for lo, _ in ranges[:cpt]]
    else:
        assert teams == 1 and max(sizes) - min(sizes) <= 1
    # a block cuts at most two tiles (its first and its last): it owns two partial-result slots
    for lo, hi in ranges:
        cut = sum(1 for u in range(lo // P, (hi - 1) // P + 1) if max(lo, u * P) > u * P or min(hi, (u + 1) * P) < (u + 1) * P)
        assert cut <= 2
    # inverse map
    rng = np.random.default_rng(0)
    items = range(T) if T <= 4096 else sorted(set(rng.integers(0, T, 2048).tolist()) | {0, T - 1} | {lo for lo, _ in ranges} | {hi - 1 for _, hi in ranges})
    starts = np.array([lo for lo, _ in ranges])
    for item in items:
        assert bd.gemm_plan_item_cta(B, m, N, K, item, num_sms=sms) == step * int(np.searchsorted(starts, item, side="right") - 1)


def test_schedules_and_work_orders_of_the_measured_workloads():
    got = {w.name: bd.gemm_plan(w.B, w.m, w.N, w.K) for w in synth.WORKLOADS}
    # one tenant group, eight tokens per unit: the 4-bit decode kernel in clusters of four blocks per W_base tile
    assert got["decode_attn"]["schedule"] == 8 and got["decode_attn"]["order"] == 3 and got["decode_attn"]["blocks"] == 128
    assert got["tiny"]["schedule"] == 2
    # two tenant groups of four token rows per tenant: the 4-bit decode kernel on the flat list, one team per group
    assert got["decode_mlp_up"]["schedule"] == 7 and got["decode_mlp_up"]["order"] == 2 and got["decode_mlp_up"]["teams"] == 2
    # eight token rows per tenant, eight groups: the 8-bit decode kernel
    assert got["many_tenant_down"]["schedule"] == 1
    assert got["many_tenant_down"]["order"] == 2 and got["many_tenant_down"]["teams"] == 8 and got["many_tenant_down"]["blocks"] == 144
    assert got["prefill"]["schedule"] == 4 and got["prefill"]["order"] == 0 and got["prefill"]["blocks"] == 148
    for g in got.values():
        assert g["smem_bytes"] <= 227 * 1024 and g["w_ring"] >= 2 and g["operand_buffers"] >= 2


def test_four_bit_decode_kernel_plans(monkeypatch):
    # default: where its cluster form applies, and on the flat work list with up to four token rows per tenant;
    # BITDELTA_FP4=0 never; BITDELTA_FP4=1 wherever it applies
    assert bd.gemm_plan(8, 1, 4096, 4096)["schedule"] == 8 and bd.gemm_plan(4, 8, 4096, 4096)["schedule"] == 8
    assert bd.gemm_plan(16, 1, 4096, 4096)["schedule"] == 7          # two tenant groups: no clusters, the flat list
    assert bd.gemm_plan(16, 8, 4096, 4096)["schedule"] in (1, 2)     # ... with more than four token rows per tenant: the 8-bit kernel
    assert bd.gemm_plan(8, 9, 4096, 4096)["schedule"] == 1           # more than eight tokens per tenant
    one = bd.gemm_plan(8, 1, 4096, 4096)
    assert one["smem_bytes"] <= 227 * 1024 and one["w_ring"] >= 3
    for b in range(one["blocks"]):
        lo, hi = bd.gemm_plan_cta_items(8, 1, 4096, 4096, b)
        assert hi - lo == 8 and lo // 32 == b // 4 and bd.gemm_plan_item_cta(8, 1, 4096, 4096, lo) == b
    monkeypatch.setenv("BITDELTA_FP4", "0")
    off = bd.gemm_plan(8, 1, 4096, 4096)
    assert off["schedule"] == 2 and off["order"] == 0 and off["blocks"] == 148
    monkeypatch.setenv("BITDELTA_FP4", "1")
    assert bd.gemm_plan(16, 4, 11008, 4096)["schedule"] == 7 and bd.gemm_plan(32, 8, 4096, 14336)["schedule"] == 7
    # the workspace covers every schedule a call may take
    monkeypatch.delenv("BITDELTA_FP4")
    assert bd.gemm_workspace_bytes(8, 1, 4096, 4096) >= 32 * 9 * 1024


def test_cuda_core_path_and_bad_arguments():
    assert bd.gemm_plan(2, 3, 96, 96)["schedule"] == 3
    lib = bd.load_library()
    import ctypes
    info = (ctypes.c_int * 16)()
    assert lib.bitdelta_gemm_plan(1, 1, 128, 100, 148, info) == 2
    assert lib.bitdelta_gemm_plan(1, 1, 128, 128, 148, None) == 1
    assert lib.bitdelta_gemm_plan_item_cta(1, 1, 128, 128, 148, 5) == -1          # only one item
    a, b = ctypes.c_int(), ctypes.c_int()
    assert lib.bitdelta_gemm_plan_cta_items(1, 1, 128, 128, 148, 3, ctypes.byref(a), ctypes.byref(b)) == 2   # one block only


def test_work_lists_beyond_the_32_bit_split_arithmetic_are_refused():
    # 8192 W_base tiles x 512 tenant groups x 256 k-steps = 2^30 items: one too many for the kernel's 32-bit split
    B, m, N, K = 4096, 1, 1 << 20, 1 << 15
    assert bd.gemm_workspace_bytes(B, m, N, K) == 0
    import ctypes
    info = (ctypes.c_int * 16)()
    assert bd.load_library().bitdelta_gemm_plan(B, m, N, K, 148, info) == 2
    # just below the limit the plan exists
    assert bd.gemm_plan(B, m, N // 2, K)["units"] * bd.gemm_plan(B, m, N // 2, K)["k_steps"] == 1 << 29
