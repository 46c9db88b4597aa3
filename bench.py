#!/usr/bin/env python
"""Benchmark of the BitDelta fused GEMM on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--all] [--impl reference]

A step is one bitdelta_gemm call (the whole hot path: TMA staging, sign decode,
both contractions, fused epilogue) on one seeded synthetic batch.  The K timed
steps are captured in one CUDA graph and cycle through R independent buffer
sets whose total size exceeds twice the L2, so every launch reads its weights
from HBM.  Prints one JSON line (rank 0).

--impl reference times the fp64 CPU oracle on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_36800_b200 import synth  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
PAPER_CONTEXT = "paper: 3.34x (standard) / 2.51x (batched) over autotuned Triton 3.6.0 on B200, FP16; no absolute figure"

def load_traffic():
    """DRAM bytes per launch of the GEMM kernel from the ncu captures summarised under profiles/."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    try:
        with open(path) as f:
            return {k: v for k, v in json.load(f).items() if not k.startswith("_")}
    except Exception:
        return {}


NCU_TRAFFIC_BYTES = load_traffic()


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# --------------------------------------------------------------------------- ours
def device_sets(wl, X, W, bits, alpha, nsets):
    import torch
    sets = []
    for _ in range(nsets):
        dX = torch.from_numpy(X.view(np.int16)).cuda().view(torch.bfloat16)
        dW = torch.from_numpy(W.view(np.int16)).cuda().view(torch.bfloat16)
        db = torch.from_numpy(bits.view(np.int32)).cuda()
        da = torch.from_numpy(alpha).cuda()
        dY = torch.empty((wl.B, wl.m, wl.N), dtype=torch.bfloat16, device="cuda")
        sets.append((dX, dW, db, da, dY))
    return sets


def time_workload(wl, steps, warmup, dist=None, sampler=None, inputs=None):
    """Returns (ms_total over `steps` launches, nsets).  Device-timed with CUDA events.  `inputs`: host arrays to
    use instead of the workload's own seeded draw (a tenant shard of a larger workload)."""
    import torch
    import paper_2609_36800_b200 as bd

    X, W, bits, alpha = inputs if inputs is not None else synth.make_inputs(wl)
    nsets = max(2, -(-2 * L2_BYTES // wl.bytes))
    sets = device_sets(wl, X, W, bits, alpha, nsets)
    ws = bd.make_workspace(wl.B, wl.m, wl.N, wl.K)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for i in range(max(warmup, 3)):
            s = sets[i % nsets]
            bd.gemm(s[0], s[1], s[2], s[3], out=s[4], workspace=ws)
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for i in range(steps):
                s = sets[i % nsets]
                bd.gemm(s[0], s[1], s[2], s[3], out=s[4], workspace=ws)
        graph.replay()          # untimed replay: graph upload, clocks up
        stream.synchronize()
        st, site = bd.last_device_status()
        if st != 0:
            raise RuntimeError(f"device status {st} at site {site}")
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        if sampler is not None:
            sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        graph.replay()
        e1.record(stream)
        stream.synchronize()
        ms = e0.elapsed_time(e1)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
    return ms, nsets, (X, W, bits, alpha), sets


def batch_stats(wl, sets, batches=20):
    """Per-launch time of short cold-L2 batches (min and median over `batches`), and of a warm-L2 batch
    (one buffer set: everything that fits stays in L2), labelled as such.  Context for the headline
    number, which is the mean over the whole timed graph."""
    import torch
    import paper_2609_36800_b200 as bd

    nsets = len(sets)
    ws = bd.make_workspace(wl.B, wl.m, wl.N, wl.K)
    stream = torch.cuda.Stream()
    out = {}
    with torch.cuda.stream(stream):
        for label, order in (("cold", [i % nsets for i in range(4 * nsets)]), ("warm_l2", [0] * max(8, 2 * nsets))):
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                for i in order:
                    sx = sets[i]
                    bd.gemm(sx[0], sx[1], sx[2], sx[3], out=sx[4], workspace=ws)
            graph.replay()
            stream.synchronize()
            times = []
            for _ in range(batches):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                graph.replay()
                e1.record(stream)
                stream.synchronize()
                times.append(e0.elapsed_time(e1) * 1e3 / len(order))
            times.sort()
            out[label] = {"us_per_launch_min": times[0], "us_per_launch_median": times[len(times) // 2],
                          "launches_per_batch": len(order), "batches": batches}
    out["warm_l2"]["note"] = "one buffer set reused: inputs up to the L2 size stay resident; not a roofline number"
    return out


def host_call_cost(wl, sets, calls=200):
    """Host time of one eager bitdelta_gemm call (argument checks, plan, tensor-map look-up, launch; the ctypes
    marshalling of this binding included), in microseconds: what a caller outside a CUDA graph pays per call."""
    import torch
    import paper_2609_36800_b200 as bd

    ws = bd.make_workspace(wl.B, wl.m, wl.N, wl.K)
    s = sets[0]
    for _ in range(10):
        bd.gemm(s[0], s[1], s[2], s[3], out=s[4], workspace=ws)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(calls):
        bd.gemm(s[0], s[1], s[2], s[3], out=s[4], workspace=ws)
    dt = time.perf_counter() - t0
    torch.cuda.synchronize()
    return dt / calls * 1e6


def time_serialized(wl, sets, launches=24):
    """The same launches without the early start (BITDELTA_EARLY_START=0): every kernel begins only when the one
    before it has completed, so nothing of a call hides behind its predecessor.  Cold L2, one CUDA graph."""
    import torch
    import paper_2609_36800_b200 as bd

    nsets = len(sets)
    ws = bd.make_workspace(wl.B, wl.m, wl.N, wl.K)
    stream = torch.cuda.Stream()
    old = os.environ.get("BITDELTA_EARLY_START")
    os.environ["BITDELTA_EARLY_START"] = "0"
    try:
        with torch.cuda.stream(stream):
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                for i in range(launches):
                    s = sets[i % nsets]
                    bd.gemm(s[0], s[1], s[2], s[3], out=s[4], workspace=ws)
            graph.replay()
            stream.synchronize()
            times = []
            for _ in range(10):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                graph.replay()
                e1.record(stream)
                stream.synchronize()
                times.append(e0.elapsed_time(e1) * 1e3 / launches)
    finally:
        if old is None:
            os.environ.pop("BITDELTA_EARLY_START", None)
        else:
            os.environ["BITDELTA_EARLY_START"] = old
    times.sort()
    return {"us_per_launch_median": times[len(times) // 2], "us_per_launch_min": times[0], "launches": launches,
            "note": "early start off: launch latency, prologue and first loads of every call are exposed"}


def time_compress(peaks, B=8, N=4096, K=4096, steps=20):
    """The setup step before the GEMM (bitdelta_compress) on the headline workload's weight shape:
    HBM-bound scan; inputs (B x N x K bf16 fine weights, 268 MB) are larger than L2, so every launch is cold."""
    import torch
    import paper_2609_36800_b200 as bd

    fine, W = synth.make_fine_weights(B, N, K, seed=0)
    d_fine = torch.from_numpy(fine.view(np.int16)).cuda().view(torch.bfloat16)
    d_W = torch.from_numpy(W.view(np.int16)).cuda().view(torch.bfloat16)
    for _ in range(3):
        bd.compress(d_fine, d_W)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        bd.compress(d_fine, d_W)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / steps
    nbytes = 2 * B * N * K + 2 * N * K + B * N * K // 8 + 4 * B
    gbs = nbytes / (us * 1e-6) / 1e9
    peak = peaks["hbm_gbs"]
    return {"shape": {"B": B, "N": N, "K": K}, "us_per_call": us, "algorithmic_bytes": nbytes,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak},
            "steps": steps, "kernels_per_call": 2}


def time_gemm_ex(wl, peaks, steps=40, act="silu"):
    """The extended call (fp16 operands, bias, SiLU fused into the epilogue) on `wl`, timed like the
    headline: rotating buffer sets larger than L2, all steps in one CUDA graph, CUDA events."""
    import torch
    import paper_2609_36800_b200 as bd

    X, W, bits, alpha, bias = synth.make_inputs_f16(wl)
    nsets = max(2, -(-2 * L2_BYTES // wl.bytes))
    f16 = lambda a: torch.from_numpy(a.view(np.int16)).cuda().view(torch.float16)
    sets = [(f16(X), f16(W), torch.from_numpy(bits.view(np.int32)).cuda(), torch.from_numpy(alpha).cuda(), f16(bias),
             torch.empty((wl.B, wl.m, wl.N // 2 if act == "silu_gate" else wl.N), dtype=torch.float16, device="cuda"))
            for _ in range(nsets)]
    ws = bd.make_workspace(wl.B, wl.m, wl.N, wl.K)
    stream = torch.cuda.Stream()
    call = lambda s: bd.gemm(s[0], s[1], s[2], s[3], out=s[5], workspace=ws, bias=s[4], act=act)
    with torch.cuda.stream(stream):
        for i in range(3):
            call(sets[i % nsets])
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for i in range(steps):
                call(sets[i % nsets])
        graph.replay()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        graph.replay()
        e1.record(stream)
        stream.synchronize()
        ms = e0.elapsed_time(e1)
    st, site = bd.last_device_status()
    if st != 0:
        raise RuntimeError(f"device status {st} at site {site}")
    _, _, roof = summarize(wl, ms, steps, 1, peaks)
    roof["traffic"] = None                       # not captured separately: same loads as the bf16 call plus N bias values
    roof["algorithmic_bytes"] = wl.bytes + 2 * wl.N
    return {"us_per_launch": ms * 1e3 / steps, "steps": steps, "buffer_sets": nsets, "dtype": "f16",
            "epilogue": "bias+" + act, "roofline": roof}


def time_e2e(wl, host_inputs, steps):
    """Same metric through the host-buffer C-ABI entry point: H2D of every input and D2H of Y
    inside the timed region, every step."""
    import torch
    import paper_2609_36800_b200 as bd

    X, W, bits, alpha = host_inputs
    hX = torch.from_numpy(X.view(np.int16)).view(torch.bfloat16).pin_memory()
    hW = torch.from_numpy(W.view(np.int16)).view(torch.bfloat16).pin_memory()
    hb = torch.from_numpy(bits.view(np.int32)).pin_memory()
    ha = torch.from_numpy(alpha).pin_memory()
    hY = torch.empty((wl.B, wl.m, wl.N), dtype=torch.bfloat16).pin_memory()
    arena = torch.empty(bd.gemm_host_arena_bytes(wl.B, wl.m, wl.N, wl.K), dtype=torch.uint8, device="cuda")
    for _ in range(3):
        bd.gemm_host(hX, hW, hb, ha, hY, arena)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        bd.gemm_host(hX, hW, hb, ha, hY, arena)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    h2d = X.nbytes + W.nbytes + bits.nbytes + alpha.nbytes
    d2h = wl.B * wl.m * wl.N * 2
    return ms, h2d, d2h


def cpu_baseline(wl, host_inputs, cpu_seconds=15.0):
    """The fp64 oracle, as it stands, on the host cores over a bounded sample of the workload."""
    import oracle
    X, W, bits, alpha = host_inputs
    cores = oracle.num_threads()
    total = wl.B * wl.m * wl.N
    rng = np.random.default_rng(123)

    def sample(count):
        idx = np.stack([rng.integers(0, wl.B, count), rng.integers(0, wl.m, count),
                        rng.integers(0, wl.N, count)], axis=1).astype(np.int32)
        t0 = time.perf_counter()
        oracle.gemm_at(X, W, bits, alpha, idx)
        return time.perf_counter() - t0

    probe = min(total, 2048)
    rate = probe / max(sample(probe), 1e-9)          # outputs per second
    wall_target = cpu_seconds / max(cores, 1) * 1.5     # ~cpu_seconds CPU-seconds of work
    count = int(min(total, max(probe, rate * wall_target)))
    reps = max(1, int(round(wall_target * rate / count)))
    dt = sum(sample(count) for _ in range(reps))
    frac = count * reps / total
    return {
        "value": wl.bytes * frac / dt / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
        "sample": f"{reps} x {count} of {total} outputs (b,t,n) drawn uniformly, each a full length-{wl.K} fp64 "
                  f"dot pair; {dt:.2f} s wall on {cores} threads",
        "tflops": wl.flops * frac / dt / 1e12,
    }


def kernels_per_step(wl):
    """Kernels one bitdelta_gemm call launches, from the library's own plan: the GEMM kernel, plus an activation
    pre-pass kernel in the 4-bit decode schedule and in the 8-bit decode schedule with more than 16 token rows per
    unit (otherwise the GEMM kernel splits the activations itself)."""
    import paper_2609_36800_b200 as bd
    schedule = bd.gemm_plan(wl.B, wl.m, wl.N, wl.K)["schedule"]
    if schedule in (7, 8):
        return 1 if os.environ.get("BITDELTA_FP4_INKERNEL") else 2
    return 2 if schedule == 1 else 1


def gemm_kernel_name(wl):
    import paper_2609_36800_b200 as bd
    schedule = bd.gemm_plan(wl.B, wl.m, wl.N, wl.K)["schedule"]
    return {7: "bitdelta_gemm_fp4_kernel", 8: "bitdelta_gemm_fp4_kernel", 3: "gemm_simt_kernel"}.get(schedule, "bitdelta_gemm_tc_kernel")


def summarize(wl, ms_total, steps, n_gpus, peaks, clocks=None):
    sec = ms_total / 1e3 / steps
    gbs = wl.bytes * n_gpus / sec / 1e9
    tfl = wl.flops * n_gpus / sec / 1e12
    hbm_bound = wl.m <= 16
    per_gpu_gbs, per_gpu_tfl = gbs / n_gpus, tfl / n_gpus
    if hbm_bound:
        roof = {"bound": "hbm", "achieved": per_gpu_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": per_gpu_gbs / peaks["hbm_gbs"]}
    else:
        # A kernel timed inside a long, power-capped run is held against the sustained cuBLAS figure,
        # one timed in a short burst at full clocks against the burst figure; both fractions are printed.
        capped = bool(clocks and "sw_power_cap" in (clocks.get("reasons") or []))
        burst = peaks["bf16_tflops"]
        sustained = peaks.get("bf16_tflops_sustained", burst)
        peak = sustained if capped else burst
        roof = {"bound": "tensor", "achieved": per_gpu_tfl, "peak": peak, "unit": "TFLOP/s",
                "frac": per_gpu_tfl / peak, "peak_kind": "sustained" if capped else "burst",
                "frac_of_burst": per_gpu_tfl / burst, "frac_of_sustained": per_gpu_tfl / sustained}
    roof["peak_source"] = peaks["_source"]
    roof["traffic"] = NCU_TRAFFIC_BYTES.get(wl.name)
    roof["algorithmic_bytes"] = wl.bytes
    roof["algorithmic_flops"] = wl.flops
    roof["kernel"] = gemm_kernel_name(wl)
    roof["us_per_launch"] = sec * 1e6   # (a whole call: the GEMM kernel and, where the schedule has one, its small pre-pass kernel)
    return gbs, tfl, roof


def run_ours(args):
    import torch
    import paper_2609_36800_b200 as bd

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (sm_100a); there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist = dist_mod
    bd.load_library()
    peaks = load_peaks()
    wl = synth.WORKLOADS_BY_NAME[args.workload]

    if args.ex_only:
        if world != 1:
            raise RuntimeError("--ex-only is a single-GPU run")
        r = time_gemm_ex(wl, peaks, args.steps)
        print(json.dumps({"metric": "bitdelta_gemm_ex " + ("effective HBM GB/s" if wl.m <= 16 else "TFLOP/s"),
                          "value": r["roofline"]["achieved"], "unit": r["roofline"]["unit"], "n_gpus": 1,
                          "steps": args.steps, "warmup": 3, "ms_per_step": r["us_per_launch"] / 1e3,
                          "higher_is_better": True, "dtype": "f16", "data": "synthetic",
                          "config": {"workload": wl.name, "variant": "fp16 operands + bias + SiLU"},
                          "roofline": r["roofline"], "gpu_launches": args.steps * kernels_per_step(wl)}), flush=True)
        return

    # What this rank runs: the whole workload (replicas: every GPU serves its own copy of all tenants), or with
    # --shard-tenants its contiguous share of the workload's tenants (W_base replicated, nothing exchanged).
    full_wl = wl
    shard_inputs = None
    shard_note = None
    if args.shard_tenants and world > 1:
        from paper_2609_36800_b200 import replicas
        Xf, Wf, bitsf, alphaf = synth.make_inputs(wl)
        Xs, bs, als, start = replicas.tenant_shard(Xf, bitsf, alphaf, world, rank)
        if Xs.shape[0] == 0:
            raise RuntimeError(f"--shard-tenants: {wl.B} tenants cannot be cut over {world} GPUs")
        wl = synth.Workload(wl.name, B=int(Xs.shape[0]), m=wl.m, K=wl.K, N=wl.N, w_std=wl.w_std, alpha_lo=wl.alpha_lo,
                            alpha_hi=wl.alpha_hi, seed=wl.seed)
        shard_inputs = (np.ascontiguousarray(Xs), Wf, np.ascontiguousarray(bs), np.ascontiguousarray(als))
        shard_note = f"tenants [{start}, {start + wl.B}) of {full_wl.B} on rank {rank}"

    sampler = ClockSampler(physical_gpu_index(local_rank)) if rank == 0 else None
    launches0 = bd.kernel_launch_count()
    ms, nsets, host_inputs, _sets = time_workload(wl, args.steps, args.warmup, dist, sampler, inputs=shard_inputs)
    clocks = sampler.stop() if sampler is not None else None
    job_bytes, job_flops = float(wl.bytes * world), float(wl.flops * world)
    if dist is not None:
        from paper_2609_36800_b200 import replicas
        ms = replicas.max_over_ranks(ms, dist, device="cuda")
        if shard_inputs is not None:   # ranks may hold different numbers of tenants: add the work up
            tot = torch.tensor([float(wl.bytes), float(wl.flops)], dtype=torch.float64, device="cuda")
            dist.all_reduce(tot, op=dist.ReduceOp.SUM)
            job_bytes, job_flops = float(tot[0].item()), float(tot[1].item())
    stats = batch_stats(wl, _sets) if (rank == 0 and world == 1) else None
    host_cost = host_call_cost(wl, _sets) if (rank == 0 and world == 1) else None
    serial = time_serialized(wl, _sets) if (rank == 0 and world == 1) else None
    del _sets
    torch.cuda.empty_cache()
    gbs, tfl, roof = summarize(wl, ms, args.steps, 1, peaks, clocks)      # this rank's kernel against one GPU's roofline
    sec_per_step = ms / 1e3 / args.steps
    gbs, tfl = job_bytes / sec_per_step / 1e9, job_flops / sec_per_step / 1e12   # whole job: all ranks' work over the slowest rank's time

    out = None
    if rank == 0:
        e2e_steps = max(3, min(args.steps, 20))
        e_ms, h2d, d2h = time_e2e(wl, host_inputs, e2e_steps)
        hbm_bound = wl.m <= 16
        e_val = (wl.bytes if hbm_bound else wl.flops / 1e3) * world / (e_ms / 1e3) / 1e9
        out = {
            "metric": "bitdelta_gemm effective HBM GB/s" if hbm_bound else "bitdelta_gemm TFLOP/s",
            "value": gbs if hbm_bound else tfl,
            "unit": "GB/s" if hbm_bound else "TFLOP/s",
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "strong" if shard_inputs is not None else "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": full_wl.name, "B": full_wl.B, "m": full_wl.m, "K": full_wl.K, "N": full_wl.N,
                       "parallelism": ("single GPU" if world == 1 else
                                       (f"tenants sharded over {world} GPUs, W_base replicated, no data-path collective ({shard_note})"
                                        if shard_inputs is not None else f"{world} replicas (no data-path collective)")),
                       "l2": f"cold: steps cycle through {nsets} buffer sets ({nsets * wl.bytes / 2**20:.0f} MiB > 2x L2)",
                       "launch": "all timed steps in one CUDA graph"},
            "tflops": tfl, "gbs": gbs,
            "roofline": roof,
            "e2e": {"value": e_val, "unit": "GB/s" if hbm_bound else "TFLOP/s", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e_ms, "steps": e2e_steps,
                    "call": "bitdelta_gemm_host (pinned host buffers, stream synchronised each step)"},
            "gpu_launches": args.steps * kernels_per_step(wl),
            "library_launches_issued": bd.kernel_launch_count() - launches0,
            "clocks": clocks,
            "context": PAPER_CONTEXT,
        }
        if stats is not None:
            out["batches"] = stats
        if host_cost is not None:
            out["host_us_per_call"] = host_cost
        if serial is not None:
            out["serialized_launches"] = serial
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline(wl, host_inputs)
        if world == 1 and not args.no_workloads:
            # The other four workloads and the compress step, timed the same way (cold L2, one CUDA graph), short:
            # every configuration's roofline fraction comes out of the one default command.
            others = {}
            for w2 in synth.WORKLOADS:
                if w2.name == wl.name:
                    continue
                steps2 = max(20, min(args.steps, int(0.25 / max(w2.bytes / 6.5e12, w2.flops / 1.6e15)))) if args.all else 20
                ms2, nsets2, _, s2 = time_workload(w2, steps2, 3)
                del s2
                torch.cuda.empty_cache()
                g2, t2, r2 = summarize(w2, ms2, steps2, 1, peaks)
                if args.all:
                    others[w2.name] = {"us_per_launch": ms2 * 1e3 / steps2, "gbs": g2, "tflops": t2, "steps": steps2,
                                       "buffer_sets": nsets2, "roofline": r2}
                else:
                    others[w2.name] = {"us_per_launch": ms2 * 1e3 / steps2, "steps": steps2, "buffer_sets": nsets2,
                                       "bound": r2["bound"], "achieved": r2["achieved"], "unit": r2["unit"],
                                       "peak": r2["peak"], "frac": r2["frac"], "traffic": r2["traffic"]}
            out["workloads"] = others
            out["compress"] = time_compress(peaks)
        if args.all:
            out["gemm_ex"] = {}
            for name in ("decode_attn", "decode_mlp_up", "prefill"):
                w3 = synth.WORKLOADS_BY_NAME[name]
                steps3 = max(20, min(args.steps, int(0.25 / max(w3.bytes / 6.5e12, w3.flops / 1.6e15))))
                out["gemm_ex"][name] = time_gemm_ex(w3, peaks, steps3)
                torch.cuda.empty_cache()
            # the gated-MLP form on the MLP up projection (gate and up rows interleaved along N)
            w4 = synth.WORKLOADS_BY_NAME["decode_mlp_up"]
            out["gemm_ex"]["decode_mlp_up_silu_gate"] = time_gemm_ex(w4, peaks, max(20, min(args.steps, 4000)), act="silu_gate")
            torch.cuda.empty_cache()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if out is not None:
        print(json.dumps(out), flush=True)


# ---------------------------------------------------------------------- reference arm
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    wl = synth.WORKLOADS_BY_NAME[args.workload]
    X, W, bits, alpha = synth.make_inputs(wl)
    total = wl.B * wl.m * wl.N
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rng = np.random.default_rng(123)
    nsteps = args.steps + args.warmup
    probe = min(total, 1024)
    idx = np.stack([rng.integers(0, wl.B, probe), rng.integers(0, wl.m, probe), rng.integers(0, wl.N, probe)],
                   axis=1).astype(np.int32)
    t0 = time.perf_counter()
    oracle.gemm_at(X, W, bits, alpha, idx)
    rate = probe / max(time.perf_counter() - t0, 1e-9)
    count = int(max(64, min(total, rate * 90.0 / nsteps)))      # whole run ~90 s
    idx = np.stack([rng.integers(0, wl.B, count), rng.integers(0, wl.m, count), rng.integers(0, wl.N, count)],
                   axis=1).astype(np.int32)
    for _ in range(args.warmup):
        oracle.gemm_at(X, W, bits, alpha, idx)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.gemm_at(X, W, bits, alpha, idx)
    dt = (time.perf_counter() - t0) / args.steps
    frac = count / total
    hbm_bound = wl.m <= 16
    val = (wl.bytes * frac / dt / 1e9) if hbm_bound else (wl.flops * frac / dt / 1e12)
    unit = "GB/s" if hbm_bound else "TFLOP/s"
    sample = f"{count} of {total} outputs per step, each a full length-{wl.K} fp64 dot pair"
    out = {
        "impl": "reference",
        "metric": "bitdelta_gemm effective HBM GB/s" if hbm_bound else "bitdelta_gemm TFLOP/s",
        "value": val, "unit": unit, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "B": wl.B, "m": wl.m, "K": wl.K, "N": wl.N},
        "cpu_baseline": {"value": val, "unit": unit, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": val, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="decode_attn", choices=sorted(synth.WORKLOADS_BY_NAME))
    ap.add_argument("--all", action="store_true", help="also time the other workloads (N=1 only)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-workloads", action="store_true",
                    help="skip the short timings of the other workloads and of the compress step (N=1)")
    ap.add_argument("--shard-tenants", action="store_true",
                    help="N > 1: every GPU serves its share of the workload's tenants (strong scaling) instead of "
                         "a full replica (weak scaling)")
    ap.add_argument("--ex-only", action="store_true",
                    help="time only the extended call (fp16 operands, bias, SiLU) on --workload and print its "
                         "line; N=1, no end-to-end or CPU leg (used for profiling that kernel instantiation)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # Started as a plain `python bench.py --gpus N`: become N processes, one per GPU, under torchrun
        # (NCCL is used for the barrier and the MAX of the per-rank times only).
        import socket
        import subprocess
        with socket.socket() as s:
            s.bind(("127.0.0.1", 0))
            port = s.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.run(cmd).returncode)
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != max(args.gpus, 1):
        print(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={world}; running {world} rank(s)", file=sys.stderr)
    run_ours(args)


if __name__ == "__main__":
    main()
