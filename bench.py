#!/usr/bin/env python
"""Benchmark of the prob-sparse attention forward path (steps (a)-(e) of Sec. 3 of the paper).

One "step" = one psattn_forward over one batch of a seeded synthetic workload.
  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]
For N > 1 launch with torch.distributed.run; every rank runs the same per-GPU batch (weak
scaling, no collective on the data path: (batch, head) units are independent).
Prints ONE JSON line on rank 0.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2106_09236_b200 import sharding  # noqa: E402
from paper_2106_09236_b200 import workloads as wl  # noqa: E402

METRIC = "prob-sparse attention queries/s"
UNIT = "queries/s"
L2_BYTES = 126e6


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def tensor_peak():
    """Dense bf16 tensor throughput (TFLOP/s) for a kernel timed alone: the measured burst figure."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops"]), "measured"
    except Exception:
        return 1590.0, "fallback"


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum per launch) of the dominant kernel from the
# ncu capture summarised under profiles/, valid only while the kernel's sources are unchanged.
_FUSED_SOURCES = ["psattn_fused.cu", "psattn_measure_mma.cuh", "psattn_attend64.cuh", "psattn_select.cuh",
                  "psattn_sm100.cuh", "psattn_common.cuh"]
_STREAM_SOURCES = ["psattn_measure_mma.cu", "psattn_measure_stream.cuh", "psattn_measure_mma.cuh",
                   "psattn_sm100.cuh", "psattn_common.cuh"]
TRAFFIC = {
    "large_bf16": {"kernel": "k_forward_fused", "bytes": 53625856, "sources": _FUSED_SOURCES,
                   "profile": "profiles/ncu_full_k_forward_fused_large_bf16.txt",
                   "sources_sha1": "30622772007f5c0e35b61ed38bfeef9d342cf0d9"},
    "long_bf16": {"kernel": "k_measure_stream", "bytes": 76343808, "sources": _STREAM_SOURCES,
                  "profile": "profiles/ncu_full_k_measure_stream_long_bf16.txt",
                  "sources_sha1": "2cefd328bfe39e8941e1eea3f3e682bc492120bf"},
}


def sources_sha1(files):
    import hashlib
    h = hashlib.sha1()
    for f in files:
        with open(os.path.join(ROOT, "paper_2106_09236_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def recorded_traffic(workload):
    """Bytes per launch from the recorded capture, or None if there is none or the kernel changed."""
    rec = TRAFFIC.get(workload)
    if rec is None:
        return None
    try:
        return rec["bytes"] if sources_sha1(rec["sources"]) == rec["sources_sha1"] else None
    except OSError:
        return None


def algorithmic_bytes(w, lengths, count, elem):
    """Bytes the method itself must move: Q, K, V read once, O written once, the used part of
    sample_idx (shared by heads), sel_idx, lengths."""
    total = 0
    for L in lengths:
        L = int(L)
        n = count(w.c, L)
        total += w.H * L * w.d * (3 * elem + elem) + L * n * 4 + w.H * n * 4
    return total + 4 * len(lengths)


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                break
            time.sleep(0.002)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def cpu_oracle_timing(w, n_cols, steps=None, warmup=0, budget_s=12.0):
    """Times the CPU oracle (as it stands, all host cores over (batch, head) units) on the whole
    batch of the workload.  steps=None: one pass to calibrate, then as many passes as fit in about
    `budget_s` seconds of CPU work."""
    from oracle import psattn_oracle as orc
    inp = wl.make_inputs(w, n_cols)
    cores = orc.max_threads()
    queries = int(inp["lengths"].sum()) * w.H

    def one():
        orc.forward(inp["Q"], inp["K"], inp["V"], inp["sample_idx"], inp["lengths"], c=w.c, nthreads=cores)

    for _ in range(warmup):
        one()
    if steps is None:
        t0 = time.perf_counter()
        one()
        first = time.perf_counter() - t0
        steps = int(max(1, min(200, budget_s / max(first, 1e-3))))
    t0 = time.perf_counter()
    for _ in range(steps):
        one()
    dt = (time.perf_counter() - t0) / steps
    return queries / dt, cores, dt, queries, steps


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import psattn_oracle as orc
    n_cols = max(orc.count(w.c, L) for L in range(1, w.T + 1))
    steps = max(1, min(args.steps, 50))
    warm = max(0, min(args.warmup, 2))
    qps, cores, dt, queries, _ = cpu_oracle_timing(w, n_cols, steps, warm)
    sample = "whole batch of %s (%d valid queries) per step" % (w.name, queries)
    line = {
        "impl": "reference", "metric": METRIC, "value": qps, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "T": w.T, "d_head": w.d, "c": w.c},
        "cpu_baseline": {"value": qps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": qps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def time_events(fn, steps, torch, grouped=False):
    """Runs fn(k) for k in range(steps) between two CUDA events on the current stream."""
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    start.record()
    for k in range(steps):
        if grouped:
            fn(k, steps)
        else:
            fn(k)
    end.record()
    torch.cuda.synchronize()
    return start.elapsed_time(end) / steps      # ms per step


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="large_bf16", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--path", default="auto", choices=["auto", "staged", "fused"])
    ap.add_argument("--no-graph", action="store_true", help="time direct calls instead of CUDA-graph replays")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle timing")
    ap.add_argument("--no-dense", action="store_true", help="skip the dense comparator timing")
    ap.add_argument("--no-variants", action="store_true",
                    help="skip the selection-reuse and paper-literal timings")
    args = ap.parse_args()
    w = wl.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    from paper_2106_09236_b200 import binding as ps

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    tdt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    elem = 2 if w.dtype == "bf16" else 4
    n_cols = max(ps.psattn_count(w.c, L) for L in range(1, w.T + 1))
    path = {"auto": ps.PSATTN_PATH_AUTO, "staged": ps.PSATTN_PATH_STAGED, "fused": ps.PSATTN_PATH_FUSED}[args.path]
    plan = ps.Plan(w.B, w.H, w.T, dtype=tdt, c=w.c, idx_cols=n_cols, path=path)

    # enough independent buffer sets that a set is evicted from L2 before it is used again
    per_set = 4 * w.B * w.H * w.T * w.d * elem + w.B * w.T * n_cols * 4
    n_sets = max(2, int(np.ceil(2.2 * L2_BYTES / per_set)) + 1)
    sets, host_sets, queries_per_step, alg_bytes = [], [], None, None
    for s in range(n_sets):
        inp = wl.make_inputs(w, n_cols, seed=sharding.rank_seed(w.seed, rank, s))
        if s == 0:
            host_sets.append(inp)
            queries_per_step = int(inp["lengths"].sum()) * w.H
            alg_bytes = algorithmic_bytes(w, inp["lengths"], ps.psattn_count, elem)
        d = {k: torch.from_numpy(inp[k]).to("cuda", tdt) for k in ("Q", "K", "V")}
        d["lengths"] = torch.from_numpy(inp["lengths"]).cuda()
        d["sample_idx"] = torch.from_numpy(inp["sample_idx"]).cuda()
        d["O"] = torch.empty((w.B, w.H, w.T, w.d), dtype=tdt, device="cuda")
        d["sel"] = torch.empty((w.B, w.H, plan.u_max), dtype=torch.int32, device="cuda")
        sets.append(d)

    def step(k):
        d = sets[k % n_sets]
        plan.psattn_forward(d["Q"], d["K"], d["V"], d["lengths"], d["sample_idx"], d["O"], d["sel"])

    l0 = ps.psattn_launch_count()
    step(0)
    torch.cuda.synchronize()
    launches_per_step = ps.psattn_launch_count() - l0

    def capture(fn):
        """CUDA graphs around fn(set index): one per buffer set, plus one that runs all sets in turn
        (fewer graph launches per timed step).  None when graphs are switched off."""
        if args.no_graph:
            return None
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for s in range(n_sets):
                fn(s)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        singles = []
        for s in range(n_sets):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                fn(s)
            singles.append(g)
        group = torch.cuda.CUDAGraph()
        with torch.cuda.graph(group):
            for s in range(n_sets):
                fn(s)
        return singles, group

    def replayer(fn, gs):
        """k -> runs step k.  With graphs: the group graph replays n_sets consecutive steps when k is
        a multiple of n_sets and enough steps remain; the tail runs through the single graphs."""
        if gs is None:
            return lambda k, total=None: fn(k)
        singles, group = gs

        def run(k, total=None):
            if total is None:
                singles[k % n_sets].replay()
                return
            full = (total // n_sets) * n_sets
            if k < full:
                if k % n_sets == 0:
                    group.replay()
            else:
                singles[k % n_sets].replay()
        return run

    graphs = capture(step)
    timed_step = replayer(step, graphs)

    for k in range(max(args.warmup, 3)):
        timed_step(k)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    sampler = ClockSampler(local)
    sampler.start()
    ms = time_events(timed_step, args.steps, torch, grouped=True)
    clocks = sampler.stop()
    if world > 1:
        dist.barrier()
        ms = sharding.max_over_ranks(ms, device="cuda")
    status = plan.psattn_read_status()
    value = queries_per_step * world / (ms * 1e-3)

    # direct (non-graph) C-ABI calls, for the record
    direct_ms = time_events(step, min(args.steps, 200), torch)

    # per-entry-point times (same kernels), rotating buffers, to find the dominant kernel
    M_buf = torch.empty((w.B, w.H, w.T), dtype=torch.float32, device="cuda")

    def k_measure(k):
        d = sets[k % n_sets]
        plan.psattn_measure(d["Q"], d["K"], d["lengths"], d["sample_idx"], M_buf)

    def k_rest(k):
        d = sets[k % n_sets]
        plan.psattn_forward_with_selection(d["Q"], d["K"], d["V"], d["lengths"], d["sel"], d["O"])

    nk = min(args.steps, 200)
    r_measure, r_rest = replayer(k_measure, capture(k_measure)), replayer(k_rest, capture(k_rest))
    for k in range(3):
        r_measure(k); r_rest(k)
    kernel_ms = {"measure(a+b)": time_events(r_measure, nk, torch, grouped=True),
                 "mean_v+attend+fill(d+e)": time_events(r_rest, nk, torch, grouped=True)}
    variants = None
    if not args.no_variants:
        variants = {}
        # Sec. 4.4: N_share consecutive layers share one index set: one full pass, then N_share - 1
        # passes of steps (d)+(e) on other layers' Q, K, V (the rotating buffer sets stand in for layers)
        for n_share in (4, 8):
            def group(k, n=n_share):
                d0 = sets[(k * n) % n_sets]
                plan.psattn_forward(d0["Q"], d0["K"], d0["V"], d0["lengths"], d0["sample_idx"], d0["O"], d0["sel"])
                for j in range(1, n):
                    d = sets[(k * n + j) % n_sets]
                    plan.psattn_forward_with_selection(d["Q"], d["K"], d["V"], d["lengths"], d0["sel"], d["O"])
            r_group = replayer(group, capture(group))
            for k in range(3):
                r_group(k)
            g_ms = time_events(r_group, max(n_sets, nk // n_share), torch, grouped=True)
            variants["selection_reuse_n_share_%d" % n_share] = {
                "ms_per_layer": g_ms / n_share, "value": queries_per_step / (g_ms / n_share * 1e-3), "unit": UNIT}
        # Sec. 3.2 / Eq. 12 as printed: u = ceil(r_sparse * T) selected queries, the others output v_i
        for r_sparse in (0.35, 0.5):
            u_lit = int(np.ceil(r_sparse * w.T))
            plan2 = ps.Plan(w.B, w.H, w.T, dtype=tdt, c=w.c, idx_cols=n_cols, u_override=u_lit,
                            fill_mode=ps.PSATTN_FILL_OWN_V)
            sel2 = torch.empty((w.B, w.H, plan2.u_max), dtype=torch.int32, device="cuda")

            def literal(k):
                d = sets[k % n_sets]
                plan2.psattn_forward(d["Q"], d["K"], d["V"], d["lengths"], d["sample_idx"], d["O"], sel2)
            r_lit = replayer(literal, capture(literal))
            for k in range(3):
                r_lit(k)
            l_ms = time_events(r_lit, max(n_sets, min(nk, 50)), torch, grouped=True)
            flops = 4.0 * w.d * sum(int(L) * min(u_lit, int(L)) for L in host_sets[0]["lengths"]) * w.H
            variants["paper_literal_r_sparse_%.2f" % r_sparse] = {
                "u": u_lit, "fill": "own value row", "ms_per_step": l_ms,
                "value": queries_per_step / (l_ms * 1e-3), "unit": UNIT,
                "attention_tflops": flops / (l_ms * 1e-3) / 1e12,
                "device_status": plan2.psattn_read_status()}
            plan2.close()
        # Sec. 3.2 read with ONE sampled key matrix per sequence: step (a) is a dense product on tcgen05
        plan3 = ps.Plan(w.B, w.H, w.T, dtype=tdt, c=w.c, idx_cols=n_cols, idx_shared=True)
        sel3 = torch.empty((w.B, w.H, plan3.u_max), dtype=torch.int32, device="cuda")
        shared_idx = [d["sample_idx"][:, 0, :].contiguous() for d in sets]

        def shared_forward(k):
            d = sets[k % n_sets]
            plan3.psattn_forward(d["Q"], d["K"], d["V"], d["lengths"], shared_idx[k % n_sets], d["O"], sel3)

        def shared_measure(k):
            d = sets[k % n_sets]
            plan3.psattn_measure(d["Q"], d["K"], d["lengths"], shared_idx[k % n_sets], M_buf)
        r_sf, r_sm = replayer(shared_forward, capture(shared_forward)), replayer(shared_measure, capture(shared_measure))
        for k in range(3):
            r_sf(k); r_sm(k)
        sf_ms = time_events(r_sf, nk, torch, grouped=True)
        sm_ms = time_events(r_sm, nk, torch, grouped=True)
        sm_bytes = w.B * w.H * w.T * (w.d * elem + 4)          # Q read once, M written; the sampled keys are small
        pk, _ = measured_peaks()
        variants["shared_sample"] = {
            "ms_per_step": sf_ms, "value": queries_per_step / (sf_ms * 1e-3), "unit": UNIT,
            "measure_ms": sm_ms, "measure_gbs": sm_bytes / (sm_ms * 1e-3) / 1e9,
            "measure_frac_of_hbm": sm_bytes / (sm_ms * 1e-3) / 1e9 / pk,
            "device_status": plan3.psattn_read_status()}
        plan3.close()
        # Eq. 10 over all keys: a dense tensor-core pass, the quantity Eq. 11 approximates
        def exact(k):
            d = sets[k % n_sets]
            plan.psattn_exact_measure(d["Q"], d["K"], d["lengths"], M_buf)
        exact(0)
        x_ms = time_events(exact, 5, torch)
        x_flops = 2.0 * w.d * sum(int(L) * int(L) for L in host_sets[0]["lengths"]) * w.H
        variants["exact_measure"] = {"ms_per_step": x_ms, "tflops": x_flops / (x_ms * 1e-3) / 1e12}
        # Sec. 3.1: the projections in front of the path (one tcgen05 GEMM writing Q, K, V in the layout
        # the path reads, plus mean(V)); reported against the measured dense bf16 peak
        if w.dtype == "bf16":
            dx = w.H * w.d
            pin = wl.make_projection_inputs(w, seed=sharding.rank_seed(w.seed, rank, 0))
            pX = [torch.from_numpy(pin["X"]).to("cuda", tdt) for _ in range(n_sets)]
            pW = torch.from_numpy(pin["Wt"]).to("cuda", tdt)
            vb = torch.empty((w.B, w.H, w.d), dtype=torch.float32, device="cuda")
            pO = [[torch.empty((w.B, w.H, w.T, w.d), dtype=tdt, device="cuda") for _ in range(3)] for _ in range(n_sets)]

            p_flops = 2.0 * dx * 3 * dx * sum(int(L) for L in host_sets[0]["lengths"])
            tf_peak = tensor_peak()
            for key, want_vbar in (("qkv_projection", True), ("qkv_projection_without_mean_v", False)):
                def project(k, want_vbar=want_vbar):
                    o = pO[k % n_sets]
                    plan.psattn_project_qkv(pX[k % n_sets], pW, sets[k % n_sets]["lengths"], o[0], o[1], o[2],
                                            vb if want_vbar else None)
                r_pj = replayer(project, capture(project))
                for k in range(3):
                    r_pj(k)
                p_ms = time_events(r_pj, nk, torch, grouped=True)
                variants[key] = {
                    "ms_per_step": p_ms, "tflops": p_flops / (p_ms * 1e-3) / 1e12, "peak_tflops": tf_peak[0],
                    "frac_of_tensor_peak": p_flops / (p_ms * 1e-3) / 1e12 / tf_peak[0],
                    "peak_kind": "of " + tf_peak[1], "d_x": dx, "device_status": plan.psattn_read_status()}
            del pO, pX
    peak, peak_kind = measured_peaks()
    units = w.B * w.H
    measure_bytes = units * w.T * w.d * elem * 2 + w.B * w.T * n_cols * 4 + units * w.T * 4
    if launches_per_step == 1:
        roof_kernel, roof_bytes, roof_ms = "fused forward", alg_bytes, ms
    else:
        roof_kernel, roof_bytes, roof_ms = "measure (steps a+b)", measure_bytes, kernel_ms["measure(a+b)"]
    achieved = roof_bytes / (roof_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": roof_kernel, "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak,
                "traffic": recorded_traffic(w.name),
                "peak_kind": "of " + peak_kind,
                "algorithmic_bytes_per_launch": roof_bytes}
    path_gbs = alg_bytes / (ms * 1e-3) / 1e9

    # end to end through the host-buffer entry point (pinned host memory, copies timed)
    e2e = None
    if True:
        plan.psattn_plan_enable_host_io()
        inp = host_sets[0]
        hQ, hK, hV = (torch.from_numpy(inp[k]).to(tdt).pin_memory() for k in ("Q", "K", "V"))
        hl = torch.from_numpy(inp["lengths"]).pin_memory()
        hi = torch.from_numpy(inp["sample_idx"]).pin_memory()
        hO = torch.empty((w.B, w.H, w.T, w.d), dtype=tdt).pin_memory()
        hs = torch.empty((w.B, w.H, plan.u_max), dtype=torch.int32).pin_memory()
        ne = max(3, min(args.steps, 20))
        for _ in range(3):
            plan.psattn_forward_host(hQ, hK, hV, hl, hi, hO, hs)
        if world > 1:
            dist.barrier()
        e_ms = time_events(lambda k: plan.psattn_forward_host(hQ, hK, hV, hl, hi, hO, hs), ne, torch)
        if world > 1:
            e_ms = sharding.max_over_ranks(e_ms, device="cuda")
        h2d = sum(x.numel() * x.element_size() for x in (hQ, hK, hV, hl, hi))
        d2h = sum(x.numel() * x.element_size() for x in (hO, hs))
        e2e = {"value": queries_per_step * world / (e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e_ms, "steps": ne}

    dense = None
    if not args.no_dense and rank == 0:
        d = sets[0]
        plan.psattn_dense_forward(d["Q"], d["K"], d["V"], d["lengths"], d["O"])
        nd = 3
        d_ms = time_events(lambda k: plan.psattn_dense_forward(
            sets[k % n_sets]["Q"], sets[k % n_sets]["K"], sets[k % n_sets]["V"],
            sets[k % n_sets]["lengths"], sets[k % n_sets]["O"]), nd, torch)
        dense = {"ms_per_step": d_ms, "speedup_sparse_vs_dense": d_ms / ms,
                 "workspace_bytes_sparse": plan.workspace_bytes}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        qps, cores, dt, q, n_pass = cpu_oracle_timing(w, n_cols)
        cpu = {"value": qps, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": "whole batch of %s (%d valid queries), %d passes of %.3f s each" % (w.name, q, n_pass, dt)}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32",
            "data": "synthetic",
            "config": {"workload": w.name, "B": w.B, "H": w.H, "T": w.T, "d_head": w.d, "c": w.c,
                       "U": n_cols, "path": args.path, "graph_replay": graphs is not None,
                       "l2": "rotating %d independent buffer sets (%.0f MB > 126 MB L2)" % (
                           n_sets, n_sets * per_set / 1e6)},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches_per_step * args.steps),
            "roofline": roofline, "cpu_baseline": cpu,
            "path_effective_gbs": path_gbs, "path_frac_of_hbm": path_gbs / peak,
            "algorithmic_bytes_per_step": alg_bytes, "queries_per_step": queries_per_step,
            "kernel_ms": kernel_ms, "direct_call_ms_per_step": direct_ms, "dense": dense,
            "variants": variants,
            "device_status": status,
        }
        print(json.dumps(line), flush=True)
    plan.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
