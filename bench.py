#!/usr/bin/env python
"""Benchmark of the CoCoD-SGD parameter engine on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A "step" is one communication round of Algorithm 1 over all K workers: comm_begin (stored copy +
averaging on the side stream), k local momentum-SGD steps, comm_end (merge).  The metric is
worker-parameter updates per second = K * P * k * rounds / time, whole job over all ranks.
Prints ONE JSON line (rank 0).  The headline runs the three kernels the path is defined by; the same
rounds with the last local step and the merge fused into one pass are reported under fusion_variants,
the VGG16-sized and the end-to-end MLP workloads under other_workloads.

N > 1 (torchrun): the path shards by parameter index with no exchange at all, so every rank
runs the same per-GPU workload on its own column range (weak scaling); time is the max over
ranks of the device-timed region.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "worker-param updates/sec (K*P*steps/s)"
UNIT = "updates/s"


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000, help="timed rounds")
    ap.add_argument("--warmup", type=int, default=3, help="untimed rounds (>= 3)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet18", choices=["tiny", "resnet18", "vgg16", "mlp"])
    ap.add_argument("--K", type=int, default=None, help="override the workload's worker count (profiling, sweeps)")
    ap.add_argument("--P", type=int, default=None, help="override the workload's model size")
    ap.add_argument("--k", type=int, default=None, help="override the workload's local steps per round")
    ap.add_argument("--snapshot", default="flip", choices=["flip", "copy"])
    ap.add_argument("--ring", type=int, default=4, help="distinct gradient buffers cycled through")
    ap.add_argument("--graph", action="store_true",
                    help="replay the timed rounds from a CUDA graph of two rounds (launch-bound workloads)")
    ap.add_argument("--fused", action="store_true",
                    help="mlp workload: gradients and local step in one call (update inside the weight-gradient GEMMs)")
    ap.add_argument("--shard", default="columns", choices=["columns", "workers"],
                    help="N > 1: split the columns (default, no exchange) or the workers (the paper's layout: "
                         "every rank holds K workers of K*N, Step I's mean spans the GPUs on the side stream)")
    ap.add_argument("--exchange", default="allreduce", choices=["allreduce", "gather"],
                    help="--shard workers: finish the mean with an all-reduce of P floats, or with the gather kernel "
                         "over peer addresses")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--repeats", type=int, default=5, help="how many times the timed block of --steps rounds is repeated "
                                                           "(the line reports the median block, and min and max)")
    ap.add_argument("--alternate-sweep", action="store_true",
                    help="experiment: consecutive streaming kernels walk the vector in alternating directions (COCOD_OPT_SWEEP)")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="default run only: skip the VGG16-sized and MLP digests added under other_workloads")
    ap.add_argument("--cpu-sample-cols", type=int, default=1 << 20)
    ap.add_argument("--sweep-K", default="2,8,16,32,64")
    ap.add_argument("--sweep-logP", default="20,24,26,28")
    ap.add_argument("--sweep", action="store_true",
                    help="scaling sweep P in {2^20,2^24,2^26,2^28} x K in {2,8,16,32,64} x k in {1,8}: one JSON line per cell")
    return ap.parse_args()


# ---------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc = None
        ident = str(index)
        try:        # nvidia-smi numbers GPUs physically; under CUDA_VISIBLE_DEVICES only the UUID is safe
            import torch
            ident = "GPU-" + str(torch.cuda.get_device_properties(index).uuid)
        except Exception:
            pass
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-i", ident, "-lms", "25"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(names, f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------------- CPU oracle leg
def time_oracle(wl, cols: int, steps: int, warmup: int):
    """The oracle as it stands (ref mode, all host cores) on a column sample of the workload:
    rounds of Algorithm 1 over K workers x `cols` columns.  Gradient generation is outside the
    timed region.  Returns (updates/s, seconds per round, cores)."""
    import numpy as np
    from oracle import cocod_oracle as O
    from paper_1906_12043_b200 import inputs as I
    cores = O.max_threads()
    O.set_threads(cores)
    K, k = wl.K, wl.k
    col_idx = np.arange(cols, dtype=np.uint64)
    eng = O.OracleEngine(K, cols, wl.lr, wl.mu, wl.wd, mode="ref")
    eng.set_params(I.initial_point(wl.P, wl.sigma_x0, cols=col_idx))
    ring = [I.gradients(K, wl.P, t, wl.sigma_g, cols=col_idx) for t in range(max(2, k))]

    def one_round(r):
        eng.comm_begin()
        for s in range(k):
            eng.local_step(ring[(r * k + s) % len(ring)])
        eng.comm_end()

    for r in range(warmup):
        one_round(r)
    t0 = time.perf_counter()
    for r in range(steps):
        one_round(warmup + r)
    dt = time.perf_counter() - t0
    O.set_threads(1)
    return K * cols * k * steps / dt, dt / steps, cores


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cols = min(args.cpu_sample_cols, wl.P)
    value, s_per_round, cores = time_oracle(wl, cols, args.steps, args.warmup)
    sample = (f"{wl.K} workers x first {cols} of {wl.P} columns, {args.steps} rounds of k={wl.k} local steps "
              f"(ref-mode oracle, OpenMP over columns); gradients pre-generated")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": s_per_round * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": wl.name, "K": wl.K, "P": wl.P, "k": wl.k, "lr": wl.lr, "mu": wl.mu, "wd": wl.wd,
                   "sampled_columns": cols},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ---------------------------------------------------------------------------------------------- our arm
def summarize_profile(recs, names):
    by = {}
    for kind, a, b in recs:
        by.setdefault(names[kind], []).append((a, b))
    return by


def overlap_fraction(by):
    """Share of the mean kernels' lifetime that lies inside some local-step kernel's lifetime."""
    steps = sorted(by.get("local_step", []))
    tot = cov = 0.0
    for a, b in by.get("mean", []):
        tot += b - a
        for c, d in steps:
            lo, hi = max(a, c), min(b, d)
            if hi > lo:
                cov += hi - lo
    return cov / tot if tot > 0 else None


def median(xs):
    xs = sorted(xs)
    n = len(xs)
    return xs[n // 2] if n % 2 else 0.5 * (xs[n // 2 - 1] + xs[n // 2])


def load_peaks():
    try:
        return json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except OSError:
        return {}


def measure_param_workload(args, wl, ctx, *, ring_n, do_e2e, cpu_seconds, do_graph, do_schemes, sampler=None):
    """One parameter-path workload on this rank: the timed blocks, the per-kernel passes, and the optional legs.
    ctx: dict(rank, world, barrier, dist).  Returns the pieces of the JSON line."""
    import torch
    from paper_1906_12043_b200 import engine as E, inputs as I, workloads as W
    rank, world, barrier, dist = ctx["rank"], ctx["world"], ctx["barrier"], ctx["dist"]
    K, P, k = wl.K, wl.P, wl.k
    p0 = rank * P                                       # this rank's columns of the global vector
    peaks = load_peaks()
    hbm_peak = float(peaks.get("hbm_gbs", 6650.0))
    peak_kind = "measured" if "hbm_gbs" in peaks else "fallback"

    eng = E.Engine(K, P, wl.lr, wl.mu, wl.wd)
    eng.set_option(E.OPT_SNAPSHOT, E.SNAPSHOT_FLIP if args.snapshot == "flip" else E.SNAPSHOT_COPY)
    if args.alternate_sweep:
        eng.set_option(E.OPT_SWEEP, 1)
    x0 = torch.empty(P, dtype=torch.float32, device="cuda")
    I.device_gaussian_into(x0, I.X0_SEED, I.STREAM_X0, 0, 0, p0, wl.sigma_x0)
    eng.set_params(x0)
    ring = []
    for t in range(max(1, ring_n)):
        g = torch.empty((K, P), dtype=torch.float32, device="cuda")
        I.device_gradients_into(g, t, wl.sigma_g, p0=p0)
        ring.append(g)
    side = torch.cuda.Stream(priority=-1)
    compute = torch.cuda.current_stream()
    step_no = [0]

    def one_round(side_stream):
        eng.comm_begin(side_stream)
        for _ in range(k):
            eng.local_step(ring[step_no[0] % len(ring)])
            step_no[0] += 1
        eng.comm_end()

    # ---- device-resident timed region: `repeats` blocks of exactly `steps` rounds, each bracketed by a barrier and a
    #      synchronize on both sides; no per-kernel events inside (those are taken in passes of their own below)
    warm = max(3, args.warmup)
    for _ in range(warm):
        one_round(side)
    graph = None
    steps = args.steps
    if args.graph and do_graph:
        # two rounds = one full cycle of the buffer flip; the side-stream mean is captured with them
        cap = torch.cuda.Stream()
        eng.sync()
        eng.set_stream(cap)
        with torch.cuda.stream(cap):
            one_round(side)
            one_round(side)
        torch.cuda.synchronize()
        step_no[0] = 0
        l_before = eng.launch_count
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=cap):
            one_round(side)
            one_round(side)
        launches_per_replay = eng.launch_count - l_before
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        steps = max(2, steps // 2 * 2)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    block_ms, launches = [], 0
    for rep in range(max(1, args.repeats)):
        barrier()
        launches0 = eng.launch_count
        ev0.record(compute)
        if graph is not None:
            for _ in range(steps // 2):
                graph.replay()
        else:
            for _ in range(steps):
                one_round(side)
        ev1.record(compute)
        barrier()
        ms = ev0.elapsed_time(ev1)
        if world > 1:
            t = torch.tensor([ms], dtype=torch.float64, device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        block_ms.append(ms)
        launches = launches_per_replay * (steps // 2) if graph is not None else eng.launch_count - launches0
    if graph is not None:
        eng.sync()
        eng.set_stream(compute)
    ms = median(block_ms)
    value = world * K * P * k * steps / (ms * 1e-3)
    clocks = sampler.stop() if sampler else None

    alg_bytes = {"local_step": W.BYTES_LOCAL_STEP * K * P, "snapshot": W.BYTES_SNAPSHOT * K * P,
                 "mean": W.bytes_mean(K) * K * P, "merge": W.bytes_merge(K) * K * P}

    def kernel_table(by_kind):
        out = {}
        for name, iv in by_kind.items():
            avg_ms = sum(b - a for a, b in iv) / len(iv)
            gbs = alg_bytes[name] / (avg_ms * 1e-3) / 1e9
            out[name] = {"launches": len(iv), "avg_ms": round(avg_ms, 5), "gbs": round(gbs, 1),
                         "frac_of_peak": round(gbs / hbm_peak, 4)}
        return out

    # ---- the same rounds with per-kernel CUDA events and the kernels' own time stamps (overlapped, then serial)
    n_prof = min(steps, 50)
    eng.set_option(E.OPT_PROFILE, 1)
    eng.profile_reset()
    torch.cuda.synchronize()
    ev0.record(compute)
    for _ in range(n_prof):
        one_round(side)
    ev1.record(compute)
    torch.cuda.synchronize()
    ms_profiled = ev0.elapsed_time(ev1) / n_prof
    by = summarize_profile(eng.profile_records(), E.KERNEL_NAMES)
    by_dev = summarize_profile(eng.profile_device_records(), E.KERNEL_NAMES)
    in_loop = kernel_table(by)
    in_loop_dev = kernel_table(by_dev)
    overlap = overlap_fraction(by)
    overlap_dev = overlap_fraction(by_dev)
    eng.profile_reset()
    torch.cuda.synchronize()
    n_ser = min(steps, 50)
    ev0.record(compute)
    for _ in range(n_ser):
        one_round(compute)
    ev1.record(compute)
    torch.cuda.synchronize()
    ms_serial = ev0.elapsed_time(ev1) / n_ser
    isolated = kernel_table(summarize_profile(eng.profile_records(), E.KERNEL_NAMES))
    eng.set_option(E.OPT_PROFILE, 0)
    # serial round WITHOUT the event brackets: the figure that compares with the headline block
    for _ in range(2):
        one_round(compute)
    torch.cuda.synchronize()
    ev0.record(compute)
    for _ in range(n_ser):
        one_round(compute)
    ev1.record(compute)
    torch.cuda.synchronize()
    ms_serial_plain = ev0.elapsed_time(ev1) / n_ser

    # ---- the paper's sequential counterparts on the same kernels: k local steps + blocking averaging
    #      (Local-SGD) and k steps of gradient averaging (S-SGD); for context next to the decoupled round
    def timed(fn, n):
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        ev0.record(compute)
        for _ in range(n):
            fn()
        ev1.record(compute)
        torch.cuda.synchronize()
        return ev0.elapsed_time(ev1) / n

    def local_sgd_round():
        for _ in range(k):
            eng.local_step(ring[step_no[0] % len(ring)])
            step_no[0] += 1
        eng.local_sgd_average()

    def ssgd_round():
        for _ in range(k):
            eng.ssgd_step(ring[step_no[0] % len(ring)])
            step_no[0] += 1

    schemes = None
    if do_schemes:
        n_cmp = min(steps, 30)
        schemes = {"cocod": ms / steps, "local_sgd": timed(local_sgd_round, n_cmp), "ssgd": timed(ssgd_round, n_cmp)}

    # ---- the same rounds replayed from a CUDA graph (extra figure; the contract value stays the eager one)
    graph_extra = None
    if graph is None and world == 1 and do_graph:
        cap = torch.cuda.Stream()
        eng.sync()
        eng.set_stream(cap)
        with torch.cuda.stream(cap):
            one_round(side)
            one_round(side)
        torch.cuda.synchronize()
        g2 = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g2, stream=cap):
            one_round(side)
            one_round(side)
        for _ in range(3):
            g2.replay()
        torch.cuda.synchronize()
        n_rep = max(1, min(steps, 200) // 2)
        ev0.record(compute)
        for _ in range(n_rep):
            g2.replay()
        ev1.record(compute)
        torch.cuda.synchronize()
        ms_g = ev0.elapsed_time(ev1) / (2 * n_rep)
        graph_extra = {"ms_per_step": ms_g, "value": K * P * k / (ms_g * 1e-3), "rounds": 2 * n_rep}
        eng.sync()
        eng.set_stream(compute)
        del g2

    # ---- fusion variant of the round: the last local step and the merge in one pass (cocod_local_step_end)
    def one_round_fused_end():
        eng.comm_begin(side)
        for j in range(k):
            gbuf = ring[step_no[0] % len(ring)]
            step_no[0] += 1
            if j < k - 1:
                eng.local_step(gbuf)
            else:
                eng.local_step_end(gbuf)

    fusion = None
    if do_schemes or do_graph is False:
        for _ in range(3):
            one_round_fused_end()
        blocks = []
        for rep in range(max(1, args.repeats)):
            torch.cuda.synchronize()
            ev0.record(compute)
            for _ in range(steps):
                one_round_fused_end()
            ev1.record(compute)
            torch.cuda.synchronize()
            blocks.append(ev0.elapsed_time(ev1) / steps)
        eng.set_option(E.OPT_PROFILE, 1)
        eng.profile_reset()
        for _ in range(min(steps, 20)):
            one_round_fused_end()
        byf = summarize_profile(eng.profile_records(), E.KERNEL_NAMES)
        eng.set_option(E.OPT_PROFILE, 0)
        ms_f = median(blocks)
        sm_bytes = (24.0 + 4.0 / K) * K * P
        iv = byf.get("step_merge", [])
        sm_ms = sum(b - a for a, b in iv) / max(1, len(iv))
        fusion = {"last_step_and_merge_in_one_pass": {
            "ms_per_step": ms_f, "ms_per_step_min": min(blocks), "ms_per_step_max": max(blocks),
            "value": world * K * P * k / (ms_f * 1e-3), "speedup_over_the_three_kernels": (ms / steps) / ms_f,
            "bytes_per_worker_parameter_per_round": 20 * (k - 1) + 24 + 4.0 / K + W.bytes_mean(K),
            "kernel": {"name": "step_merge_vec8", "avg_ms": round(sm_ms, 5), "launches": len(iv),
                       "algorithmic_bytes_per_launch": sm_bytes,
                       "gbs": round(sm_bytes / (sm_ms * 1e-3) / 1e9, 1) if iv else None,
                       "frac_of_peak": round(sm_bytes / (sm_ms * 1e-3) / 1e9 / hbm_peak, 4) if iv else None},
            "note": "same values bit for bit; the headline value above is the explicit local step / mean / merge path"}}

    dom = "local_step"
    traffic = W.NCU_DRAM_BYTES_PER_WORKER_PARAM.get(dom)
    traffic = traffic * K * P if traffic is not None else None
    dom_tab = in_loop.get(dom) or isolated.get(dom, {})
    roofline = {"bound": "hbm", "kernel": dom, "achieved": dom_tab.get("gbs"), "peak": hbm_peak,
                "unit": "GB/s", "frac": dom_tab.get("frac_of_peak"), "traffic": traffic,
                "peak_kind": peak_kind, "algorithmic_bytes_per_launch": alg_bytes[dom],
                "avg_launch_ms": dom_tab.get("avg_ms"), "isolated": isolated.get(dom),
                "measured_in": "a pass of its own with per-kernel CUDA events, mean kernel overlapping on the side stream"}

    # ---- end to end through the host-buffer entry point
    e2e = None
    if do_e2e:
        host_ring = []
        for t in range(2):
            hbuf = torch.empty((K, P), dtype=torch.float32, pin_memory=True)
            hbuf.copy_(ring[t % len(ring)])
            host_ring.append(hbuf)
        mean_out = torch.empty(P, dtype=torch.float32, pin_memory=True)
        hs = [0]

        def one_round_host():
            eng.comm_begin(side)
            for _ in range(k):
                eng.local_step_host(host_ring[hs[0] % 2])
                hs[0] += 1
            eng.comm_end()
            eng.get_mean(mean_out)                      # device -> host read of the round's result

        n_e2e = max(1, min(steps, 20))
        for _ in range(2):
            one_round_host()
        barrier()
        t0 = time.perf_counter()
        ev0.record(compute)
        for _ in range(n_e2e):
            one_round_host()
        ev1.record(compute)
        barrier()
        wall = time.perf_counter() - t0
        ms_e2e = max(ev0.elapsed_time(ev1), 0.0)
        if world > 1:
            t = torch.tensor([ms_e2e], dtype=torch.float64, device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms_e2e = float(t.item())
        e2e = {"value": world * K * P * k * n_e2e / (ms_e2e * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": k * K * P * 4, "d2h_bytes_per_step": P * 4,
               "rounds": n_e2e, "ms_per_step": ms_e2e / n_e2e, "wall_ms_per_step": wall * 1e3 / n_e2e}
        del host_ring, mean_out

    eng.destroy()
    del ring, x0
    torch.cuda.empty_cache()

    # ---- CPU oracle beside it (rank 0, N = 1 only)
    cpu_baseline = None
    if rank == 0 and world == 1 and cpu_seconds > 0:
        cols = min(args.cpu_sample_cols, P)
        probe, s_per_round, cores = time_oracle(wl, cols, 2, 1)
        n_rounds = max(2, min(200, int(cpu_seconds / max(s_per_round, 1e-6))))
        v, s_per_round, cores = time_oracle(wl, cols, n_rounds, 1)
        cpu_baseline = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": f"{K} workers x first {cols} of {P} columns, {n_rounds} rounds of k={k} "
                                  f"(ref-mode oracle, OpenMP over columns, gradients pre-generated)"}

    return {
        "value": value, "steps": steps, "ms_per_step": ms / steps,
        "timed_blocks": {"repeats": len(block_ms), "rounds_per_block": steps,
                         "ms_per_step": [b / steps for b in block_ms], "ms_per_step_median": ms / steps,
                         "ms_per_step_min": min(block_ms) / steps, "ms_per_step_max": max(block_ms) / steps,
                         "reported": "median block"},
        "config": {"workload": wl.name, "K": K, "P": P, "k": k, "lr": wl.lr, "mu": wl.mu, "wd": wl.wd,
                   "snapshot": args.snapshot, "alternate_sweep": bool(args.alternate_sweep), "gradient_ring": max(1, ring_n),
                   "cuda_graph": bool(graph is not None),
                   "l2": "inputs larger than L2 (each K x P buffer is %.0f MB, L2 is 126 MB)" % (K * P * 4 / 1e6)
                         if K * P * 4 > 126e6 else "L2-resident workload: not an HBM number",
                   "sharding": "columns, no exchange" if world > 1 else "single GPU"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "cpu_baseline": cpu_baseline,
        "kernels_in_loop": in_loop, "kernels_in_loop_device_stamps": in_loop_dev, "kernels_isolated": isolated,
        "overlap_fraction": overlap, "overlap_fraction_device_stamps": overlap_dev,
        "ms_per_round_overlapped": ms / steps, "ms_per_round_serial": ms_serial_plain,
        "ms_per_round_profiled": {"overlapped": ms_profiled, "serial": ms_serial},
        "cuda_graph_replay": graph_extra, "ms_per_round_by_scheme": schemes, "fusion_variants": fusion,
        "hbm_gbs_whole_round": wl.bytes_per_round(args.snapshot == "copy") / (ms / steps * 1e-3) / 1e9,
    }


def run_ours(args, wl):
    import torch
    import torch.distributed as dist
    from paper_1906_12043_b200 import build, engine as E
    from paper_1906_12043_b200.workloads import WORKLOADS

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the engine has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    E.load()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    ctx = {"rank": rank, "world": world, "barrier": barrier, "dist": dist}
    sampler = ClockSampler(local_rank) if rank == 0 else None
    res = measure_param_workload(args, wl, ctx, ring_n=args.ring, do_e2e=not args.no_e2e,
                                 cpu_seconds=0 if args.no_cpu_baseline else 12.0, do_graph=True, do_schemes=True,
                                 sampler=sampler)
    # ---- digests of the other stated workloads, so that one default run shows all of them (N = 1 only; their
    #      end-to-end legs are left to `--workload vgg16` / `--workload mlp`)
    other = None
    default_run = (wl.name == "resnet18" and world == 1 and not args.graph and not args.no_other_workloads)
    if default_run:
        other = {}
        saved = (args.steps, args.repeats)
        try:
            args.steps = max(2, min(saved[0], 10))
            v = measure_param_workload(args, WORKLOADS["vgg16"], ctx, ring_n=2, do_e2e=False,
                                       cpu_seconds=0 if args.no_cpu_baseline else 6.0, do_graph=False, do_schemes=False,
                                       sampler=ClockSampler(local_rank))
            other["vgg16"] = {key: v[key] for key in ("value", "steps", "ms_per_step", "timed_blocks", "config", "clocks",
                                                      "gpu_launches", "roofline", "cpu_baseline", "kernels_in_loop",
                                                      "kernels_isolated", "overlap_fraction", "overlap_fraction_device_stamps",
                                                      "ms_per_round_serial", "hbm_gbs_whole_round", "fusion_variants")}
            other["vgg16"].update(metric=METRIC, unit=UNIT)
        except Exception as e:                              # e.g. a smaller GPU: say so instead of losing the headline
            other["vgg16"] = {"unavailable": f"{type(e).__name__}: {e}"}
        finally:
            args.steps, args.repeats = saved
        try:                                                # a digest of the scaling sweep: six of its 38 cells
            digest = []
            sweep_cells([(2, 1 << 24), (16, 1 << 24), (64, 1 << 24)], digest.append)
            other["sweep_digest"] = {"cells": digest, "note": "timing only; the whole sweep is `bench.py --sweep`"}
        except Exception as e:
            other["sweep_digest"] = {"unavailable": f"{type(e).__name__}: {e}"}
        try:
            args.steps = max(2, min(saved[0], 20))
            other["mlp"] = measure_mlp(args, digest=True)
        except Exception as e:
            other["mlp"] = {"unavailable": f"{type(e).__name__}: {e}"}
        finally:
            args.steps, args.repeats = saved

    if rank == 0:
        line = {
            "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": world, "steps": res["steps"],
            "warmup": max(3, args.warmup), "ms_per_step": res["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        }
        line.update({key: res[key] for key in res if key not in ("value", "steps", "ms_per_step")})
        fv = (res.get("fusion_variants") or {}).get("last_step_and_merge_in_one_pass")
        if fv:                           # the fastest way through the library that ends on the same bits
            line["best_value"] = {"value": fv["value"], "ms_per_step": fv["ms_per_step"],
                                  "path": "cocod_local_step_end for the round's last step (fusion_variants)"}
        if other is not None:
            line["other_workloads"] = other
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_reference_mlp(args):
    """Reference arm of the MLP workload: the oracle as it stands on the host cores.  A step is one round
    (Step I, k x (numpy fp64 gradient with the bf16 rounding points + reference-mode update), line 6) of a
    SAMPLE of two of the 16 workers."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import numpy as np
    from oracle import mlp_oracle as MO
    from oracle.cocod_oracle import OracleEngine
    from paper_1906_12043_b200 import inputs as I
    nw, k, lr, mu, wd = 2, args.k or 4, 0.05, 0.9, 0.0
    dims = I.MLP_DIMS
    x0 = I.mlp_init_params(I.MLP_STUDENT_SEED)
    teacher = I.mlp_init_params(I.MLP_TEACHER_SEED)
    P_raw = x0.size
    oe = OracleEngine(nw, P_raw, lr, mu, wd, mode="ref")
    oe.set_params(x0)
    args.steps = min(args.steps, 10)                      # every (worker, step) has its own minibatch: keep the run bounded
    ring = (args.warmup + args.steps) * k
    Xo = [[I.mlp_batch(w, t) for w in range(nw)] for t in range(ring)]
    yo = [[I.mlp_teacher_labels(Xo[t][w], teacher) for w in range(nw)] for t in range(ring)]
    tau = [0]

    def one_round():
        oe.comm_begin()
        for _ in range(k):
            t = tau[0] % ring
            g = np.stack([MO.loss_and_grad(oe.x[w], Xo[t][w], yo[t][w], dims, emulate_bf16=True)[1] for w in range(nw)])
            oe.local_step(g)
            tau[0] += 1
        oe.comm_end()

    for _ in range(args.warmup):
        one_round()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        one_round()
    dt = time.perf_counter() - t0
    value = nw * P_raw * k * args.steps / dt
    sample = (f"{nw} of 16 workers, {args.steps} rounds of k={k} local steps (numpy fp64 gradient with bf16 rounding "
              f"points + reference-mode parameter path)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 contractions / f32 state", "data": "synthetic",
        "config": {"workload": "mlp", "K": 16, "P": P_raw, "k": k, "lr": lr, "mu": mu, "wd": wd, "mlp": list(dims),
                   "batch": I.MLP_BATCH, "sampled_workers": nw},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def _mlp_oracle_job(job):
    """Child process of the MLP CPU-baseline leg: one worker's oracle gradient (numpy fp64, bf16 rounding points)."""
    import numpy as np
    from oracle import mlp_oracle as MO
    from paper_1906_12043_b200 import inputs as I
    flat, xbits, y = job
    X = (xbits.astype(np.uint32) << np.uint32(16)).view(np.float32)
    loss, g = MO.loss_and_grad(flat, X, y, I.MLP_DIMS, emulate_bf16=True)
    return float(loss), g


def time_mlp_oracle(K, k, rounds, lr, mu, wd, x0_raw, X_bits, y, procs):
    """The oracle as it stands on the host cores for the first `rounds` rounds of the MLP workload, all K workers:
    Step I, k x (numpy fp64 gradient of every worker, one process per worker, + reference-mode update), line 6.
    X_bits: [rounds * k][K][batch][d_in] uint16 (bf16 patterns), y: [rounds * k][K][batch] int32 -- the bytes the
    device consumed.  Returns (seconds, per-step mean losses, bf16-rounded parameters after every round)."""
    import multiprocessing as mp
    import numpy as np
    from oracle.cocod_oracle import OracleEngine
    from paper_1906_12043_b200 import inputs as I
    P_raw = x0_raw.size
    oe = OracleEngine(K, P_raw, lr, mu, wd, mode="ref")
    oe.set_params(x0_raw)
    saved = {v: os.environ.get(v) for v in ("OMP_NUM_THREADS", "OPENBLAS_NUM_THREADS", "MKL_NUM_THREADS")}
    for v in saved:                                      # one BLAS thread per process: the pool is the parallelism
        os.environ[v] = "1"
    try:
        pool = mp.get_context("spawn").Pool(procs)
    finally:
        for v, old in saved.items():
            if old is None:
                os.environ.pop(v, None)
            else:
                os.environ[v] = old
    pool.map(_mlp_oracle_job, [(oe.x[w], X_bits[0][w], y[0][w]) for w in range(min(K, procs))])      # start-up, untimed
    losses, params = [], []
    t0 = time.perf_counter()
    for r in range(rounds):
        oe.comm_begin()
        for s_ in range(k):
            t = r * k + s_
            res = pool.map(_mlp_oracle_job, [(oe.x[w], X_bits[t][w], y[t][w]) for w in range(K)], chunksize=1)
            oe.local_step(np.stack([g for _, g in res]))
            losses.append(float(np.mean([l for l, _ in res])))
        oe.comm_end()
        params.append(I.round_to_bf16(oe.x))
    dt = time.perf_counter() - t0
    pool.close()
    pool.join()
    return dt, losses, params


def measure_mlp(args, digest=False):
    """End-to-end synthetic training: K = 16 workers each train the 784-1024-1024-10 ReLU MLP (bf16 weights, fp32
    master copy and momentum) on minibatches of 128; gradients come from the tensor-core path, the parameter path is
    the same engine with its bf16 shadow switched on.  A step (round) = comm_begin, k = 4 x (batched gradients +
    local step), comm_end.  Every (worker, global step) has its own seeded minibatch (a pool of up to 2048 steps,
    generated on the device, labels from the teacher in fp64; a longer run goes through the pool again, like epochs
    over a data set).  Four variants are timed, each from the common initial point: the two calls; the two calls with the
    round's last local step and the merge in one pass (cocod_local_step_end); the fused gradient + update call; and the
    fused call replayed from CUDA graphs of two rounds each (one graph per pair of rounds of the pool)."""
    import numpy as np
    import torch
    from paper_1906_12043_b200 import build, engine as E, inputs as I, mlp as M, workloads as W
    build.build()
    M.load()
    K, k, lr, mu, wd = (16 if digest else (args.K or 16)), (4 if digest else (args.k or 4)), 0.05, 0.9, 0.0
    dims, B = I.MLP_DIMS, I.MLP_BATCH
    mg = M.MLPGrad(K, B, dims[0], dims[1], dims[3])
    P, P_raw = mg.P, mg.P_raw
    x0 = np.zeros(P, np.float32)
    x0[:P_raw] = I.mlp_init_params(I.MLP_STUDENT_SEED)
    teacher = I.mlp_init_params(I.MLP_TEACHER_SEED)
    peaks = load_peaks()
    hbm_peak = float(peaks.get("hbm_gbs", 6650.0))
    peak_kind = "measured" if "hbm_gbs" in peaks else "fallback"
    steps, repeats = max(2, args.steps // 2 * 2), max(1, args.repeats)
    n_cpu_rounds = 0 if args.no_cpu_baseline else 6
    warm = max(3, args.warmup, n_cpu_rounds)
    warm += warm % 2
    need = (warm + repeats * steps) * k
    pool_n = min(need, 2048) // (2 * k) * (2 * k)
    pool_x = torch.empty((pool_n, K, B, dims[0]), dtype=torch.bfloat16, device="cuda")
    I.device_mlp_batches_into(pool_x, 0)
    pool_y = I.device_mlp_teacher_labels(pool_x, teacher)
    side = torch.cuda.Stream(priority=-1)
    compute = torch.cuda.current_stream()
    grads = torch.empty((K, P), dtype=torch.float32, device="cuda")
    flops_step = K * 2 * B * (2 * dims[0] * dims[1] + 3 * dims[1] * dims[2] + 3 * dims[2] * dims[3])
    n_w12 = dims[1] * dims[0] + dims[2] * dims[1]                 # parameters the persistent kernel updates

    def run_variant(name):
        fused = name.startswith("fused")              # gradient + update in one call (all steps but, with step_end, the last)
        graphed = name.endswith("+graph")
        fuse_end = "+step_end" in name                # the round's last local step and the merge in one pass
        eng = E.Engine(K, P, lr, mu, wd)
        eng.set_option(E.OPT_BF16_SHADOW, 1)
        eng.set_params(x0)
        shadow = eng.bf16_shadow()
        n_rec = (warm + repeats * steps) * k
        loss_all = torch.zeros((n_rec + 1, K), dtype=torch.float32, device="cuda")      # last row: calls that are not recorded
        step_no = [0]
        snaps = []

        def one_round(xs, ys, first, record_at=None):
            eng.comm_begin(side)
            for j in range(k):
                out = loss_all[record_at + j] if (record_at is not None and record_at + k <= n_rec) else loss_all[n_rec]
                if fused and not (fuse_end and j == k - 1):
                    mg.grad_step(eng, xs[first + j], ys[first + j], out)
                else:
                    mg.grad(shadow, xs[first + j], ys[first + j], grads, out)
                    if fuse_end and j == k - 1:
                        eng.local_step_end(grads)
                    else:
                        eng.local_step(grads)
            if not fuse_end:
                eng.comm_end()

        def eager_round():
            i = step_no[0]
            one_round(pool_x, pool_y, i % pool_n, record_at=i)
            step_no[0] += k

        for r in range(warm):
            eager_round()
            if name == "two-call" and r < n_cpu_rounds:
                snaps.append(shadow.clone())
        torch.cuda.synchronize()
        graph = None
        if graphed:
            # One captured graph per pair of rounds of the minibatch pool (two rounds = one full cycle of the buffer
            # flip), each reading its own 2 k minibatches in place: replaying them in turn walks through the pool with
            # nothing but graph launches in the timed region.
            cap = torch.cuda.Stream()
            eng.sync()
            eng.set_stream(cap)
            graphs, per_replay = [], 0
            n_graphs = min(pool_n // (2 * k), (repeats * steps + 4) // 2 + 2)
            base = step_no[0]
            for gi in range(n_graphs):
                first = (base + gi * 2 * k) % pool_n
                lb = eng.launch_count + mg.launch_count
                g_ = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g_, stream=cap):
                    one_round(pool_x, pool_y, first)
                    one_round(pool_x, pool_y, first + k)
                per_replay = eng.launch_count + mg.launch_count - lb
                graphs.append(g_)
            graph = graphs
            plays = [0]

            def replay():
                graphs[plays[0] % n_graphs].replay()
                plays[0] += 1
                step_no[0] += 2 * k

            for _ in range(2):
                replay()
            torch.cuda.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        block_ms, launches = [], 0
        for rep in range(repeats):
            torch.cuda.synchronize()
            l0 = eng.launch_count + mg.launch_count
            ev0.record(compute)
            if graph is not None:
                for _ in range(steps // 2):
                    replay()
            else:
                for _ in range(steps):
                    eager_round()
            ev1.record(compute)
            torch.cuda.synchronize()
            block_ms.append(ev0.elapsed_time(ev1))
            launches = per_replay * (steps // 2) if graph is not None else eng.launch_count + mg.launch_count - l0
        mg.check()
        if graph is not None:
            eng.sync()
            eng.set_stream(compute)
        ms = median(block_ms)
        out = {"value": K * P_raw * k * steps / (ms * 1e-3), "ms_per_step": ms / steps, "ms_per_local_step": ms / (k * steps),
               "local_steps_per_s": k * steps / (ms * 1e-3), "gpu_launches": launches,
               "timed_blocks": {"repeats": repeats, "rounds_per_block": steps, "ms_per_step": [b_ / steps for b_ in block_ms],
                                "ms_per_step_min": min(block_ms) / steps, "ms_per_step_max": max(block_ms) / steps,
                                "reported": "median block"},
               "tensor_tflops": flops_step * k * steps / (ms * 1e-3) / 1e12}
        # ---- per-kernel pass of its own (events break the programmatic launch edges, so never inside the timed blocks)
        if not graphed:
            n_prof = min(steps, 25)
            mg.set_profile(True)
            eng.set_option(E.OPT_PROFILE, 1)
            eng.profile_reset()
            for _ in range(n_prof):
                eager_round()
            calls, pass_ms, upd_ms = mg.profile()
            by = summarize_profile(eng.profile_records(), E.KERNEL_NAMES)
            eng.set_option(E.OPT_PROFILE, 0)
            mg.set_profile(False)
            if fused:
                # the same kernel inside the undisturbed chain, by its own stamps (no events, launches unchanged)
                mg.set_profile(2)
                for _ in range(n_prof):
                    eager_round()
                n_dev, upd_dev_ms = mg.profile_device()
                mg.set_profile(0)
                alg = 18 * K * n_w12
                gbs = alg / (upd_ms * 1e-3) / 1e9 if upd_ms > 0 else None
                out["roofline"] = {"bound": "hbm", "kernel": "gemm_update_persistent (weight gradients of W1, W2 + their momentum update)",
                                   "achieved": round(gbs, 1) if gbs else None, "peak": hbm_peak, "unit": "GB/s",
                                   "frac": round(gbs / hbm_peak, 4) if gbs else None,
                                   "traffic": W.NCU_DRAM_BYTES_MLP_UPDATE_KERNEL_K16 if K == 16 else None, "peak_kind": peak_kind,
                                   "algorithmic_bytes_per_launch": alg, "avg_launch_ms": round(upd_ms, 5),
                                   "bytes_per_parameter": 18,
                                   "measured_in": "a pass of its own with CUDA events around the kernel (launched without its "
                                                  "programmatic overlap)",
                                   "inside_the_chain": {"avg_launch_ms": round(upd_dev_ms, 5), "launches": n_dev,
                                                        "achieved": round(alg / (upd_dev_ms * 1e-3) / 1e9, 1) if upd_dev_ms > 0 else None,
                                                        "frac": round(alg / (upd_dev_ms * 1e-3) / 1e9 / hbm_peak, 4) if upd_dev_ms > 0 else None,
                                                        "measured_in": "the undisturbed eager chain, by the kernel's own first-start / "
                                                                       "last-end stamps on the GPU's clock"}}
                out["gradient_pass_ms"] = {"whole_call": round(pass_ms, 5), "update_kernel": round(upd_ms, 5),
                                           "everything_else": round(pass_ms - upd_ms, 5), "calls": calls}
            else:
                iv = by.get("local_step", [])
                avg_ms = sum(b_ - a_ for a_, b_ in iv) / max(1, len(iv))
                gbs = 22.0 * K * P / (avg_ms * 1e-3) / 1e9 if iv else None
                out["roofline"] = {"bound": "hbm", "kernel": "local_step (with bf16 shadow)", "achieved": round(gbs, 1) if gbs else None,
                                   "peak": hbm_peak, "unit": "GB/s", "frac": round(gbs / hbm_peak, 4) if gbs else None,
                                   "traffic": None, "peak_kind": peak_kind, "algorithmic_bytes_per_launch": 22 * K * P,
                                   "avg_launch_ms": round(avg_ms, 5), "bytes_per_parameter": 22,
                                   "measured_in": "a pass of its own with per-kernel CUDA events"}
                out["gradient_pass_ms"] = {"whole_call": round(pass_ms, 5), "weight_gradient_kernel": round(upd_ms, 5),
                                           "everything_else": round(pass_ms - upd_ms, 5), "calls": calls}
        torch.cuda.synchronize()
        n_done = min(step_no[0], n_rec) if not graphed else warm * k
        curve = loss_all[:n_done].double().mean(dim=1).cpu().numpy()
        out["loss_first_steps"] = [round(float(v), 5) for v in curve[:4 * k]]
        out["loss_last"] = round(float(curve[-1]), 5) if not graphed else None
        return out, eng, curve, snaps

    variants = {}
    curve2, snaps2 = None, None
    sampler = ClockSampler(0)
    names = ["two-call", "two-call+step_end", "fused", "fused+graph", "fused+step_end", "fused+step_end+graph"]
    engines = {}
    for name in names:
        variants[name], engines[name], curve, snaps = run_variant(name)
        if name == "two-call":
            curve2, snaps2 = curve, snaps
        if name != "fused" or digest:
            engines.pop(name).destroy()
    clocks = sampler.stop()

    # ---- end to end (stand-alone run only): minibatches and labels start in pinned host memory, the loss comes back every
    #      step; the upload of step t + 1 (copy stream, two device buffers) runs under the kernels of step t
    e2e = None
    if not digest and not args.no_e2e:
        eng = engines.pop("fused")
        ring_n = min(pool_n, 256)
        xs_h = pool_x[:ring_n].cpu().pin_memory()
        ys_h = pool_y[:ring_n].cpu().pin_memory()
        copy_stream = torch.cuda.Stream()
        x_buf = [torch.empty_like(pool_x[0]) for _ in range(2)]
        y_buf = [torch.empty_like(pool_y[0]) for _ in range(2)]
        ev_up = [torch.cuda.Event() for _ in range(2)]
        ev_used = [torch.cuda.Event() for _ in range(2)]
        loss = torch.empty(K, dtype=torch.float32, device="cuda")
        loss_h = torch.empty(K, dtype=torch.float32, pin_memory=True)
        n_e2e = max(1, min(steps, 50))
        up_no, host_step = [0], [0]

        def upload():
            slot, i = up_no[0] % 2, up_no[0] % ring_n
            with torch.cuda.stream(copy_stream):
                if up_no[0] >= 2:
                    copy_stream.wait_event(ev_used[slot])          # the kernels that read this buffer are done
                x_buf[slot].copy_(xs_h[i], non_blocking=True)
                y_buf[slot].copy_(ys_h[i], non_blocking=True)
                ev_up[slot].record(copy_stream)
            up_no[0] += 1

        def one_round_host():
            eng.comm_begin(side)
            for _ in range(k):
                slot = host_step[0] % 2
                upload()                                           # next step's inputs
                compute.wait_event(ev_up[slot])
                mg.grad_step(eng, x_buf[slot], y_buf[slot], loss)
                ev_used[slot].record(compute)
                loss_h.copy_(loss, non_blocking=True)
                host_step[0] += 1
            eng.comm_end()

        torch.cuda.synchronize()
        upload()
        for _ in range(2):
            one_round_host()
        torch.cuda.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(compute)
        for _ in range(n_e2e):
            one_round_host()
        ev1.record(compute)
        torch.cuda.synchronize()
        ms_e2e = ev0.elapsed_time(ev1)
        e2e = {"value": K * P_raw * k * n_e2e / (ms_e2e * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": k * (xs_h[0].numel() * 2 + ys_h[0].numel() * 4), "d2h_bytes_per_step": k * K * 4,
               "rounds": n_e2e, "ms_per_step": ms_e2e / n_e2e, "path": "fused gradient + update call"}
        eng.destroy()
    for e_ in engines.values():
        e_.destroy()

    # ---- the oracle beside it: the first rounds of the SAME run (same minibatch and label bytes), all K workers, one
    #      process per worker on the host's cores; gives the paired loss curve and the per-round parameter distance
    cpu_baseline, paired = None, None
    if n_cpu_rounds > 0:
        procs = max(1, min(K, os.cpu_count() or 1))
        nst = n_cpu_rounds * k
        Xb = pool_x[:nst].view(torch.int16).cpu().numpy().view(np.uint16)
        yb = pool_y[:nst].cpu().numpy()
        dt, o_losses, o_params = time_mlp_oracle(K, k, n_cpu_rounds, lr, mu, wd, x0[:P_raw], Xb, yb, procs)
        cpu_baseline = {"value": K * P_raw * k * n_cpu_rounds / dt, "unit": UNIT, "cores": procs, "kind": "oracle",
                        "sample": f"the first {n_cpu_rounds} rounds (k={k}) of the same run, all {K} workers: numpy fp64 gradient "
                                  f"with the bf16 rounding points (one process per worker) + reference-mode parameter path"}
        worst, first_break = [], None
        for r in range(n_cpu_rounds):
            got = snaps2[r].float().cpu().numpy()[:, :P_raw]
            want = o_params[r]
            scale = np.maximum(np.abs(want), np.sqrt(np.mean(want.astype(np.float64) ** 2)))
            e_ = float((np.abs(got - want) / scale).max())
            worst.append(round(e_, 5))
            if e_ > 1e-2 and first_break is None:
                first_break = r + 1
        paired = {"steps": nst, "gpu": [round(float(v), 5) for v in curve2[:nst]], "oracle": [round(v, 5) for v in o_losses],
                  "max_relative_gap": float(max(abs(a_ - b_) / abs(b_) for a_, b_ in zip(curve2[:nst], o_losses))),
                  "bf16_parameters_max_scaled_error_per_round_free_running": worst,
                  "first_round_outside_1e-2": first_break,
                  "note": "free-running device run against the canonical oracle; the per-round parity run with the "
                          "restarted engines over all 200 rounds is tests/c4_loss_curve.py"}
    head = "fused+graph" if (args.fused and args.graph) else "fused" if args.fused else "fused+graph" if args.graph else "two-call"
    if digest:
        head = "fused"
    hv = variants[head]
    res = {
        "metric": METRIC, "value": hv["value"], "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": warm,
        "ms_per_step": hv["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 contractions / f32 state", "data": "synthetic",
        "config": {"workload": "mlp", "K": K, "P": P_raw, "P_padded": P, "k": k, "lr": lr, "mu": mu, "wd": wd,
                   "mlp": list(dims), "batch": B, "minibatch_pool_steps": pool_n,
                   "minibatches": "one per (worker, global step), seeded; the pool repeats after minibatch_pool_steps steps",
                   "headline_variant": head,
                   "l2": "the K x P state is 119 MB fp32 + 119 MB momentum + 60 MB bf16 copy: larger than the 126 MB L2"},
        "clocks": clocks, "gpu_launches": hv["gpu_launches"], "roofline": hv.get("roofline") or variants["fused"].get("roofline"),
        "cpu_baseline": cpu_baseline, "variants": variants, "loss_curve_vs_oracle": paired,
        "local_steps_per_s": hv["local_steps_per_s"], "ms_per_local_step": hv["ms_per_local_step"],
        "tensor_peak_tflops": peaks.get("bf16_tflops"), "e2e": e2e,
    }
    mg.destroy()
    del pool_x, pool_y, grads
    torch.cuda.empty_cache()
    return res


def run_mlp(args):
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the engine has no CPU fallback")
    torch.cuda.set_device(0)
    print(json.dumps(measure_mlp(args, digest=False)))


# ---------------------------------------------------------------------------------------------- workers over GPUs
def run_worker_sharded(args, wl):
    """Every rank holds wl.K workers of K_global = wl.K * N (weak scaling in the workers, the paper's
    layout).  Step II and the merge are local; Step I's mean over all K_global workers is completed on
    the side stream by an all-reduce of P floats or by the gather kernel."""
    import socket
    import torch
    import torch.distributed as dist
    from paper_1906_12043_b200 import build, engine as E, inputs as I, workloads as W
    from paper_1906_12043_b200.sharded import WorkerShardedEngine

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the engine has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if "MASTER_ADDR" not in os.environ:                 # plain `python bench.py`: a group of one
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(sk.getsockname()[1]))
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=torch.device("cuda", local_rank))
    if rank == 0:
        build.build()
    dist.barrier()
    E.load()
    K, P, k = wl.K, wl.P, wl.k
    K_global = K * world
    hbm_peak, peak_kind = 6650.0, "fallback"
    try:
        hbm_peak, peak_kind = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["hbm_gbs"]), "measured"
    except (OSError, KeyError):
        pass
    eng = WorkerShardedEngine(K_global, P, wl.lr, wl.mu, wl.wd, exchange=args.exchange, sync="stream")
    x0 = torch.empty(P, dtype=torch.float32, device="cuda")
    I.device_gaussian_into(x0, I.X0_SEED, I.STREAM_X0, 0, 0, 0, wl.sigma_x0)
    eng.set_params(x0)
    ring = []
    for t in range(max(1, args.ring)):
        g = torch.empty((K, P), dtype=torch.float32, device="cuda")
        I.device_gradients_into(g, t, wl.sigma_g, first_worker=eng.first)
        ring.append(g)
    side = torch.cuda.Stream(priority=-1)
    compute = torch.cuda.current_stream()
    step_no = [0]

    def one_round():
        eng.comm_begin(side)
        for _ in range(k):
            eng.local_step(ring[step_no[0] % len(ring)])
            step_no[0] += 1
        eng.comm_end()

    def barrier():
        dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        one_round()
    eng.engine.set_option(E.OPT_PROFILE, 1)
    eng.engine.profile_reset()
    barrier()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    launches0 = eng.engine.launch_count
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(compute)
    for _ in range(args.steps):
        one_round()
    ev1.record(compute)
    barrier()
    clocks = sampler.stop() if sampler else None
    t = torch.tensor([ev0.elapsed_time(ev1)], dtype=torch.float64, device="cuda")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms = float(t.item())
    launches = eng.engine.launch_count - launches0
    by = summarize_profile(eng.engine.profile_records(), E.KERNEL_NAMES)
    eng.engine.set_option(E.OPT_PROFILE, 0)
    # what one GPU's mean kernel moves: its K stored copies -> P partial sums, or K_global rows of its
    # share of the columns -> that share in every GPU's buffer
    mean_bytes = (4 * K * P + 4 * P) if args.exchange == "allreduce" else (4 * K_global * P / world + 4 * P)
    alg_bytes = {"local_step": W.BYTES_LOCAL_STEP * K * P, "mean": mean_bytes, "merge": W.bytes_merge(K) * K * P}
    table = {}
    for name, iv in by.items():
        avg_ms = sum(b - a for a, b in iv) / len(iv)
        gbs = alg_bytes[name] / (avg_ms * 1e-3) / 1e9
        table[name] = {"launches": len(iv), "avg_ms": round(avg_ms, 5), "gbs": round(gbs, 1),
                       "frac_of_peak": round(gbs / hbm_peak, 4)}
    dom = table.get("local_step", {})
    if rank == 0:
        if world == 1:
            link_bytes = 0
        elif args.exchange == "allreduce":
            link_bytes = 8 * P * (world - 1) / world
        else:
            link_bytes = 4 * P * (K_global - K) / world + 4 * P * (world - 1) / world
        print(json.dumps({
            "metric": METRIC, "value": world * K * P * k * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name, "K": K, "K_global": K_global, "P": P, "k": k, "lr": wl.lr, "mu": wl.mu,
                       "wd": wl.wd, "snapshot": "flip", "gradient_ring": len(ring),
                       "sharding": f"workers ({K} per GPU), mean over GPUs by {args.exchange} on the side stream",
                       "l2": "inputs larger than L2" if K * P * 4 > 126e6 else "L2-resident workload: not an HBM number"},
            "clocks": clocks, "e2e": None, "gpu_launches": launches,
            "roofline": {"bound": "hbm", "kernel": "local_step", "achieved": dom.get("gbs"), "peak": hbm_peak,
                         "unit": "GB/s", "frac": dom.get("frac_of_peak"), "traffic": None, "peak_kind": peak_kind,
                         "algorithmic_bytes_per_launch": alg_bytes["local_step"], "avg_launch_ms": dom.get("avg_ms")},
            "cpu_baseline": None, "kernels_in_loop": table, "overlap_fraction": overlap_fraction(by),
            "link_bytes_per_round_per_gpu": link_bytes,
        }))
    eng.close()
    dist.destroy_process_group()


def sweep_cells(cells, emit):
    """Timing-only measurement of (K, P) cells at k = 1 and k = 8.  Values do not affect timing, so each cell reuses
    one generated gradient buffer.  `emit(record)` is called per (K, P, k)."""
    import torch
    from paper_1906_12043_b200 import engine as E, inputs as I, workloads as W
    side = torch.cuda.Stream(priority=-1)
    compute = torch.cuda.current_stream()
    for K, P in cells:
        g = torch.empty((K, P), dtype=torch.float32, device="cuda")
        I.device_gradients_into(g, 0)
        x0 = torch.empty(P, dtype=torch.float32, device="cuda")
        I.device_gaussian_into(x0, I.X0_SEED, I.STREAM_X0, 0, 0, 0, 0.01)
        for k in (1, 8):
            eng = E.Engine(K, P, 0.1, 0.9, 5e-4)
            eng.set_params(x0)
            wl = W.Workload("sweep", K, P, k, 0, 0.1, 0.9, 5e-4)
            rounds = max(3, min(200, int(0.25 / (wl.bytes_per_round() / 6.5e12))))

            def one_round(s):
                eng.comm_begin(s)
                for _ in range(k):
                    eng.local_step(g)
                eng.comm_end()

            res = {}
            for mode, s in (("overlapped", side), ("serial", compute)):
                for _ in range(3):
                    one_round(s)
                eng.set_option(E.OPT_PROFILE, 1)
                eng.profile_reset()
                torch.cuda.synchronize()
                ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                ev0.record(compute)
                for _ in range(rounds):
                    one_round(s)
                ev1.record(compute)
                torch.cuda.synchronize()
                by = summarize_profile(eng.profile_records(), E.KERNEL_NAMES)
                eng.set_option(E.OPT_PROFILE, 0)
                alg = {"local_step": W.BYTES_LOCAL_STEP * K * P, "mean": W.bytes_mean(K) * K * P,
                       "merge": W.bytes_merge(K) * K * P}
                res[mode] = {"ms_per_round": ev0.elapsed_time(ev1) / rounds,
                             "gbs": {n: round(alg[n] / (sum(b - a for a, b in iv) / len(iv) * 1e-3) / 1e9, 1)
                                     for n, iv in by.items()},
                             "overlap_fraction": overlap_fraction(by)}

            # the same rounds with the last local step and the merge in one pass
            def one_round_fused_end():
                eng.comm_begin(side)
                for j in range(k):
                    if j < k - 1:
                        eng.local_step(g)
                    else:
                        eng.local_step_end(g)

            for _ in range(3):
                one_round_fused_end()
            torch.cuda.synchronize()
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record(compute)
            for _ in range(rounds):
                one_round_fused_end()
            ev1.record(compute)
            torch.cuda.synchronize()
            ms_fe = ev0.elapsed_time(ev1) / rounds
            ms = res["overlapped"]["ms_per_round"]
            emit({
                "sweep": True, "K": K, "P": P, "k": k, "rounds": rounds,
                "ms_per_round_fused_end": ms_fe, "updates_per_s_fused_end": K * P * k / (ms_fe * 1e-3),
                "hbm_gbs_whole_round_fused_end": (wl.bytes_per_round() - 8 * K * P) / (ms_fe * 1e-3) / 1e9,
                "updates_per_s": K * P * k / (ms * 1e-3),
                "hbm_gbs_whole_round": wl.bytes_per_round() / (ms * 1e-3) / 1e9,
                "ms_per_round": ms, "ms_per_round_serial": res["serial"]["ms_per_round"],
                "kernel_gbs_isolated": res["serial"]["gbs"], "kernel_gbs_overlapped": res["overlapped"]["gbs"],
                "overlap_fraction": res["overlapped"]["overlap_fraction"],
                "l2_resident": bool(K * P * 16 < 126e6)})
            eng.destroy()
        del g, x0
        torch.cuda.empty_cache()


def run_sweep(args):
    """The scaling sweep over (P, K, k): one JSON line per cell.  Cells whose four K x P buffers exceed 160 GB are
    skipped."""
    import torch
    from paper_1906_12043_b200 import build
    build.build()
    torch.cuda.set_device(0)
    cells = [(K, 1 << logP) for logP in [int(v) for v in args.sweep_logP.split(",")]
             for K in [int(v) for v in args.sweep_K.split(",")] if K * (1 << logP) * 16 <= 160e9]
    sweep_cells(cells, lambda rec: print(json.dumps(rec), flush=True))


def main():
    args = parse()
    if args.sweep:
        run_sweep(args)
        return
    from paper_1906_12043_b200.workloads import WORKLOADS
    if args.workload == "mlp":
        if args.impl == "reference":
            run_reference_mlp(args)
            return
        run_mlp(args)
        return
    wl = WORKLOADS[args.workload]
    if args.K or args.P or args.k:
        from dataclasses import replace
        wl = replace(wl, name=wl.name + "-custom", K=args.K or wl.K, P=args.P or wl.P, k=args.k or wl.k)
    if args.impl == "reference":
        run_reference(args, wl)
    elif args.shard == "workers":
        run_worker_sharded(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
