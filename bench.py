#!/usr/bin/env python
"""Benchmark of the DropCompute threshold sweep on B200.

One "step" is one pass of the whole path over one batch of synthetic latencies:
dc_simulate_ex (the sweep) + dc_reduce_trials + dc_argmax_tau, through the C ABI.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is latency samples per second over the timed steps with the
latency tensor already resident in HBM; `e2e` is the same metric through dc_sweep_host with the
samples in pinned HOST memory (copies inside the timed region); `roofline` is the sweep kernel's
algorithmic bytes over its CUDA-event duration against the measured HBM copy bandwidth;
`cpu_baseline` times the CPU oracle on a bounded sample of the same workload.
With --gpus N > 1 (under torchrun) every rank sweeps its own tensor of the same shape (trials are
independent: weak scaling, no data-path collective); the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2306_10598_b200 import sharding  # noqa: E402
from paper_2306_10598_b200 import workloads as W  # noqa: E402

METRIC = "latency samples/s (tau-sweep: dc_simulate + dc_reduce_trials + dc_argmax_tau)"
UNIT = "samples/s"
FALLBACK_HBM_GBS = 6650.0


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def mark(self):
        return time.time()

    def stop(self, t0=None, t1=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        rows = [r for (ts, r) in self.rows if (t0 is None or ts >= t0) and (t1 is None or ts <= t1 + 0.2)] or [r for _, r in self.rows]
        sm, smax, reasons = [], None, set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0]))
                smax = float(r[1])
            except ValueError:
                continue
            for name, val in zip(names, r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": smax, "reasons": sorted(reasons),
                "samples": len(sm)}


def cpu_baseline(w: W.Workload, lat_dev, taus: np.ndarray, budget_s: float = 15.0):
    """Times the CPU oracle (as it stands) on a bounded sample of whole trials of the same workload."""
    import oracle
    probe = min(w.T, 16)
    lat = lat_dev[:probe].cpu().numpy()
    oracle.sweep(lat[:1], taus, w.t_comm)  # loads the library and starts the thread pool
    t = time.perf_counter()
    oracle.sweep(lat, taus, w.t_comm)
    dt = max(time.perf_counter() - t, 1e-4)
    n = int(max(probe, min(w.T, budget_s / (dt / probe))))
    # keep the host copy of the sample modest
    n = min(n, max(probe, (16 << 30) // (4 * w.N * w.M)))
    lat = lat_dev[:n].cpu().numpy()
    t = time.perf_counter()
    sw = oracle.sweep(lat, taus, w.t_comm)
    st = oracle.reduce_trials(sw.step, sw.done, sw.sync, w.N, w.M)
    oracle.argmax(st.stats[4])
    dt = time.perf_counter() - t
    return {"value": n * w.N * w.M / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"first {n} of {w.T} trials of '{w.name}' (N={w.N}, M={w.M}, K={w.K}), {dt:.2f} s, row-order oracle with OpenMP",
            "seconds": dt}


def run_reference(args, w: W.Workload):
    """The reference arm: the CPU oracle on the machine's host cores, each step a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    taus = W.make_taus(w)
    # size the per-step sample so that (steps + warmup) steps take about a minute in total
    probe = min(w.T, 16)
    lat = W.fill_latencies(w, "cpu", t0=0, t1=probe).numpy()
    oracle.sweep(lat[:1], taus, w.t_comm)  # loads the library and starts the thread pool
    t = time.perf_counter()
    oracle.sweep(lat, taus, w.t_comm)
    per_trial = max(time.perf_counter() - t, 1e-4) / probe
    total_steps = args.steps + args.warmup
    n = int(max(1, min(w.T, (60.0 / total_steps) / per_trial)))
    n = min(n, max(1, (4 << 30) // (4 * w.N * w.M)))
    lat = W.fill_latencies(w, "cpu", t0=0, t1=n).numpy()

    def step():
        sw = oracle.sweep(lat, taus, w.t_comm)
        st = oracle.reduce_trials(sw.step, sw.done, sw.sync, w.N, w.M)
        return oracle.argmax(st.stats[4])

    for _ in range(args.warmup):
        step()
    t = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t
    value = args.steps * n * w.N * w.M / dt
    sample = f"first {n} of {w.T} trials of '{w.name}' per step (CPU-generated, same law and seed)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "T": w.T, "N": w.N, "M": w.M, "K": w.K, "t_comm": w.t_comm},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


def read_traffic(workload: str, kernel_version: str):
    """DRAM bytes per sweep launch from the ncu capture filed in profiles/traffic.txt, or None when there is
    no capture of this workload taken on the kernel version the library reports."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.txt")) as f:
            for ln in f:
                parts = ln.split()
                if len(parts) == 3 and not ln.startswith("#") and parts[0] == workload and parts[1] == kernel_version:
                    return int(parts[2])
    except (OSError, ValueError):
        pass
    return None


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
    parts = [x.strip() for x in vis.split(",") if x.strip()]
    if local_rank < len(parts) and parts[local_rank].isdigit():
        return int(parts[local_rank])
    return local_rank


def host_mem_available_bytes() -> int:
    try:
        with open("/proc/meminfo") as f:
            for line in f:
                if line.startswith("MemAvailable:"):
                    return int(line.split()[1]) * 1024
    except OSError:
        pass
    return 0


def time_other_workloads(api, dev, peak: float, max_trials: int = 0):
    """The four smaller workloads under both completion rules and the bench workload under rule 1: one
    dc_simulate_ex launch each, 3 warm-ups and 10 timed launches, under the same regime as the headline
    measurement (a 256 MiB buffer is written between launches when the input is smaller than 512 MB; larger
    inputs exceed the L2 cache by themselves), with a plain read-only pass over the same bytes beside each.  Three of
    the workloads are also run through dc_simulate_scaled (rows with an "entry" key)."""
    rows = []
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    sink = torch.zeros((1,), dtype=torch.float32, device=dev)
    for name, rules in (("tiny", (0, 1)), ("paper_scale", (0, 1)), ("extrapolation", (0, 1)), ("correlated", (0, 1)),
                        ("bandwidth_stress", (1,))):
        w = W.WORKLOADS[name]
        if max_trials and w.T > max_trials:
            w = w.with_trials(max_trials)
        free, _ = torch.cuda.mem_get_info(dev)
        if free < w.latency_bytes + (2 << 30):
            rows.append({"workload": name, "skipped": "not enough free device memory"})
            continue
        lat = W.fill_latencies(w, dev)
        taus = torch.from_numpy(W.make_taus(w)).to(dev)
        step = torch.empty((w.T, w.K), dtype=torch.float32, device=dev)
        done = torch.empty((w.T, w.K), dtype=torch.int32, device=dev)
        sync = torch.empty((w.T,), dtype=torch.float32, device=dev)
        fl = flush if w.latency_bytes < (512 << 20) else None

        def timed(fn):
            ms = []
            for i in range(13):
                if fl is not None:
                    fl.zero_()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                fn()
                e1.record()
                torch.cuda.synchronize(dev)
                if i >= 3:
                    ms.append(e0.elapsed_time(e1))
            return sum(ms) / len(ms), min(ms)

        probe_ms, _ = timed(lambda: api.dc_read_probe(lat, sink))
        alg_bytes = 4 * w.samples + 8 * w.T * w.K + 4 * w.T
        for rule in rules:
            avg_ms, best_ms = timed(lambda: api.dc_simulate_ex(lat, taus, w.t_comm, step, done, sync, rule))
            gbs = alg_bytes / (avg_ms * 1e-3) / 1e9
            rows.append({"workload": name, "rule": rule, "T": w.T, "N": w.N, "M": w.M, "K": w.K,
                         "kernel": ("dc_sweep_tiled", "dc_sweep_plain", "dc_sweep_flat")[api.dc_simulate_plan(lat, w.K)],
                         "sweep_ms": avg_ms, "sweep_ms_best": best_ms, "hbm_gbs": gbs, "frac": gbs / peak,
                         "read_only_pass_ms": probe_ms, "sweep_over_read_only_pass": avg_ms / probe_ms,
                         "l2": "inputs larger than L2" if fl is None else "256 MiB buffer written between launches"})
        if name in ("paper_scale", "extrapolation", "correlated"):
            # workers with thresholds of their own (s_n tau_k, s_n uniform on [0.8, 1.2]): dc_simulate_scaled
            scale = torch.from_numpy(W.worker_scales(w.N, w.seed)).to(dev)
            for rule in rules:
                avg_ms, best_ms = timed(lambda: api.dc_simulate_scaled(lat, taus, scale, w.t_comm, step, done, sync, rule))
                gbs = (alg_bytes + 4 * w.N) / (avg_ms * 1e-3) / 1e9
                rows.append({"workload": name, "rule": rule, "T": w.T, "N": w.N, "M": w.M, "K": w.K,
                             "entry": "dc_simulate_scaled", "kernel": "dc_sweep_scaled",
                             "sweep_ms": avg_ms, "sweep_ms_best": best_ms, "hbm_gbs": gbs, "frac": gbs / peak,
                             "read_only_pass_ms": probe_ms, "sweep_over_read_only_pass": avg_ms / probe_ms,
                             "l2": "inputs larger than L2" if fl is None else "256 MiB buffer written between launches"})
        del lat, step, done, sync
        torch.cuda.empty_cache()
    api.dc_device_status()
    return rows


def shape_grid(args):
    """`--shape-grid`: a table (text, not the JSON line) of GB/s of latency bytes per dc_simulate_ex launch over worker
    counts N and micro-batch counts M at fixed numbers of latency bytes, rule 0 / rule 1.  Uniform latencies, 64 evenly
    spaced thresholds over [0.6, 1.4] x the mean row total, median of five launches by CUDA events, a 256 MiB buffer
    written between launches.  Shows what few workers per trial, very short rows and ragged row lengths cost."""
    from paper_2306_10598_b200 import build
    build.build_library()
    from paper_2306_10598_b200 import api
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    K = 64

    def cell(T, N, M, rule):
        g = torch.Generator(device=dev).manual_seed(1)
        lat = torch.rand(T, N, M, device=dev, generator=g) * 0.01 + 0.02
        taus = torch.linspace(0.6 * 0.025 * M, 1.4 * 0.025 * M, K, device=dev)
        step = torch.empty(T, K, dtype=torch.float32, device=dev)
        done = torch.empty(T, K, dtype=torch.int32, device=dev)
        sync = torch.empty(T, dtype=torch.float32, device=dev)
        ms = []
        for i in range(7):
            flush.fill_(i)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            api.dc_simulate_ex(lat, taus, 0.1, step, done, sync, rule)
            e1.record()
            torch.cuda.synchronize(dev)
            if i >= 2:
                ms.append(e0.elapsed_time(e1))
        return 4 * T * N * M / statistics.median(ms) / 1e6

    workers = (8, 32, 100, 200, 256, 300, 512, 1000, 2048, 5000)
    micro = (4, 8, 12, 16, 24, 32, 48, 64, 100, 128, 256, 512)
    for total in args.shape_grid:
        print(f"{total:.1e} latency bytes; rows: workers N, columns: micro-batches M; GB/s under rule 0 / rule 1")
        print("N\\M   " + "".join(f"{m:>12d}" for m in micro))
        for N in workers:
            cells = []
            for M in micro:
                T = max(1, int(total / (4 * N * M)))
                cells.append(f"{cell(T, N, M, 0):6.0f}/{cell(T, N, M, 1):5.0f}")
            print(f"{N:5d} " + "".join(f"{c:>12s}" for c in cells), flush=True)
    api.dc_device_status()
    return 0


def run_ours(args, w: W.Workload):
    from paper_2306_10598_b200 import build
    if int(os.environ.get("LOCAL_RANK", "0")) == 0:
        build.build_library()   # compiles the library in-tree if it is missing or older than its sources
    else:                       # the other ranks of the node wait for it (the build replaces the file atomically)
        deadline = time.time() + 900
        while build.is_stale() and time.time() < deadline:
            time.sleep(0.5)
    from paper_2306_10598_b200 import api

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus != world:
        if world == 1 and args.gpus > 1:
            raise SystemExit("--gpus N > 1 must be launched with torch.distributed.run (one rank per GPU)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1 or ("RANK" in os.environ and "MASTER_ADDR" in os.environ):  # launched by torch.distributed.run
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    # every rank sweeps its own tensor of the same shape (independent trials: weak scaling)
    wr = sharding.rank_workload(w, rank)
    lat = W.fill_latencies(wr, dev)
    taus_np = W.make_taus(wr)
    taus = torch.from_numpy(taus_np).to(dev)
    T, N, M, K = wr.T, wr.N, wr.M, wr.K
    out_step = torch.empty((T, K), dtype=torch.float32, device=dev)
    out_done = torch.empty((T, K), dtype=torch.int32, device=dev)
    out_sync = torch.empty((T,), dtype=torch.float32, device=dev)
    stats = torch.empty((api.NSTATS, K), dtype=torch.float64, device=dev)
    baseline = torch.empty((2,), dtype=torch.float64, device=dev)
    ws = torch.empty((api.dc_reduce_workspace_bytes(T, K),), dtype=torch.uint8, device=dev)
    k_star = torch.empty((), dtype=torch.int32, device=dev)
    tau_star = torch.empty((), dtype=torch.float32, device=dev)
    value = torch.empty((), dtype=torch.float64, device=dev)
    # --worker-scales: the heterogeneous-worker sweep (worker n against s_n tau_k) in place of the common-threshold one
    scale = torch.from_numpy(W.worker_scales(N, wr.seed)).to(dev) if args.worker_scales else None
    flush = None
    if wr.latency_bytes < (512 << 20):  # inputs not much larger than L2: write a 256 MiB buffer between steps
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def step(ev=None):
        if flush is not None:
            flush.zero_()
        if ev:
            ev[0].record()
        if scale is not None:
            api.dc_simulate_scaled(lat, taus, scale, wr.t_comm, out_step, out_done, out_sync, args.rule)
        else:
            api.dc_simulate_ex(lat, taus, wr.t_comm, out_step, out_done, out_sync, args.rule)
        if ev:
            ev[1].record()
        api.dc_reduce_trials(out_step, out_done, out_sync, N, M, stats, baseline, ws)
        api.dc_argmax_tau(stats, taus, api.STAT_S_EFF, k_star, tau_star, value)
        if ev:
            ev[2].record()

    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    api.dc_device_status()

    events = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sampler = ClockSampler(physical_gpu_index(local_rank))
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    t_mark0 = sampler.mark()
    for i in range(args.steps):
        step(events[i])
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    t_mark1 = sampler.mark()
    # the flush (if any) sits before ev[0], so step time = ev[0]..ev[2] summed over steps
    step_ms = [e[0].elapsed_time(e[2]) for e in events]
    sim_ms = [e[0].elapsed_time(e[1]) for e in events]
    total_ms = sum(step_ms)
    total_ms = sharding.max_over_ranks(total_ms, dev)
    clocks = sampler.stop(t_mark0, t_mark1) if rank == 0 else None
    api.dc_device_status()

    # a plain read-only pass over the same latency bytes, under the same flush regime (context for the roofline
    # fraction: short passes do not reach the bandwidth a long copy measures)
    sink = torch.zeros((1,), dtype=torch.float32, device=dev)
    probe_ms = []
    for i in range(8):
        if flush is not None:
            flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        api.dc_read_probe(lat, sink)
        e1.record()
        torch.cuda.synchronize()
        if i >= 3:
            probe_ms.append(e0.elapsed_time(e1))
    read_probe_ms = statistics.median(probe_ms)

    samples = T * N * M
    value_sps = world * args.steps * samples / (total_ms * 1e-3)
    sim_avg_s = (sum(sim_ms) / len(sim_ms)) * 1e-3
    alg_bytes = 4 * samples + 8 * T * K + 4 * T + (4 * N if scale is not None else 0)
    peak, peak_kind = measured_hbm_peak()
    achieved = alg_bytes / sim_avg_s / 1e9
    traffic = read_traffic(w.name, api.dc_kernel_version()) if not (args.trials or args.worker_scales) else None
    kernel_name = ("dc_sweep_scaled" if scale is not None
                   else ("dc_sweep_tiled", "dc_sweep_plain", "dc_sweep_flat")[api.dc_simulate_plan(lat, K)])

    line = {
        "metric": METRIC, "value": value_sps, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "T": T, "N": N, "M": M, "K": K, "t_comm": wr.t_comm,
                   "latency_bytes": wr.latency_bytes,
                   "l2": "inputs larger than L2" if flush is None else "256 MiB buffer written between steps",
                   "parallelism": f"{world} x independent trials", "rule": args.rule,
                   "entry": "dc_simulate_scaled (s_n uniform on [0.8, 1.2])" if scale is not None else "dc_simulate_ex"},
        "hbm_gbs": achieved,
        "sweep_ms": sim_avg_s * 1e3,
        "sweep_ms_best": min(sim_ms),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": traffic, "kernel": kernel_name,
                     "peak_kind": f"of {peak_kind} (a copy: half reads, half writes; this kernel almost only reads, which HBM "
                                  "does a little faster, so the fraction can pass 1)",
                     "algorithmic_bytes_per_launch": alg_bytes,
                     "frac_of_nominal_8TBs": achieved / 8000.0,
                     "read_only_pass_ms": read_probe_ms, "read_only_pass_gbs": 4 * samples / (read_probe_ms * 1e-3) / 1e9,
                     "sweep_over_read_only_pass": (sim_avg_s * 1e3) / read_probe_ms},
        "sweep_ms_x_sm_ghz": None,
        "gpu_launches": args.steps * (api.dc_launch_count(api.ENTRY_SIMULATE, T, N, M, K) +
                                      api.dc_launch_count(api.ENTRY_REDUCE_TRIALS, T, N, M, K) +
                                      api.dc_launch_count(api.ENTRY_ARGMAX_TAU, T, N, M, K)),
        "clocks": clocks,
    }

    if rank == 0 and clocks and clocks.get("sm_mhz"):
        line["sweep_ms_x_sm_ghz"] = sim_avg_s * 1e3 * clocks["sm_mhz"] / 1e3
    if rank == 0 and world == 1:
        tau_k = int(k_star.item())
        line["result"] = {"k_star": tau_k, "tau_star": float(tau_star.item()), "s_eff": float(value.item()),
                          "mean_sync": float(baseline[0].item())}

    # ---- end to end: samples in pinned host memory, through dc_sweep_host -------------------------
    e2e = None
    if not args.no_e2e and not args.worker_scales:   # (dc_sweep_host runs the common-threshold sweep)
        avail = host_mem_available_bytes()
        Te = T
        if wr.latency_bytes > 0.6 * avail / max(world, 1):
            Te = max(1, int(0.5 * avail / max(world, 1)) // (4 * N * M))
        chunk = max(1, min(Te, (1 << 30) // (4 * N * M)))   # 1 GiB per copy
        host = torch.empty((Te, N, M), dtype=torch.float32, pin_memory=True)
        host.copy_(lat[:Te])
        taus_h = torch.from_numpy(taus_np).pin_memory()
        stats_h = torch.empty((api.NSTATS, K), dtype=torch.float64).pin_memory()
        base_h = torch.empty((2,), dtype=torch.float64).pin_memory()
        wbytes = api.dc_sweep_host_workspace_bytes(Te, N, M, K, chunk)
        wsh = torch.empty((wbytes + 1024,), dtype=torch.uint8, device=dev)
        off = (-wsh.data_ptr()) % 1024
        wsv = wsh[off:]
        torch.cuda.synchronize()
        n_e2e = max(1, min(args.steps, 3))
        api.dc_sweep_host(host, taus_h, wr.t_comm, wsv, chunk, stats_out=stats_h, baseline_out=base_h)  # warm-up
        if dist:
            dist.barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            hs = api.dc_sweep_host(host, taus_h, wr.t_comm, wsv, chunk, stats_out=stats_h, baseline_out=base_h)
        e2e_s = time.perf_counter() - t0   # dc_sweep_host is synchronous: results are in host memory on return
        e2e_s = sharding.max_over_ranks(e2e_s, dev)
        e2e = {"value": world * n_e2e * Te * N * M / e2e_s, "unit": UNIT,
               "h2d_bytes_per_step": 4 * Te * N * M + 4 * K, "d2h_bytes_per_step": 8 * api.NSTATS * K + 16 + 8,
               "steps": n_e2e, "trials_per_step": Te, "chunk_trials": chunk, "ms_per_step": 1e3 * e2e_s / n_e2e,
               "api": "dc_sweep_host (pinned host samples, chunked copies overlapped with the kernels)",
               "k_star": hs.k_star}
        del host, wsh
    line["e2e"] = e2e

    if rank == 0 and world == 1 and not args.no_cpu_baseline and not args.worker_scales:
        line["cpu_baseline"] = cpu_baseline(wr, lat, taus_np)
    if (rank == 0 and world == 1 and not args.no_other_workloads and w.name == "bandwidth_stress" and not args.trials
            and args.rule == 0 and not args.worker_scales):
        del lat
        torch.cuda.empty_cache()
        line["other_workloads"] = time_other_workloads(api, dev, peak, args.other_trials)
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist:
        dist.barrier()
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=("ours", "reference"), default="ours")
    ap.add_argument("--workload", default="bandwidth_stress",
                    help="one of " + ", ".join(sorted(W.WORKLOADS)) + "; or c3:<law> for the paper's own synthetic setting "
                         "(App. C.3: 12 accumulations of 0.45 s + eps; laws: " + ", ".join(sorted(W.C3_NOISE)) +
                         "), or b1 (App. B.1 delay); these two take --workers and --trials")
    ap.add_argument("--workers", type=int, default=200, help="workers N of a c3:<law> or b1 workload")
    ap.add_argument("--trials", type=int, default=0, help="override the number of trials (profiling small cases)")
    ap.add_argument("--rule", type=int, default=0, choices=(0, 1),
                    help="completion rule: 0 = Algorithm 2 (finish before tau, the benchmark), 1 = start before tau")
    ap.add_argument("--worker-scales", action="store_true",
                    help="time dc_simulate_scaled (workers with thresholds s_n tau_k of their own) instead of dc_simulate_ex; "
                         "the end-to-end and CPU legs are skipped")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--other-trials", type=int, default=0, help="cap the trials of those extra workloads (for tests)")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="skip the extra per-workload sweep timings that the default run adds to its JSON line")
    ap.add_argument("--shape-grid", type=float, nargs="+", default=None, metavar="BYTES",
                    help="instead of the benchmark: print a table of sweep GB/s over worker and micro-batch counts at "
                         "these numbers of latency bytes (e.g. 4e8 3e9), one GPU")
    args = ap.parse_args()
    if args.shape_grid:
        return shape_grid(args)
    if args.workload.startswith("c3:"):
        w = W.c3_workload(args.workload[3:], N=args.workers, T=args.trials or 16384)
        args.trials = w.T
    elif args.workload == "b1":
        w = W.b1_workload(N=args.workers, T=args.trials or 16384)
        args.trials = w.T
    else:
        if args.workload not in W.WORKLOADS:
            ap.error(f"unknown workload {args.workload!r}")
        w = W.WORKLOADS[args.workload]
        if args.trials:
            w = w.with_trials(args.trials)
    if args.impl == "reference":
        return run_reference(args, w)
    return run_ours(args, w)


if __name__ == "__main__":
    sys.exit(main())
