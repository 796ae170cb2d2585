#!/usr/bin/env python
"""Benchmark of the Solon encode + robust-decode path on synthetic gradients.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload vgg13] [--impl ours|reference]

One step = encode all P partition gradients, let the Byzantine nodes overwrite their coded rows, decode
(projections, locator, recovery + sum).  Prints ONE JSON line (rank 0).  With N > 1 (under torchrun) every
rank runs its own independent problem on its own GPU: the path has no collective, scaling is weak.
"""

from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2110_01595_b200 import dist_util, synth

METRIC = "encode+decode gradient GB/s"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0


# ----------------------------------------------------------------------------- helpers


def algorithmic_bytes(wl, n_rec_rows: int, eb: int = 4):
    """Bytes each kernel must move (eb bytes per element: 4 or 8): encode eb P d + eb P d_c; projections eb P d_c + 4 K d_c
    (the vectors f are float32); recovery eb n_rows d_c + eb d with n_rows the trusted rows the locator selected."""
    d_c = wl.d_c
    enc = eb * wl.P * wl.d + eb * wl.P * d_c
    proj = eb * wl.P * d_c + 4 * 2 * d_c
    rec = eb * n_rec_rows * d_c + eb * wl.d
    return enc, proj, rec


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines: list[str] = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_step_seconds(wl, G_host: np.ndarray, nodes, byz_rows_host, f_host: np.ndarray):
    """One pass of the float64 oracle (encode, attack, decode) over the given gradient slice; returns seconds."""
    from oracle import solon_oracle as so

    sizes = so.group_sizes(wl.P, wl.r)
    w = so.node_scalars(sizes)
    t0 = time.perf_counter()
    Z = so.encode(G_host, wl.m, sizes, w).astype(np.float32)
    if len(nodes):
        Z[nodes] = byz_rows_host
    u, mask, status = so.decode(Z, G_host.shape[1], wl.m, wl.s, sizes, w, f_host, tau=1e-5)
    dt = time.perf_counter() - t0
    if status != 0 or mask.nonzero()[0].tolist() != sorted(nodes):
        raise RuntimeError("oracle failed to decode its sample")
    return dt


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info

        counts = [info.get("num_threads", 1) for info in threadpool_info()]
        return max(counts) if counts else 1
    except Exception:
        return os.cpu_count() or 1


def oracle_sample(wl, d_sample: int, device):
    """A bounded sample of the workload for the CPU oracle: its first d_sample coordinates."""
    import dataclasses

    d_sample = min(d_sample, wl.d)
    d_sample -= d_sample % wl.m
    small = dataclasses.replace(wl, d=d_sample)
    G = synth.make_grads(small, device)
    G_host = G.cpu().numpy()
    nodes = synth.byzantine_nodes(small)
    from oracle import solon_oracle as so

    sizes = so.group_sizes(wl.P, wl.r)
    Z = torch.from_numpy(so.encode(G_host, wl.m, sizes, so.node_scalars(sizes)).astype(np.float32))
    rows = synth.byzantine_rows(small, Z, nodes).numpy()
    rng = np.random.default_rng(wl.seed)
    f = (1.0 + rng.normal(size=(2, small.d_c))).astype(np.float32)
    return small, G_host, nodes, rows, f


# ----------------------------------------------------------------------------- arms


def config_of(wl, whole_d, n_byz, sharded, eb=4):
    """The workload description both arms print (identical keys and values, so the two lines can be compared)."""
    return {"workload": wl.name, "P": wl.P, "s": wl.s, "m": wl.m, "r": wl.r, "d": whole_d, "n_byz": n_byz,
            "attack": wl.attack, "element_bytes": eb,
            "arithmetic": ("float64 elements at the boundary, float64 throughout" if eb == 8 else
                           "encode and recovery in f32 for m <= 6 (f64 above), projections and locator in f64"),
            "l2": "inputs (%.2f GB of gradients per step) are larger than L2" % (wl.P * whole_d * eb / 1e9),
            "parallelism": ("one problem, coordinates sharded over the GPUs, one all-reduce of (K+1) x P float64 per decode"
                            if sharded else "independent problems per GPU, no collective")}


def host_memory_allows(wl, d_sample: int) -> bool:
    """The oracle holds the float32 sample plus float64 copies of a group of gradients and of the coded matrix."""
    try:
        import psutil

        need = wl.P * d_sample * 4 * 3.5 + 4e9
        return psutil.virtual_memory().available >= need
    except Exception:
        return d_sample <= 4_000_000


def oracle_speed_probe(wl) -> float:
    """Gradient bytes per second of the oracle on a small sample (1 M coordinates), to size the timed samples."""
    small, G_host, nodes, rows, f = oracle_sample(wl, 1_000_000, "cpu")
    dt = oracle_step_seconds(small, G_host, nodes, rows, f)
    return small.P * small.d * 4 / dt


def run_reference(args, wl):
    """The oracle as it stands, timed on the host cores.  Every step is one pass of the oracle (encode, attack,
    decode) over a sample of the workload: the whole of it when steps + warm-up passes over the whole fit in about
    three minutes, else its first coordinates, as many as do."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    warm = min(args.warmup, 1)
    if args.oracle_d is None:
        budget_s = 170.0 / (args.steps + warm)
        d_fit = int(oracle_speed_probe(wl) * budget_s / (wl.P * 4))
        args.oracle_d = max(wl.m * 1000, min(wl.d, d_fit))
    while not host_memory_allows(wl, args.oracle_d) and args.oracle_d > 1_000_000:
        args.oracle_d //= 2
    small, G_host, nodes, rows, f = oracle_sample(wl, args.oracle_d, "cpu")
    for _ in range(warm):
        oracle_step_seconds(small, G_host, nodes, rows, f)
    times = [oracle_step_seconds(small, G_host, nodes, rows, f) for _ in range(args.steps)]
    total = float(sum(times))
    eb = 8 if args.dtype == "f64" else 4
    value = small.P * small.d * eb * args.steps / total / 1e9
    cores = blas_threads()
    whole = "the whole workload" if small.d >= wl.d - wl.m else f"first {small.d} of {wl.d} coordinates of every partition gradient"
    sample = f"{whole}, all {wl.P} nodes, per step (sized so that {args.steps} steps take about three minutes at most)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True,
        "scaling": "strong" if args.sharded else "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(wl, wl.d, len(nodes), args.sharded, 8 if args.dtype == "f64" else 4),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample, "sample_d": small.d},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_ours(args, wl):
    from paper_2110_01595_b200 import binding, build

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist_util.init("nccl", device_id=local_rank)
    build.build()

    import dataclasses

    sp = None
    if args.sharded:
        # one problem for all ranks: rank i holds the coordinates [lo_i, hi_i) of every gradient; the decode's
        # single exchange is an all-reduce of (K + 1) x P float64 values between the projection and the locator
        from paper_2110_01595_b200 import sharded

        sp = sharded.ShardedPlan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=wl.seed, rank=rank, world=world)
        G_all = synth.make_grads(wl, "cuda")
        G = G_all[:, sp.lo:sp.hi].contiguous()
        del G_all
        whole, wl_rank = wl, wl
        wl = dataclasses.replace(wl, d=sp.d_local)               # this rank's share, for the byte counts below
        plan = sp.plan
    else:
        whole = wl
        wl_rank = dataclasses.replace(wl, seed=wl.seed + 17 * rank)      # every rank its own problem
        G = synth.make_grads(wl_rank, "cuda")
        if args.dtype == "f64":
            G = G.double()
        plan = binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=wl_rank.seed, dtype=args.dtype)
    if args.optimistic is not None and sp is None:
        plan.set_optimistic(args.optimistic)
    coded = plan.encode(G)
    nodes = synth.byzantine_nodes(wl_rank)
    byz_rows = synth.byzantine_rows(wl_rank, coded, nodes)
    nodes_dev = torch.tensor(nodes, dtype=torch.int32, device="cuda")
    eb = 8 if args.dtype == "f64" else 4
    agg = torch.empty(wl.d, dtype=G.dtype, device="cuda")
    mask = torch.empty(wl.P, dtype=torch.uint8, device="cuda")

    def step(events=None):
        # events: two (around the encode call: the roofline's kernel) or four (around the decode call as well)
        n_ev = 0 if events is None else len(events)
        if n_ev:
            events[0].record()
        plan.encode(G, coded)
        if n_ev:
            events[1].record()
        plan.overwrite_rows(coded, nodes_dev, byz_rows)       # the adversary: one device-to-device row copy
        if n_ev == 4:
            events[2].record()
        if sp is not None:
            sp.decode(coded, agg, mask)
        else:
            plan.decode(coded, agg, mask)
        if n_ev == 4:
            events[3].record()

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    status = plan.decode_status()
    if status != 0 or mask.nonzero().flatten().tolist() != nodes:
        raise RuntimeError(f"warm-up decode failed: status {status}")
    n_rec, _, _, _ = plan.recovery()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    # The timed region is EXACTLY args.steps steps; it is repeated until at least a second of GPU time has passed, so that
    # the clocks are those of sustained work (the power cap needs a few hundred milliseconds to act).  The value reported is
    # the median region; the fastest and slowest are given beside it.
    launches0 = plan.kernel_launches()
    regions, enc_all = [], []
    total_ms = 0.0
    while True:
        # (events around the encode call only: every event recorded between two kernels costs the step about 3 us)
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
        dist_util.barrier()
        torch.cuda.synchronize()
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        for i in range(args.steps):
            step(evs[i])
        stop.record()
        torch.cuda.synchronize()
        dist_util.barrier()
        region_ms, _ = dist_util.combine(start.elapsed_time(stop), 0.0)        # max over ranks: all ranks take the same decision
        regions.append(region_ms)
        enc_all.append(float(np.mean([e[0].elapsed_time(e[1]) for e in evs])))
        total_ms += region_ms
        if total_ms >= args.min_timed_ms or len(regions) >= 2000:
            break
    launches = (plan.kernel_launches() - launches0) // len(regions)
    # the decode call's own time: a pass of its own after the timed region, same steps, events around both calls
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(min(args.steps, 100))]
    for ev in evs:
        step(ev)
    torch.cuda.synchronize()
    dec_pass_ms = float(np.mean([e[2].elapsed_time(e[3]) for e in evs]))
    clocks = sampler.stop() if rank == 0 else None
    status = plan.decode_status()
    if status != 0 or mask.nonzero().flatten().tolist() != nodes:
        raise RuntimeError(f"timed decode failed: status {status}")
    # optimistic decode: when the recovery kernel had nothing to do (asked after the last timed decode: a steady state
    # reached during the warm-up holds from then on), the decode read the received matrix once
    skipped = bool(plan.optimistic_outcome()) if sp is None else False
    enc_b, proj_b, rec_b = algorithmic_bytes(wl, 0 if skipped else int(n_rec.sum()), eb)
    rec_two_pass_b = algorithmic_bytes(wl, int(n_rec.sum()), eb)[2]      # what Algorithm 1 as written (locate, then recover) moves

    # the same decode with projection vectors drawn anew for every decode (solon_plan_set_fresh_projections; Algorithm 1
    # draws its random vector inside the decoder) instead of reused
    dec_fresh_ms = None
    if sp is None:
        plan.set_fresh_projections(True)
        for _ in range(3):
            step()
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(min(args.steps, 50))]
        for ev in evs:
            step(ev)
        torch.cuda.synchronize()
        dec_fresh_ms = float(np.mean([e[2].elapsed_time(e[3]) for e in evs]))
        plan.set_fresh_projections(False)

    order = int(np.argsort(regions)[len(regions) // 2])                         # the median region
    max_ms = float(regions[order])
    enc_ms, dec_ms = enc_all[order], dec_pass_ms
    _, total_units = dist_util.combine(0.0, wl.P * wl.d * eb * args.steps)          # gradient bytes all ranks processed per region
    repeats = {"n": len(regions), "timed_ms_total": total_ms, "ms_per_step_median": max_ms / args.steps,
               "ms_per_step_min": min(regions) / args.steps, "ms_per_step_max": max(regions) / args.steps,
               "ms_per_step_first": regions[0] / args.steps}

    # end to end through the host-buffer entry point: pinned host memory in, host results out
    e2e = None
    if not args.no_e2e and sp is None:
        G_host = torch.empty((wl.P, wl.d), dtype=G.dtype).pin_memory()
        G_host.copy_(G)
        rows_host = byz_rows.cpu().pin_memory() if nodes else torch.empty((0, wl.d_c))
        agg_host = torch.empty(wl.d, dtype=G.dtype).pin_memory()
        mask_host = torch.empty(wl.P, dtype=torch.uint8).pin_memory()
        plan.step_host(G_host, nodes, rows_host, agg_host, mask_host)             # allocates staging, warms up
        dist_util.barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            st = plan.step_host(G_host, nodes, rows_host, agg_host, mask_host)
        torch.cuda.synchronize()
        e2e_ms = (time.perf_counter() - t0) * 1e3
        if st != 0 or mask_host.nonzero().flatten().tolist() != nodes:
            raise RuntimeError("host-buffer step failed")
        e2e_max_ms, e2e_units = dist_util.combine(e2e_ms, wl.P * wl.d * eb * args.e2e_steps)
        e2e = {"value": e2e_units / (e2e_max_ms * 1e-3) / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": wl.P * wl.d * eb + len(nodes) * wl.d_c * eb, "d2h_bytes_per_step": wl.d * eb + wl.P,
               "steps": args.e2e_steps}
        del G_host, agg_host

    if rank != 0:
        dist_util.shutdown()
        return

    peak, peak_kind = measured_peak()
    enc_gbs = enc_b / (enc_ms * 1e-3) / 1e9
    total_b = enc_b + proj_b + rec_b
    path_gbs = total_b / ((enc_ms + dec_ms) * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": total_units / (max_ms * 1e-3) / 1e9, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": max_ms / args.steps, "higher_is_better": True,
        "scaling": "strong" if sp is not None else "weak",
        "vs_baseline": None, "dtype": "f64" if (args.dtype == "f64" or wl.m > 6) else "f32", "data": "synthetic",
        "config": config_of(whole, whole.d, len(nodes), sp is not None, eb),
        "repeats": repeats,
        "roofline": {"bound": "hbm", "kernel": "encode_direct_kernel", "achieved": enc_gbs, "peak": peak, "unit": "GB/s",
                     "frac": enc_gbs / peak, "peak_kind": f"of {peak_kind}", "traffic": encode_traffic(wl) if (sp is None and eb == 4) else None,
                     "algorithmic_bytes": enc_b, "ms": enc_ms},
        "path": {"encode_ms": enc_ms, "decode_ms": dec_ms, "decode_ms_fresh_f": dec_fresh_ms, "recovery_skipped": skipped,
                 "decodes_per_s": 1e3 / dec_ms,
                 "algorithmic_bytes": total_b,
                 "hbm_gbs": path_gbs, "frac_of_peak": path_gbs / peak, "frac_of_8TBs": path_gbs / 8000.0,
                 # the same time against the bytes of the method as written (projection pass, then recovery pass over the
                 # trusted rows): equal to the figures above unless the recovery was done inside the projection pass
                 "two_pass_bytes": enc_b + proj_b + rec_two_pass_b,
                 "frac_of_8TBs_on_two_pass_bytes": (enc_b + proj_b + rec_two_pass_b) / ((enc_ms + dec_ms) * 1e-3) / 1e9 / 8000.0},
        "clocks": clocks,
        "e2e": e2e,
        "gpu_launches": int(launches),
    }
    if not args.no_cpu_baseline and world == 1 and sp is None:
        d_oracle = args.oracle_d if args.oracle_d is not None else wl.d          # the whole workload: one pass, 10-30 s
        note = ""
        while not host_memory_allows(wl, d_oracle) and d_oracle > 1_000_000:
            d_oracle //= 2
            note = " (the host's free memory does not hold the whole workload)"
        small, G_s, nodes_s, rows_s, f_s = oracle_sample(wl, d_oracle, "cpu")
        dt = oracle_step_seconds(small, G_s, nodes_s, rows_s, f_s)
        whole_txt = "the whole workload" if small.d >= wl.d - wl.m else f"first {small.d} of {wl.d} coordinates of every partition gradient"
        line["cpu_baseline"] = {"value": small.P * small.d * eb / dt / 1e9, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                                "sample": f"{whole_txt}, all {wl.P} nodes, one step ({dt:.1f} s){note}", "sample_d": small.d}
    print(json.dumps(line), flush=True)
    dist_util.shutdown()


def run_lsq(args, wl):
    """solon_lsq_grads alone on the least-squares configuration (a parity case, not the benchmark step): CUDA events around
    every call, L2 flushed between calls (the 1.54 GB matrix is larger than L2 anyway), algorithmic bytes = two passes
    over X.  Prints one JSON line of its own."""
    from paper_2110_01595_b200 import binding, build

    torch.cuda.set_device(0)
    build.build()
    X, y, w = synth.make_lsq_problem(wl, "cuda")
    w = torch.randn(wl.d, device="cuda", generator=torch.Generator(device="cuda").manual_seed(wl.seed + 3))
    flush = torch.empty(160 * 1024 * 1024 // 4, dtype=torch.float32, device="cuda")
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=wl.seed) as plan:
        G = plan.lsq_grads(X, y, w, rows=wl.lsq_rows)
        for _ in range(max(args.warmup, 3)):
            plan.lsq_grads(X, y, w, G, rows=wl.lsq_rows)
        times = []
        for _ in range(args.steps):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            plan.lsq_grads(X, y, w, G, rows=wl.lsq_rows)
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        # a property that holds at any size: against a float64 device-side evaluation of X_i^T (X_i w - y_i)
        rows = wl.lsq_rows
        ref = torch.stack([X[i * rows:(i + 1) * rows].double().T @ (X[i * rows:(i + 1) * rows].double() @ w.double() - y[i * rows:(i + 1) * rows].double())
                           for i in range(wl.P)])
        err = float((G.double() - ref).abs().max() / ref.abs().max())
    peak, peak_kind = measured_peak()
    ms = float(np.median(times))
    algo = 2 * 4 * wl.P * wl.lsq_rows * wl.d
    print(json.dumps({"workload": wl.name, "kernel": "solon_lsq_grads", "steps": args.steps, "ms_median": ms, "ms_min": float(min(times)),
                      "algorithmic_bytes": algo, "hbm_gbs": algo / (ms * 1e-3) / 1e9, "frac_of_peak": algo / (ms * 1e-3) / 1e9 / peak,
                      "peak_kind": f"of {peak_kind}", "max_rel_err_vs_float64": err, "l2": "flushed between calls"}), flush=True)


def run_sweep(args):
    """The grid P in {15,45,105} x s in {1,3,5} x m in {1,2,5,10} x d: s random nodes send N(0,100^2).

    Every point is checked (mask equal to the attacked set; aggregate against a float64 device-side sum of the
    partition gradients, the definition of the result) and timed with CUDA events; GB/s figures use each
    kernel's algorithmic bytes.  One JSON line per point goes to the file; one summary line is printed.
    """
    from paper_2110_01595_b200 import binding, build

    torch.cuda.set_device(0)
    build.build()
    peak, peak_kind = measured_peak()
    ds = tuple(int(x) for x in args.sweep_d.split(","))
    points = synth.sweep_points(ds)
    worst_err, failures, rows = 0.0, 0, []
    with open(args.sweep, "a") as out:
        for wl in points:
            G = synth.make_grads(wl, "cuda")
            plan = binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=wl.seed)
            coded = plan.encode(G)
            nodes = synth.byzantine_nodes(wl)
            byz_rows = synth.byzantine_rows(wl, coded, nodes)
            nodes_dev = torch.tensor(nodes, dtype=torch.int32, device="cuda")
            agg = torch.empty(wl.d, dtype=torch.float32, device="cuda")
            mask = torch.empty(wl.P, dtype=torch.uint8, device="cuda")

            def step(ev=None):
                if ev:
                    ev[0].record()
                plan.encode(G, coded)
                if ev:
                    ev[1].record()
                plan.overwrite_rows(coded, nodes_dev, byz_rows)
                if ev:
                    ev[2].record()
                plan.decode(coded, agg, mask)
                if ev:
                    ev[3].record()

            for _ in range(4):      # the single-pass decode, where a plan has one, is the steady state from the fourth decode on
                step()
            torch.cuda.synchronize()
            n_steps = max(3, min(args.steps, 10))
            evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(n_steps)]
            for ev in evs:
                step(ev)
            torch.cuda.synchronize()
            status = plan.decode_status()
            enc_ms = float(np.median([e[0].elapsed_time(e[1]) for e in evs]))
            dec_ms = float(np.median([e[2].elapsed_time(e[3]) for e in evs]))
            n_rec = int(plan.recovery()[0].sum())
            # optimistic decode: when the recovery kernel had nothing to do, the decode read the received matrix once
            skipped = bool(plan.optimistic_outcome())
            enc_b, proj_b, rec_b = algorithmic_bytes(wl, 0 if skipped else n_rec)
            two_pass_b = enc_b + proj_b + algorithmic_bytes(wl, n_rec)[2]      # the bytes of locate-then-recover as written
            ref = G.sum(dim=0, dtype=torch.float64)
            scale = float(ref.abs().max())
            err = float((agg.double() - ref).abs().max()) / scale
            mask_ok = mask.nonzero().flatten().tolist() == nodes
            ok = bool(status == 0 and mask_ok and err <= 1e-4)
            failures += 0 if ok else 1
            worst_err = max(worst_err, err)
            total_b = enc_b + proj_b + rec_b
            row = {"workload": wl.name, "P": wl.P, "s": wl.s, "m": wl.m, "r": wl.r, "d": wl.d, "q": plan.q, "ok": ok,
                   "status": status, "mask_exact": mask_ok, "agg_err": err, "encode_ms": enc_ms, "decode_ms": dec_ms,
                   "gradient_gbs": wl.P * wl.d * 4 / ((enc_ms + dec_ms) * 1e-3) / 1e9,
                   "hbm_gbs": total_b / ((enc_ms + dec_ms) * 1e-3) / 1e9,
                   "frac_of_peak": total_b / ((enc_ms + dec_ms) * 1e-3) / 1e9 / peak,
                   "frac_of_8TBs": total_b / ((enc_ms + dec_ms) * 1e-3) / 1e9 / 8000.0,
                   "encode_gbs": enc_b / (enc_ms * 1e-3) / 1e9, "decodes_per_s": 1e3 / dec_ms, "recovery_skipped": skipped,
                   "frac_of_8TBs_on_two_pass_bytes": two_pass_b / ((enc_ms + dec_ms) * 1e-3) / 1e9 / 8000.0}
            out.write(json.dumps(row) + "\n")
            out.flush()
            rows.append(row)
            plan.close()
            del G, coded, byz_rows, agg, mask, ref, plan
            torch.cuda.empty_cache()
    big = [r for r in rows if r["d"] >= 10_000_000]
    summary = {"sweep_points": len(rows), "failures": failures, "worst_agg_err": worst_err, "peak_gbs": peak,
               "peak_kind": peak_kind,
               "median_frac_of_peak_d_ge_10M": float(np.median([r["frac_of_peak"] for r in big])) if big else None,
               "min_frac_of_8TBs_d_ge_10M": min((r["frac_of_8TBs"] for r in big), default=None),
               "max_frac_of_8TBs_d_ge_10M": max((r["frac_of_8TBs"] for r in big), default=None),
               "median_frac_of_8TBs_on_two_pass_bytes_d_ge_10M":
                   float(np.median([r["frac_of_8TBs_on_two_pass_bytes"] for r in big])) if big else None,
               "points_below_0.70_on_two_pass_bytes_d_ge_10M": sum(1 for r in big if r["frac_of_8TBs_on_two_pass_bytes"] < 0.70)}
    print(json.dumps(summary), flush=True)


def encode_traffic(wl):
    """DRAM bytes (read + write) of one encode launch on this workload, from the ncu capture recorded in
    profiles/encode_kernel_traffic.json: the capture's bytes scaled by the units processed (P * d; the kernel makes one
    pass, so traffic grows in proportion).  None when no capture of the kernel as it stands is on record."""
    try:
        with open(os.path.join(ROOT, "profiles", "encode_kernel_traffic.json")) as fh:
            rec = json.load(fh)
        if not rec.get("valid_for_current_kernel", False) or rec.get("m") != wl.m:
            return None
        return float(rec["dram_bytes_read"] + rec["dram_bytes_write"]) * (wl.P * wl.d) / (rec["P"] * rec["d"])
    except Exception:
        return None


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="vgg13")
    ap.add_argument("--dtype", default="f32", choices=["f32", "f64"],
                    help="element type of gradients, coded vectors and aggregate (f64: the paper's 8-byte wire format)")
    ap.add_argument("--optimistic", type=int, default=None, choices=[0, 1, 2],
                    help="solon_plan_set_optimistic mode (default: the library's, 1)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sharded", action="store_true",
                    help="with --gpus N: ONE problem whose coordinates are spread over the N GPUs (strong scaling; the "
                         "decode's only exchange is a small all-reduce) instead of N independent problems; no e2e leg")
    ap.add_argument("--sweep", default=None, metavar="FILE",
                    help="run the (P, s, m, d) grid instead: one JSON line per point is appended to FILE, a summary is printed")
    ap.add_argument("--sweep-d", default="1000000,10000000,50000000", help="gradient lengths of the grid")
    ap.add_argument("--oracle-d", type=int, default=None,
                    help="coordinates per gradient in the oracle's sample (default: the whole workload for the cpu_baseline "
                         "leg; for --impl reference as many as let steps + warm-up passes finish in about three minutes)")
    ap.add_argument("--min-timed-ms", type=float, default=1000.0,
                    help="the timed region of --steps steps is repeated until this much GPU time has passed")
    args = ap.parse_args()
    if args.workload in synth.WORKLOADS:
        wl = synth.WORKLOADS[args.workload]
    else:
        match = [p for p in synth.sweep_points() if p.name == args.workload]
        if not match:
            raise SystemExit(f"unknown workload {args.workload}")
        wl = match[0]
    if wl.grads == "lsq":
        if args.steps == 200:
            args.steps = 20
        run_lsq(args, wl)
        return
    if args.sweep:
        run_sweep(args)
        return
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
