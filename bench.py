#!/usr/bin/env python
"""Benchmark of the HBF service-model hot path on B200.

One step = one pass of the whole hot path over one batch: ``hbf_submit_batch`` (classify, decode,
queue order, max-plus scan, scatter, per-die stats) followed by ``hbf_thermal_step`` (power map, RC
stencil, throttle controller).  The workload is the capacity-mode stream (200 M accesses in one batch,
64 channels x 8 dies x 4 planes); with N > 1 every rank runs an independent replica on its own stream
(replicas only: the path needs no exchange at one GPU per model instance).

Prints ONE JSON line.  ``--impl reference`` times the CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import datetime
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2609_09800_b200 import workloads as wl  # noqa: E402

METRIC = "simulated HBF accesses/s"
UNIT = "accesses/s"
ALGO_BYTES_PER_ACCESS = 41            # 24 B record in, 8 B completion + 8 B stall + 1 B status out
# algorithmic bytes per access of each kernel group (what the kernel itself must move)
STAGE_BYTES = {"classify": 24 + 8 + 1, "plan_hist": 8, "scan": 8 + 4 + 24 + 16, "inorder": 24 + 16 + 1}
# Profiler counters of the dominant kernel (DRAM bytes and warp instructions per access) are not typed in here: they come
# from a small tracked file that names the kernel source it was captured on; when that source has changed since, the
# bench reports no traffic and no instruction roofline rather than stale ones.
COUNTERS_FILE = os.path.join(ROOT, "profiles", "inorder_serve_capacity_200M.json")
KERNEL_SOURCES = {"inorder": os.path.join(ROOT, "paper_2609_09800_b200", "csrc", "inorder_kernels.cu")}


def profiled_counters(kernel: str):
    """{'dram_bytes_per_access', 'warp_instr_per_access', ...} of an ncu capture of this kernel's present source, or None."""
    import hashlib
    try:
        with open(COUNTERS_FILE) as f:
            rec = json.load(f)
        with open(KERNEL_SOURCES[kernel], "rb") as f:
            sha = hashlib.sha256(f.read()).hexdigest()
    except Exception:
        return None
    return rec if rec.get("kernel") == kernel and rec.get("source_sha256") == sha else None


SM_COUNT, SCHEDULERS_PER_SM = 148, 4
FALLBACK_HBM_GBS = 6650.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--n", type=int, default=200_000_000, help="accesses per batch (default: the capacity-mode config)")
    ap.add_argument("--path", default="auto", choices=["auto", "sort", "sort_full"])
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--e2e-chunk", type=int, default=4_000_000, help="records per chunk of the end-to-end pipeline")
    ap.add_argument("--cpu-sample", type=int, default=20_000_000)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the per-configuration block (other streams, coupled run)")
    ap.add_argument("--shuffle", action="store_true", help="submit the records in a random order: the sort path has to serve the batch")
    ap.add_argument("--profile", default="nominal", choices=["nominal", "aggressive"], help="timing profile of the coupled_thermal run")
    ap.add_argument("--workload", default="capacity_mode", choices=["capacity_mode", "coupled_thermal", "capacity_paged", "rom", "capacity_retention"],
                    help="coupled_thermal: the prefix-KV stream in 1 ms batches, each followed by a thermal step; "
                         "capacity_paged: the capacity-mode batch through the page-granular submit; rom: fit the reduced-order "
                         "thermal model of the package floorplan and time its step against the full grid; capacity_retention: the "
                         "capacity-mode batch with retention on: a batch without debt, an epoch (damage, eligibility, plan), the "
                         "same batch paying refresh claims (none is the headline)")
    ap.add_argument("--horizon-ms", type=int, default=1000, help="simulated time of the coupled_thermal run")
    ap.add_argument("--channel-bus", action="store_true",
                    help="capacity_mode: also run the channel-bus stage (reads' transfers queue per channel); not the headline")
    ap.add_argument("--retention", action="store_true",
                    help="coupled_thermal: retention on, one epoch per thermal step with the temperatures of the field "
                         "(reliability time accelerated 2e6 times so that blocks come due within the simulated second)")
    ap.add_argument("--energy-bins", action="store_true",
                    help="coupled_thermal: book event energies into 1 ms bins (time-bin power integration) instead of at submit")
    return ap.parse_args()


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            with open(p) as f:
                return float(json.load(f)["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons, sampled every 20 ms.  The sampler is started early (it needs a few
    hundred ms to come up); only samples taken between mark_start() and mark_end() are reported."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.proc, self.t0, self.t1 = gpu_index, None, None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def mark_start(self):
        self.t0 = datetime.datetime.now()

    def mark_end(self):
        self.t1 = datetime.datetime.now()

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill(); out = ""
        sm, smax, reasons, all_sm = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f")
                mhz, mx = float(f[1]), float(f[2])
            except ValueError:
                continue
            all_sm.append(mhz)
            if self.t0 is not None and self.t1 is not None and not (self.t0 <= ts <= self.t1):
                continue
            sm.append(mhz); smax.append(mx)
            for name, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "samples_whole_run": len(all_sm), "reasons": sorted(reasons)}


# The batch spans seconds of simulated time while the thermal window that follows it is 1 ms, so the
# window's power is far above anything physical.  The kernels' work does not depend on the values; the
# four thresholds are raised so that the controller stays in Normal mode and every step does full work.
BENCH_THRESHOLDS = dict(rtt_c=1e6, ltt_c=2e6, stt_c=3e6, shutdown_c=4e6)


def make_stream(n: int, seed: int):
    t = time.time()
    w = wl.capacity_mode(n=n, seed=seed)
    w.profile.update(BENCH_THRESHOLDS)
    return w, time.time() - t


def cpu_oracle_rate(w, sample: int, repeats: int = 1):
    """The oracle as it stands, on one host core, on the first ``sample`` accesses of the stream."""
    from oracle import hbfo
    acc = w.acc[:sample]
    o = hbfo.Oracle(w.profile, wl.package_floorplan(channels=w.profile["channels"], dies=w.profile["dies"]))
    for r in w.ranges:
        o.register_range(*r)
    times = []
    for _ in range(repeats):
        o.reset()
        t = time.perf_counter()
        o.submit(acc)
        o.thermal_step(1_000_000, None)
        times.append(time.perf_counter() - t)
    return acc.shape[0] / min(times), times


def cpu_oracle_rate_all_cores(w, sample: int):
    """The same oracle on all host cores: queues are independent, so the sample is dealt to one oracle instance per core
    by channel (a channel's queues stay together) and the instances run side by side (plain threads around the C call).
    Returns (accesses/s, cores, seconds, sum of stalls) -- the sum lets the caller check the dealing against the one-core run."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import hbfo
    cores = max(1, len(os.sched_getaffinity(0)))
    acc = w.acc[:sample]
    stripe = int(w.profile["stripe_bytes"]).bit_length() - 1
    channel = ((acc["addr"] - np.uint64(w.ranges[0][0])) >> np.uint64(stripe)) % np.uint64(w.profile["channels"])
    groups = min(cores, int(w.profile["channels"]))
    subs = [np.ascontiguousarray(acc[(channel % np.uint64(groups)) == np.uint64(g)]) for g in range(groups)]
    oracles = []
    for _ in range(groups):
        o = hbfo.Oracle(w.profile)
        for r in w.ranges:
            o.register_range(*r)
        oracles.append(o)
    with ThreadPoolExecutor(groups) as pool:
        t = time.perf_counter()
        outs = list(pool.map(lambda g: oracles[g].submit(subs[g]), range(groups)))
        dt = time.perf_counter() - t
    return acc.shape[0] / dt, groups, dt, int(sum(int(o[2].sum()) for o in outs))


def host_memory_bytes() -> int:
    try:
        return os.sysconf("SC_PAGE_SIZE") * os.sysconf("SC_PHYS_PAGES")
    except (ValueError, OSError):
        return 0


def run_reference(args, rank: int):
    """The CPU oracle, as it stands, on this machine's host cores, on the same step as the library's arm: the whole batch
    (queues idle at the start of every step) and one thermal step.  Queues are independent, so the batch is dealt by channel
    to one oracle instance per core and the instances run side by side (plain threads around the C call); the first of
    them also carries the package grid and takes the thermal step.  On a host too small to hold the batch and the oracle's
    per-access arrays (about 100 bytes per access) a step is the first 20 M accesses of the stream, and `sample` says so."""
    if rank != 0:
        return
    from concurrent.futures import ThreadPoolExecutor
    from oracle import hbfo
    n = args.n
    if host_memory_bytes() < 140 * n:
        n = min(n, 20_000_000)
    w, gen_s = make_stream(n, 0)
    cores = max(1, len(os.sched_getaffinity(0)))
    stripe = int(w.profile["stripe_bytes"]).bit_length() - 1
    channel = ((w.acc["addr"] - np.uint64(w.ranges[0][0])) >> np.uint64(stripe)) % np.uint64(w.profile["channels"])
    groups = min(cores, int(w.profile["channels"]))
    subs = [np.ascontiguousarray(w.acc[(channel % np.uint64(groups)) == np.uint64(g)]) for g in range(groups)]
    del channel
    fp = wl.package_floorplan(channels=w.profile["channels"], dies=w.profile["dies"])
    oracles = []
    for g in range(groups):
        o = hbfo.Oracle(w.profile, fp if g == 0 else None)
        for r in w.ranges:
            o.register_range(*r)
        oracles.append(o)

    def step(pool):
        for o in oracles:
            o.reset()
        t = time.perf_counter()
        list(pool.map(lambda g: oracles[g].submit(subs[g])[0], range(groups)))
        oracles[0].thermal_step(1_000_000, fp["ext_power_w"])
        return time.perf_counter() - t

    with ThreadPoolExecutor(groups) as pool:
        for _ in range(args.warmup):
            step(pool)
        dt = sum(step(pool) for _ in range(args.steps))
    value = args.steps * n / dt
    sample_txt = ("the whole batch of %d accesses per step" % n if n == args.n else
                  "the first %d accesses of the stream per step (host memory)" % n) + \
                 ", dealt by channel to one oracle instance per core, 1 thermal step per batch"
    config = headline_config(args, n)
    config["l2"] = "host run: the batch (%.1f GB) is larger than every cache" % (n * 24 / 1e9)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int64", "data": "synthetic", "config": config, "gen_seconds": round(gen_s, 1),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": groups, "kind": "oracle", "sample": sample_txt},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def headline_config(args, n: int) -> dict:
    """What the headline step is run on: the same dictionary in the library's line and in the reference arm's."""
    return {"workload": "capacity_mode", "accesses_per_step": n, "geometry": "64x8x4", "queues": 2048,
            "path": args.path, "input_order": "shuffled" if args.shuffle else "issue order",
            "channel_bus_stage": bool(args.channel_bus), "thermal_grid": "128x128",
            "multi_gpu": "replicas only",
            "state": "queues idle at the start of every step (reset outside the timed region)"}


def time_one_batch(hbf, w, path, repeats: int = 3):
    """hbf_submit_batch alone on one stream of records, device-resident, on idle queues: best of `repeats` after a warm-up."""
    import torch
    ctx = hbf.Context(w.profile)
    for r in w.ranges:
        ctx.register_range(*r)
    ctx.set_path(path)
    n = w.n
    d_acc = torch.from_numpy(w.acc.view(np.int64).reshape(-1)).cuda()
    d_comp = torch.empty(n, dtype=torch.int64, device="cuda"); d_stall = torch.empty_like(d_comp)
    d_status = torch.empty(n, dtype=torch.uint8, device="cuda")
    d_stats = torch.empty(ctx.n_dies * 6, dtype=torch.int64, device="cuda")
    ws = ctx.workspace(n)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    best = None
    for k in range(repeats + 1):
        ctx.reset(); flush.fill_(1)
        e0.record(); rc = ctx.submit_batch(d_acc, n, d_comp, d_stall, d_status, d_stats, ws); e1.record(); e1.synchronize()
        assert rc == 0 and ctx.last_result()["code"] == 0
        if k:
            best = e0.elapsed_time(e1) if best is None else min(best, e0.elapsed_time(e1))
    ctx.destroy()
    del d_acc, d_comp, d_stall, d_status, d_stats, ws, flush
    return {"accesses": n, "ms": round(best, 4), "accesses_per_s": n / (best * 1e-3)}


def other_configs(hbf, args):
    """The other configurations of the benchmark definition, one batch each on idle queues (in-order path as the library
    chooses it, and the sort path forced), and the long coupled run per step.  Reported beside the headline."""
    out = {}
    streams = [("tiny_uniform_65k", lambda: wl.tiny_uniform()), ("decode_weights_256_tokens", lambda: wl.decode_weights(256)),
               ("decode_weights_48_tokens", lambda: wl.decode_weights(48)), ("prefix_kv", lambda: wl.prefix_kv())]
    kv = None
    for name, make in streams:
        w = make()
        out[name] = {"auto": time_one_batch(hbf, w, hbf.PATH_AUTO), "sort_forced": time_one_batch(hbf, w, hbf.PATH_SORT)}
        if name == "prefix_kv":
            kv = w
    out["coupled_thermal_10s"] = coupled_run(hbf, kv, 10_000, hbf.PATH_AUTO)
    return out


def coupled_run(hbf, w, n_steps: int, path, energy_bins=False, retention=False):
    """1 ms batches of the prefix-KV stream, device-resident, a thermal step after each: device time per (submit + step)."""
    import torch
    fp = wl.package_floorplan()
    batches = [b for _, b in wl.timed_batches(w, n_steps * 1_000_000)]
    sizes = [b.shape[0] for b in batches]
    allrec = np.concatenate(batches)
    ctx = hbf.Context(w.profile, fp)
    for r in w.ranges:
        ctx.register_range(*r)
    ctx.set_path(path)
    if energy_bins:
        ctx.enable_energy_bins(1_000_000, 64)
    if retention:
        ctx.enable_retention(pages_per_block=64, blocks_per_plane=64, blocks_per_zone=8, max_pec=3000, disturb_limit=0,
                             l_ref_s=3.15e7, t_ref_c=40.0, ea_ev=1.04, accel=2.0e6, lead_threshold=0.8)
    d_all = torch.from_numpy(allrec.view(np.int64).reshape(-1, 3)).cuda()
    nmax = max(sizes)
    d_comp = torch.empty(nmax, dtype=torch.int64, device="cuda"); d_stall = torch.empty_like(d_comp)
    d_stats = torch.empty(ctx.n_dies * 6, dtype=torch.int64, device="cuda")
    ws = ctx.workspace(nmax)
    offs = np.concatenate([[0], np.cumsum(sizes)])
    ext = fp["ext_power_w"]

    def run():
        refused = 0
        for k, nk in enumerate(sizes):
            rc = ctx.submit_batch(d_all[offs[k]:offs[k + 1]], nk, d_comp, d_stall, None, d_stats, ws)
            if rc != 0:                                      # (the controller shut the link down: later batches are refused)
                refused += 1
            ctx.thermal_step(1_000_000, ext, None, want_hot=False)
            if retention:
                ctx.retention_advance(1_000_000)
        return refused
    ctx.reset(); run(); torch.cuda.synchronize()               # warm-up pass over the same horizon
    ctx.reset()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    l0 = hbf.kernel_launches()
    t_host = time.perf_counter()
    e0.record(); refused = run(); e1.record(); torch.cuda.synchronize()
    wall = time.perf_counter() - t_host
    ms = e0.elapsed_time(e1)
    hot = ctx.thermal_step(1_000_000, ext)
    mode, q = ctx.get_mode()
    res = {"steps": len(sizes), "accesses": int(offs[-1]), "us_per_submit_plus_step": ms * 1e3 / len(sizes), "device_ms": ms,
           "host_wall_s": round(wall, 3), "gpu_launches": int(hbf.kernel_launches() - l0), "batches_refused_at_launch": refused,
           "path": "auto" if path == hbf.PATH_AUTO else "inorder (declared by the caller)",
           "final": {"hot_c": [round(float(x), 3) for x in hot], "mode": mode, "q_ppm": q}}
    if retention:
        res["retention"] = ctx.retention_totals()
    ctx.destroy()
    return res


def run_coupled(args):
    """Long-run coupled mode on one GPU: 1 ms batches of the prefix-KV stream, a thermal step after each."""
    from paper_2609_09800_b200 import build as hbf_build, hbf
    hbf_build.build()
    t0 = time.time()
    w = wl.prefix_kv(profile=args.profile)
    gen_s = time.time() - t0
    r = coupled_run(hbf, w, args.horizon_ms, hbf.PATH_INORDER, energy_bins=args.energy_bins, retention=args.retention)
    line = {"metric": METRIC, "value": r["accesses"] / (r["device_ms"] * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": r["steps"],
            "warmup": r["steps"], "ms_per_step": r["device_ms"] / r["steps"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int64", "data": "synthetic",
            "config": {"workload": "coupled_thermal", "profile": args.profile, "accesses": r["accesses"],
                       "mean_accesses_per_step": r["accesses"] / r["steps"],
                       "simulated_ms": args.horizon_ms, "geometry": "32x8x4", "path": r["path"],
                       "thermal_grid": "128x128", "gen_seconds": round(gen_s, 1),
                       "energy": "1 ms bins, split by time overlap" if args.energy_bins else "charged at submit"},
            "gpu_launches": r["gpu_launches"], "host_wall_s": r["host_wall_s"], "final": r["final"]}
    if args.retention:
        line["retention"] = r["retention"]
        line["config"]["retention"] = "one epoch per thermal step, region temperatures from the field, a_t = 2e6"
    print(json.dumps(line), flush=True)


def run_paged(args):
    """The capacity-mode batch through hbf_submit_batch_paged on one GPU: every page of a read queued on its own."""
    import torch
    from paper_2609_09800_b200 import build as hbf_build, hbf
    hbf_build.build()
    n = args.n
    w, gen_s = make_stream(n, seed=0)
    fp = wl.package_floorplan(channels=w.profile["channels"], dies=w.profile["dies"])
    ctx = hbf.Context(w.profile, fp)
    for r in w.ranges:
        ctx.register_range(*r)
    page = w.profile["page_bytes"]
    off = w.acc["addr"] - np.uint64(w.ranges[0][0])
    parts = int(((off % np.uint64(page) + w.acc["bytes"] + np.uint64(page - 1)) // np.uint64(page)).sum())
    d_acc = torch.from_numpy(w.acc.view(np.int64).reshape(-1)).cuda()
    d_comp = torch.empty(n, dtype=torch.int64, device="cuda"); d_stall = torch.empty_like(d_comp)
    d_status = torch.empty(n, dtype=torch.uint8, device="cuda")
    d_stats = torch.empty(ctx.n_dies * 6, dtype=torch.int64, device="cuda")
    ws = torch.empty(ctx.workspace_bytes_paged(n, parts), dtype=torch.uint8, device="cuda")
    ext = fp["ext_power_w"]
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def step():
        rc = ctx.submit_batch_paged(d_acc, n, parts, d_comp, d_stall, d_status, d_stats, ws)
        assert rc == 0, rc
        ctx.thermal_step(1_000_000, ext, None, want_hot=False)

    def timed(k):
        total = 0.0
        for _ in range(k):
            ctx.reset()
            e0.record(stream); step(); e1.record(stream)
            e1.synchronize()
            total += e0.elapsed_time(e1)
        return total
    timed(args.warmup)
    res = ctx.last_result()
    assert res["code"] == 0, res
    l0 = hbf.kernel_launches()
    ms = timed(args.steps)
    launches = hbf.kernel_launches() - l0
    peak, kind = measured_peak()
    rate = n * args.steps / (ms * 1e-3)
    # The method's bytes: 41 per queued request (a part), whatever the implementation moves.  What this implementation moves
    # (records in, part records out and in again, their results out and in, results out) is reported beside it.
    algo = ALGO_BYTES_PER_ACCESS * parts
    moved = 24 * n + 2 * 24 * parts + 2 * 17 * parts + 17 * n
    line = {"metric": METRIC, "value": rate, "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64",
            "data": "synthetic",
            "config": {"workload": "capacity_mode_paged", "accesses_per_step": n, "parts_per_step": parts, "geometry": "64x8x4",
                       "queues": 2048, "thermal_grid": "128x128",
                       "gen_seconds": round(gen_s, 1), "state": "queues idle at the start of every step"},
            "gpu_launches": int(launches),
            "roofline": {"bound": "hbm", "kernel": "paged submit, all kernels", "achieved": algo * args.steps / (ms * 1e-3) / 1e9,
                         "peak": peak, "peak_kind": kind, "unit": "GB/s",
                         "frac": algo * args.steps / (ms * 1e-3) / 1e9 / peak, "traffic": None,
                         "algorithmic_bytes_per_part": ALGO_BYTES_PER_ACCESS,
                         "implementation_bytes_moved_per_step": moved},
            "batch_result": {k: res[k] for k in ("n_modeled", "n_native", "max_completion_ns")}}
    print(json.dumps(line), flush=True)


def run_retention(args):
    """The capacity-mode batch with retention, refresh and wear on (one GPU).  A step: reset; the batch on a device without
    refresh debt (claim window, service, read disturb, commit scan); one epoch at 60 C with a read-disturb limit of one
    page read, so that every block the batch touched becomes eligible and its pages join the plan; the same batch again,
    its first accesses now claiming one refresh quantum each."""
    import torch
    from paper_2609_09800_b200 import build as hbf_build, hbf
    hbf_build.build()
    n = args.n
    w, gen_s = make_stream(n, seed=0)
    fp = wl.package_floorplan(channels=w.profile["channels"], dies=w.profile["dies"])
    ctx = hbf.Context(w.profile, fp)
    for r in w.ranges:
        ctx.register_range(*r)
    ret = dict(pages_per_block=256, blocks_per_plane=64, blocks_per_zone=8, max_pec=3000, disturb_limit=1,
               l_ref_s=3.15e7, t_ref_c=40.0, ea_ev=1.04, accel=1.0, lead_threshold=0.8)
    ctx.enable_retention(**ret)
    temps = np.full(len(fp["region_kind"]), 60.0)
    d_acc = torch.from_numpy(w.acc.view(np.int64).reshape(-1)).cuda()
    d_comp = torch.empty(n, dtype=torch.int64, device="cuda"); d_stall = torch.empty_like(d_comp)
    d_status = torch.empty(n, dtype=torch.uint8, device="cuda")
    d_stats = torch.empty(ctx.n_dies * 6, dtype=torch.int64, device="cuda")
    ws = torch.empty(ctx.workspace_bytes(n), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]

    def submit():
        rc = ctx.submit_batch(d_acc, n, d_comp, d_stall, d_status, d_stats, ws)
        assert rc == 0, rc

    def timed(k):
        t = np.zeros(3)
        for _ in range(k):
            ctx.reset()
            ev[0].record(stream); submit()
            ev[1].record(stream); ctx.retention_advance(1_000_000_000, temps)
            ev[2].record(stream); submit()
            ev[3].record(stream); ev[3].synchronize()
            t += [ev[i].elapsed_time(ev[i + 1]) for i in range(3)]
        return t
    timed(args.warmup)
    res = ctx.last_result()
    assert res["code"] == 0, res
    tot = ctx.retention_totals()
    l0 = hbf.kernel_launches()
    t = timed(args.steps)
    launches = hbf.kernel_launches() - l0
    ms = float(t.sum())
    peak, kind = measured_peak()
    rate = 2 * n * args.steps / (ms * 1e-3)
    # the method's bytes: 41 per access and batch (two batches per step)
    moved = 2 * ALGO_BYTES_PER_ACCESS * n
    line = {"metric": METRIC, "value": rate, "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64",
            "data": "synthetic",
            "config": {"workload": "capacity_mode_retention", "accesses_per_step": 2 * n, "geometry": "64x8x4", "queues": 2048,
                       "blocks": tot["n_blocks"], "pages_per_block": ret["pages_per_block"], "gen_seconds": round(gen_s, 1),
                       "state": "reset at the start of every step; two batches and one epoch per step"},
            "gpu_launches": int(launches),
            "retention": {"batch_without_debt_ms": t[0] / args.steps, "epoch_ms": t[1] / args.steps,
                          "batch_with_claims_ms": t[2] / args.steps, "quanta_planned_per_epoch": tot["planned"],
                          "quanta_claimed_by_the_batch": tot["claimed"], "blocks_committed": tot["commits"]},
            "roofline": {"bound": "hbm", "kernel": "submit with retention, all kernels", "achieved": moved * args.steps / (ms * 1e-3) / 1e9,
                         "peak": peak, "peak_kind": kind, "unit": "GB/s",
                         "frac": moved * args.steps / (ms * 1e-3) / 1e9 / peak, "traffic": None,
                         "algorithmic_bytes_per_access": ALGO_BYTES_PER_ACCESS},
            "batch_result": {k: res[k] for k in ("n_modeled", "n_native", "max_completion_ns")}}
    print(json.dumps(line), flush=True)


def run_rom(args):
    """Fits the 224-state reduced-order thermal model (Eq. 2) of the package floorplan from the CUDA grid's unit-step
    responses (10 ms steps), compares it with the grid on three input shapes, and times both."""
    import torch
    from paper_2609_09800_b200 import build as hbf_build, hbf, era
    hbf_build.build()
    fp0 = wl.package_floorplan()
    fp = dict(fp0); fp["region_idle_w"] = np.zeros_like(fp["region_idle_w"])
    prof = wl.load_profile("nominal", **wl.GEOMETRY["serving"]); prof["n_sub"] = 160
    prof.update(rtt_c=500.0, ltt_c=600.0, stt_c=700.0, shutdown_c=800.0)
    g = hbf.Context(prof, fp)
    dt = 10_000_000
    region = np.asarray(fp["cell_region"]); m = len(fp["region_kind"])
    sel = list(range(m))[::6][:11]
    probes = [int(np.flatnonzero(region == k)[len(np.flatnonzero(region == k)) // 2]) for k in sel]
    t0 = time.time(); steps = era.unit_step_responses(g, probes, 420, dt); resp_s = time.time() - t0
    t0 = time.time(); fit = era.era(era.markov_from_steps(steps), n_states=224, rows=200, cols=200); fit_s = time.time() - t0
    rom = hbf.Rom(fit["A"], fit["B"], fit["C"], D=fit["D"], d=np.full(len(probes), prof["ambient_c"]))
    n_run = 400
    k = np.arange(n_run)[:, None]; amp = np.asarray(fp0["ext_power_w"], np.float64)[None, :] + 0.2
    shapes = dict(step=np.ones((n_run, 1)) * amp, ramp=(k / n_run) * amp, pulses=((k // 40) % 2) * amp)
    d_T = torch.empty(g.n_cells, dtype=torch.float32, device="cuda"); pt = torch.as_tensor(probes, device="cuda")
    errs = {}
    for name, p in shapes.items():
        g.reset(); full = np.empty((n_run, len(probes)))
        for i in range(n_run):
            g.thermal_step(dt, p[i].astype(np.float32), d_T, want_hot=False); full[i] = d_T[pt].cpu().numpy()
        rom.reset(); red = rom.step(p.astype(np.float32).astype(np.float64))
        errs[name] = {"worst_k": float(np.abs(red - full).max()), "swing_k": float(full.max() - prof["ambient_c"])}
    d_p = torch.from_numpy(shapes["step"]).cuda(); d_o = torch.empty((n_run, len(probes)), dtype=torch.float64, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    rom.step_device(d_p, n_run, d_o); torch.cuda.synchronize()
    e0.record(); rom.step_device(d_p, n_run, d_o); e1.record(); torch.cuda.synchronize()
    rom_us = e0.elapsed_time(e1) * 1e3 / n_run
    ext = shapes["step"][0].astype(np.float32)
    g.thermal_step(dt, ext, None, want_hot=False); torch.cuda.synchronize()
    e0.record()
    for _ in range(50):
        g.thermal_step(dt, ext, None, want_hot=False)
    e1.record(); torch.cuda.synchronize()
    grid_us = e0.elapsed_time(e1) * 1e3 / 50
    print(json.dumps({"metric": "thermal steps/s (reduced-order model, 10 ms steps)", "value": 1e6 / rom_us, "unit": "steps/s",
                      "n_gpus": 1, "steps": n_run, "warmup": n_run, "ms_per_step": rom_us * 1e-3, "higher_is_better": True,
                      "dtype": "f64", "data": "synthetic",
                      "config": {"workload": "rom", "states": 224, "inputs": m, "outputs": len(probes), "grid": "128x128",
                                 "unit_step_samples": 420, "responses_seconds": round(resp_s, 1), "fit_seconds": round(fit_s, 1)},
                      "full_grid_us_per_step": grid_us, "rom_us_per_step": rom_us, "model_vs_grid": errs}), flush=True)


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.workload == "capacity_paged":
        if rank == 0:
            run_paged(args)
        return
    if args.workload == "rom":
        if rank == 0:
            run_rom(args)
        return
    if args.workload == "capacity_retention":
        if rank == 0:
            run_retention(args)
        return
    if args.workload == "coupled_thermal":
        if rank == 0:
            run_coupled(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2609_09800_b200 import build as hbf_build, hbf, replicas

    assert torch.cuda.is_available(), "bench.py needs a CUDA device (no CPU fallback)"
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if local_rank == 0:
        hbf_build.build()
    if world > 1:
        dist.barrier()

    sampler = ClockSampler(local_rank)         # started now: it takes a few hundred ms before the first sample
    sampler.start()
    n = args.n
    w, gen_s = make_stream(n, seed=replicas.rank_seed(0, rank))   # every rank: an independent replica on its own stream
    if args.shuffle:                           # the same records in a random order (seeded): nothing is in issue order any more
        w.acc = w.acc[np.random.Generator(np.random.PCG64([7, rank])).permutation(n)]
    fp = wl.package_floorplan(channels=w.profile["channels"], dies=w.profile["dies"])
    ctx = hbf.Context(w.profile, fp)
    for r in w.ranges:
        ctx.register_range(*r)
    ctx.set_path({"auto": hbf.PATH_AUTO, "sort": hbf.PATH_SORT, "sort_full": hbf.PATH_SORT_FULL}[args.path])
    if args.channel_bus:
        ctx.enable_channel_bus()

    # inputs resident in HBM before the timed region
    h_acc = torch.from_numpy(w.acc.view(np.int64).reshape(-1))
    d_acc = h_acc.cuda()
    d_comp = torch.empty(n, dtype=torch.int64, device="cuda")
    d_stall = torch.empty(n, dtype=torch.int64, device="cuda")
    d_status = torch.empty(n, dtype=torch.uint8, device="cuda")
    d_stats = torch.empty(ctx.n_dies * 6, dtype=torch.int64, device="cuda")
    ws = ctx.workspace(n)
    ext = fp["ext_power_w"]
    stream = torch.cuda.current_stream()

    def step():
        rc = ctx.submit_batch(d_acc, n, d_comp, d_stall, d_status, d_stats, ws)
        assert rc == 0, rc
        ctx.thermal_step(1_000_000, ext, None, want_hot=False)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(k, fn):
        """k steps, each on idle queues (the reset is outside the timed region); device time summed over the steps."""
        total = 0.0
        for _ in range(k):
            ctx.reset()
            flush.fill_(1)                     # L2 flush (a write larger than the L2); the step is enqueued behind it, so the
            e0.record(stream); fn(); e1.record(stream)   # timed region begins on the device, not with the host's launch latency
            e1.synchronize()
            total += e0.elapsed_time(e1)
        return total

    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.mark_start()                       # the warm-up runs the same load as the timed steps
    timed(args.warmup, step)
    sync_all()
    res = ctx.last_result()
    assert res["code"] == 0, res
    launches0 = hbf.kernel_launches()
    stage_ms = {k: [] for k in hbf.PROF_STAGES}
    sync_all()
    total_ms = timed(args.steps, step)
    sync_all()
    sampler.mark_end()
    clocks = sampler.stop()
    launches = hbf.kernel_launches() - launches0
    # per-stage device times of a few more steps (events recorded between kernel groups on the same stream)
    ctx.set_profiling(True)
    for _ in range(min(3, args.steps)):
        ctx.reset()
        step()
        prof = ctx.get_profile()
        for k, v in prof.items():
            stage_ms[k].append(v)
    # the same batch replayed on the queues it has just filled: every queue is backlogged from its first access on
    e0.record(stream); step(); e1.record(stream); e1.synchronize()
    replay_ms = e0.elapsed_time(e1)
    units, total_ms = replicas.combine(n * args.steps, total_ms, device="cuda")     # sum of units, max of device times
    value = units / (total_ms * 1e-3)

    # end to end through the C ABI with host buffers: H2D of the records, submit + thermal step, D2H of results
    e2e = None
    if not args.no_e2e and not args.shuffle:   # (the chunked host call equals one batch only for records in issue order)
        h_in = h_acc.pin_memory()
        h_comp = torch.empty(n, dtype=torch.int64).pin_memory()
        h_stall = torch.empty(n, dtype=torch.int64).pin_memory()
        h_stats = torch.empty(ctx.n_dies * 6, dtype=torch.int64).pin_memory()

        e2e_chunk = max(1, min(n, args.e2e_chunk))

        def e2e_step():
            # the public host-buffer call: chunks of the batch are copied in, served and read back on three streams
            rc, _ = ctx.submit_pinned(h_in, n, h_comp, h_stall, h_stats, chunk=e2e_chunk)
            assert rc == 0, rc
            ctx.thermal_step(1_000_000, ext, None, want_hot=False)
        ctx.reset(); e2e_step(); sync_all()
        assert ctx.last_result()["code"] == 0
        ms = timed(args.e2e_steps, e2e_step)
        sync_all()
        e2e_units, ms = replicas.combine(n * args.e2e_steps, ms, device="cuda")
        e2e = {"value": e2e_units / (ms * 1e-3), "unit": UNIT, "steps": args.e2e_steps,
               "h2d_bytes_per_step": n * 24, "d2h_bytes_per_step": n * 16 + ctx.n_dies * 48,
               "call": "hbf_submit_host (C ABI, pinned host buffers): %d chunks, copy-in / service / read-back overlapped on three streams" % (-(-n // e2e_chunk))}

    if rank == 0:
        peak, peak_kind = measured_peak()
        med = {k: (statistics.median(v) if v else 0.0) for k, v in stage_ms.items()}
        timed = {k: v for k, v in med.items() if k in STAGE_BYTES or k == "sort"}
        dom = max(timed, key=lambda k: timed[k])
        if dom == "sort":
            n_pass = 2 if args.path != "sort_full" else 6
            dom_bytes = (8 + 12) + (n_pass - 1) * 24            # first pass reads keys only
            per_launch_ms = med["sort"]
        else:
            dom_bytes = STAGE_BYTES[dom]; per_launch_ms = med[dom]
        achieved = dom_bytes * n / (per_launch_ms * 1e-3) / 1e9 if per_launch_ms > 0 else 0.0
        counters = profiled_counters(dom) if dom in KERNEL_SOURCES else None
        roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                    "frac": achieved / peak, "traffic": counters["dram_bytes_per_access"] * n if counters else None,
                    "traffic_source": (os.path.relpath(COUNTERS_FILE, ROOT) if counters else
                                       "none: no capture of the present kernel source under profiles/"),
                    "algorithmic_bytes_per_access": dom_bytes, "ms_per_launch": per_launch_ms}
        if counters and per_launch_ms > 0:
            # the same kernel against the issue rate at the clock sampled during the timed region: what actually binds it
            mhz = (clocks or {}).get("sm_mhz") or 1965.0
            issue_peak = SM_COUNT * SCHEDULERS_PER_SM * mhz * 1e6
            issued = counters["warp_instr_per_access"] * n / (per_launch_ms * 1e-3)
            roofline["alu"] = {"achieved": issued / 1e12, "peak": issue_peak / 1e12, "unit": "T warp instructions/s",
                               "frac": issued / issue_peak, "warp_instructions_per_access": counters["warp_instr_per_access"],
                               "note": "instruction count from an ncu capture, time measured live"}
        path_gbs = ALGO_BYTES_PER_ACCESS * value / world / 1e9
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "int64", "data": "synthetic",
                "config": dict(headline_config(args, n),
                               l2="inputs (%.1f GB) larger than L2, and a 256 MB write before every timed step" % (n * 24 / 1e9)),
                "gen_seconds": round(gen_s, 1),
                "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
                "path_algorithmic": {"bytes_per_access": ALGO_BYTES_PER_ACCESS, "achieved": path_gbs, "unit": "GB/s",
                                     "frac": path_gbs / peak, "frac_of_8tbs_nominal": path_gbs / 8000.0},
                "stage_ms": {k: round(v, 4) for k, v in med.items()},
                "replay_on_backlogged_queues_ms": round(replay_ms, 4),
                "batch_result": {k: res[k] for k in ("n_modeled", "n_native", "max_completion_ns")}}
        if world == 1 and not args.no_cpu_baseline:
            sample = min(n, args.cpu_sample)
            rate, times = cpu_oracle_rate(w, sample)
            rate_all, cores, dt_all, _ = cpu_oracle_rate_all_cores(w, sample)
            line["cpu_baseline"] = {"value": rate_all, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": "first %d accesses of the same stream, one pass, dealt by channel to one oracle "
                                              "instance per core (%.1f s)" % (sample, dt_all),
                                    "one_core": {"value": rate, "cores": 1, "seconds": round(min(times), 2)}}
        if world == 1 and not args.no_configs:
            shuffled = None
            if not args.shuffle and not args.channel_bus:
                # the headline batch once more with its records in a random order (a seeded permutation made on the device):
                # nothing is in issue order, so the sort path has to serve it; best of two after a warm-up
                gen = torch.Generator(device="cuda"); gen.manual_seed(7)
                perm = torch.randperm(n, device="cuda", generator=gen)
                d_shuf = d_acc.view(n, 3)[perm].contiguous().view(-1)
                del perm
                ctx.set_profiling(False)
                ctx.set_path(hbf.PATH_SORT)
                best = None
                for k in range(3):
                    ctx.reset(); flush.fill_(1)
                    e0.record(stream)
                    rc = ctx.submit_batch(d_shuf, n, d_comp, d_stall, d_status, d_stats, ws)
                    e1.record(stream); e1.synchronize()
                    assert rc == 0 and ctx.last_result()["code"] == 0
                    if k:
                        best = e0.elapsed_time(e1) if best is None else min(best, e0.elapsed_time(e1))
                shuffled = {"accesses": n, "ms": round(best, 4), "accesses_per_s": n / (best * 1e-3),
                            "what": "hbf_submit_batch alone, sort path, the headline batch in a seeded random order"}
                del d_shuf
            del d_acc, d_comp, d_stall, d_status, ws
            ctx.destroy()
            torch.cuda.empty_cache()
            line["configs"] = other_configs(hbf, args)
            if shuffled:
                line["configs"]["capacity_mode_shuffled_order"] = {"sort": shuffled}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
