#!/usr/bin/env python
"""Benchmark of the Local AdaAlter hot path (Algorithm 3 of arXiv 1911.09030) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl ours|reference]

A "step" is one `la_run(T)` of the chosen configuration: T iterations of Algorithm 3 for all
W workers over all N coordinates, including the synchronisations that fall in it.  Prints ONE
JSON line.  With N > 1 GPUs (torchrun) each rank runs the same configuration on its own
coordinate range (coordinates never interact, so there is no data-path collective): weak
scaling.  `--impl reference` times the CPU oracle, as it stands, on a bounded sample.
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

METRIC = "worker_param_updates_per_sec"
UNIT = "worker*param updates/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
# DRAM bytes per launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum from
# the ncu capture summarised in profiles/), valid only for the kernel sources they were taken on.
KERNEL_HASH_AT_CAPTURE = "f7182c402edd33c4"
NCU_TRAFFIC_BYTES = {"c2": 2.2240e9}


def kernel_source_hash():
    """Hash of what defines the la_sweep kernels: the two headers and the tuning macros."""
    import hashlib
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_1911_09030_b200", "csrc")
    for name in ("grad_source.cuh", "la_sweep.cuh"):
        with open(os.path.join(d, name), "rb") as fh:
            h.update(fh.read())
    with open(os.path.join(d, "la_sweep_inst.inc")) as fh:
        for line in fh:
            if line.startswith("#define LA_VEC") or line.startswith("#define LA_MINB"):
                h.update(line.encode())
    return h.hexdigest()[:16]


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs (read-only)."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: str):
        self.idx = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.idx)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._pump, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        rows = [l for (ts, l) in self.lines if t0 <= ts <= t1 + 0.2] or [l for _, l in self.lines]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in rows:
            f = [v.strip() for v in l.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for nm, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------- oracle leg
def oracle_rate(wl, n_slice: int, threads: int = 1, T=None):
    """worker*param updates/s of the CPU oracle on the first n_slice coordinates at full W and T."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle.oracle import Oracle
    T = wl.T if T is None else T
    per = n_slice // threads
    jobs = []
    for k in range(threads):
        lo = k * per
        arr = wl.arrays(lo, per)
        o = Oracle(per, wl.W, wl.eta, wl.eps, wl.H, wl.b0sq, j_base=lo)
        if wl.grad == "quadratic":
            o.set_grad_quadratic(wl.noise_seed, arr["a"], arr["c"], wl.sigma)
        elif wl.grad == "noise_scaled":
            o.set_grad_noise(wl.noise_seed, arr["s"])
        else:
            o.set_grad_noise(wl.noise_seed, None)
        if wl.bf16_grads:
            o.set_grad_bf16(True)
        jobs.append(o)
    t0 = time.perf_counter()
    if threads == 1:
        jobs[0].run(T)
    else:
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(lambda o: o.run(T), jobs))
    dt = time.perf_counter() - t0
    return per * threads * wl.W * T / dt, dt


def run_reference(args, wl):
    """The reference arm: the oracle (plain single-threaded C++), timed as it stands."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_slice = min(wl.N, 1 << 14)
    for _ in range(args.warmup):
        oracle_rate(wl, 1024)
    rates, t_all = [], 0.0
    for _ in range(args.steps):
        r, dt = oracle_rate(wl, n_slice)
        rates.append(r); t_all += dt
    value = float(np.mean(rates))
    sample = f"first {n_slice} coordinates of {wl.name} at full W={wl.W}, T={wl.T}, per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_all / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(wl, args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# Issue-slot roofline of the temporal-blocking kernel (la_period): 148 SMs x 4 schedulers x 32
# lanes = 18 944 lane-instructions per clock; lane-instructions per worker*param update from the
# ncu capture summarised in profiles/ (smsp__inst_executed.sum x 32 / updates per launch).
LANE_INSTR_PER_CLOCK = 148 * 4 * 32
PERIOD_LANE_INSTR_PER_UPDATE = {"c2": 50.5}


def alu_roofline(period, wl, clocks):
    if period is None:
        return None
    out = dict(period)
    ipu = PERIOD_LANE_INSTR_PER_UPDATE.get(wl.name)
    max_mhz = (clocks or {}).get("sm_max_mhz") or 1965.0
    peak = LANE_INSTR_PER_CLOCK * max_mhz * 1e6 / 1e12          # T lane-instr/s at the maximum SM clock
    if ipu:
        ach = period["value"] * ipu / 1e12
        out["roofline"] = {"bound": "alu", "achieved": ach, "peak": peak, "unit": "T lane-instr/s",
                           "frac": ach / peak, "lane_instr_per_update": ipu, "traffic": None}
    return out


def workload_config(wl, args):
    return {"workload": f"{wl.name}: W={wl.W}, N={wl.N} fp32 in {len(wl.sizes)} tensor(s), grad={wl.grad}"
                        f"{'+bf16' if wl.bf16_grads else ''}, eta={wl.eta}, eps={wl.eps}, H={wl.H}, T={wl.T} per step",
            "W": wl.W, "N": wl.N, "H": wl.H, "T": wl.T, "fusion": getattr(args, "fusion", None),
            "l2": "inputs larger than L2 (state %.2f GiB per GPU)" % (wl.N * 4 * (2 * wl.W + 1) / 2 ** 30),
            "sharding": "by coordinate range, no collective"}


# --------------------------------------------------------------------------- CUDA leg
def run_ours(args, wl):
    import torch
    import torch.distributed as dist
    from paper_1911_09030_b200 import local_adaalter as la

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    use_dist = world > 1 or ("RANK" in os.environ and "MASTER_PORT" in os.environ)   # launched by torchrun
    if use_dist:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize()

    # this rank's coordinate range: the same configuration, shifted (weak scaling)
    from paper_1911_09030_b200 import sharding
    j_base = sharding.weak_scaling_base(wl.N, rank)
    arr = wl.arrays()            # same per-coordinate inputs on every rank; noise differs through j_base
    stream = torch.cuda.current_stream()
    ctx = la.LocalAdaAlter.with_torch_arena(wl.sizes, wl.W, wl.eta, wl.eps, wl.H, b0sq=wl.b0sq, j_base=j_base)

    pinned = {k: torch.from_numpy(v).pin_memory() for k, v in arr.items()}
    x0_pin = torch.zeros(wl.N, dtype=torch.float32).pin_memory()
    out_pin = {k: torch.empty(wl.N, dtype=torch.float32).pin_memory() for k in ("x", "b2", "bs")}

    def upload():
        ctx._ck(ctx.L.la_set_init(ctx.h, x0_pin.data_ptr(), float(wl.b0sq)))
        if wl.grad == "quadratic":
            ctx._ck(ctx.L.la_set_grad_quadratic(ctx.h, wl.noise_seed, pinned["a"].data_ptr(),
                                                 pinned["c"].data_ptr(), float(wl.sigma)))
        elif wl.grad == "noise_scaled":
            ctx._ck(ctx.L.la_set_grad_noise(ctx.h, wl.noise_seed, pinned["s"].data_ptr()))
        else:
            ctx._ck(ctx.L.la_set_grad_noise(ctx.h, wl.noise_seed, None))
    h2d = 4 * wl.N * (1 + len(arr))
    d2h = 4 * wl.N * 3

    upload()
    if wl.bf16_grads:
        ctx.set_grad_dtype(la.LA_BF16)
    ctx.set_fusion(args.fusion)
    if args.blocks_per_sm:
        ctx.set_launch_shape(args.blocks_per_sm)

    # ---- device-resident timing -----------------------------------------------------------
    for _ in range(args.warmup):
        ctx.run(wl.T)
    barrier()
    ctx.get_stats(reset=True)
    ctx.set_profiling(True)
    vis = [v for v in os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",") if v]
    sampler = ClockSampler(vis[local_rank] if local_rank < len(vis) else str(local_rank))
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_wall0 = time.time()
    e0.record(stream)
    for _ in range(args.steps):
        ctx.run(wl.T)
    e1.record(stream)
    barrier()
    t_wall1 = time.time()
    ms_total = e0.elapsed_time(e1)
    stats = ctx.get_stats(reset=True)
    ctx.set_profiling(False)
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None

    # ---- the same job with temporal blocking (LA_FUSE_PERIOD): issue-bound instead of HBM-bound
    period = None
    if args.fusion != la.LA_FUSE_PERIOD and not args.no_period:
        ctx.set_fusion(la.LA_FUSE_PERIOD)
        for _ in range(2):
            ctx.run(wl.T)
        barrier()
        ctx.get_stats(reset=True)
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        p0.record(stream)
        for _ in range(args.steps):
            ctx.run(wl.T)
        p1.record(stream)
        barrier()
        pst = ctx.get_stats(reset=True)
        pms = sharding.max_over_ranks(p0.elapsed_time(p1) / args.steps, dist if use_dist else None)
        period = {"ms_per_step": pms, "value": wl.W * wl.N * wl.T * world / (pms * 1e-3), "unit": UNIT,
                  "launches_per_step": pst["launches_fused"] // args.steps,
                  "hbm_GBps": pst["bytes_fused"] / args.steps / (pms * 1e-3) / 1e9}
        ctx.set_fusion(args.fusion)

    # ---- end to end through the C-ABI with host buffers -------------------------------------
    def e2e_step():
        upload()
        ctx.run(wl.T)
        ctx._ck(ctx.L.la_read_state(ctx.h, 0, out_pin["x"].data_ptr(), out_pin["b2"].data_ptr(),
                                    out_pin["bs"].data_ptr()))
    e2e_step()
    barrier()
    t0 = time.perf_counter()
    e2e_steps = max(1, min(args.steps, 3))
    for _ in range(e2e_steps):
        e2e_step()                               # la_read_state synchronises the stream
    barrier()
    e2e_ms = 1e3 * (time.perf_counter() - t0) / e2e_steps

    ms_total = sharding.max_over_ranks(ms_total, dist if use_dist else None)
    e2e_ms = sharding.max_over_ranks(e2e_ms, dist if use_dist else None)
    ms_per_step = ms_total / args.steps
    units = wl.W * wl.N * wl.T * world
    value = units / (ms_per_step * 1e-3)

    if rank == 0:
        peak, peak_kind = measured_peak()
        launches = {k: stats[k] for k in ("launches_local", "launches_sync", "launches_fused")}
        n_local = max(1, stats["launches_local"])
        ms_local = stats["ms_local"] / n_local
        bytes_local = stats["bytes_local"] / n_local
        achieved = bytes_local / (ms_local * 1e-3) / 1e9 if ms_local > 0 else None
        roofline = {
            "bound": "hbm", "kernel": "la_sweep<STEP> (K1 local step)", "achieved": achieved, "peak": peak,
            "peak_kind": peak_kind, "unit": "GB/s", "frac": (achieved / peak) if achieved else None,
            "traffic": (NCU_TRAFFIC_BYTES.get(wl.name) if kernel_source_hash() == KERNEL_HASH_AT_CAPTURE
                        and args.H is None and args.N is None else None),
            "frac_of_nominal_8TBps": (achieved / NOMINAL_HBM_GBS) if achieved else None,
            "bytes_per_launch": bytes_local, "ms_per_launch": ms_local,
            "bytes_per_update": bytes_local / (wl.W * wl.N),
        }
        per_class = {}
        for cls in ("local", "sync", "fused"):
            n = stats[f"launches_{cls}"]
            if n:
                ms = stats[f"ms_{cls}"] / n
                per_class[cls] = {"launches": n, "ms_per_launch": ms,
                                  "GBps": stats[f"bytes_{cls}"] / n / (ms * 1e-3) / 1e9 if ms > 0 else None,
                                  "share_of_device_time": None}
        tot = sum(stats[f"ms_{c}"] for c in ("local", "sync", "fused"))
        for cls in per_class:
            per_class[cls]["share_of_device_time"] = stats[f"ms_{cls}"] / tot if tot > 0 else None
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            n_slice = min(wl.N, 1 << 16)
            v, dt = oracle_rate(wl, n_slice)
            cpu = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "seconds": dt,
                   "sample": f"first {n_slice} coordinates of {wl.name} at full W={wl.W}, T={wl.T}"}
            ncores = os.cpu_count() or 1
            if ncores > 1:      # the same loop on disjoint coordinate ranges, one per host core
                va, dta = oracle_rate(wl, n_slice * min(ncores, 16) // 2, threads=min(ncores, 16))
                cpu["all_cores"] = {"value": va, "cores": min(ncores, 16), "seconds": dta}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": workload_config(wl, args),
            "clocks": clocks,
            "e2e": {"value": units / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms},
            "gpu_launches": int(sum(launches.values())),
            "roofline": roofline, "cpu_baseline": cpu, "kernels": per_class,
            "temporal_blocking": alu_roofline(period, wl, clocks),
            "hbm_GBps_whole_step": (stats["bytes_local"] + stats["bytes_sync"] + stats["bytes_fused"]) / (ms_total * 1e-3) / 1e9,
        }
        print(json.dumps(line), flush=True)
    ctx.close()
    if use_dist:
        dist.destroy_process_group()


def run_report(args):
    """All five configurations plus the synchronisation-period sweep of configuration 4
    (H in {1,4,16,64} x {unfused, step+sync, sync+step, temporal blocking}): per-kernel-class device time, GB/s
    against the measured and the nominal HBM peak, share of time spent synchronising.
    Writes one JSON document to --report-out and a markdown table to stdout."""
    import torch
    from paper_1911_09030_b200 import local_adaalter as la
    from paper_1911_09030_b200 import workloads
    torch.cuda.set_device(0)
    peak, peak_kind = measured_peak()
    rows = []

    def one(wl, H, fusion, reps):
        arr = wl.arrays()
        ctx = la.LocalAdaAlter.with_torch_arena(wl.sizes, wl.W, wl.eta, wl.eps, H, b0sq=wl.b0sq)
        if wl.grad == "quadratic":
            ctx.set_grad_quadratic(wl.noise_seed, arr["a"], arr["c"], wl.sigma)
        elif wl.grad == "noise_scaled":
            ctx.set_grad_noise(wl.noise_seed, arr["s"])
        else:
            ctx.set_grad_noise(wl.noise_seed, None)
        del arr
        if wl.bf16_grads:
            ctx.set_grad_dtype(la.LA_BF16)
        ctx.set_fusion(fusion)
        ctx.run(wl.T)                                   # warm-up: one full run
        ctx.run(wl.T)
        ctx.run(wl.T)
        ctx.sync_stream()
        ctx.get_stats(reset=True)
        ctx.set_profiling(True)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        st = torch.cuda.current_stream()
        e0.record(st)
        for _ in range(reps):
            ctx.run(wl.T)
        e1.record(st)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        stats = ctx.get_stats(reset=True)
        ctx.close()
        row = {"config": wl.name, "W": wl.W, "N": wl.N, "H": H, "T": wl.T, "fusion": fusion,
               "ms_per_run": ms, "updates_per_s": wl.W * wl.N * wl.T / (ms * 1e-3)}
        tot_ms = sum(stats[f"ms_{c}"] for c in ("local", "sync", "fused"))
        tot_b = sum(stats[f"bytes_{c}"] for c in ("local", "sync", "fused"))
        row["GBps_all"] = tot_b / reps / (ms * 1e-3) / 1e9
        for c in ("local", "sync", "fused"):
            n = stats[f"launches_{c}"]
            row[f"n_{c}"] = n // reps
            row[f"us_{c}"] = 1e3 * stats[f"ms_{c}"] / n if n else None
            row[f"GBps_{c}"] = stats[f"bytes_{c}"] / n / (stats[f"ms_{c}"] / n * 1e-3) / 1e9 if n else None
            row[f"share_{c}"] = stats[f"ms_{c}"] / tot_ms if tot_ms else None
        # time attributable to synchronising: stand-alone syncs, plus for fused passes the
        # excess over a plain local step
        us_local = row["us_local"] or row["us_fused"]
        extra = 0.0
        if row["n_sync"]:
            extra += row["n_sync"] * row["us_sync"]
        if row["n_fused"] and row["us_local"]:
            extra += row["n_fused"] * max(0.0, row["us_fused"] - row["us_local"])
        row["sync_share_of_time"] = extra / (1e3 * tot_ms / reps) if tot_ms else None
        rows.append(row)
        return row

    for name in ("c1", "c2", "c3", "c5"):
        wl = workloads.config(name)
        one(wl, wl.H, args.fusion, reps=3 if name != "c1" else 20)
        one(wl, wl.H, 3, reps=3 if name != "c1" else 20)          # temporal blocking
    wl4 = workloads.config("c4")
    for H in wl4.H_sweep:
        for fusion in (0, 1, 2, 3):
            one(wl4, H, fusion, reps=2)
    doc = {"peak_GBps": peak, "peak_kind": peak_kind, "nominal_GBps": NOMINAL_HBM_GBS, "rows": rows}
    if args.report_out:
        os.makedirs(os.path.dirname(os.path.abspath(args.report_out)), exist_ok=True)
        with open(args.report_out, "w") as f:
            json.dump(doc, f, indent=1)
    f2 = lambda v, d=0: "-" if v is None else f"{v:.{d}f}"
    print(f"| cfg | W | H | fusion | updates/s | GB/s all | pct of {peak:.0f} | pct of 8000 | K1 us (GB/s) | K2 us (GB/s) | "
          "fused us (GB/s) | sync share |")
    print("|---|---|---|---|---|---|---|---|---|---|---|---|")
    for r in rows:
        print(f"| {r['config']} | {r['W']} | {r['H']} | {r['fusion']} | {r['updates_per_s']:.3e} | {r['GBps_all']:.0f} | "
              f"{100 * r['GBps_all'] / peak:.1f} | {100 * r['GBps_all'] / NOMINAL_HBM_GBS:.1f} | "
              f"{f2(r['us_local'], 1)} ({f2(r['GBps_local'])}) | {f2(r['us_sync'], 1)} ({f2(r['GBps_sync'])}) | "
              f"{f2(r['us_fused'], 1)} ({f2(r['GBps_fused'])}) | {f2(100 * r['sync_share_of_time'], 1)} % |")


def run_tradeoff(args):
    """Single-GPU analogue of the paper's Table 2 (quality and time against the synchronisation
    period): the noisy quadratic of configuration 3 at N = 2^24, T = 256 iterations, for Local
    AdaAlter with H in {1,4,8,16,64,never} (unfused, so that the synchronisation cost is visible,
    and fused) and for the two baseline rules.  Prints objective at the mean iterate, replica
    spread before the last synchronisation, and time."""
    import torch
    from paper_1911_09030_b200 import local_adaalter as la
    from paper_1911_09030_b200 import workloads
    torch.cuda.set_device(0)
    wl = workloads.config("c3")
    wl.sizes = [1 << 24]
    arr = wl.arrays()
    T = 256
    rows = []

    def one(label, rule, H, fusion):
        ctx = la.LocalAdaAlter.with_torch_arena(wl.sizes, wl.W, wl.eta, wl.eps, H, b0sq=1.0)
        ctx.set_init(None, 1.0)
        ctx.set_grad_quadratic(wl.noise_seed, arr["a"], arr["c"], wl.sigma)
        ctx.set_rule(rule)
        ctx.set_fusion(fusion)
        f0 = ctx.diagnostics()[0]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        st = torch.cuda.current_stream()
        e0.record(st)
        ctx.run(T - 1)
        e1.record(st)
        torch.cuda.synchronize()
        spread = ctx.diagnostics()[1]
        ctx.run(1)
        f = ctx.diagnostics()[0]
        rows.append((label, H, fusion, f / f0, spread / wl.N, e0.elapsed_time(e1) * T / (T - 1), ctx.get_counters()[2]))
        ctx.close()

    for H in (1, 4, 8, 16, 64, la.LA_H_NEVER):
        one("Local AdaAlter", la.LA_RULE_ADAALTER, H, 0)
    for H in (4, 16):
        one("Local AdaAlter", la.LA_RULE_ADAALTER, H, 1)
        one("Local AdaAlter", la.LA_RULE_ADAALTER, H, 3)
    one("Distributed AdaGrad", la.LA_RULE_ADAGRAD, 1, 0)
    for H in (1, 16):
        one("Local SGD", la.LA_RULE_LOCAL_SGD, H, 0)
    print("| rule | H | fusion | F(x-bar_T)/F(x_0) | replica spread per coordinate at T-1 | ms for T=256 | exchanges |")
    print("|---|---|---|---|---|---|---|")
    for label, H, fusion, f, sp, ms, ns in rows:
        hs = "never" if H == la.LA_H_NEVER else str(H)
        print(f"| {label} | {hs} | {fusion} | {f:.5f} | {sp:.3e} | {ms:.1f} | {ns} |")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--H", type=int, default=None, help="override the synchronisation period")
    ap.add_argument("--T", type=int, default=None, help="override iterations per step")
    ap.add_argument("--N", type=int, default=None, help="override the size (one flat tensor), e.g. for small ncu captures")
    ap.add_argument("--fusion", type=int, default=1, help="0 unfused, 1 step+sync, 2 sync+next step")
    ap.add_argument("--blocks-per-sm", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-period", action="store_true", help="skip the extra temporal-blocking measurement")
    ap.add_argument("--report", action="store_true", help="all configurations + the H sweep (not the JSON line)")
    ap.add_argument("--report-out", default=None)
    ap.add_argument("--tradeoff", action="store_true", help="quality/time against H on a noisy quadratic (table)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.report:
        return run_report(args)
    if args.tradeoff:
        return run_tradeoff(args)
    from paper_1911_09030_b200 import workloads
    wl = workloads.config(args.workload)
    if args.H is not None:
        wl.H = args.H
    if args.T is not None:
        wl.T = args.T
    if args.N is not None:
        wl.sizes = [args.N]
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
