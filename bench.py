#!/usr/bin/env python
"""Benchmark of the Local AdaAlter hot path (Algorithm 3 of arXiv 1911.09030) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c5] [--impl ours|reference]

A "step" is one `la_run(T)` of the chosen configuration: T iterations of Algorithm 3 for all
W workers over all N coordinates, including the synchronisations that fall in it.  The default
workload is the largest single-GPU configuration (c5: 200 ragged tensors, 4e8 coordinates, four
workers, bf16-rounded gradients, 13.4 GiB of state), run with the per-step kernels and the
synchronised state stored once (LA_FUSE_MEAN_ONCE).  Prints ONE JSON line: the whole-run rate,
per-kernel durations and HBM roofline fractions of the local step (K1), the stand-alone
synchronisation (K2) and both fusions (K3, K4), the temporal-blocking mode, the end-to-end rate
with host buffers, the CPU oracle on the host cores, and — on one GPU — configuration 2 and the
synchronisation-period sweep of configuration 4, and the by-worker layout (`--sharding worker`
runs that layout alone, across ranks).  With N > 1 GPUs (torchrun) each rank runs the
same configuration on its own coordinate range (coordinates never interact, so there is no
data-path collective): weak scaling.  `--impl reference` times the CPU oracle, as it stands, on
a bounded sample.
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
# Figures taken from the ncu captures summarised in profiles/, valid only for the kernel sources
# they were taken on (KERNEL_HASH_AT_CAPTURE):
#   NCU_TRAFFIC_BYTES             dram__bytes_read.sum + dram__bytes_write.sum per K1 launch.  c2: captured at
#                                 full size.  c5: captured at N = 2^25 (1.5 GiB of state; the full 13.4 GiB is too
#                                 much to save and restore around ncu's replay passes) and scaled by
#                                 400 007 886 / 2^25 — every byte is touched once, so traffic grows with N.
#   PERIOD_LANE_INSTR_PER_UPDATE  smsp__inst_executed.sum x 32 / updates per la_period launch
KERNEL_HASH_AT_CAPTURE = "f309962a307aeecc"
NCU_TRAFFIC_BYTES = {"c2": 2.2235e9, "c5": 29.742e9}
PERIOD_LANE_INSTR_PER_UPDATE = {"c2": 43.15, "c5": 50.89}   # c5: captured at N = 2^25 (the count per update does not depend on N)


def kernel_source_hash():
    """Hash of what defines the kernels: the device headers and the tuning macros."""
    import hashlib
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_1911_09030_b200", "csrc")
    for name in ("grad_source.cuh", "la_sweep.cuh", "la_period.cuh", "la_exchange.cuh"):
        with open(os.path.join(d, name), "rb") as fh:
            h.update(fh.read())
    import glob
    for path in [os.path.join(d, "la_sweep_inst.inc")] + sorted(glob.glob(os.path.join(d, "la_sweep_w*.cu"))):
        with open(path) as fh:
            for line in fh:
                if line.startswith("#define LA_"):
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
    """Samples nvidia-smi clocks and throttle reasons for the whole invocation (read-only);
    `window(t0, t1)` summarises the samples that fell inside one timed region."""
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

    def stop(self):
        if not self.proc:
            return
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()

    def window(self, t0: float, t1: float):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        rows = [l for (ts, l) in list(self.lines) if t0 <= ts <= t1 + 0.2]
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
ORACLE_UPDATES_PER_CORE_S = 4.5e7     # order of magnitude, only used to bound the sample size


def oracle_rate(wl, j0: int, n_slice: int, threads: int = 1, T=None):
    """worker*param updates/s of the CPU oracle on coordinates [j0, j0 + n_slice) at full W and T,
    the slice cut into `threads` contiguous ranges, one per host thread."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle.oracle import Oracle
    T = wl.T if T is None else T
    per = n_slice // threads
    jobs = []
    for k in range(threads):
        lo = j0 + k * per
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


def bounded_slice(wl, want: int, seconds: float) -> int:
    """Largest power of two <= want whose single-core oracle run stays near `seconds`."""
    n = min(want, wl.N)
    while n > 1024 and n * wl.W * wl.T / ORACLE_UPDATES_PER_CORE_S > seconds:
        n //= 2
    return n


def cpu_baseline(wl):
    """The oracle as it stands on a contiguous slice of the workload (2^22 coordinates when one
    core finishes that in about half a minute) at full W and T: one core, then all cores."""
    n_slice = bounded_slice(wl, 1 << 22, 40.0)
    v, dt = oracle_rate(wl, 0, n_slice)
    cpu = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "seconds": dt,
           "sample": f"contiguous slice of {n_slice} coordinates [0, {n_slice}) of {wl.name} at full W={wl.W}, T={wl.T}"}
    ncores = os.cpu_count() or 1
    if ncores > 1:      # the same loop on disjoint coordinate ranges, one per host core
        th = min(ncores, 32)
        va, dta = oracle_rate(wl, 0, n_slice // th * th, threads=th)
        cpu["all_cores"] = {"value": va, "cores": th, "seconds": dta,
                            "sample": f"the same slice cut into {th} contiguous ranges, one host thread each"}
    return cpu


def run_reference(args, wl):
    """The reference arm: the oracle (plain single-threaded C++), timed as it stands."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_slice = bounded_slice(wl, 1 << 18, 1.5)
    for _ in range(args.warmup):
        oracle_rate(wl, 0, 1024)
    rates, t_all = [], 0.0
    for _ in range(args.steps):
        r, dt = oracle_rate(wl, 0, n_slice)
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
# ncu captures summarised in profiles/ (smsp__inst_executed.sum x 32 / updates per launch), valid
# only while the kernel sources hash to the captured version.
LANE_INSTR_PER_CLOCK = 148 * 4 * 32


def alu_roofline(period, wl, clocks):
    if period is None:
        return None
    out = dict(period)
    ipu = PERIOD_LANE_INSTR_PER_UPDATE.get(wl.name) if kernel_source_hash() == KERNEL_HASH_AT_CAPTURE else None
    max_mhz = (clocks or {}).get("sm_max_mhz") or 1965.0
    sm_mhz = (clocks or {}).get("sm_mhz")
    peak = LANE_INSTR_PER_CLOCK * max_mhz * 1e6 / 1e12          # T lane-instr/s at the maximum SM clock
    out["clocks"] = clocks
    if ipu:
        ach = period["value"] / period["n_gpus"] * ipu / 1e12
        out["roofline"] = {"bound": "alu", "achieved": ach, "peak": peak, "unit": "T lane-instr/s",
                           "frac": ach / peak, "lane_instr_per_update": ipu, "traffic": None,
                           "peak_at_sampled_clock": (LANE_INSTR_PER_CLOCK * sm_mhz * 1e6 / 1e12) if sm_mhz else None,
                           "frac_at_sampled_clock": (ach / (LANE_INSTR_PER_CLOCK * sm_mhz * 1e6 / 1e12)) if sm_mhz else None}
    return out


def workload_config(wl, args):
    return {"workload": f"{wl.name}: W={wl.W}, N={wl.N} fp32 in {len(wl.sizes)} tensor(s), grad={wl.grad}"
                        f"{'+bf16' if wl.bf16_grads else ''}, eta={wl.eta}, eps={wl.eps}, H={wl.H}, T={wl.T} per step",
            "W": wl.W, "N": wl.N, "H": wl.H, "T": wl.T, "fusion": getattr(args, "fusion", None),
            "l2": "inputs larger than L2 (state %.2f GiB per GPU)" % (wl.N * 4 * (2 * wl.W + 1) / 2 ** 30),
            "sharding": "by coordinate range, no collective"}


# --------------------------------------------------------------------------- CUDA leg
KERNEL_NAMES = {"local": "K1 local step", "sync": "K2 sync", "step_sync": "K3 step+sync",
                "sync_step": "K4 sync+next step", "period": "temporal blocking"}
# With LA_FUSE_MEAN_ONCE the two passes next to a synchronisation move about half the bytes of K3 / K4
# (one side of the replicas is a single copy) for the same arithmetic, so they are reported apart.
MEAN_ONCE_NAMES = {"step_sync": ("step_sums", "step t'=H storing only the sums over the workers"),
                   "sync_step": ("means_step", "step t'=1 reading the one stored copy")}


def per_kernel(stats, peak, leg):
    """Per-kernel figures from the library's event-timed statistics of one profiled leg."""
    out = {}
    for cls in KERNEL_NAMES:
        n = stats[f"launches_{cls}"]
        ms_all = stats[f"ms_{cls}"]
        if not n or ms_all <= 0:
            continue
        ms = ms_all / n
        b = stats[f"bytes_{cls}"] / n
        gbs = b / (ms * 1e-3) / 1e9
        out[cls] = {"kernel": KERNEL_NAMES[cls], "launches": int(n), "ms_per_launch": ms, "bytes_per_launch": b,
                    "GBps": gbs, "frac": gbs / peak, "frac_of_nominal_8TBps": gbs / NOMINAL_HBM_GBS,
                    "ms_total": ms_all, "leg": leg}
    return out


class Job:
    """One configuration resident on this rank's GPU."""

    def __init__(self, la, wl, j_base=0, pinned=False):
        import torch
        self.la, self.wl, self.torch = la, wl, torch
        arr = wl.arrays()        # same per-coordinate inputs on every rank; noise differs through j_base
        self.ctx = la.LocalAdaAlter.with_torch_arena(wl.sizes, wl.W, wl.eta, wl.eps, wl.H, b0sq=wl.b0sq, j_base=j_base)
        self.stream = torch.cuda.current_stream()
        self.pinned = None
        if pinned:
            self.pinned = {k: torch.from_numpy(v).pin_memory() for k, v in arr.items()}
            self.x0_pin = torch.zeros(wl.N, dtype=torch.float32).pin_memory()
            self.out_pin = {k: torch.empty(wl.N, dtype=torch.float32).pin_memory() for k in ("x", "b2", "bs")}
            self.h2d = 4 * wl.N * (1 + len(arr))
            self.d2h = 4 * wl.N * 3
            self.upload()
        else:
            c = self.ctx
            if wl.grad == "quadratic":
                c.set_grad_quadratic(wl.noise_seed, arr["a"], arr["c"], wl.sigma)
            elif wl.grad == "noise_scaled":
                c.set_grad_noise(wl.noise_seed, arr["s"])
            else:
                c.set_grad_noise(wl.noise_seed, None)
        if wl.bf16_grads:
            self.ctx.set_grad_dtype(la.LA_BF16)

    def upload(self):
        """The step's inputs from pinned host memory, through the C-ABI (enqueued on the stream)."""
        c, wl, p = self.ctx, self.wl, self.pinned
        c._ck(c.L.la_set_init(c.h, self.x0_pin.data_ptr(), float(wl.b0sq)))
        if wl.grad == "quadratic":
            c._ck(c.L.la_set_grad_quadratic(c.h, wl.noise_seed, p["a"].data_ptr(), p["c"].data_ptr(), float(wl.sigma)))
        elif wl.grad == "noise_scaled":
            c._ck(c.L.la_set_grad_noise(c.h, wl.noise_seed, p["s"].data_ptr()))
        else:
            c._ck(c.L.la_set_grad_noise(c.h, wl.noise_seed, None))

    def download(self):
        c, o = self.ctx, self.out_pin
        c._ck(c.L.la_read_state(c.h, 0, o["x"].data_ptr(), o["b2"].data_ptr(), o["bs"].data_ptr()))

    def timed(self, fusion, steps, warmup, barrier, profiling=False, H=None, T=None):
        """`steps` x la_run(T) on the device; returns (ms per step, library statistics, wall window)."""
        torch, c = self.torch, self.ctx
        T = self.wl.T if T is None else T
        c.set_fusion(fusion)
        for _ in range(warmup):
            c.run(T)
        barrier()
        c.get_stats(reset=True)
        c.set_profiling(profiling)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        w0 = time.time()
        e0.record(self.stream)
        for _ in range(steps):
            c.run(T)
        e1.record(self.stream)
        barrier()
        w1 = time.time()
        ms = e0.elapsed_time(e1) / steps
        stats = c.get_stats(reset=True)
        c.set_profiling(False)
        return ms, stats, (w0, w1)

    def close(self):
        self.ctx.close()
        self.pinned = self.out_pin = self.x0_pin = None
        self.torch.cuda.empty_cache()


def run_ours(args, wl):
    import torch
    import torch.distributed as dist
    from paper_1911_09030_b200 import local_adaalter as la
    from paper_1911_09030_b200 import sharding, workloads

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    use_dist = world > 1 or ("RANK" in os.environ and "MASTER_PORT" in os.environ)   # launched by torchrun
    if use_dist:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dd = dist if use_dist else None

    def barrier():
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize()

    vis = [v for v in os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",") if v]
    sampler = ClockSampler(vis[local_rank] if local_rank < len(vis) else str(local_rank))
    if rank == 0:
        sampler.start()

    # this rank's coordinate range: the same configuration, shifted (weak scaling)
    job = Job(la, wl, j_base=sharding.weak_scaling_base(wl.N, rank), pinned=True)
    if args.blocks_per_sm:
        job.ctx.set_launch_shape(args.blocks_per_sm)
    units = wl.W * wl.N * wl.T * world
    peak, peak_kind = measured_peak()

    # ---- headline: device-resident, per-launch profiling off --------------------------------
    ms_step, stats_main, win_main = job.timed(args.fusion, args.steps, args.warmup, barrier)
    ms_step = sharding.max_over_ranks(ms_step, dd)
    launches_main = int(stats_main["launches_local"] + stats_main["launches_sync"] + stats_main["launches_fused"])
    bytes_main = stats_main["bytes_local"] + stats_main["bytes_sync"] + stats_main["bytes_fused"]

    # ---- the same run again with CUDA events around every launch: per-kernel durations -------
    kernels = {}
    _, st, _ = job.timed(args.fusion, args.steps, 1, barrier, profiling=True)
    for k, v in per_kernel(st, peak, f"la_run, fusion {args.fusion}, {args.steps} steps").items():
        if args.fusion == la.LA_FUSE_MEAN_ONCE and k in MEAN_ONCE_NAMES:
            k, v["kernel"] = MEAN_ONCE_NAMES[k]
            v["bound"] = "instruction issue (half the bytes of K3 / K4 for the same arithmetic)"
        kernels[k] = v
    short = max(1, min(args.steps, 3))
    if not args.main_only:
        for fusion in (la.LA_FUSE_NONE, la.LA_FUSE_STEP_SYNC, la.LA_FUSE_SYNC_STEP):
            if fusion == args.fusion:
                continue
            _, st, _ = job.timed(fusion, short, 1, barrier, profiling=True)
            for k, v in per_kernel(st, peak, f"la_run, fusion {fusion}, {short} steps").items():
                kernels.setdefault(k, v)
    kernels.pop("period", None)

    # ---- the same job with temporal blocking (LA_FUSE_PERIOD): issue-bound instead of HBM-bound
    period = None
    if args.fusion != la.LA_FUSE_PERIOD and not args.no_period:
        psteps = max(1, min(args.steps, 5))
        pms, pst, pwin = job.timed(la.LA_FUSE_PERIOD, psteps, 2, barrier)
        pms = sharding.max_over_ranks(pms, dd)
        period = {"ms_per_step": pms, "steps": psteps, "value": units / (pms * 1e-3), "unit": UNIT, "n_gpus": world,
                  "launches_per_step": int(pst["launches_fused"]) // psteps,
                  "hbm_GBps": pst["bytes_fused"] / psteps / (pms * 1e-3) / 1e9}
        period = alu_roofline(period, wl, sampler.window(*pwin) if rank == 0 else None)

    # ---- end to end through the C-ABI with host buffers -------------------------------------
    job.ctx.set_fusion(args.fusion)

    def e2e_plain():                             # three calls, one after the other
        job.upload()
        job.ctx.run(wl.T)
        job.download()                           # la_read_state synchronises the stream

    def e2e_streamed():                          # one call, the same work pipelined over coordinate ranges
        p, o = job.pinned, job.out_pin
        job.ctx.run_streamed(wl.T, worker=0, x0=job.x0_pin, a=p.get("a"), c=p.get("c"), s=p.get("s"),
                             x_out=o["x"], b2_out=o["b2"], bs_out=o["bs"], chunks=args.e2e_chunks)

    def e2e_time(step, n):
        step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(n):
            step()
        barrier()
        return sharding.max_over_ranks(1e3 * (time.perf_counter() - t0) / n, dd)
    e2e_steps = max(1, min(args.steps, 5))
    e2e_ms = e2e_time(e2e_streamed, e2e_steps)
    e2e_plain_ms = e2e_time(e2e_plain, max(1, min(args.steps, 2)))
    h2d, d2h = job.h2d, job.d2h
    job.close()

    # ---- the other bandwidth-bound configurations, on one GPU only ---------------------------
    extras = {}
    if world == 1 and not args.main_only:
        if wl.name != "c2":
            extras["c2"] = side_config(la, workloads.config("c2"), peak, barrier, sampler)
        extras["c4_sync_period_sweep"] = sync_period_sweep(la, workloads.config("c4"), peak, barrier)
        # the by-worker layout with this one rank (exchange kernels and host-ordered phases included)
        extras["by_worker"] = by_worker_leg(la, workloads.config("c2"), dd, rank, world, barrier, T=64)

    if rank == 0:
        sampler.stop()
        clocks = sampler.window(*win_main)
        k1 = kernels.get("local")
        roofline = {"bound": "hbm", "kernel": "la_sweep<STEP> (K1 local step)", "achieved": None, "peak": peak,
                    "peak_kind": peak_kind, "unit": "GB/s", "frac": None, "traffic": None}
        if k1:
            roofline.update({
                "achieved": k1["GBps"], "frac": k1["frac"], "frac_of_nominal_8TBps": k1["frac_of_nominal_8TBps"],
                "bytes_per_launch": k1["bytes_per_launch"], "ms_per_launch": k1["ms_per_launch"],
                "bytes_per_update": k1["bytes_per_launch"] / (wl.W * wl.N), "launches": k1["launches"],
                "timed": "CUDA events around every launch on the launching stream, in a repeat of the timed "
                         "region with the library's per-launch profiling on (the headline value is timed with it off)",
                "traffic": (NCU_TRAFFIC_BYTES.get(wl.name) if kernel_source_hash() == KERNEL_HASH_AT_CAPTURE
                            and args.H is None and args.N is None else None)})
        for cls, key in (("sync", "sync"), ("step_sync", "step_sync"), ("sync_step", "sync_step")):
            k = kernels.get(cls)
            if k:
                roofline[key] = {"kernel": k["kernel"], "achieved": k["GBps"], "peak": peak, "unit": "GB/s",
                                 "frac": k["frac"], "bytes_per_launch": k["bytes_per_launch"],
                                 "ms_per_launch": k["ms_per_launch"], "launches": k["launches"]}
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            cpu = cpu_baseline(wl)
        line = {
            "metric": METRIC, "value": units / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": workload_config(wl, args),
            "clocks": clocks,
            "e2e": {"value": units / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": e2e_steps,
                    "call": f"la_run_streamed: pinned host inputs -> T iterations -> pinned host outputs, "
                            f"{args.e2e_chunks or 16} coordinate ranges pipelined on three streams",
                    "unpipelined": {"value": units / (e2e_plain_ms * 1e-3), "ms_per_step": e2e_plain_ms,
                                    "call": "la_set_init + la_set_grad_* + la_run + la_read_state"}},
            "gpu_launches": launches_main,
            "roofline": roofline, "cpu_baseline": cpu, "kernels": kernels,
            "temporal_blocking": period,
            "hbm_GBps_whole_step": bytes_main / args.steps / (ms_step * 1e-3) / 1e9,
        }
        line.update(extras)
        print(json.dumps(line), flush=True)
    if use_dist:
        dist.destroy_process_group()


def side_config(la, wl, peak, barrier, sampler, steps=3):
    """A further configuration in the same invocation: whole-run rate, K1/K3 figures, temporal blocking."""
    job = Job(la, wl)
    ms, _, _ = job.timed(la.LA_FUSE_STEP_SYNC, steps, 3, barrier)
    _, st, _ = job.timed(la.LA_FUSE_STEP_SYNC, steps, 1, barrier, profiling=True)
    units = wl.W * wl.N * wl.T
    out = {"workload": workload_config(wl, None)["workload"], "steps": steps, "ms_per_step": ms,
           "value": units / (ms * 1e-3), "unit": UNIT,
           "kernels": per_kernel(st, peak, f"la_run, fusion 1, {steps} steps")}
    mms, _, _ = job.timed(la.LA_FUSE_MEAN_ONCE, steps, 2, barrier)
    out["mean_once"] = {"ms_per_step": mms, "value": units / (mms * 1e-3), "unit": UNIT}
    pms, pst, pwin = job.timed(la.LA_FUSE_PERIOD, steps, 2, barrier)
    period = {"ms_per_step": pms, "steps": steps, "value": units / (pms * 1e-3), "unit": UNIT, "n_gpus": 1,
              "launches_per_step": int(pst["launches_fused"]) // steps,
              "hbm_GBps": pst["bytes_fused"] / steps / (pms * 1e-3) / 1e9}
    out["temporal_blocking"] = alu_roofline(period, wl, sampler.window(*pwin))
    job.close()
    return out


def sync_period_sweep(la, wl, peak, barrier):
    """Configuration 4: for every synchronisation period H, one full la_run(T) unfused (K1 + K2),
    with the step fused into its synchronisation (K3), with the synchronisation folded into the
    next step (K4), and with the synchronised state stored once (LA_FUSE_MEAN_ONCE, where the
    passes next to a synchronisation are cheaper than a plain step); share of device time spent
    synchronising.  The single-GPU analogue of the
    2/H communication claim of Section 4.2."""
    import copy
    rows = []
    for H in wl.H_sweep:
        w = copy.copy(wl)
        w.H = H
        job = Job(la, w)
        for fusion in (la.LA_FUSE_NONE, la.LA_FUSE_STEP_SYNC, la.LA_FUSE_SYNC_STEP, la.LA_FUSE_MEAN_ONCE):
            if fusion == la.LA_FUSE_MEAN_ONCE and H < 2:
                continue                                    # with H = 1 it is LA_FUSE_STEP_SYNC
            job.ctx.set_fusion(fusion)
            job.ctx.run(2 * H if 2 * H < w.T else w.T)      # warm-up: two periods
            ms, st, _ = job.timed(fusion, 1, 0, barrier, profiling=True)
            ker = per_kernel(st, peak, f"H={H}, fusion {fusion}")
            tot = sum(st[f"ms_{c}"] for c in ("local", "sync", "fused"))
            ms_k1 = ker["local"]["ms_per_launch"] if "local" in ker else None
            sync_ms = st["ms_sync"]
            if ms_k1 is not None:   # a fused pass is charged its excess over a plain local step
                for c in ("step_sync", "sync_step"):
                    if c in ker:
                        sync_ms += st[f"launches_{c}"] * max(0.0, ker[c]["ms_per_launch"] - ms_k1)
            if fusion == la.LA_FUSE_MEAN_ONCE:
                ker = {MEAN_ONCE_NAMES.get(c, (c,))[0]: v for c, v in ker.items()}
            rows.append({"H": H, "fusion": fusion, "T": w.T, "ms_per_run": ms,
                         "value": w.W * w.N * w.T / (ms * 1e-3),
                         "sync_share_of_device_time": sync_ms / tot if tot > 0 else None,
                         "GBps": {c: round(v["GBps"], 1) for c, v in ker.items()},
                         "launches": {c: v["launches"] for c, v in ker.items()}})
        job.close()
    return {"workload": workload_config(wl, None)["workload"].split(", H=")[0], "unit": UNIT, "rows": rows}


def by_worker_leg(la, wl, dd, rank, world, barrier, T=None, periods=(1, 4, 16), exchanges=("peer", "allreduce")):
    """Sharding BY WORKER (the paper's layout, Section 4.2): every rank holds wl.W replicas of the
    W_total = wl.W x world workers and the ranks exchange x and B^2 every H steps — export of the
    local tree sums, exchange (peer-load combine kernel, or an all-reduce of the buffer by
    torch.distributed), import; the steps next to a synchronisation are fused with it.  Times T
    iterations per (H, exchange): whole-job rate, host time per exchange and its share."""
    import torch
    from paper_1911_09030_b200 import sharding
    from paper_1911_09030_b200.worker_sharded import CudaEngine, WorkerShardedJob
    T = int(T or wl.T)
    arr = wl.arrays()
    rows = []
    for H in periods:
        for exch in exchanges:
            ctx = la.LocalAdaAlter.with_torch_arena(wl.sizes, wl.W, wl.eta, wl.eps, la.LA_H_NEVER, b0sq=wl.b0sq)
            if wl.grad == "quadratic":
                ctx.set_grad_quadratic(wl.noise_seed, arr["a"], arr["c"], wl.sigma)
            elif wl.grad == "noise_scaled":
                ctx.set_grad_noise(wl.noise_seed, arr["s"])
            else:
                ctx.set_grad_noise(wl.noise_seed, None)
            if wl.bf16_grads:
                ctx.set_grad_dtype(la.LA_BF16)
            eng = CudaEngine(ctx, rank, world)
            if dd is not None and exch == "peer":
                eng.attach_peers(dd)
            job = WorkerShardedJob(eng, H, exchange=exch, dist=dd, fused=True)
            job.run(2 * H if 2 * H < T else T)          # warm-up: two periods
            barrier()
            job.exchange_seconds, syncs0 = 0.0, job.syncs
            t0 = time.perf_counter()
            job.run(T)
            barrier()
            sec = sharding.max_over_ranks(time.perf_counter() - t0, dd)
            exs = sharding.max_over_ranks(job.exchange_seconds, dd)
            nsync = job.syncs - syncs0
            rows.append({"H": H, "exchange": exch, "T": T, "syncs": nsync, "ms_per_iteration": 1e3 * sec / T,
                         "value": wl.W * world * wl.N * T / sec,
                         "exchange_ms_per_sync": 1e3 * exs / nsync if nsync else None,
                         "exchange_share_of_time": exs / sec,
                         "exchange_bytes_per_rank_per_sync": 8 * wl.N})
            ctx.close()
            torch.cuda.empty_cache()
    return {"sharding": "by worker: %d local replicas per rank, W_total = %d" % (wl.W, wl.W * world),
            "workload": workload_config(wl, None)["workload"], "unit": UNIT, "ranks": world,
            "exchange_fused_steps": True, "rows": rows}


def run_by_worker(args, wl):
    """`--sharding worker`: the by-worker layout alone, one JSON line."""
    import torch
    import torch.distributed as dist
    from paper_1911_09030_b200 import local_adaalter as la
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    use_dist = world > 1 or ("RANK" in os.environ and "MASTER_PORT" in os.environ)
    if use_dist:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        # keep the communicator's own log lines (ranks, transports) on stderr, next to the numbers
        os.environ.setdefault("NCCL_DEBUG", "INFO")
        os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        os.environ.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dd = dist if use_dist else None

    def barrier():
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize()

    doc = by_worker_leg(la, wl, dd, rank, world, barrier, T=args.T)
    if rank == 0:
        best = max(doc["rows"], key=lambda r: r["value"])
        line = {"metric": METRIC, "value": best["value"], "unit": UNIT, "n_gpus": world, "steps": 1, "warmup": 1,
                "ms_per_step": best["ms_per_iteration"] * best["T"], "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": dict(workload_config(wl, args), sharding=doc["sharding"], H=best["H"], exchange=best["exchange"]),
                "by_worker": doc}
        print(json.dumps(line), flush=True)
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


def run_kernel_report(args):
    """Per-kernel GB/s away from the benchmark configurations: worker counts with their own
    instantiation (1 ... 16, 32, 64), worker counts known only at run time (17, 20, 24, 48), and
    caller-supplied gradient tables in fp32 and bf16 (W = 2, 4, 8, 16).  N = 2^24 (more for W < 4), pure-noise gradients
    (the shape of configuration 4), every pass timed by CUDA events around the launch.
    Markdown table to stdout, JSON to --report-out."""
    import torch
    from paper_1911_09030_b200 import local_adaalter as la
    torch.cuda.set_device(0)
    peak, peak_kind = measured_peak()
    rows = []

    def classes(ctx, W, what, once=False):
        st = ctx.get_stats(reset=True)
        for cls in ("local", "sync", "step_sync", "sync_step"):
            n = st[f"launches_{cls}"]
            if once and cls not in MEAN_ONCE_NAMES:
                continue
            if n and st[f"ms_{cls}"] > 0:
                ms = st[f"ms_{cls}"] / n
                gbs = st[f"bytes_{cls}"] / n / (ms * 1e-3) / 1e9
                rows.append({"W": W, "N": ctx.N, "gradients": what,
                             "kernel": MEAN_ONCE_NAMES[cls][1] if once else KERNEL_NAMES[cls], "launches": int(n),
                             "us_per_launch": 1e3 * ms, "GBps": gbs, "frac": gbs / peak})

    for W in args.workers:
        # at least 2^26 worker*params per pass, so that a launch lasts long enough to be bandwidth-bound
        N = args.N or max(1 << 24, 1 << (26 - max(0, W.bit_length() - 1)))
        ctx = la.LocalAdaAlter.with_torch_arena([N], W, 0.01, 1e-2, 4)
        ctx.set_grad_noise(4, None)
        if args.blocks_per_sm:
            ctx.set_launch_shape(args.blocks_per_sm)
        for fusion in (la.LA_FUSE_NONE, la.LA_FUSE_STEP_SYNC, la.LA_FUSE_SYNC_STEP):
            ctx.set_fusion(fusion)
            ctx.run(8)
        ctx.sync_stream()
        ctx.get_stats(reset=True)
        ctx.set_profiling(True)
        for fusion in (la.LA_FUSE_NONE, la.LA_FUSE_STEP_SYNC, la.LA_FUSE_SYNC_STEP):
            ctx.set_fusion(fusion)
            ctx.run(24)
        ctx.set_profiling(False)
        classes(ctx, W, "generated (noise)")
        if W in args.table_workers:
            for dtype, name, tdt in ((la.LA_F32, "fp32 table", torch.float32), (la.LA_BF16, "bf16 table", torch.bfloat16)):
                G = torch.randn(W, N, device="cuda", dtype=torch.float32).to(tdt)
                ctx.set_fusion(la.LA_FUSE_STEP_SYNC)
                for _ in range(8):
                    ctx.step_grads(G.data_ptr(), dtype)
                ctx.sync_stream()
                ctx.get_stats(reset=True)
                ctx.set_profiling(True)
                for _ in range(24):
                    ctx.step_grads(G.data_ptr(), dtype)
                ctx.set_profiling(False)
                classes(ctx, W, name)
                ctx.sync()
                ctx.set_fusion(la.LA_FUSE_MEAN_ONCE)      # the same table with the synchronised state stored once
                for _ in range(8):
                    ctx.step_grads(G.data_ptr(), dtype)
                ctx.sync_stream()
                ctx.get_stats(reset=True)
                ctx.set_profiling(True)
                for _ in range(24):
                    ctx.step_grads(G.data_ptr(), dtype)
                ctx.set_profiling(False)
                classes(ctx, W, name, once=True)
                ctx.sync()
                del G
        ctx.close()
        torch.cuda.empty_cache()
    doc = {"peak_GBps": peak, "peak_kind": peak_kind, "rows": rows}
    if args.report_out:
        os.makedirs(os.path.dirname(os.path.abspath(args.report_out)), exist_ok=True)
        with open(args.report_out, "w") as f:
            json.dump(doc, f, indent=1)
    print(f"| W | N | gradients | kernel | launches | us per launch | GB/s | of {peak:.0f} ({peak_kind}) |")
    print("|---|---|---|---|---|---|---|---|")
    for r in rows:
        print(f"| {r['W']} | {r['N']} | {r['gradients']} | {r['kernel']} | {r['launches']} | {r['us_per_launch']:.1f} | "
              f"{r['GBps']:.0f} | {r['frac']:.3f} |")


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
    ap.add_argument("--workload", default="c5", help="c1..c5; default: the largest single-GPU configuration")
    ap.add_argument("--H", type=int, default=None, help="override the synchronisation period")
    ap.add_argument("--T", type=int, default=None, help="override iterations per step")
    ap.add_argument("--W", type=int, default=None, help="override the worker count (replicas per rank)")
    ap.add_argument("--N", type=int, default=None, help="override the size (one flat tensor), e.g. for small ncu captures")
    ap.add_argument("--fusion", type=int, default=4,
                    help="0 unfused, 1 step+sync, 2 sync+next step, 3 temporal blocking, 4 synchronised state stored once")
    ap.add_argument("--blocks-per-sm", type=int, default=0)
    ap.add_argument("--e2e-chunks", type=int, default=0, help="coordinate ranges of the pipelined end-to-end call (0 = 16)")
    ap.add_argument("--sharding", default="coordinate", choices=["coordinate", "worker"],
                    help="coordinate: every rank owns a coordinate range, no collective (the headline); "
                         "worker: every rank owns W replicas and the ranks exchange x, B^2 every H steps")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-period", action="store_true", help="skip the extra temporal-blocking measurement")
    ap.add_argument("--main-only", action="store_true",
                    help="only the chosen workload in its fusion mode (no other fusion legs, no c2 / c4 extras)")
    ap.add_argument("--report", action="store_true", help="all configurations + the H sweep (not the JSON line)")
    ap.add_argument("--report-out", default=None)
    ap.add_argument("--tradeoff", action="store_true", help="quality/time against H on a noisy quadratic (table)")
    ap.add_argument("--report-kernels", action="store_true",
                    help="per-kernel GB/s for worker counts and gradient tables outside the five configurations")
    ap.add_argument("--workers", type=lambda v: [int(x) for x in v.split(",")], default=[1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 12, 13, 14, 15, 16, 32, 64, 17, 20, 24, 48])
    ap.add_argument("--table-workers", type=lambda v: [int(x) for x in v.split(",")], default=[2, 4, 8, 16])
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.report:
        return run_report(args)
    if args.tradeoff:
        return run_tradeoff(args)
    if args.report_kernels:
        return run_kernel_report(args)
    from paper_1911_09030_b200 import workloads
    wl = workloads.config(args.workload)
    if args.H is not None:
        wl.H = args.H
    if args.T is not None:
        wl.T = args.T
    if args.N is not None:
        wl.sizes = [args.N]
    if args.W is not None:
        wl.W = args.W
    if args.impl == "reference":
        run_reference(args, wl)
    elif args.sharding == "worker":
        run_by_worker(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
