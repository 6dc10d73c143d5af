#!/usr/bin/env python
"""Benchmark of the Server quasi-Newton step (arXiv 1709.05069, Section 2) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--m M] [--impl ours|reference]
                    [--shard n] [--no-per-config] [--gram-path auto|alu|fp64]

One step = one pass of the whole hot path (Gram pass, solve, combine; for the asynchronous config the row refresh
of one Write followed by the update) over one resident synthetic input.  Prints ONE JSON line: updates/s of the
headline configuration over exactly K timed steps, the roofline of its dominant kernel, `per_config` (all five
configurations and the m sweep of the last one, each timed for at least two seconds so that the figure is the one
under the board's power limit, each labelled with the storage type and the Gram kernel that was dispatched), the
CPU oracle's time on a bounded sample, and the end-to-end figure with host buffers.

N > 1 (launched by torch.distributed.run, one rank per GPU).  Default: the method runs on one GPU with all m
Workers' vectors resident, so the ranks are independent replicas of the same workload ("replicas only", weak
scaling): no data-path collective; the barrier and the max-over-ranks of the device time use NCCL.
With `--shard n` the ranks share ONE problem instead (strong scaling): each holds a contiguous slice of the columns
of all m Workers, and a step is the Gram pass on the slice, one all-reduce of m*m + m doubles (NCCL), the
replicated eigen-solve and the combine pass on the slice.
"""
from __future__ import annotations

import argparse
import gc
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# The CPU legs time an OpenMP program: bind its threads to cores before the OpenMP runtime starts (it reads these
# once), so that repetitions and the two arms of a run see the same placement.
os.environ.setdefault("OMP_PROC_BIND", "close")
os.environ.setdefault("OMP_PLACES", "cores")

import numpy as np  # noqa: E402
import torch  # noqa: E402

import workloads as W  # noqa: E402

METRIC = "qn_update/s"
UNIT = "updates/s"
DEFAULT_CONFIG = 2
NOMINAL_HBM_GBS = 8000.0  # B200 data-sheet figure (7.7 TB/s on HGX boards); context beside the measured copy peak
TARGET_MIN_N = 25_600_000  # the >= 80 % end-to-end target applies from this n on
MIN_TIMED_SECONDS = 2.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


# DRAM bytes (read + written) per algorithmic byte of one launch, from the ncu captures of small cases summarised
# under profiles/ (traffic grows in proportion to n: every element is read once per pass).  Keyed by kernel kind,
# storage type and Gram kernel; a kernel without a capture of its current form reports no traffic.
MEASURED_TRAFFIC_RATIO = {
    ("combine", "f32", "tcgen05"): 0.997,   # combine_vec_kernel<float>, config 2's generator at n = 4,194,304
    ("gram", "f32", "tcgen05"): 1.007,      # gram_tc_kernel<float, 32>, same capture
    ("gram", "bf16", "tcgen05"): 1.006,     # gram_tc_kernel<bf16, 64>, config 4's generator at n = 8,388,608
    ("row", "bf16", "row"): 0.979,          # row_stream_kernel<bf16>, config 3's generator at n = 33,554,432
    ("combine", "bf16", "bulk-copy"): 0.986,  # combine_vec_kernel<bf16>, config 4's generator at m = 8, n = 33,554,432
    ("combine", "bf16", "tcgen05"): 0.986,    # the same kernel (the Gram kernel does not change the combine pass)
    ("combine", "bf16", "row"): 0.986,
    ("gram", "bf16", "bulk-copy"): 1.008,     # gram_stream_kernel<bf16, 8, true>, same capture
}


def algorithmic_bytes(cfg: W.Config):
    """Per update: Gram pass reads m*n, combine reads 2*m*n and writes n elements."""
    b = cfg.elem_bytes
    gram = cfg.m * cfg.n * b
    combine = (2 * cfg.m * cfg.n + cfg.n) * b
    row = (cfg.m * cfg.n + cfg.n) * b  # asynchronous row refresh: m-1 window rows + new column, lands n
    return {"gram": gram, "combine": combine, "row": row, "solve": 0}


def step_bytes_of(cfg: W.Config) -> int:
    b = algorithmic_bytes(cfg)
    return (b["row"] + b["combine"]) if cfg.writes else (b["gram"] + b["combine"])


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    REASONS = {
        0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
        0x80: "hw_power_brake", 0x2: "applications_clocks_setting", 0x100: "display_clock_setting", 0x10: "sync_boost",
    }

    def __init__(self, index: int, period: float = 0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml

            pynvml.nvmlInit()
            self.nv = pynvml
            uuid = None
            try:
                uuid = torch.cuda.get_device_properties(index).uuid
            except Exception:
                pass
            self.handle = None
            if uuid is not None:
                try:
                    self.handle = pynvml.nvmlDeviceGetHandleByUUID(("GPU-%s" % uuid).encode())
                except Exception:
                    self.handle = None
            if self.handle is None:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        while not self._stop_evt.is_set():
            try:
                self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.handle, self.nv.NVML_CLOCK_SM))
                mask = self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop_evt.wait(self.period)

    def stop(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2)
        return {
            "sm_mhz": float(np.median(self.samples)) if self.samples else None,
            "sm_max_mhz": float(self.max_mhz) if self.max_mhz else None,
            "reasons": sorted(self.reasons),
            "samples": len(self.samples),
        }


def max_over_ranks(x: float, world: int, device) -> float:
    """The slowest rank's figure: the job is as slow as its slowest rank."""
    if world <= 1:
        return float(x)
    t = torch.tensor([x], device=device, dtype=torch.float64)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(ms_per_step: float, world: int) -> float:
    """updates/s of the whole job: every rank finishes one update per step (weak scaling, replicas only)."""
    return world * 1e3 / ms_per_step


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def workload_name(cfg: W.Config) -> str:
    mode = "async sliding window, one Write + update per step" if cfg.writes else "synchronous update"
    return "config %d: n=%d, m=%d, %s storage, %s" % (cfg.index, cfg.n, cfg.m, cfg.dtype, mode)


def arithmetic_label(kernel: str) -> str:
    return "Gram/row pass: %s; eigen-solve: fp64 Jacobi (fp32 pre-sweeps for m >= 12); combine: fp32" % kernel


def kernel_key(kernel: str) -> str:
    for key in ("tcgen05", "bulk-copy", "tiled", "direct"):
        if kernel.startswith(key):
            return key
    return "row" if kernel.startswith("row refresh") else kernel


# ---------------------------------------------------------------------------------------------------------- CPU legs
class OracleSample:
    """The first `target_cols` columns of the workload on the host, and the CPU oracle, as it stands, timed on them."""

    def __init__(self, cfg: W.Config, target_cols: int):
        import oracle

        self.oracle = oracle
        self.cfg = cfg
        sub = cfg.with_shape(n=min(cfg.n, target_cols))
        theta, g = W.generate(sub, "cpu")
        self.tb, self.gb = W.to_bits(theta), W.to_bits(g)
        self.ncols = sub.n
        self.cores = oracle.threads_used(0)

    def time_once(self, nthreads: int = 0, cols=None) -> float:
        tb, gb = (self.tb, self.gb) if cols is None else (np.ascontiguousarray(self.tb[:, :cols]),
                                                         np.ascontiguousarray(self.gb[:, :cols]))
        t0 = time.perf_counter()
        self.oracle.update(tb, gb, self.cfg.tau, self.cfg.lam, nthreads=nthreads)
        return time.perf_counter() - t0

    def times_for(self, seconds: float, max_reps: int = 64):
        """Times of repeated oracle updates filling about `seconds` of CPU work, after one warm-up update."""
        first = self.time_once()
        reps = max(3, min(max_reps, int(math.ceil(seconds / max(first, 1e-3)))))
        return [self.time_once() for _ in range(reps)]


def cpu_spread(times, scale):
    """Per-update seconds -> updates/s at the full n: the median, and the fastest and slowest repetition."""
    t = np.asarray(times) * scale
    return {"value": float(1.0 / np.median(t)), "min": float(1.0 / t.max()), "median": float(1.0 / np.median(t)),
            "max": float(1.0 / t.min())}


def cpu_baseline_leg(cfg: W.Config, ref_cols: int, seconds: float):
    import oracle

    oracle.build()
    sample = OracleSample(cfg, ref_cols)
    times = sample.times_for(seconds)
    scale = cfg.n / sample.ncols
    out = {"unit": UNIT, "cores": sample.cores, "kind": "oracle", "threads": "bound to cores (OMP_PROC_BIND=close)"}
    out.update(cpu_spread(times, scale))
    out["sample"] = ("%d oracle updates on the first %d of %d columns (%.1f s of CPU work after one warm-up update), "
                     "median time scaled by n/sample" % (len(times), sample.ncols, cfg.n, float(np.sum(times))))
    # one thread, on an eighth of the sample
    cols1 = max(1, sample.ncols // 8)
    t1 = sample.time_once(nthreads=1, cols=cols1)
    out["single_thread"] = {"value": float(1.0 / (t1 * cfg.n / cols1)), "unit": UNIT, "cores": 1,
                            "sample": "1 oracle update on the first %d columns, time scaled by n/sample" % cols1}
    return out


def run_reference(args, cfg: W.Config):
    rank, world, _ = dist_env()
    if rank != 0:
        return 0
    import oracle

    oracle.build()
    sample = OracleSample(cfg, args.ref_cols)
    ncols, cores = sample.ncols, sample.cores
    times = []
    for it in range(args.warmup + args.steps):
        dt = sample.time_once()
        if it >= args.warmup:
            times.append(dt)
    scale = cfg.n / ncols
    spread = cpu_spread(times, scale)
    value = spread["value"]
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 / value, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(cfg), "n": cfg.n, "m": cfg.m, "storage": cfg.dtype,
                   "note": "CPU oracle timed on a sample of the columns, median step scaled linearly in n"},
        "cpu_baseline": {"value": value, "min": spread["min"], "median": spread["median"], "max": spread["max"],
                         "unit": UNIT, "cores": cores, "kind": "oracle",
                         "threads": "bound to cores (OMP_PROC_BIND=close)",
                         "sample": "first %d of %d columns per step, time scaled by n/sample" % (ncols, cfg.n)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# ---------------------------------------------------------------------------------------------------------- GPU legs
class Problem:
    """One configuration resident in HBM with its handle: `step(i)` enqueues one update."""

    def __init__(self, qn, cfg: W.Config, dev, gram_path: int = 0):
        self.qn, self.cfg, self.dev = qn, cfg, dev
        self.theta, self.g = W.generate(cfg, dev)
        self.out = torch.empty(cfg.n, dtype=cfg.torch_dtype, device=dev)
        self.h = qn.qn_create(cfg.n, cfg.m, cfg.torch_dtype)
        qn.qn_set_gram_path(self.h, gram_path)
        self.writes = None
        if cfg.writes:
            # the window starts as the generated (theta, g); Writes cycle through a small pool of columns
            self.writes = [W.write_column(cfg, cfg.m + t, dev) for t in range(4)]
            for k in range(cfg.m):
                qn.qn_push(self.h, -1, self.theta[k], self.g[k])
            self.theta = self.g = None

    def step(self, i: int):
        cfg, qn = self.cfg, self.qn
        if cfg.writes:
            th, gr = self.writes[i % len(self.writes)]
            qn.qn_push(self.h, -1, th, gr)
            qn.qn_update_window(self.h, cfg.tau, cfg.lam, self.out, want_host=False)
        else:
            qn.qn_update(self.h, self.theta, self.g, cfg.tau, cfg.lam, self.out, want_host=False)

    def close(self):
        self.h.close()
        self.theta = self.g = self.out = self.writes = None
        gc.collect()
        torch.cuda.empty_cache()


def timed_region(prob: Problem, steps: int, warmup: int, world: int, local: int, min_seconds: float = 0.0):
    """W warm-up steps, then `steps` timed steps between barriers (CUDA events on the launching stream, clocks
    sampled meanwhile).  With `min_seconds` the step count is raised until the region lasts that long."""
    qn, h, dev = prob.qn, prob.h, prob.dev

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    for i in range(warmup):
        prob.step(i)
    barrier()
    if min_seconds > 0.0:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        probe = 5
        e0.record()
        for i in range(probe):
            prob.step(i)
        e1.record()
        torch.cuda.synchronize()
        est = max(e0.elapsed_time(e1) / probe, 1e-3)
        steps = int(max(steps, min(200_000, math.ceil(min_seconds * 1e3 / est * 1.05))))
    launches0 = h.total_launches
    qn.qn_timing_begin(h, min(steps, 4000) * 6 + 8)  # per-kernel events for (at least) the first 4000 steps
    sampler = ClockSampler(local)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for i in range(steps):
        prob.step(i)
    e1.record()
    barrier()
    clocks = sampler.stop()
    total_ms = e0.elapsed_time(e1)
    timing = qn.qn_timing_end(h)
    launches = h.total_launches - launches0
    kernel = h.last_gram_kernel
    status = qn.qn_status_sync(h)
    total_ms = max_over_ranks(total_ms, world, dev)
    return {"steps": steps, "total_ms": total_ms, "timing": timing, "launches": int(launches), "kernel": kernel,
            "status": int(status), "clocks": clocks}


def describe(cfg: W.Config, res, peak: float, peak_kind: str, world: int = 1):
    """The figures of one timed region: per-kernel times, the dominant kernel's roofline, the step against the HBM
    roofline (measured copy peak and data-sheet figure)."""
    bytes_per = algorithmic_bytes(cfg)
    step_bytes = step_bytes_of(cfg)
    ms_per_step = res["total_ms"] / res["steps"]
    # per step and kind of kernel (a step may launch two kernels of a kind: the conditional fp64 repeat of the Gram
    # pass and of the solve return at once unless the spectrum asks for them, and are counted with their kind)
    timed_steps = max(1, res["timing"]["combine"][1])  # one combine pass per step: the steps whose kernels were timed
    per_kernel = {k: (ms / timed_steps, cnt) for k, (ms, cnt) in res["timing"].items()}
    dominant = max(per_kernel, key=lambda k: per_kernel[k][0])
    dom_ms = per_kernel[dominant][0]
    achieved = bytes_per[dominant] / (dom_ms * 1e-3) / 1e9 if dom_ms > 0 and bytes_per[dominant] else 0.0
    ratio = MEASURED_TRAFFIC_RATIO.get((dominant, cfg.dtype, kernel_key(res["kernel"])))
    step_gbs = step_bytes / (ms_per_step * 1e-3) / 1e9
    frac = step_gbs / peak
    if cfg.n < TARGET_MIN_N:
        target = "n/a (n < 25.6 M: latency-bound)"
    else:
        target = "met" if frac >= 0.8 else "not met"
    sm = res["clocks"].get("sm_mhz")
    roofline = {
        "bound": "hbm", "kernel": dominant, "achieved": achieved, "peak": peak, "unit": "GB/s",
        "frac": achieved / peak if peak else None, "peak_kind": "of " + peak_kind,
        "traffic": ratio * bytes_per[dominant] if ratio else None,
        "algorithmic_bytes_per_launch": bytes_per[dominant], "ms_per_launch": dom_ms,
        "launches_per_step": {k: round(v[1] / timed_steps, 3) for k, v in per_kernel.items() if v[1]},
        "per_kernel_ms": {k: round(v[0], 6) for k, v in per_kernel.items() if v[1]},
        "step_algorithmic_bytes": step_bytes, "step_gbs": step_gbs, "step_frac_of_hbm_peak": frac,
        "step_frac_of_nominal_hbm": step_gbs / NOMINAL_HBM_GBS, "nominal_hbm_gbs": NOMINAL_HBM_GBS,
    }
    return {
        "workload": workload_name(cfg), "n": cfg.n, "m": cfg.m, "dtype": cfg.dtype,
        "gram_kernel": res["kernel"], "steps": res["steps"], "timed_ms": res["total_ms"],
        "ms_per_step": ms_per_step, "value": whole_job_value(ms_per_step, world), "unit": UNIT,
        "per_kernel_ms": roofline["per_kernel_ms"], "step_gbs": step_gbs, "step_frac_of_hbm_peak": frac,
        "step_frac_of_nominal_hbm": step_gbs / NOMINAL_HBM_GBS,
        "target_80pct_of_measured_peak": target,
        "dominant": {"kernel": dominant, "achieved_gbs": achieved, "frac": achieved / peak if peak else None},
        "clocks": res["clocks"], "ms_x_ghz": ms_per_step * sm / 1e3 if sm else None,
        "device_status": res["status"], "gpu_launches": res["launches"],
    }, roofline


def per_config_entries():
    cfgs = [W.CONFIGS[0], W.CONFIGS[1], W.CONFIGS[2], W.CONFIGS[3]]
    cfgs += [W.CONFIGS[4].with_shape(m=m) for m in W.CONFIG4_M_SWEEP]
    return cfgs


def fits(cfg: W.Config) -> bool:
    need = 2 * cfg.m * cfg.n * cfg.elem_bytes * (2 if cfg.writes else 1) + 4 * cfg.n * cfg.elem_bytes + (3 << 30)
    free, _ = torch.cuda.mem_get_info()
    return free >= need


def e2e_leg(prob: Problem, world: int, steps: int):
    """The same metric through the library's host-buffer entry point: pinned host inputs copied in, theta_new (and
    j, sigma) copied out, every step."""
    qn, cfg, dev, h = prob.qn, prob.cfg, prob.dev, prob.h
    try:
        if not cfg.writes:
            th_h = torch.empty((cfg.m, cfg.n), dtype=cfg.torch_dtype, pin_memory=True)
            g_h = torch.empty((cfg.m, cfg.n), dtype=cfg.torch_dtype, pin_memory=True)
            out_h = torch.empty(cfg.n, dtype=cfg.torch_dtype, pin_memory=True)
            th_h.copy_(prob.theta)
            g_h.copy_(prob.g)
            torch.cuda.synchronize()
            qn.qn_update_host(h, th_h, g_h, cfg.tau, cfg.lam, out_h)  # warm-up: allocates the staging
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for _ in range(steps):
                qn.qn_update_host(h, th_h, g_h, cfg.tau, cfg.lam, out_h)
            torch.cuda.synchronize()
            dt = max_over_ranks((time.perf_counter() - t0) / steps, world, dev)
            return {"value": world / dt, "unit": UNIT, "h2d_bytes_per_step": 2 * cfg.m * cfg.n * cfg.elem_bytes,
                    "d2h_bytes_per_step": cfg.n * cfg.elem_bytes + 528, "ms_per_step": dt * 1e3, "steps": steps,
                    "api": "qn_update_host (pinned host buffers in, theta_new + j + sigma out)"}
        cols_h = [(a.cpu().pin_memory(), b.cpu().pin_memory()) for a, b in prob.writes]
        out_h = torch.empty(cfg.n, dtype=cfg.torch_dtype, pin_memory=True)
        stage = [torch.empty(cfg.n, dtype=cfg.torch_dtype, device=dev) for _ in range(2)]

        def e2e_step(i):
            a, b = cols_h[i % len(cols_h)]
            stage[0].copy_(a, non_blocking=True)
            stage[1].copy_(b, non_blocking=True)
            qn.qn_push(h, -1, stage[0], stage[1])
            r = qn.qn_update_window(h, cfg.tau, cfg.lam, prob.out, want_host=True)
            out_h.copy_(prob.out, non_blocking=True)
            torch.cuda.synchronize()
            return r

        e2e_step(0)
        t0 = time.perf_counter()
        for i in range(steps):
            e2e_step(i)
        dt = max_over_ranks((time.perf_counter() - t0) / steps, world, dev)
        return {"value": world / dt, "unit": UNIT, "h2d_bytes_per_step": 2 * cfg.n * cfg.elem_bytes,
                "d2h_bytes_per_step": cfg.n * cfg.elem_bytes + 528, "ms_per_step": dt * 1e3, "steps": steps,
                "api": "pinned Write copied in, qn_push + qn_update_window, theta_new out"}
    except Exception as ex:  # noqa: BLE001
        return {"value": None, "unit": UNIT, "error": str(ex)[:200]}


def default_steps(cfg: W.Config, peak: float) -> int:
    ideal_ms = step_bytes_of(cfg) / (peak * 1e9) * 1e3
    return int(max(20, min(2000, 4000.0 / max(ideal_ms * 1.5, 0.05))))  # a few seconds of timed work


# ---------------------------------------------------------------------------------------------------------- sharded
def run_sharded(args, cfg: W.Config, qn, dev, rank: int, world: int, local: int, peak: float, peak_kind: str):
    """ONE problem over all ranks: this rank generates and keeps only its column slice."""
    import torch.distributed as dist

    b, e = qn.shard_columns(cfg.n, world, rank)
    wt = None
    if cfg.rank:
        nchunks = (cfg.n + W.CHUNK - 1) // W.CHUNK
        c0, c1 = nchunks * rank // world, nchunks * (rank + 1) // world
        wt = W.low_rank_products(cfg, dev, min(c0 * W.CHUNK, cfg.n), min(c1 * W.CHUNK, cfg.n))
        dist.all_reduce(wt)  # input generation (the quadratic's low-rank part couples the columns), not the method
    theta, g = W.generate_slice(cfg, dev, b, e, wt)
    n_local = e - b
    out = torch.empty(n_local, dtype=cfg.torch_dtype, device=dev)
    buf = torch.empty(cfg.m * cfg.m + cfg.m, dtype=torch.float64, device=dev)
    h = qn.qn_create(n_local, cfg.m, cfg.torch_dtype)

    def step(_i):
        qn.qn_update_sharded(h, theta, g, cfg.tau, cfg.lam, out, buf, want_host=False)

    def barrier():
        dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    barrier()
    launches0 = h.total_launches
    qn.qn_timing_begin(h, args.steps * 6 + 8)
    sampler = ClockSampler(local)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for i in range(args.steps):
        step(i)
    e1.record()
    barrier()
    clocks = sampler.stop()
    total_ms = max_over_ranks(e0.elapsed_time(e1), world, dev)
    timing = qn.qn_timing_end(h)
    launches = h.total_launches - launches0
    kernel = h.last_gram_kernel
    status = qn.qn_status_sync(h)
    h.close()
    ms_per_step = total_ms / args.steps
    step_bytes = step_bytes_of(cfg)
    per_kernel = {k: round(ms / args.steps, 6) for k, (ms, cnt) in timing.items() if cnt}
    gbs = step_bytes / (ms_per_step * 1e-3) / 1e9
    if rank == 0:
        line = {
            "metric": METRIC, "value": 1e3 / ms_per_step, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong",
            "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": workload_name(cfg) + ", ONE problem sharded by columns over the ranks",
                       "n": cfg.n, "m": cfg.m, "storage": cfg.dtype, "tau": cfg.tau, "lambda": cfg.lam,
                       "columns_per_rank": n_local, "l2": "inputs larger than L2",
                       "parallelism": "n-sharded: per step one all-reduce of m*m + m doubles (%d bytes)" % (
                           8 * (cfg.m * cfg.m + cfg.m)),
                       "arithmetic": arithmetic_label(kernel)},
            "roofline": {"bound": "hbm", "kernel": "step", "achieved": gbs, "peak": peak * world, "unit": "GB/s",
                         "frac": gbs / (peak * world), "peak_kind": "of " + peak_kind + " (x ranks)",
                         "traffic": None, "per_kernel_ms": per_kernel, "step_algorithmic_bytes": step_bytes},
            "cpu_baseline": None, "e2e": None, "gpu_launches": int(launches), "kernels_per_step": round(launches / args.steps, 3),
            "clocks": clocks, "device_status": int(status),
        }
        print(json.dumps(line), flush=True)
    return 0


# ---------------------------------------------------------------------------------------------------------- main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--config", type=int, default=None, choices=range(len(W.CONFIGS)))
    ap.add_argument("--m", type=int, default=None, help="override the number of Workers (config 4's m sweep)")
    ap.add_argument("--n", type=int, default=None, help="override n (profiling on a small case)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--shard", default=None, choices=["n"], help="share ONE problem over the ranks by columns")
    ap.add_argument("--gram-path", default="auto", choices=["auto", "alu", "fp64"],
                    help="alu: plain-ALU Gram kernels only (A/B runs); fp64: those with fp64 products whatever n")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-per-config", action="store_true")
    ap.add_argument("--ref-cols", type=int, default=6_400_000, help="columns per oracle sample")
    ap.add_argument("--ref-seconds", type=float, default=12.0, help="CPU work of the cpu_baseline leg, seconds")
    args = ap.parse_args()

    if args.config is None:
        # the sharded form is measured on the largest configuration unless told otherwise
        args.config = 4 if args.shard else DEFAULT_CONFIG
    cfg = W.CONFIGS[args.config].with_shape(n=args.n, m=args.m)
    if args.impl == "reference":
        if args.steps is None:
            args.steps = 5
        if args.warmup is None:
            args.warmup = 1
        return run_reference(args, cfg)

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1 or args.shard:
        import torch.distributed as dist

        if "MASTER_ADDR" in os.environ and "RANK" in os.environ:
            dist.init_process_group("nccl", device_id=dev)
        else:
            import socket

            with socket.socket() as s:
                s.bind(("127.0.0.1", 0))
                port = s.getsockname()[1]
            dist.init_process_group("nccl", init_method="tcp://127.0.0.1:%d" % port, rank=0, world_size=1, device_id=dev)

    from paper_1709_05069_b200 import qn

    qn.lib()
    peak, peak_kind = measured_peaks()
    if args.steps is None:
        args.steps = default_steps(cfg, peak)
    if args.warmup is None:
        args.warmup = max(3, min(20, args.steps // 10))
    args.warmup = max(args.warmup, 3)
    gram_path = {"auto": qn.QN_GRAM_PATH_AUTO, "alu": qn.QN_GRAM_PATH_PLAIN_ALU, "fp64": qn.QN_GRAM_PATH_FP64}[args.gram_path]

    if args.shard:
        rc = run_sharded(args, cfg, qn, dev, rank, world, local, peak, peak_kind)
        torch.distributed.destroy_process_group()
        return rc

    # ------------------------------------------------------------------ CPU baseline (rank 0, before GPU work)
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu_baseline = cpu_baseline_leg(cfg, args.ref_cols, args.ref_seconds)

    # ------------------------------------------------------------------ headline: exactly K timed steps
    prob = Problem(qn, cfg, dev, gram_path)
    res = timed_region(prob, args.steps, args.warmup, world, local)
    head, roofline = describe(cfg, res, peak, peak_kind, world)
    e2e = None if args.no_e2e else e2e_leg(prob, world, args.e2e_steps)
    prob.close()

    # ------------------------------------------------------------------ every configuration, >= 2 s each
    per_config = None
    if rank == 0 and world == 1 and not args.no_per_config:
        per_config = []
        for c in per_config_entries():
            if not fits(c):
                per_config.append({"workload": workload_name(c), "skipped": "not enough free device memory"})
                continue
            p = Problem(qn, c, dev, gram_path)
            r = timed_region(p, 5, 3, 1, local, min_seconds=MIN_TIMED_SECONDS)
            entry, _ = describe(c, r, peak, peak_kind)
            per_config.append(entry)
            p.close()

    if rank == 0:
        line = {
            "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": workload_name(cfg), "n": cfg.n, "m": cfg.m, "storage": cfg.dtype, "tau": cfg.tau,
                       "lambda": cfg.lam, "l2": "inputs (%.2f GB) larger than L2" % (
                           (2 * cfg.m * cfg.n * cfg.elem_bytes) / 1e9),
                       "parallelism": "replicas only (one GPU holds all m Workers' vectors)",
                       "gram_kernel": head["gram_kernel"], "arithmetic": arithmetic_label(head["gram_kernel"])},
            "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": head["gpu_launches"],
            "kernels_per_step": round(head["gpu_launches"] / args.steps, 3), "clocks": head["clocks"], "ms_x_ghz": head["ms_x_ghz"],
            "device_status": head["device_status"],
            "target": {"what": ">= 80 %% of peak HBM bandwidth end to end at n >= 25.6 M, read against the measured "
                               "copy peak (%.0f GB/s); the fraction of the data-sheet %.0f GB/s is given beside it"
                               % (peak, NOMINAL_HBM_GBS),
                       "this_run": head["target_80pct_of_measured_peak"]},
            "per_config": per_config,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
