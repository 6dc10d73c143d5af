#!/usr/bin/env python
"""Benchmark of the Server quasi-Newton step (arXiv 1709.05069, Section 2) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]

One step = one pass of the whole hot path (Gram pass, solve, combine; for the asynchronous config
the row refresh of one Write followed by the update) over one resident synthetic input.  Prints one
JSON line: updates/s over all ranks, the roofline of the dominant kernel, the CPU oracle's time on a
bounded sample, and the end-to-end figure with host buffers.

N > 1 (launched by torch.distributed.run, one rank per GPU): the method runs on one GPU with all m
Workers' vectors resident, so ranks are independent replicas of the same workload ("replicas
only"): there is no data-path collective; the barrier and the max-over-ranks of the device time
use NCCL.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

import workloads as W  # noqa: E402

METRIC = "qn_update/s"
UNIT = "updates/s"
DEFAULT_CONFIG = 2


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
# storage type and Gram path; a kernel without a capture of its current form reports no traffic.
MEASURED_TRAFFIC_RATIO = {
    ("combine", "f32", "tc"): 0.997,   # combine_vec_kernel<float>, config 2's generator at n = 4,194,304
    ("gram", "f32", "tc"): 1.007,      # gram_tc_kernel<float, 32>, same capture
    ("gram", "bf16", "tc"): 1.006,     # gram_tc_kernel<bf16, 64>, config 4's generator at n = 8,388,608
    ("row", "bf16", "direct"): 0.979,  # row_stream_kernel<bf16>, config 3's generator at n = 33,554,432
    ("combine", "bf16", "direct"): 0.986,  # combine_vec_kernel<bf16>, config 4's generator at m = 8, n = 33,554,432
    ("combine", "bf16", "tc"): 0.986,      # the same kernel (the Gram path does not change the combine pass)
    ("gram", "bf16", "direct"): 1.008,     # gram_stream_kernel<bf16, 8, true>, same capture
}


def algorithmic_bytes(cfg: W.Config):
    """Per update: Gram pass reads m*n, combine reads 2*m*n and writes n elements."""
    b = cfg.elem_bytes
    gram = cfg.m * cfg.n * b
    combine = (2 * cfg.m * cfg.n + cfg.n) * b
    row = (cfg.m * cfg.n + cfg.n) * b  # asynchronous row refresh: m-1 window rows + new column, lands n
    return {"gram": gram, "combine": combine, "row": row, "solve": 0}


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    REASONS = {
        0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
        0x80: "hw_power_brake", 0x2: "applications_clocks_setting", 0x100: "display_clock_setting", 0x10: "sync_boost",
    }

    def __init__(self, index: int, period: float = 0.05):
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
    """The slowest rank's figure: ranks are independent replicas, the job is as slow as its slowest one."""
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

    def time_once(self) -> float:
        t0 = time.perf_counter()
        self.oracle.update(self.tb, self.gb, self.cfg.tau, self.cfg.lam)
        return time.perf_counter() - t0

    def time_for(self, seconds: float, max_reps: int = 64):
        """Mean time of one oracle update over enough repetitions to fill about `seconds` of CPU work."""
        first = self.time_once()
        reps = max(1, min(max_reps, int(math.ceil(seconds / max(first, 1e-3))) - 1))
        times = [self.time_once() for _ in range(reps)]
        return float(np.mean(times)), reps


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
    per_update = float(np.mean(times)) * (cfg.n / ncols)
    value = 1.0 / per_update
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": per_update * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(cfg), "n": cfg.n, "m": cfg.m, "storage": cfg.dtype,
                   "note": "CPU oracle timed on a sample of the columns, scaled linearly in n"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": "first %d of %d columns per step, time scaled by n/sample" % (ncols, cfg.n)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


def workload_name(cfg: W.Config) -> str:
    mode = "async sliding window, one Write + update per step" if cfg.writes else "synchronous update"
    return "config %d: n=%d, m=%d, %s storage, %s" % (cfg.index, cfg.n, cfg.m, cfg.dtype, mode)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--config", type=int, default=DEFAULT_CONFIG, choices=range(len(W.CONFIGS)))
    ap.add_argument("--m", type=int, default=None, help="override the number of Workers (config 4's m sweep)")
    ap.add_argument("--n", type=int, default=None, help="override n (profiling on a small case)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--ref-cols", type=int, default=6_400_000, help="columns per oracle sample")
    ap.add_argument("--ref-seconds", type=float, default=12.0, help="CPU work of the cpu_baseline leg, seconds")
    args = ap.parse_args()

    cfg = W.CONFIGS[args.config].with_shape(n=args.n, m=args.m)
    if args.impl == "reference":
        if args.steps is None:
            args.steps = 3
        if args.warmup is None:
            args.warmup = 1
        return run_reference(args, cfg)

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=dev)

    from paper_1709_05069_b200 import qn

    qn.lib()
    bytes_per = algorithmic_bytes(cfg)
    step_bytes = (bytes_per["row"] + bytes_per["combine"]) if cfg.writes else (bytes_per["gram"] + bytes_per["combine"])
    peak, peak_kind = measured_peaks()
    ideal_ms = step_bytes / (peak * 1e9) * 1e3
    if args.steps is None:  # aim at a few seconds of timed work
        args.steps = int(max(20, min(2000, 4000.0 / max(ideal_ms * 1.5, 0.05))))
    if args.warmup is None:
        args.warmup = max(3, min(20, args.steps // 10))
    args.warmup = max(args.warmup, 3)

    # ------------------------------------------------------------------ CPU baseline (rank 0, before GPU work)
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu:
        import oracle

        oracle.build()
        sample = OracleSample(cfg, args.ref_cols)
        dt, reps = sample.time_for(args.ref_seconds)
        per_update = dt * (cfg.n / sample.ncols)
        cpu_baseline = {"value": 1.0 / per_update, "unit": UNIT, "cores": sample.cores, "kind": "oracle",
                        "sample": "%d oracle updates on the first %d of %d columns (%.1f s of CPU work after one warm-up "
                                  "update), mean time scaled by n/sample" % (reps, sample.ncols, cfg.n, dt * reps)}
        del sample

    # ------------------------------------------------------------------ inputs resident in HBM
    theta, g = W.generate(cfg, dev)
    out = torch.empty(cfg.n, dtype=cfg.torch_dtype, device=dev)
    h = qn.qn_create(cfg.n, cfg.m, cfg.torch_dtype)
    writes = None
    if cfg.writes:
        # the window starts as the generated (theta, g); Writes cycle through a small pool of columns
        pool = 4
        writes = [W.write_column(cfg, cfg.m + t, dev) for t in range(pool)]
        for k in range(cfg.m):
            qn.qn_push(h, -1, theta[k], g[k])
        del theta, g
        theta = g = None

    def step(i):
        if cfg.writes:
            th, gr = writes[i % len(writes)]
            qn.qn_push(h, -1, th, gr)
            qn.qn_update_window(h, cfg.tau, cfg.lam, out, want_host=False)
        else:
            qn.qn_update(h, theta, g, cfg.tau, cfg.lam, out, want_host=False)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    barrier()
    launches0 = h.total_launches
    kernels_per_step = 3
    qn.qn_timing_begin(h, args.steps * 4 + 8)
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
    total_ms = e0.elapsed_time(e1)
    timing = qn.qn_timing_end(h)
    launches = h.total_launches - launches0
    status = qn.qn_status_sync(h)
    total_ms = max_over_ranks(total_ms, world, dev)
    ms_per_step = total_ms / args.steps
    value = whole_job_value(ms_per_step, world)

    # dominant kernel and its roofline
    per_kernel = {k: (ms / cnt if cnt else 0.0, cnt) for k, (ms, cnt) in timing.items()}
    dominant = max(per_kernel, key=lambda k: per_kernel[k][0] * per_kernel[k][1])
    dom_ms = per_kernel[dominant][0]
    achieved = bytes_per[dominant] / (dom_ms * 1e-3) / 1e9 if dom_ms > 0 and bytes_per[dominant] else 0.0
    path = "tc" if (cfg.m > 8 and cfg.n >= (1 << 22)) else "direct" if cfg.m <= 8 else "alu"
    ratio = MEASURED_TRAFFIC_RATIO.get((dominant, cfg.dtype, path))
    roofline = {
        "bound": "hbm", "kernel": dominant, "achieved": achieved, "peak": peak, "unit": "GB/s",
        "frac": achieved / peak if peak else None, "peak_kind": "of " + peak_kind,
        "traffic": ratio * bytes_per[dominant] if ratio else None,
        "algorithmic_bytes_per_launch": bytes_per[dominant], "ms_per_launch": dom_ms,
        "per_kernel_ms": {k: round(v[0], 6) for k, v in per_kernel.items() if v[1]},
        "step_algorithmic_bytes": step_bytes, "step_gbs": step_bytes / (ms_per_step * 1e-3) / 1e9,
        "step_frac_of_hbm_peak": step_bytes / (ms_per_step * 1e-3) / 1e9 / peak,
    }

    # ------------------------------------------------------------------ end to end with host buffers
    e2e = None
    if not args.no_e2e and not cfg.writes:
        try:
            th_h = torch.empty((cfg.m, cfg.n), dtype=cfg.torch_dtype, pin_memory=True)
            g_h = torch.empty((cfg.m, cfg.n), dtype=cfg.torch_dtype, pin_memory=True)
            out_h = torch.empty(cfg.n, dtype=cfg.torch_dtype, pin_memory=True)
            th_h.copy_(theta)
            g_h.copy_(g)
            torch.cuda.synchronize()
            qn.qn_update_host(h, th_h, g_h, cfg.tau, cfg.lam, out_h)  # warm-up: allocates the staging
            barrier()
            t0 = time.perf_counter()
            for _ in range(args.e2e_steps):
                qn.qn_update_host(h, th_h, g_h, cfg.tau, cfg.lam, out_h)
            torch.cuda.synchronize()
            dt = (time.perf_counter() - t0) / args.e2e_steps
            dt = max_over_ranks(dt, world, dev)
            e2e = {"value": world / dt, "unit": UNIT, "h2d_bytes_per_step": 2 * cfg.m * cfg.n * cfg.elem_bytes,
                   "d2h_bytes_per_step": cfg.n * cfg.elem_bytes + 528, "ms_per_step": dt * 1e3,
                   "steps": args.e2e_steps, "api": "qn_update_host (pinned host buffers in, theta_new + j + sigma out)"}
            del th_h, g_h, out_h
        except Exception as ex:  # noqa: BLE001
            e2e = {"value": None, "unit": UNIT, "error": str(ex)[:200]}
    elif cfg.writes and not args.no_e2e:
        try:
            cols_h = [(a.cpu().pin_memory(), b.cpu().pin_memory()) for a, b in writes]
            out_h = torch.empty(cfg.n, dtype=cfg.torch_dtype, pin_memory=True)
            stage = [torch.empty(cfg.n, dtype=cfg.torch_dtype, device=dev) for _ in range(2)]

            def e2e_step(i):
                a, b = cols_h[i % len(cols_h)]
                stage[0].copy_(a, non_blocking=True)
                stage[1].copy_(b, non_blocking=True)
                qn.qn_push(h, -1, stage[0], stage[1])
                r = qn.qn_update_window(h, cfg.tau, cfg.lam, out, want_host=True)
                out_h.copy_(out, non_blocking=True)
                torch.cuda.synchronize()
                return r

            e2e_step(0)
            t0 = time.perf_counter()
            for i in range(args.e2e_steps):
                e2e_step(i)
            dt = (time.perf_counter() - t0) / args.e2e_steps
            e2e = {"value": world / dt, "unit": UNIT, "h2d_bytes_per_step": 2 * cfg.n * cfg.elem_bytes,
                   "d2h_bytes_per_step": cfg.n * cfg.elem_bytes + 528, "ms_per_step": dt * 1e3,
                   "steps": args.e2e_steps, "api": "pinned Write copied in, qn_push + qn_update_window, theta_new out"}
        except Exception as ex:  # noqa: BLE001
            e2e = {"value": None, "unit": UNIT, "error": str(ex)[:200]}

    h.close()
    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": workload_name(cfg), "n": cfg.n, "m": cfg.m, "storage": cfg.dtype, "tau": cfg.tau,
                       "lambda": cfg.lam, "l2": "inputs (%.2f GB) larger than L2" % (
                           (2 * cfg.m * cfg.n * cfg.elem_bytes) / 1e9),
                       "parallelism": "replicas only (one GPU holds all m Workers' vectors)",
                       "accumulation": "fp32 products, fp64 accumulation, fp64 eigen-solve"},
            "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": int(launches),
            "kernels_per_step": kernels_per_step, "clocks": clocks, "device_status": int(status),
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
