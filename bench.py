#!/usr/bin/env python
"""Benchmark of the A2CiD2 event-update engine.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config cfg4]

A step is one pass of the whole hot path over one chunk of the seeded event stream: host
scheduling, the fused event kernel over the chunk's batches, then the consensus-distance reduction.
The default workload is the 64-worker ring with ResNet-50-sized rows (d = 25.6e6, fp32), 500 events
per step and a consensus distance after every step.

Printed JSON line (rank 0):
  value     events/s with the step's descriptors already resident on the device (plans built
            and uploaded before the timed region), timed with CUDA events on the engine's stream
  e2e       the same through a2cid2_apply_events with host event arrays: validation,
            scheduling, descriptor upload and the consensus result read back are inside the
            timed region
  roofline  of the event kernel: bytes its items must move / its measured time, against the
            measured copy bandwidth of this machine's B200s
  clocks    SM clock and throttle reasons sampled (NVML) inside the timed region of `value`
  fresh_gradients   the same workload with a pool of gradient rows per worker, so that consecutive
            gradient events of a worker use different rows (fetched inside chained items)
  round_per_store   the same workload with x rounded once per store instead of once per event
            (a2cid2_set_rounding): the arithmetic that keeps every element within 1e-5, and its price
  other_configs     the other four workloads, a few timed steps each
  cpu_baseline  the CPU checker timed on a column slice of the same workload (reported only)
With N > 1 every rank runs an independent replica (the path has no exchange between GPUs) and only
the main figures are taken. `--impl reference` times the CPU checker alone, as the reference arm.
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
from concurrent.futures import ThreadPoolExecutor
from dataclasses import replace

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2306_08289_b200 import workload as W  # noqa: E402
from paper_2306_08289_b200.distutil import Ranks, aggregate_throughput  # noqa: E402

FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum of one event-kernel launch as a ratio to the bytes the
# launch's items must move, from the committed ncu summary named beside it; None while the kernel has
# changed since the counters were taken.
NCU_TRAFFIC_RATIO = 0.986
NCU_TRAFFIC_SOURCE = ("ncu dram__bytes_read.sum + dram__bytes_write.sum of three whole-step launches of the four-worker instance "
                      "on a d = 2e6 case of cfg4 (15.04 GB against 15.25 GB the items move: profiles/k_apply_events_cfg4_d2m.md), "
                      "scaled to this launch by its bytes; not a counter of this run")
LAUNCH_MODES = {"auto": 0, "per-batch": 1, "column-slices": 2}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=17)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="cfg4", choices=sorted(W.CONFIGS))
    ap.add_argument("--d", type=int, default=None, help="override the row width (for quick checks)")
    ap.add_argument("--events-per-step", type=int, default=500)
    ap.add_argument("--grad-pool", type=int, default=None,
                    help="gradient rows per worker, used round-robin by its gradient events (default: the workload's own)")
    ap.add_argument("--launch-mode", default="auto", choices=sorted(LAUNCH_MODES),
                    help="how a whole step is put on the GPU (a2cid2_set_launch_mode)")
    ap.add_argument("--no-fuse", action="store_true", help="one event per item (no gradient fusion)")
    ap.add_argument("--no-chain", action="store_true", help="gradient fusion only (A2_SCHED_FUSE), no item chaining")
    ap.add_argument("--cpu-sample-cols", type=int, default=None)
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--skip-resident-mode", action="store_true")
    ap.add_argument("--skip-baseline-dynamic", action="store_true")
    ap.add_argument("--skip-other-configs", action="store_true")
    ap.add_argument("--skip-fresh-gradients", action="store_true")
    ap.add_argument("--skip-round-per-store", action="store_true")
    ap.add_argument("--fresh-pool", type=int, default=4, help="gradient rows per worker of the fresh_gradients figure")
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


def config_dict(cfg, args, world):
    """The workload and how it is run; the same keys in both arms."""
    eb = 2 if cfg.storage == "bf16" else 4
    return {"workload": f"{cfg.name}: {cfg.note}", "n": cfg.n, "d": cfg.d, "graph": cfg.graph, "storage": cfg.storage,
            "events_per_step": args.events_per_step, "consensus_every_events": args.events_per_step,
            "gradient_rows_per_worker": cfg.grad_pool, "gradient_fusion": not args.no_fuse,
            "item_chaining": not (args.no_fuse or args.no_chain), "launch_mode": args.launch_mode,
            "parallelism": "replicas only" if world > 1 else "1 gpu",
            "l2": "state 2*n*d*elem bytes per replica exceeds L2; no flush needed" if 2 * cfg.n * cfg.d * eb > 3 * 126e6
                  else "state fits L2: figures are L2-assisted"}


def dtype_string(cfg):
    return "f32" if cfg.storage == "f32" else "bf16 storage, f32 math"


class ClockSampler:
    """SM clock, power and throttle reasons of one GPU, polled from a thread for the whole run (NVML reads
    only; nvidia-smi as a fallback); `window(t0, t1)` summarises the samples taken between two
    time.perf_counter() stamps, so the timed region has samples however short it is."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown"}

    def __init__(self, torch_device, period_s=0.004):
        self.samples = []  # (stamp, sm_mhz, power_w, reasons bitmask)
        self.max_mhz = None
        self.period = period_s
        self._stop = threading.Event()
        self._thread = None
        self._nvml = None
        self._handle = None
        self._smi_index = None
        try:
            import pynvml
            import torch

            pynvml.nvmlInit()
            props = torch.cuda.get_device_properties(torch_device)
            try:
                self._handle = pynvml.nvmlDeviceGetHandleByUUID(f"GPU-{props.uuid}")
            except Exception:
                vis = os.environ.get("CUDA_VISIBLE_DEVICES")
                idx = torch_device.index or 0
                self._handle = pynvml.nvmlDeviceGetHandleByIndex(int(vis.split(",")[idx]) if vis and vis.split(",")[idx].isdigit() else idx)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self._handle, pynvml.NVML_CLOCK_SM))
            self._nvml = pynvml
        except Exception:
            self._nvml = None
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            idx = getattr(torch_device, "index", 0) or 0
            self._smi_index = vis.split(",")[idx] if vis else str(idx)

    def _read_nvml(self):
        n, h = self._nvml, self._handle
        sm = float(n.nvmlDeviceGetClockInfo(h, n.NVML_CLOCK_SM))
        try:
            mask = int(n.nvmlDeviceGetCurrentClocksEventReasons(h))
        except Exception:
            mask = int(n.nvmlDeviceGetCurrentClocksThrottleReasons(h))
        try:
            power = n.nvmlDeviceGetPowerUsage(h) / 1e3
        except Exception:
            power = float("nan")
        return sm, power, mask

    def _read_smi(self):
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.sw_power_cap,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.hw_thermal_slowdown")
        out = subprocess.run(["nvidia-smi", "-i", self._smi_index, f"--query-gpu={q}", "--format=csv,noheader,nounits"],
                             capture_output=True, text=True, timeout=5).stdout.strip().splitlines()[0]
        f = [s.strip() for s in out.split(",")]
        self.max_mhz = float(f[1])
        mask = 0
        for bit, v in zip((0x4, 0x8, 0x20, 0x40), f[3:7]):
            if v.lower().startswith("active"):
                mask |= bit
        return float(f[0]), float(f[2]), mask

    def _loop(self):
        read = self._read_nvml if self._nvml is not None else self._read_smi
        while not self._stop.is_set():
            try:
                sm, power, mask = read()
                self.samples.append((time.perf_counter(), sm, power, mask))
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        self._thread = threading.Thread(target=self._loop, daemon=True)
        self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=5)

    def window(self, t0, t1):
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        if not inside:  # nearest samples on either side: better than nothing, and said so
            inside = sorted(self.samples, key=lambda s: min(abs(s[0] - t0), abs(s[0] - t1)))[:2]
            note = "no sample fell inside the timed region; nearest samples used"
        else:
            note = None
        if not inside:
            return None
        mask = 0
        for s in inside:
            mask |= s[3]
        out = {"sm_mhz": statistics.median(s[1] for s in inside), "sm_mhz_min": min(s[1] for s in inside),
               "sm_max_mhz": self.max_mhz, "power_w_max": max(s[2] for s in inside), "samples": len(inside),
               "window_s": t1 - t0, "source": "nvml" if self._nvml is not None else "nvidia-smi",
               "reasons": sorted(name for bit, name in self.REASONS.items() if mask & bit)}
        if note:
            out["note"] = note
        return out


def fill_engine(eng, cfg, threads):
    """x0 and the gradient rows, generated row by row on the host and copied in; x~ <- x."""
    def job(a):
        which, row = a
        stored, _ = (W.x0_row if which == "x" else W.grad_row)(cfg, row)
        return which, row, stored

    jobs = [("x", i) for i in range(cfg.n)] + [("g", i) for i in range(cfg.n_grad_slots)]
    with ThreadPoolExecutor(max(1, threads)) as ex:
        for which, row, stored in ex.map(job, jobs):
            eng.fill_row(which, row, stored)
    if eng.xt is not None:
        eng.xt.copy_(eng.x)
    eng.set_times(np.zeros(cfg.n))
    eng.sync()


def sample_inputs(cfg, n_cols, threads):
    """Widened (fp64) first n_cols columns of x0 and of the gradient rows."""
    cols = np.arange(n_cols)
    with ThreadPoolExecutor(max(1, threads)) as ex:
        xw = np.stack(list(ex.map(lambda i: W.x0_row(cfg, i, cols)[1], range(cfg.n))))
        gw = np.stack(list(ex.map(lambda i: W.grad_row(cfg, i, cols)[1], range(cfg.n_grad_slots))))
    return xw, gw


def oracle_params(cfg):
    from oracle import spectral

    if cfg.fixed_params is not None:
        return cfg.fixed_params
    return spectral.prescribe(cfg.n, cfg.edges(), cfg.rates())[:3]


def cpu_baseline(cfg, ev, n_cols, threads):
    """The CPU checker, as it stands, on the first n_cols columns of the workload and the given
    events; events/s is scaled to the full width by the column fraction (columns never interact,
    so the work is proportional to the width)."""
    from oracle.sim import OracleSim

    xw, gw = sample_inputs(cfg, n_cols, threads)
    sim = OracleSim(xw, *oracle_params(cfg), cfg.gamma, grads=gw)
    t0 = time.perf_counter()
    sim.apply_stream(ev, threads=threads)
    cons = sim.consensus()
    dt = time.perf_counter() - t0
    return len(ev) / dt * (n_cols / cfg.d), dt, cons


def run_reference(args, cfg):
    """Reference arm: the CPU checker on the host cores (rank 0 only)."""
    from oracle.sim import OracleSim

    threads = max(1, min(os.cpu_count() or 1, 32))
    n_cols = args.cpu_sample_cols or max(1, min(cfg.d, 256_000))
    eps = args.events_per_step
    ev_all = W.config_events(cfg, n_events=(args.warmup + args.steps) * eps)
    xw, gw = sample_inputs(cfg, n_cols, threads)
    sim = OracleSim(xw, *oracle_params(cfg), cfg.gamma, grads=gw)
    t_timed = 0.0
    for s in range(args.warmup + args.steps):
        chunk = ev_all.slice(s * eps, (s + 1) * eps)
        t0 = time.perf_counter()
        sim.apply_stream(chunk, threads=threads)
        sim.consensus()
        if s >= args.warmup:
            t_timed += time.perf_counter() - t0
    value = args.steps * eps / t_timed * (n_cols / cfg.d)
    sample = (f"first {n_cols} of {cfg.d} columns, all {cfg.n} workers, {eps} events + one consensus distance per step; "
              f"events/s scaled to the full width by the column fraction, ms_per_step as run")
    line = {
        "impl": "reference", "metric": "gossip_events_per_s", "value": value, "unit": "events/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * t_timed / args.steps,  # as run, on the column sample
        "ms_per_step_full_width_equivalent": 1e3 * t_timed / args.steps * (cfg.d / n_cols),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(cfg, args, max(1, args.gpus)),
        "cpu_baseline": {"value": value, "unit": "events/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "events/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


class Bench:
    """One workload on one engine: the timed passes share the engine, the event stream and the ranks."""

    def __init__(self, cfg, args, ranks, device, threads, n_warm, n_timed, stretches, rounding=None):
        import torch

        from paper_2306_08289_b200 import binding as B

        self.torch, self.B = torch, B
        self.cfg, self.args, self.ranks, self.device = cfg, args, ranks, device
        self.W_, self.K, self.eps = n_warm, n_timed, args.events_per_step
        self.n_steps = n_warm + n_timed
        self.flags = 0 if args.no_fuse else (B.A2_SCHED_FUSE if args.no_chain else B.A2_SCHED_CHAIN)
        self.eng = B.Engine(cfg.n, cfg.d, *B.config_params(cfg), cfg.gamma, storage=cfg.storage,
                            n_grad_slots=cfg.n_grad_slots, device=str(device))
        self.eng.set_launch_mode(LAUNCH_MODES[args.launch_mode])
        if rounding is not None:
            self.eng.set_rounding(rounding)
        fill_engine(self.eng, cfg, threads)
        self.ev_all = W.config_events(cfg, n_events=stretches * self.n_steps * self.eps)
        self.stretch = 0
        self.cons = []

    def _chunk(self, s):
        k = self.stretch * self.n_steps + s
        return self.ev_all.slice(k * self.eps, (k + 1) * self.eps)

    def _plans(self, flags):
        plans, t_start = [], self.eng.times()
        for s in range(self.n_steps):
            c = self._chunk(s)
            p = self.eng.plan(c.times, c.wi, c.wj, c.slot, flags=flags, t_start=t_start)
            t_start = p.sched.t_final(self.cfg.n)
            plans.append(p)
        return plans

    def plans_pass(self, flags=None):
        """Descriptors resident on the device; CUDA events around every plan run and every consensus distance."""
        torch, dev, W_, n = self.torch, self.device, self.W_, self.n_steps
        plans = self._plans(self.flags if flags is None else flags)
        stream = self.eng.stream
        marks = [tuple(torch.cuda.Event(enable_timing=True) for _ in range(3)) for _ in range(n)]
        stats = []
        t0 = t1 = None
        for s in range(n):
            if s == W_:
                torch.cuda.synchronize(dev)
                self.ranks.barrier()
                torch.cuda.synchronize(dev)
                t0 = time.perf_counter()
            a, b, c = marks[s]
            a.record(stream)
            stats.append(plans[s].run(want_stats=True))
            b.record(stream)
            self.cons.append(self.eng.consensus_distance())
            c.record(stream)
        torch.cuda.synchronize(dev)
        t1 = time.perf_counter()
        self.ranks.barrier()
        timed = range(W_, n)
        out = {
            "total_ms": marks[W_][0].elapsed_time(marks[n - 1][2]),
            "k1_ms": sum(marks[s][0].elapsed_time(marks[s][1]) for s in timed),
            "k2_ms": sum(marks[s][1].elapsed_time(marks[s][2]) for s in timed),
            "launches": sum(stats[s]["n_launches"] for s in timed),
            "bytes": sum(stats[s]["bytes_moved"] for s in timed),
            "bytes_single": sum(stats[s]["bytes_one_by_one"] for s in timed),
            "events": sum(stats[s]["n_events"] for s in timed),
            "batches": sum(stats[s]["n_batches"] for s in timed),
            "items": sum(stats[s]["n_items"] for s in timed),
            "window": (t0, t1),
        }
        for p in plans:
            p.close()
        self.stretch += 1
        return out

    def e2e_pass(self):
        """Through a2cid2_apply_events with host arrays; wall clock around the timed steps."""
        torch, dev = self.torch, self.device
        h2d = []
        torch.cuda.synchronize(dev)
        t0 = None
        for s in range(self.n_steps):
            if s == self.W_:
                torch.cuda.synchronize(dev)
                self.ranks.barrier()
                t0 = time.perf_counter()
            c = self._chunk(s)
            st = self.eng.apply_events(c.times, c.wi, c.wj, c.slot, flags=self.flags, want_stats=True)
            self.cons.append(self.eng.consensus_distance())  # waits for the stream and reads the result back
            if s >= self.W_:
                h2d.append(st["descriptor_bytes"])
        torch.cuda.synchronize(dev)
        secs = time.perf_counter() - t0
        self.ranks.barrier()
        self.stretch += 1
        value, _ = aggregate_throughput(self.ranks, self.K * self.eps, secs)
        return {"value": value, "unit": "events/s", "h2d_bytes_per_step": int(np.mean(h2d)) if h2d else 0, "d2h_bytes_per_step": 8}

    def check(self):
        if not all(np.isfinite(self.cons)):
            raise SystemExit("non-finite consensus distance: the run is invalid")

    def close(self):
        self.eng.close()
        self.eng = None
        self.torch.cuda.empty_cache()


def kernel_figures(p, peak):
    gbs = p["bytes"] / (p["k1_ms"] / 1e3) / 1e9
    return {"achieved_gbs": gbs, "frac": gbs / peak, "avg_launch_ms": p["k1_ms"] / max(1, p["launches"]), "launches": p["launches"]}


def light_run(cfg, args, ranks, device, threads, peak, n_warm=3, n_timed=5, rounding=None):
    """A few timed steps of another workload: events/s (plans resident), end to end, the event kernel."""
    t0 = time.perf_counter()
    b = Bench(cfg, args, ranks, device, threads, n_warm, n_timed, stretches=2, rounding=rounding)
    p = b.plans_pass()
    value, slowest = aggregate_throughput(ranks, p["events"], p["total_ms"] / 1e3)
    e2e = b.e2e_pass()
    b.check()
    b.close()
    out = {"value": value, "unit": "events/s", "ms_per_step": 1e3 * slowest / n_timed, "e2e": e2e["value"],
           "dtype": dtype_string(cfg), "steps": n_timed, "warmup": n_warm, "events_per_step": args.events_per_step,
           "rows_per_event": p["bytes"] / (cfg.d * (2 if cfg.storage == "bf16" else 4)) / max(1, p["events"]),
           "batches_per_step": p["batches"] / n_timed, "seconds_spent": None}
    out.update(kernel_figures(p, peak))
    out["seconds_spent"] = round(time.perf_counter() - t0, 1)
    return out


def main():
    args = parse_args()
    cfg = W.CONFIGS[args.config]
    if args.d is not None:
        cfg = cfg.scaled(d=args.d, name=f"{cfg.name}-d{args.d}")
    if args.grad_pool is not None:
        cfg = replace(cfg, grad_pool=int(args.grad_pool))
    if args.impl == "reference":
        # rank 0 alone times the CPU checker; the other ranks have nothing to do and no group is formed
        if int(os.environ.get("RANK", "0")) == 0:
            run_reference(args, cfg)
        return

    import torch

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the engine has no CPU path")
    from paper_2306_08289_b200 import binding as B
    from paper_2306_08289_b200 import build as cuda_build

    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    ranks = Ranks(backend="nccl", device=device)
    if ranks.rank == 0:
        cuda_build.build()
    ranks.barrier()
    sampler = ClockSampler(device)
    sampler.start()

    W_, K, eps = args.warmup, args.steps, args.events_per_step
    threads = max(1, min(os.cpu_count() or 1, 32) // max(1, ranks.world))
    peak, peak_src = measured_peak()

    # four stretches of the stream: plans resident on the device, end to end, shared-memory-resident mode,
    # and the asynchronous baseline without the momentum buffer
    b = Bench(cfg, args, ranks, device, threads, W_, K, stretches=4)
    eng = b.eng

    # ---- pass 1: descriptors resident on the device ---------------------------------------------
    p1 = b.plans_pass()
    clocks = sampler.window(*p1["window"])
    value, slowest_s = aggregate_throughput(ranks, p1["events"], p1["total_ms"] / 1e3)

    # ---- pass 2: end to end through a2cid2_apply_events with host arrays --------------------------
    e2e = b.e2e_pass()
    b.check()

    # ---- pass 3: the shared-memory-resident mode (one launch per step), reported beside the main figure ---
    resident = None
    if not args.skip_resident_mode:
        try:
            r = b.plans_pass(flags=B.A2_SCHED_RESIDENT)
            r_value, r_slow = aggregate_throughput(ranks, r["events"], r["total_ms"] / 1e3)
            resident = {"value": r_value, "unit": "events/s", "ms_per_step": 1e3 * r_slow / K,
                        "hbm_gbs": r["bytes"] / (r["total_ms"] / 1e3) / 1e9,
                        "note": "A2_SCHED_RESIDENT: one launch per step, column tile of all workers in shared "
                                "memory; needs every gradient of the step up front; not HBM-bound"}
        except B.A2Error as exc:
            resident = {"unavailable": str(exc)}

    # ---- pass 4: the asynchronous baseline (no momentum buffer, half the rows), reported beside the main figure ---
    plain = None
    if not args.skip_baseline_dynamic:
        eng.set_variant(B.A2_NO_MOMENTUM)
        q = b.plans_pass()
        eng.set_variant(B.A2_MSG_AFTER_MIX)
        q_value, q_slow = aggregate_throughput(ranks, q["events"], q["total_ms"] / 1e3)
        plain = {"value": q_value, "unit": "events/s", "ms_per_step": 1e3 * q_slow / K, "kernel": "k_apply_events_plain",
                 "note": "A2_NO_MOMENTUM: the paper's asynchronous baseline on the same stream recipe; x only, so "
                         "an event moves half the bytes"}
        plain.update(kernel_figures(q, peak))
        b.check()
    elem_bytes = eng.elem_bytes
    b.close()

    # ---- roofline of the event kernel ------------------------------------------------------------
    achieved = p1["bytes"] / (p1["k1_ms"] / 1e3) / 1e9
    per_launch_bytes = p1["bytes"] / max(1, p1["launches"])
    roofline = {
        "kernel": "k_apply_events", "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
        "frac": achieved / peak, "peak_source": f"of {peak_src} copy bandwidth",
        "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
        "traffic": None if NCU_TRAFFIC_RATIO is None else NCU_TRAFFIC_RATIO * per_launch_bytes,
        "traffic_source": NCU_TRAFFIC_SOURCE,
        "bytes_per_launch": per_launch_bytes, "avg_launch_ms": p1["k1_ms"] / max(1, p1["launches"]), "launches": p1["launches"],
        "rows_per_event": p1["bytes"] / (cfg.d * elem_bytes) / max(1, p1["events"]),
        "effective_gbs_one_event_per_item": p1["bytes_single"] / (p1["k1_ms"] / 1e3) / 1e9,
        "share_of_step_time": p1["k1_ms"] / p1["total_ms"],
        "note": "HBM is the roofline every instance of the event kernel is measured against; the four-worker instance on "
                "static gradient rows (ten events on 20 rows per item) is held back by instruction issue and latency "
                "before DRAM and follows the SM clock, with a gradient row per gradient event (fresh_gradients) it sits "
                "at the copy bandwidth",
    }
    consensus_gbs = K * cfg.n * cfg.d * elem_bytes / (p1["k2_ms"] / 1e3) / 1e9

    line = {
        "metric": "gossip_events_per_s", "value": value, "unit": "events/s", "n_gpus": ranks.world, "steps": K,
        "warmup": W_, "ms_per_step": 1e3 * slowest_s / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": dtype_string(cfg), "data": "synthetic",
        "config": config_dict(cfg, args, ranks.world),
        "clocks": clocks, "roofline": roofline, "e2e": e2e,
        "gpu_launches": int(p1["launches"] + 2 * K),
        "consensus_kernel": {"ms": p1["k2_ms"] / K, "gbs": consensus_gbs, "frac": consensus_gbs / peak},
        "batches_per_step": p1["batches"] / K, "items_per_step": p1["items"] / K,
        "resident_mode": resident,
        "baseline_dynamic": plain,
    }

    solo = ranks.world == 1
    # ---- the same workload with fresh gradient rows (a pool per worker, used round robin) ---------
    if solo and not args.skip_fresh_gradients and args.fresh_pool != cfg.grad_pool:
        try:
            fc = replace(cfg, grad_pool=args.fresh_pool, name=f"{cfg.name}-pool{args.fresh_pool}")
            fr = light_run(fc, args, ranks, device, threads, peak)
            fr["gradient_rows_per_worker"] = args.fresh_pool
            fr["note"] = ("consecutive gradient events of a worker name different rows; chained items fetch a worker's "
                          "next row inside the item, and every row fetched is counted in the kernel's bytes")
            line["fresh_gradients"] = fr
        except Exception as exc:  # e.g. not enough device memory for the pool
            line["fresh_gradients"] = {"unavailable": f"{type(exc).__name__}: {exc}"}
    # ---- the same workload with x rounded once per store instead of once per event ----------------
    if solo and not args.skip_round_per_store and cfg.storage == "f32":
        try:
            rs = light_run(cfg, args, ranks, device, threads, peak, rounding=B.A2_ROUND_PER_STORE)
            rs["note"] = ("A2_ROUND_PER_STORE: inside an item x is carried as a two-word value and rounded once, when the "
                          "row is stored; with it every element of this workload stays within 1e-5 of the fp64 checker "
                          "(the default, one rounding per event, ends 5 % above on the worst of 3.3e9 elements)")
            line["round_per_store"] = rs
        except Exception as exc:
            line["round_per_store"] = {"unavailable": f"{type(exc).__name__}: {exc}"}
    # ---- the other workloads, a few timed steps each ---------------------------------------------
    if solo and not args.skip_other_configs:
        others, budget_s, t_begin = {}, 150.0, time.perf_counter()
        for name in sorted(W.CONFIGS):
            if name == args.config:
                continue
            if time.perf_counter() - t_begin > budget_s:
                others[name] = {"skipped": f"time budget of {budget_s:.0f} s for the other workloads used up"}
                continue
            try:
                others[name] = light_run(W.CONFIGS[name], args, ranks, device, threads, peak)
            except Exception as exc:
                others[name] = {"unavailable": f"{type(exc).__name__}: {exc}"}
        line["other_configs"] = others

    if ranks.rank == 0 and solo and not args.skip_cpu_baseline:
        cores = max(1, min(os.cpu_count() or 1, 32))
        n_cols = args.cpu_sample_cols or max(1, min(cfg.d, 2_560_000))
        sample_ev = W.config_events(cfg, n_events=4 * eps)
        v, dt, _ = cpu_baseline(cfg, sample_ev, n_cols, cores)
        line["cpu_baseline"] = {
            "value": v, "unit": "events/s", "cores": cores, "kind": "oracle", "seconds": dt,
            "sample": f"first {n_cols} of {cfg.d} columns, all {cfg.n} workers, {4 * eps} events + one consensus "
                      f"distance; events/s scaled by the column fraction"}
        # the same checker strictly sequential on one thread, on a smaller slice
        n1 = max(1, min(cfg.d, n_cols // 10))
        v1, dt1, _ = cpu_baseline(cfg, W.config_events(cfg, n_events=eps), n1, 1)
        line["cpu_baseline"]["one_thread"] = {"value": v1, "seconds": dt1,
                                              "sample": f"first {n1} columns, {eps} events + one consensus distance"}
    sampler.stop()
    if ranks.rank == 0:
        print(json.dumps(line), flush=True)
    ranks.close()


if __name__ == "__main__":
    main()
