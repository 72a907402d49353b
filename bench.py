#!/usr/bin/env python
"""Benchmark of the A2CiD2 event-update engine.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config cfg4]

A step is one pass of the whole hot path over one chunk of the seeded event stream: host
scheduling, one fused event kernel per batch, then the consensus-distance reduction. The default
workload is the 64-worker ring with ResNet-50-sized rows (d = 25.6e6, fp32), 500 events per step
and a consensus distance after every step; 3 warm-up + 17 timed steps are its 10,000 events.

Printed JSON line (rank 0):
  value     events/s with the step's descriptors already resident on the device (plans built
            and uploaded before the timed region), timed with CUDA events on the engine's stream
  e2e       the same through a2cid2_apply_events with host event arrays: validation,
            scheduling, descriptor upload and the consensus result read back are inside the
            timed region
  roofline  of the event kernel: bytes its items must move / its measured time, against the
            measured copy bandwidth of this machine's B200s
  cpu_baseline  the CPU checker timed on a column slice of the same workload (reported only)
With N > 1 every rank runs an independent replica (the path has no exchange between GPUs).
`--impl reference` times the CPU checker alone, as the reference arm.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2306_08289_b200 import workload as W  # noqa: E402
from paper_2306_08289_b200.distutil import Ranks, aggregate_throughput  # noqa: E402

FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum per event-kernel launch from the committed ncu
# summary (profiles/k_apply_events_cfg4_d2m.md: two launches of the four-worker instance on a
# d = 2e6 case), as a ratio to the bytes the launch's items must move: reads 1.000, writes 0.93
# (the rest was still in L2 when the small launches ended). None once the kernel has changed
# since the counters were taken.
NCU_TRAFFIC_RATIO = 0.973


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
    ap.add_argument("--launch-mode", default="auto", choices=["auto", "per-batch", "column-slices"],
                    help="how a whole step is put on the GPU (a2cid2_set_launch_mode)")
    ap.add_argument("--no-fuse", action="store_true", help="one event per item (no gradient fusion)")
    ap.add_argument("--cpu-sample-cols", type=int, default=None)
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--no-chain", action="store_true", help="gradient fusion only (A2_SCHED_FUSE), no item chaining")
    ap.add_argument("--skip-resident-mode", action="store_true")
    ap.add_argument("--skip-baseline-dynamic", action="store_true")
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
    """nvidia-smi clocks and throttle reasons, sampled while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return None
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            return None
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            f = [s.strip() for s in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        if not sm:
            return None
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "samples": len(sm), "reasons": sorted(reasons)}


def fill_engine(eng, cfg, threads):
    """x0 and the gradient rows, generated row by row on the host and copied in; x~ <- x."""
    def job(args):
        which, row = args
        stored, _ = (W.x0_row if which == "x" else W.grad_row)(cfg, row)
        return which, row, stored

    jobs = [("x", i) for i in range(cfg.n)] + [("g", i) for i in range(cfg.n_grad_slots)]
    with ThreadPoolExecutor(max(1, threads)) as ex:
        for which, row, stored in ex.map(job, jobs):
            eng.fill_row(which, row, stored)
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


def cpu_baseline(cfg, ev, n_cols, threads):
    """The CPU checker, as it stands, on the first n_cols columns of the workload and the given
    events; events/s is scaled to the full width by the column fraction (columns never interact,
    so the work is proportional to the width)."""
    from oracle import spectral
    from oracle.sim import OracleSim

    xw, gw = sample_inputs(cfg, n_cols, threads)
    if cfg.fixed_params is not None:
        params = cfg.fixed_params
    else:
        params = spectral.prescribe(cfg.n, cfg.edges(), cfg.rates())[:3]
    sim = OracleSim(xw, *params, cfg.gamma, grads=gw)
    t0 = time.perf_counter()
    sim.apply_stream(ev, threads=threads)
    cons = sim.consensus()
    dt = time.perf_counter() - t0
    return len(ev) / dt * (n_cols / cfg.d), dt, cons


def run_reference(args, cfg):
    """Reference arm: the CPU checker on the host cores (rank 0 only)."""
    threads = max(1, min(os.cpu_count() or 1, 32))
    n_cols = args.cpu_sample_cols or max(1, min(cfg.d, 256_000))
    eps = args.events_per_step
    ev_all = W.config_events(cfg, n_events=(args.warmup + args.steps) * eps)
    from oracle import spectral
    from oracle.sim import OracleSim

    xw, gw = sample_inputs(cfg, n_cols, threads)
    params = cfg.fixed_params if cfg.fixed_params is not None else spectral.prescribe(cfg.n, cfg.edges(), cfg.rates())[:3]
    sim = OracleSim(xw, *params, cfg.gamma, grads=gw)
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
              f"events/s scaled by the column fraction")
    line = {
        "impl": "reference", "metric": "gossip_events_per_s", "value": value, "unit": "events/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * t_timed / args.steps * (cfg.d / n_cols), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: {cfg.note}", "n": cfg.n, "d": cfg.d, "graph": cfg.graph,
                   "events_per_step": eps},
        "cpu_baseline": {"value": value, "unit": "events/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "events/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    args = parse_args()
    cfg = W.CONFIGS[args.config]
    if args.d is not None:
        cfg = cfg.scaled(d=args.d, name=f"{cfg.name}-d{args.d}")
    if args.grad_pool is not None:
        from dataclasses import replace

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

    W_, K, eps = args.warmup, args.steps, args.events_per_step
    flags = 0 if args.no_fuse else (B.A2_SCHED_FUSE if args.no_chain else B.A2_SCHED_CHAIN)
    n_steps = W_ + K
    threads = max(1, min(os.cpu_count() or 1, 32) // max(1, ranks.world))

    eng = B.Engine(cfg.n, cfg.d, *B.config_params(cfg), cfg.gamma, storage=cfg.storage, n_grad_slots=cfg.n_grad_slots,
                   device=str(device))
    eng.set_launch_mode({"auto": B.A2_LAUNCH_AUTO, "per-batch": B.A2_LAUNCH_PER_BATCH,
                         "column-slices": B.A2_LAUNCH_COLUMN_SLICES}[args.launch_mode])
    fill_engine(eng, cfg, threads)
    # four stretches of the stream: plans resident on the device, end to end, shared-memory-resident mode,
    # and the asynchronous baseline without the momentum buffer
    ev_all = W.config_events(cfg, n_events=4 * n_steps * eps)

    # ---- pass 1: descriptors resident on the device ---------------------------------------------
    plans, t_start = [], np.zeros(cfg.n)
    for s in range(n_steps):
        c = ev_all.slice(s * eps, (s + 1) * eps)
        p = eng.plan(c.times, c.wi, c.wj, c.slot, flags=flags, t_start=t_start)
        t_start = p.sched.t_final(cfg.n)
        plans.append(p)
    stream = eng.stream
    ev_pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True),
                 torch.cuda.Event(enable_timing=True)) for _ in range(n_steps)]
    stats, cons = [], []
    sampler = ClockSampler(local_rank if os.environ.get("CUDA_VISIBLE_DEVICES") is None else
                           os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local_rank])
    for s in range(n_steps):
        if s == W_:
            torch.cuda.synchronize(device)
            ranks.barrier()
            sampler.start()
            torch.cuda.synchronize(device)
        a, b, c_ = ev_pairs[s]
        a.record(stream)
        stats.append(plans[s].run(want_stats=True))
        b.record(stream)
        cons.append(eng.consensus_distance())
        c_.record(stream)
    torch.cuda.synchronize(device)
    ranks.barrier()
    clocks = sampler.stop()
    timed = range(W_, n_steps)
    total_ms = ev_pairs[W_][0].elapsed_time(ev_pairs[n_steps - 1][2])
    k1_ms = sum(ev_pairs[s][0].elapsed_time(ev_pairs[s][1]) for s in timed)
    k2_ms = sum(ev_pairs[s][1].elapsed_time(ev_pairs[s][2]) for s in timed)
    k1_launches = sum(stats[s]["n_launches"] for s in timed)
    k1_bytes = sum(stats[s]["bytes_moved"] for s in timed)
    k1_bytes_single = sum(stats[s]["bytes_one_by_one"] for s in timed)
    n_events_timed = sum(stats[s]["n_events"] for s in timed)
    for p in plans:
        p.close()
    value, slowest_s = aggregate_throughput(ranks, n_events_timed, total_ms / 1e3)

    # ---- pass 2: end to end through a2cid2_apply_events with host arrays --------------------------
    h2d = []
    torch.cuda.synchronize(device)
    for s in range(n_steps):
        if s == W_:
            torch.cuda.synchronize(device)
            ranks.barrier()
            t0 = time.perf_counter()
        c = ev_all.slice((n_steps + s) * eps, (n_steps + s + 1) * eps)
        st = eng.apply_events(c.times, c.wi, c.wj, c.slot, flags=flags, want_stats=True)
        cons.append(eng.consensus_distance())  # waits for the stream and reads the result back
        if s >= W_:
            h2d.append(st["descriptor_bytes"])
    torch.cuda.synchronize(device)
    e2e_s = time.perf_counter() - t0
    ranks.barrier()
    e2e_value, _ = aggregate_throughput(ranks, K * eps, e2e_s)

    if not all(np.isfinite(cons)):
        raise SystemExit("non-finite consensus distance: the run is invalid")

    # ---- pass 3: the shared-memory-resident mode (one launch per step), reported beside the main figure ---
    resident = None
    if not args.skip_resident_mode:
        try:
            r_plans, t_start = [], eng.times()
            for s in range(n_steps):
                c = ev_all.slice((2 * n_steps + s) * eps, (2 * n_steps + s + 1) * eps)
                p = eng.plan(c.times, c.wi, c.wj, c.slot, flags=B.A2_SCHED_RESIDENT, t_start=t_start)
                t_start = p.sched.t_final(cfg.n)
                r_plans.append(p)
            r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            r_bytes = 0
            for s in range(n_steps):
                if s == W_:
                    torch.cuda.synchronize(device)
                    ranks.barrier()
                    r0.record(stream)
                st = r_plans[s].run(want_stats=True)
                cons.append(eng.consensus_distance())
                if s >= W_:
                    r_bytes += st["bytes_moved"]
            r1.record(stream)
            torch.cuda.synchronize(device)
            ranks.barrier()
            r_ms = r0.elapsed_time(r1)
            for p in r_plans:
                p.close()
            r_value, r_slow = aggregate_throughput(ranks, K * eps, r_ms / 1e3)
            resident = {"value": r_value, "unit": "events/s", "ms_per_step": 1e3 * r_slow / K,
                        "hbm_gbs": r_bytes / (r_ms / 1e3) / 1e9,
                        "note": "A2_SCHED_RESIDENT: one launch per step, column tile of all workers in shared "
                                "memory; needs every gradient of the step up front; not HBM-bound"}
        except B.A2Error as exc:
            resident = {"unavailable": str(exc)}

    # ---- pass 4: the asynchronous baseline (no momentum buffer, half the rows), reported beside the main figure ---
    plain = None
    if not args.skip_baseline_dynamic:
        eng.set_variant(B.A2_NO_MOMENTUM)
        p_plans, t_start = [], eng.times()
        for s in range(n_steps):
            c = ev_all.slice((3 * n_steps + s) * eps, (3 * n_steps + s + 1) * eps)
            p = eng.plan(c.times, c.wi, c.wj, c.slot, flags=flags, t_start=t_start)
            t_start = p.sched.t_final(cfg.n)
            p_plans.append(p)
        marks = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_steps)]
        q_end = torch.cuda.Event(enable_timing=True)
        p_bytes = p_launches = 0
        for s in range(n_steps):
            if s == W_:
                torch.cuda.synchronize(device)
                ranks.barrier()
            marks[s][0].record(stream)
            st = p_plans[s].run(want_stats=True)
            marks[s][1].record(stream)
            cons.append(eng.consensus_distance())
            if s >= W_:
                p_bytes += st["bytes_moved"]
                p_launches += st["n_launches"]
        q_end.record(stream)
        torch.cuda.synchronize(device)
        ranks.barrier()
        p_ms = marks[W_][0].elapsed_time(q_end)
        p_k1_ms = sum(marks[s][0].elapsed_time(marks[s][1]) for s in timed)
        for p in p_plans:
            p.close()
        eng.set_variant(B.A2_MSG_AFTER_MIX)
        p_value, p_slow = aggregate_throughput(ranks, K * eps, p_ms / 1e3)
        plain = {"value": p_value, "unit": "events/s", "ms_per_step": 1e3 * p_slow / K,
                 "kernel": "k_apply_events_plain", "achieved_gbs": p_bytes / (p_k1_ms / 1e3) / 1e9,
                 "launches": p_launches,
                 "note": "A2_NO_MOMENTUM: the paper's asynchronous baseline on the same stream recipe; x only, so "
                         "an event moves half the bytes"}
        if not all(np.isfinite(cons)):
            raise SystemExit("non-finite consensus distance: the run is invalid")

    # ---- roofline of the event kernel ------------------------------------------------------------
    peak, peak_src = measured_peak()
    achieved = k1_bytes / (k1_ms / 1e3) / 1e9
    per_launch_bytes = k1_bytes / max(1, k1_launches)
    roofline = {
        "kernel": "k_apply_events", "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
        "frac": achieved / peak, "peak_source": f"of {peak_src} copy bandwidth",
        "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
        "traffic": None if NCU_TRAFFIC_RATIO is None else NCU_TRAFFIC_RATIO * per_launch_bytes,
        "bytes_per_launch": per_launch_bytes, "avg_launch_ms": k1_ms / max(1, k1_launches), "launches": k1_launches,
        "effective_gbs_one_event_per_item": k1_bytes_single / (k1_ms / 1e3) / 1e9,
        "share_of_step_time": k1_ms / total_ms,
    }
    consensus_gbs = K * cfg.n * cfg.d * eng.elem_bytes / (k2_ms / 1e3) / 1e9

    line = {
        "metric": "gossip_events_per_s", "value": value, "unit": "events/s", "n_gpus": ranks.world, "steps": K,
        "warmup": W_, "ms_per_step": 1e3 * slowest_s / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: {cfg.note}", "n": cfg.n, "d": cfg.d, "graph": cfg.graph,
                   "storage": cfg.storage, "events_per_step": eps, "consensus_every_events": eps,
                   "gradient_fusion": not args.no_fuse, "item_chaining": not (args.no_fuse or args.no_chain), "parallelism": "replicas only" if ranks.world > 1 else "1 gpu",
                   "l2": "state 2*n*d*elem bytes per replica exceeds L2; no flush needed" if
                   2 * cfg.n * cfg.d * eng.elem_bytes > 3 * 126e6 else "state fits L2: figures are L2-assisted"},
        "clocks": clocks, "roofline": roofline,
        "e2e": {"value": e2e_value, "unit": "events/s", "h2d_bytes_per_step": int(np.mean(h2d)) if h2d else 0,
                "d2h_bytes_per_step": 8},
        "gpu_launches": int(k1_launches + 2 * K),
        "consensus_kernel": {"ms": k2_ms / K, "gbs": consensus_gbs, "frac": consensus_gbs / peak},
        "batches_per_step": sum(stats[s]["n_batches"] for s in timed) / K,
        "resident_mode": resident,
        "baseline_dynamic": plain,
    }
    if plain is not None:
        plain["frac"] = plain["achieved_gbs"] / peak

    if ranks.rank == 0 and ranks.world == 1 and not args.skip_cpu_baseline:
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
    eng.close()
    if ranks.rank == 0:
        print(json.dumps(line), flush=True)
    ranks.close()


if __name__ == "__main__":
    main()
