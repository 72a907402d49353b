"""Helpers of the GPU parity tests: build an engine for a workload, run it batch by batch and
compare with the CPU checker element by element.

fp32 storage -- bar 1e-5, element-wise, against the plain fp64 run. Metric, per row:
    max_k |gpu_k - ref_k| / max(|ref_k|, rms(ref row)),
a relative error whose denominator is floored by the row's root-mean-square, so that elements
that happen to pass near zero do not blow it up.

bf16 storage -- bar 2e-2, applied norm-wise against the plain fp64 run:
    |gpu_row - ref_row|_2 / |ref_row|_2 for every row of x and x~ (rows of >= 256 columns).
  Element-wise the bar is below what the storage format can hold: one bf16 store costs up to
  2^-8 = 3.9e-3 of an element, x~ integrates alpha~ times the rounding errors of x at every
  averaging, and an ideal bf16-storage run (fp64 arithmetic, exact round-to-nearest-even at
  every store) already sits at 3-6e-2 in the element-wise metric after a few hundred events
  (tests/test_oracle_pins.py::test_what_bf16_storage_alone_costs).
  So that a wrong element cannot hide inside a norm, every element is compared with the fp64 run
  *with the storage modelled* (the checker's rows rounded to bf16 at the engine's documented storage
  points, i.e. when an item's rows are written back), in bf16 units in the last place of the
  element's own magnitude:
      |gpu_k - ref_k| / ulp_bf16(max(|ref_k|, rms(ref row))),   ulp_bf16(v) = 2^(floor(log2 v) - 7).
  Two correct implementations that differ only in the precision of the arithmetic between two stores
  (fp32 on the GPU, fp64 in the checker) round a store to different neighbours once in a few thousand
  stores, and such one-ulp differences are then carried along like any perturbation. The bound is what
  tests/test_parity_bounds_cpu.py measures between two such implementations on the CPU (fp64 against
  NumPy float32 arithmetic: at most 4 ulps and 98 % of the elements identical after 10,000 events on
  2e5 elements, the tail falling tenfold per ulp), extended along that tail to the 3e9 elements of the
  full-size runs: BF16_ULP_BOUND = 8 ulps on any element, at least BF16_MIN_EXACT = 95 % of the
  elements bit-equal and BF16_MIN_WITHIN_1 = 99.5 % within one ulp (the two fractions on rows of
  >= 256 columns).
"""
from __future__ import annotations

import numpy as np

from oracle import spectral
from oracle.sim import OracleSim
from paper_2306_08289_b200 import binding as B
from paper_2306_08289_b200 import workload as W

TOL = {"f32": 1e-5, "bf16": 2e-2}
BF16_ULP_BOUND = 8.0
BF16_MIN_EXACT = 0.95
BF16_MIN_WITHIN_1 = 0.995
BF16_NORM_MIN_COLS = 256
TILE_COLS = {"f32": 256 * 8, "bf16": 256 * 8}  # columns per work unit of the event kernel


def rel_err(gpu, ref):
    ref = np.asarray(ref, dtype=np.float64)
    gpu = np.asarray(gpu, dtype=np.float64)
    rms = np.sqrt((ref * ref).mean(axis=1, keepdims=True))
    den = np.maximum(np.abs(ref), np.maximum(rms, 1e-300))
    return float((np.abs(gpu - ref) / den).max()) if ref.size else 0.0


def row_norm_err(gpu, ref):
    ref = np.asarray(ref, dtype=np.float64)
    gpu = np.asarray(gpu, dtype=np.float64)
    num = np.sqrt(((gpu - ref) ** 2).sum(axis=1))
    den = np.maximum(np.sqrt((ref * ref).sum(axis=1)), 1e-300)
    return float((num / den).max()) if ref.size else 0.0


def ulp_bf16(v):
    """Spacing of bfloat16 (8 significant bits) at magnitude v > 0."""
    return np.exp2(np.floor(np.log2(v)) - 7.0)


def bf16_ulp_distance(gpu, ref):
    """Per element: |gpu - ref| in bf16 ulps of max(|ref|, rms of ref's row)."""
    ref = np.asarray(ref, dtype=np.float64)
    gpu = np.asarray(gpu, dtype=np.float64)
    rms = np.sqrt((ref * ref).mean(axis=1, keepdims=True))
    mag = np.maximum(np.abs(ref), np.maximum(rms, 1e-300))
    return np.abs(gpu - ref) / ulp_bf16(mag)


def ulp_histogram(u):
    """Counts of elements off by exactly 0, at most 1, at most 2, and more than 2 ulps; and the maximum."""
    u = np.asarray(u)
    return {"n": int(u.size), "eq": int((u == 0).sum()), "le1": int((u <= 1).sum()), "le2": int((u <= 2).sum()),
            "gt2": int((u > 2).sum()), "max": float(u.max()) if u.size else 0.0}


def widen(a, storage):
    return W.bf16_bits_to_f32(a).astype(np.float64) if storage == "bf16" else np.asarray(a, dtype=np.float64)


def oracle_params(cfg):
    if cfg.fixed_params is not None:
        return tuple(float(v) for v in cfg.fixed_params)
    return tuple(float(v) for v in spectral.prescribe(cfg.n, cfg.edges(), cfg.rates())[:3])


def per_event_groups(ev):
    """Rounding points of an implementation that stores the rows of an event's workers after every event:
    (group_end, worker_ptr, workers) for OracleSim.apply_groups."""
    n = len(ev)
    comm = ev.wj >= 0
    ptr = np.concatenate([[0], np.cumsum(1 + comm.astype(np.int64))])
    workers = np.empty(int(ptr[-1]), dtype=np.int32)
    workers[ptr[:-1]] = ev.wi
    workers[ptr[:-1][comm] + 1] = ev.wj[comm]
    return np.arange(1, n + 1, dtype=np.int64), ptr.astype(np.int64), workers


def storage_only_error(cfg, fmt, x0=None, G=None, ev=None):
    """Element-wise error (the metric of the fp32 parity tests) of a run whose arithmetic is fp64 and
    whose only loss is that the rows of an event's workers are rounded to `fmt` ("f32" or "bf16") when
    they are stored, once per event: what an ideal implementation with that storage format delivers.
    x0, G: widened inputs (default: the configuration's own, all columns)."""
    if x0 is None:
        _, x0 = W.x0_matrix(cfg)
        _, G = W.grad_matrix(cfg)
    if ev is None:
        ev = W.config_events(cfg)
    par = oracle_params(cfg)
    plain = OracleSim(x0, *par, cfg.gamma, grads=G)
    stored = OracleSim(x0, *par, cfg.gamma, grads=G)
    plain.apply_stream(ev)
    stored.apply_groups(ev.times, ev.wi, ev.wj, ev.slot, *per_event_groups(ev), fmt=fmt)
    return max(rel_err(stored.X, plain.X), rel_err(stored.Xt, plain.Xt))


class _XOnly:
    """View of a simulator in which x stands in for x~ too, for engines that hold x alone."""

    def __init__(self, sim):
        self.X = sim.X
        self.Xt = sim.X
        self.t = sim.t


class Checker:
    """The fp64 run, plus (bf16 storage only) a second fp64 run whose rows are rounded to bf16
    wherever the engine stores them."""

    def __init__(self, x0, params, gamma, grads, storage, variant=0):
        self.storage = storage
        self.plain = OracleSim(x0, *params, gamma, grads=grads, variant=variant)
        self.stored = OracleSim(x0, *params, gamma, grads=grads, variant=variant) if storage == "bf16" else None

    def apply_batch(self, ev, sched, b):
        idx = sched.batch_events(b)
        order = idx[np.argsort(ev.times[idx], kind="stable")]
        self.plain.apply(ev.times[order], ev.wi[order], ev.wj[order], ev.slot[order])
        if self.stored is not None:
            first, cnt = sched.batch_items(b)
            for k in range(first, first + cnt):
                it = sched.item(k)
                e, _ = sched.ops(it.first_op, it.n_ops)
                e = e[np.argsort(ev.times[e], kind="stable")]
                self.stored.apply(ev.times[e], ev.wi[e], ev.wj[e], ev.slot[e])
                self.stored.round_rows(it.workers())

    def compare(self, x, xt, t, where="", cols=None):
        """x, xt: widened device state (optionally only the columns `cols` of the checker). xt = None
        (an engine without a momentum buffer): x alone is compared."""
        pl, st = self.plain, self.stored
        sel = (lambda a: a) if cols is None else (lambda a: a[:, cols])
        assert np.array_equal(t, pl.t), f"times differ {where}"
        if xt is None:
            xt = x
            pl = _XOnly(pl)
            st = None if st is None else _XOnly(st)
        out = {"elem_plain": max(rel_err(x, sel(pl.X)), rel_err(xt, sel(pl.Xt)))}
        if st is None:
            assert out["elem_plain"] <= TOL["f32"], f"parity {where}: {out}"
        else:
            out["norm_plain"] = max(row_norm_err(x, sel(pl.X)), row_norm_err(xt, sel(pl.Xt)))
            u = np.concatenate([bf16_ulp_distance(x, sel(st.X)).ravel(), bf16_ulp_distance(xt, sel(st.Xt)).ravel()])
            h = ulp_histogram(u)
            out["ulps_stored_max"] = h["max"]
            out["not_exact"] = 1.0 - h["eq"] / max(1, h["n"])
            out["beyond_1_ulp"] = 1.0 - h["le1"] / max(1, h["n"])
            self.last_histogram = h
            assert h["max"] <= BF16_ULP_BOUND, f"parity {where}: {out}"
            if x.shape[1] >= BF16_NORM_MIN_COLS:
                assert out["norm_plain"] <= TOL["bf16"], f"parity {where}: {out}"
                assert out["not_exact"] <= 1.0 - BF16_MIN_EXACT, f"parity {where}: {out}"
                assert out["beyond_1_ulp"] <= 1.0 - BF16_MIN_WITHIN_1, f"parity {where}: {out}"
        return out


def make_small(cfg, variant=0, momentum=True):
    """Engine + checker for a configuration whose arrays fit the host: same stored inputs on both.
    momentum=False: an engine with no x~ buffer (the variant is then A2_NO_MOMENTUM)."""
    xs, xw = W.x0_matrix(cfg)
    gs, gw = W.grad_matrix(cfg)
    if not momentum:
        variant = B.A2_NO_MOMENTUM
    eng = B.Engine(cfg.n, cfg.d, *B.config_params(cfg), cfg.gamma, storage=cfg.storage, n_grad_slots=cfg.n_grad_slots,
                   momentum=momentum)
    eng.write_state(xs)
    eng.write_grads(gs)
    if variant and momentum:
        eng.set_variant(variant)
    chk = Checker(xw, oracle_params(cfg), cfg.gamma, gw, cfg.storage, variant=variant)
    return eng, chk


def _merge(worst, out):
    for k, v in out.items():
        worst[k] = max(worst.get(k, 0.0), v)


def run_batches_and_check(eng, chk, ev, flags, every=1):
    """Plan the stream, run it one batch at a time; advance the checker through the same events
    (sorted by time inside the batch) and, after every `every`-th batch and the last, compare the
    whole stored state."""
    worst = {}
    plan = eng.plan(ev.times, ev.wi, ev.wj, ev.slot, flags=flags)
    nb = plan.sched.num_batches
    for b in range(nb):
        plan.run(b, 1)
        chk.apply_batch(ev, plan.sched, b)
        if b % every == 0 or b == nb - 1:
            x, xt, t = eng.read_state()
            _merge(worst, chk.compare(widen(x, chk.storage), None if xt is None else widen(xt, chk.storage), t,
                                      where=f"after batch {b}/{nb}"))
    plan.close()
    return worst, nb
