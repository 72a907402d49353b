"""Sequential fp64 simulator backed by a2cid2_oracle.c -- TEST INFRASTRUCTURE.

Follows Eq. (dynamic) of Sec. 3.2 event by event in time order; see the C file's header for
the passage behind each step."""
from __future__ import annotations

import ctypes as C
from concurrent.futures import ThreadPoolExecutor

import numpy as np

from . import build as _build

_lib = None


def load(path):
    """Load a build of the C checker and declare its signatures."""
    if True:
        L = C.CDLL(path)
        dp, ip = C.POINTER(C.c_double), C.POINTER(C.c_int32)
        L.a2o_mix_coeff.restype = C.c_double
        L.a2o_mix_coeff.argtypes = [C.c_double, C.c_double]
        L.a2o_run.restype = C.c_int
        L.a2o_run.argtypes = [C.c_int32, C.c_int64, C.c_int64, C.c_double, C.c_double, C.c_double, C.c_double,
                              dp, dp, dp, dp, C.c_int32, C.c_int64,
                              C.c_int64, dp, ip, ip, ip, C.c_int32]
        lp = C.POINTER(C.c_int64)
        L.a2o_to_bf16.restype = C.c_double
        L.a2o_to_bf16.argtypes = [C.c_double]
        L.a2o_run_groups.restype = C.c_int
        L.a2o_run_groups.argtypes = [C.c_int32, C.c_int64, C.c_int64, C.c_double, C.c_double, C.c_double, C.c_double,
                                     dp, dp, dp, dp, C.c_int32, C.c_int64, dp, ip, ip, ip, C.c_int32,
                                     C.c_int64, lp, lp, ip, C.c_int32]
        L.a2o_consensus.restype = C.c_double
        L.a2o_consensus.argtypes = [C.c_int32, C.c_int64, C.c_int64, dp]
        L.a2o_consensus_at.restype = C.c_double
        L.a2o_consensus_at.argtypes = [C.c_int32, C.c_int64, C.c_int64, C.c_double, dp, dp, dp, C.c_double]
    return L


def lib():
    global _lib
    if _lib is None:
        _lib = load(_build.build())
    return _lib


def _dp(a, off=0):
    return C.cast(a.ctypes.data + 8 * off, C.POINTER(C.c_double))


def _ip(a):
    return a.ctypes.data_as(C.POINTER(C.c_int32))


class OracleError(RuntimeError):
    pass


def round_to_bf16(a):
    """Values of `a` (float64) rounded to bfloat16 -- 8 exponent bits, 7 stored mantissa bits,
    i.e. the upper half of an IEEE binary32 -- with round-to-nearest-even, returned as float64.
    The value is first rounded to binary32 (also nearest-even). Finite inputs only."""
    u = np.ascontiguousarray(a, dtype=np.float64).astype(np.float32).view(np.uint32).astype(np.uint64)
    keep_odd = (u >> np.uint64(16)) & np.uint64(1)
    u = (u + np.uint64(0x7FFF) + keep_odd) >> np.uint64(16) << np.uint64(16)
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(a))


class OracleSim:
    """State: X, Xt of shape [n, d] (fp64), t_last[n]. Initialisation as in Algorithm 1:
    x~ <- x, t <- 0, unless given."""

    def __init__(self, x0, eta, alpha, alpha_tilde, gamma, grads=None, xt0=None, t0=None, variant=0):
        self.X = np.array(x0, dtype=np.float64, order="C")
        self.n, self.d = self.X.shape
        self.Xt = self.X.copy() if xt0 is None else np.array(xt0, dtype=np.float64, order="C")
        self.t = np.zeros(self.n) if t0 is None else np.array(t0, dtype=np.float64)
        self.G = None if grads is None else np.array(grads, dtype=np.float64, order="C")
        self.eta, self.alpha, self.alpha_tilde, self.gamma = float(eta), float(alpha), float(alpha_tilde), float(gamma)
        self.variant = int(variant)

    def _run_cols(self, c0, c1, tl, times, wi, wj, slot):
        G = self.G if self.G is not None else np.zeros((1, self.d))
        rc = lib().a2o_run(self.n, c1 - c0, self.d, self.eta, self.alpha, self.alpha_tilde, self.gamma,
                           _dp(self.X, c0), _dp(self.Xt, c0), _dp(tl), _dp(G, c0), G.shape[0], self.d,
                           len(times), _dp(times), _ip(wi), _ip(wj), _ip(slot), self.variant)
        return rc

    def apply(self, times, wi, wj, slot, threads=1):
        """Apply events in the order given. threads > 1 splits the *columns* over threads
        (columns never interact); every slice still sees the events in the same order."""
        times = np.ascontiguousarray(times, dtype=np.float64)
        wi = np.ascontiguousarray(wi, dtype=np.int32)
        wj = np.ascontiguousarray(wj, dtype=np.int32)
        slot = np.ascontiguousarray(slot, dtype=np.int32)
        if len(times) == 0:
            return
        if threads <= 1 or self.d < threads:
            rc = self._run_cols(0, self.d, self.t, times, wi, wj, slot)
            if rc != 0:
                raise OracleError(f"a2o_run -> {rc}")
            return
        bounds = np.linspace(0, self.d, threads + 1).astype(np.int64)
        tls = [self.t.copy() for _ in range(threads)]
        with ThreadPoolExecutor(threads) as ex:
            rcs = list(ex.map(lambda k: self._run_cols(int(bounds[k]), int(bounds[k + 1]), tls[k],
                                                       times, wi, wj, slot), range(threads)))
        if any(rcs):
            raise OracleError(f"a2o_run -> {rcs}")
        self.t[:] = tls[0]

    def apply_groups(self, times, wi, wj, slot, group_end, worker_ptr, workers, fmt="bf16"):
        """Storage model over a whole schedule in one call: the events (already in the order they are to be
        applied) come in consecutive groups ending at group_end[k]; after group k the rows of
        workers[worker_ptr[k]:worker_ptr[k+1]] are rounded to the storage format ("bf16" or "f32"). Equal to
        apply() on each group followed by round_rows() on its workers."""
        times = np.ascontiguousarray(times, dtype=np.float64)
        wi = np.ascontiguousarray(wi, dtype=np.int32)
        wj = np.ascontiguousarray(wj, dtype=np.int32)
        slot = np.ascontiguousarray(slot, dtype=np.int32)
        group_end = np.ascontiguousarray(group_end, dtype=np.int64)
        worker_ptr = np.ascontiguousarray(worker_ptr, dtype=np.int64)
        workers = np.ascontiguousarray(workers, dtype=np.int32)
        assert len(worker_ptr) == len(group_end) + 1 and (len(group_end) == 0 or group_end[-1] == len(times))
        G = self.G if self.G is not None else np.zeros((1, self.d))
        lp = C.POINTER(C.c_int64)
        rc = lib().a2o_run_groups(self.n, self.d, self.d, self.eta, self.alpha, self.alpha_tilde, self.gamma,
                                  _dp(self.X), _dp(self.Xt), _dp(self.t), _dp(G), G.shape[0], self.d,
                                  _dp(times), _ip(wi), _ip(wj), _ip(slot), self.variant, len(group_end),
                                  group_end.ctypes.data_as(lp), worker_ptr.ctypes.data_as(lp), _ip(workers),
                                  {"bf16": 0, "f32": 1}[fmt])
        if rc != 0:
            raise OracleError(f"a2o_run_groups -> {rc}")

    def apply_stream(self, ev, threads=1):
        self.apply(ev.times, ev.wi, ev.wj, ev.slot, threads=threads)

    def flush(self, t_flush):
        """Every worker mixed forward to the common time t_flush, in place: the state Algorithm 1
        returns at the end of training."""
        if np.any(self.t > t_flush):
            raise OracleError("flush time precedes a worker's last event")
        self.X, self.Xt = self.flushed(t_flush)
        self.t[:] = t_flush

    def round_rows(self, workers, fmt="bf16", which=("x", "xt")):
        """Model of reduced-precision *storage*: the rows of these workers are rounded to the storage
        format (bfloat16, or IEEE binary32 with fmt="f32"; both to nearest even), as happens whenever
        an implementation that keeps its state in that format writes them back. The arithmetic
        between two stores stays fp64. `which` restricts the rounding to x or to x~ (to see which
        of the two buffers' roundings an error comes from)."""
        w = np.unique(np.asarray(workers, dtype=np.int64))
        if fmt == "bf16":
            rnd = round_to_bf16
        elif fmt == "f32":
            rnd = lambda a: a.astype(np.float32).astype(np.float64)  # noqa: E731
        else:
            raise ValueError(fmt)
        if "x" in which:
            self.X[w] = rnd(self.X[w])
        if "xt" in which:
            self.Xt[w] = rnd(self.Xt[w])

    def consensus(self, t_eval=None):
        if t_eval is None:
            return float(lib().a2o_consensus(self.n, self.d, self.d, _dp(self.X)))
        return float(lib().a2o_consensus_at(self.n, self.d, self.d, self.eta, _dp(self.X), _dp(self.Xt),
                                            _dp(self.t), float(t_eval)))

    def flushed(self, t_eval):
        """(x, x~) of every worker mixed forward to the common time t_eval (copies)."""
        c = np.array([lib().a2o_mix_coeff(self.eta, float(t_eval) - ti) for ti in self.t])[:, None]
        dlt = self.X - self.Xt
        return self.X - c * dlt, self.Xt + c * dlt
