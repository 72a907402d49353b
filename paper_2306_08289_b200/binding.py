"""Thin ctypes binding of liba2cid2.so: argument marshalling only.

Every function of include/a2cid2.h is exposed under its own name through `lib()`; the
classes below only keep handles alive and convert NumPy arrays / torch tensors to pointers.
All arithmetic of the update runs in the library's CUDA kernels. If the shared library is
missing, `lib()` raises: there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import math
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "liba2cid2.so")

A2_OK, A2_EINVAL, A2_EORDER, A2_ERANGE, A2_ENOMEM, A2_ECUDA, A2_ESTATE = 0, -1, -2, -3, -4, -5, -6
A2_F32, A2_BF16 = 0, 1
A2_SCHED_FUSE = 1
A2_SCHED_RESIDENT = 2
A2_SCHED_CHAIN = 4
A2_SCHED_ROW_PER_OP = 8
A2_OP_GRAD_A, A2_OP_GRAD_B, A2_OP_COMM, A2_OP_MIX_A, A2_OP_GRAD_C, A2_OP_COMM_AC, A2_OP_COMM_BC = 0, 1, 2, 3, 4, 5, 6
A2_OP_GRAD_D, A2_OP_COMM_AD, A2_OP_COMM_BD, A2_OP_COMM_CD = 7, 8, 9, 10
A2_MSG_AFTER_MIX, A2_MSG_BEFORE_MIX, A2_NO_MOMENTUM = 0, 1, 2
A2_LAUNCH_AUTO, A2_LAUNCH_PER_BATCH, A2_LAUNCH_COLUMN_SLICES = 0, 1, 2
A2_ROUND_PER_EVENT, A2_ROUND_PER_STORE = 0, 1

ERROR_NAMES = {A2_EINVAL: "A2_EINVAL", A2_EORDER: "A2_EORDER", A2_ERANGE: "A2_ERANGE", A2_ENOMEM: "A2_ENOMEM",
               A2_ECUDA: "A2_ECUDA", A2_ESTATE: "A2_ESTATE"}


class ItemInfo(C.Structure):
    _fields_ = [("a", C.c_int32), ("b", C.c_int32), ("slot_a", C.c_int32), ("slot_b", C.c_int32),
                ("first_op", C.c_int64), ("n_ops", C.c_int32), ("batch", C.c_int32),
                ("c", C.c_int32), ("slot_c", C.c_int32), ("d", C.c_int32), ("slot_d", C.c_int32)]

    def workers(self):
        return [w for w in (self.a, self.b, self.c, self.d) if w >= 0]


class Stats(C.Structure):
    _fields_ = [("n_events", C.c_int64), ("n_comm", C.c_int64), ("n_grad", C.c_int64),
                ("n_batches", C.c_int64), ("n_launches", C.c_int64), ("n_items", C.c_int64),
                ("bytes_moved", C.c_int64), ("bytes_one_by_one", C.c_int64), ("descriptor_bytes", C.c_int64),
                ("host_ms", C.c_double)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


class A2Error(RuntimeError):
    def __init__(self, code, text):
        super().__init__(f"{ERROR_NAMES.get(code, code)}: {text}")
        self.code = code


_dp = C.POINTER(C.c_double)
_ip = C.POINTER(C.c_int32)
_lp = C.POINTER(C.c_int64)
_vp = C.c_void_p

# name -> (restype, argtypes); mirrors include/a2cid2.h one to one
SIGNATURES = {
    "a2cid2_create": (C.c_int, [C.c_int32, C.c_int64, C.c_double, C.c_double, C.c_double, C.c_double, C.c_int32, C.POINTER(_vp)]),
    "a2cid2_set_variant": (C.c_int, [_vp, C.c_int32]),
    "a2cid2_set_launch_mode": (C.c_int, [_vp, C.c_int32]),
    "a2cid2_set_rounding": (C.c_int, [_vp, C.c_int32]),
    "a2cid2_bind": (C.c_int, [_vp, _vp, _vp, _vp, C.c_int32, C.c_int64, _vp]),
    "a2cid2_write_state": (C.c_int, [_vp, _vp, _vp, _dp]),
    "a2cid2_write_grads": (C.c_int, [_vp, C.c_int32, C.c_int32, _vp]),
    "a2cid2_read_state": (C.c_int, [_vp, _vp, _vp, _dp]),
    "a2cid2_times": (C.c_int, [_vp, _dp]),
    "a2cid2_set_times": (C.c_int, [_vp, _dp]),
    "a2cid2_apply_events": (C.c_int, [_vp, C.c_int64, _dp, _ip, _ip, _ip, C.c_uint32, C.POINTER(Stats)]),
    "a2cid2_flush": (C.c_int, [_vp, C.c_double]),
    "a2cid2_consensus_distance": (C.c_int, [_vp, C.c_double, _dp]),
    "a2cid2_consensus_distance_static": (C.c_int, [_vp, C.c_int32, C.c_int64, C.c_int64, C.c_int32, _vp, _vp]),
    "a2cid2_sync": (C.c_int, [_vp]),
    "a2cid2_last_error": (C.c_char_p, [_vp]),
    "a2cid2_destroy": (None, [_vp]),
    "a2cid2_plan_create": (C.c_int, [_vp, _dp, C.c_int64, _dp, _ip, _ip, _ip, C.c_uint32, C.POINTER(_vp)]),
    "a2cid2_plan_sched": (_vp, [_vp]),
    "a2cid2_plan_run": (C.c_int, [_vp, _vp, C.c_int64, C.c_int64, C.POINTER(Stats)]),
    "a2cid2_plan_destroy": (None, [_vp]),
    "a2cid2_sched_create": (C.c_int, [C.c_int32, C.c_int32, _dp, C.c_int64, _dp, _ip, _ip, _ip, C.c_uint32, C.c_int32, C.c_int32,
                                      C.POINTER(_vp)]),
    "a2cid2_sched_num_batches": (C.c_int64, [_vp]),
    "a2cid2_sched_num_items": (C.c_int64, [_vp]),
    "a2cid2_sched_num_ops": (C.c_int64, [_vp]),
    "a2cid2_sched_batch_items": (C.c_int, [_vp, C.c_int64, _lp, _lp]),
    "a2cid2_sched_item": (C.c_int, [_vp, C.c_int64, C.POINTER(ItemInfo)]),
    "a2cid2_sched_ops": (C.c_int, [_vp, C.c_int64, C.c_int64, _lp, _ip]),
    "a2cid2_sched_op_reloads": (C.c_int, [_vp, C.c_int64, C.c_int64, _ip]),
    "a2cid2_sched_t_final": (C.c_int, [_vp, _dp]),
    "a2cid2_sched_stats": (C.c_int, [_vp, C.c_int64, C.c_int64, C.c_int64, C.c_int32, C.POINTER(Stats)]),
    "a2cid2_sched_destroy": (None, [_vp]),
    "a2cid2_graph_chi": (C.c_int, [C.c_int32, C.c_int64, _ip, _ip, _dp, _dp, _dp]),
    "a2cid2_prescribe": (C.c_int, [C.c_double, C.c_double, C.c_int32, _dp, _dp, _dp]),
    "a2cid2_version": (C.c_char_p, []),
}

_lib = None


def lib():
    """The loaded shared library with typed signatures. Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2306_08289_b200.build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def _check(code, handle=None):
    if code != A2_OK:
        raise A2Error(code, lib().a2cid2_last_error(handle).decode())


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _ptr(a, typ):
    return a.ctypes.data_as(typ)


# ---------------------------------------------------------------------------------------------
# host-only pieces
# ---------------------------------------------------------------------------------------------
def graph_chi(n, edges, rates):
    edges = np.asarray(edges, dtype=np.int32).reshape(-1, 2)
    ei, ej, lam = _i32(edges[:, 0]), _i32(edges[:, 1]), _f64(rates)
    c1, c2 = C.c_double(), C.c_double()
    _check(lib().a2cid2_graph_chi(n, len(ei), _ptr(ei, _ip), _ptr(ej, _ip), _ptr(lam, _dp), C.byref(c1), C.byref(c2)))
    return c1.value, c2.value


def prescribe(chi1, chi2, accelerated=True):
    eta, alpha, at = C.c_double(), C.c_double(), C.c_double()
    _check(lib().a2cid2_prescribe(chi1, chi2, 1 if accelerated else 0, C.byref(eta), C.byref(alpha), C.byref(at)))
    return eta.value, alpha.value, at.value


def config_params(cfg):
    """(eta, alpha, alpha_tilde) of a workload configuration: the values it fixes outright, else
    the prescription of the convergence proposition of Sec. 3.4 evaluated by the library on the configuration's graph."""
    if cfg.fixed_params is not None:
        return tuple(float(v) for v in cfg.fixed_params)
    c1, c2 = graph_chi(cfg.n, cfg.edges(), cfg.rates())
    return prescribe(c1, c2, True)


def consensus_distance_static(x_ptr, n, d, row_pitch_elems, storage_dtype, cuda_stream, out_device_ptr):
    """a2cid2_consensus_distance_static: consensus distance of the rows at device address x_ptr,
    queued on cuda_stream, result written to the device double at out_device_ptr. For callers
    that may not allocate: the call itself allocates nothing (see include/a2cid2.h)."""
    _check(lib().a2cid2_consensus_distance_static(x_ptr, n, d, row_pitch_elems, storage_dtype, cuda_stream,
                                                  out_device_ptr))


class Schedule:
    """a2cid2_sched_* : batches of worker-disjoint items for an event stream (host only)."""

    def __init__(self, n, n_grad_slots, times, wi, wj, slot, flags=0, t_last=None, max_ops_per_item=0,
                 max_workers_per_item=0, _borrowed=None):
        self._owned = _borrowed is None
        if _borrowed is not None:
            self._h = _borrowed
            return
        times, wi, wj, slot = _f64(times), _i32(wi), _i32(wj), _i32(slot)
        tl = None if t_last is None else _f64(t_last)
        h = _vp()
        _check(lib().a2cid2_sched_create(n, n_grad_slots, None if tl is None else _ptr(tl, _dp), len(times),
                                         _ptr(times, _dp), _ptr(wi, _ip), _ptr(wj, _ip), _ptr(slot, _ip),
                                         flags, max_ops_per_item, max_workers_per_item, C.byref(h)))
        self._h = h
        self.n = n

    @property
    def num_batches(self):
        return lib().a2cid2_sched_num_batches(self._h)

    @property
    def num_items(self):
        return lib().a2cid2_sched_num_items(self._h)

    @property
    def num_ops(self):
        return lib().a2cid2_sched_num_ops(self._h)

    def batch_items(self, b):
        first, cnt = C.c_int64(), C.c_int64()
        _check(lib().a2cid2_sched_batch_items(self._h, b, C.byref(first), C.byref(cnt)))
        return first.value, cnt.value

    def item(self, k):
        info = ItemInfo()
        _check(lib().a2cid2_sched_item(self._h, k, C.byref(info)))
        return info

    def ops(self, first_op, n_ops):
        ev = np.empty(n_ops, dtype=np.int64)
        kind = np.empty(n_ops, dtype=np.int32)
        _check(lib().a2cid2_sched_ops(self._h, first_op, n_ops, _ptr(ev, _lp), _ptr(kind, _ip)))
        return ev, kind

    def op_reloads(self, first_op, n_ops):
        """Per operation: the gradient row fetched into the worker's registers after it, or -1."""
        out = np.empty(n_ops, dtype=np.int32)
        _check(lib().a2cid2_sched_op_reloads(self._h, first_op, n_ops, _ptr(out, _ip)))
        return out

    def batch_events(self, b):
        """Event indices applied by batch b, item by item, in the order they are applied."""
        first, cnt = self.batch_items(b)
        if cnt == 0:
            return np.empty(0, dtype=np.int64)
        i0, i1 = self.item(first), self.item(first + cnt - 1)
        ev, _ = self.ops(i0.first_op, i1.first_op + i1.n_ops - i0.first_op)
        return ev

    def t_final(self, n):
        out = np.empty(n, dtype=np.float64)
        _check(lib().a2cid2_sched_t_final(self._h, _ptr(out, _dp)))
        return out

    def stats(self, d, elem_bytes, first_batch=0, n_batches=-1):
        st = Stats()
        _check(lib().a2cid2_sched_stats(self._h, first_batch, n_batches, d, elem_bytes, C.byref(st)))
        return st.as_dict()

    def close(self):
        if self._owned and self._h:
            lib().a2cid2_sched_destroy(self._h)
        self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ---------------------------------------------------------------------------------------------
# engine
# ---------------------------------------------------------------------------------------------
class Plan:
    def __init__(self, engine, handle):
        self.engine = engine
        self._h = handle
        self.sched = Schedule(0, 0, None, None, None, None, _borrowed=_vp(lib().a2cid2_plan_sched(handle)))

    def run(self, first_batch=0, n_batches=-1, want_stats=False):
        st = Stats() if want_stats else None
        _check(lib().a2cid2_plan_run(self.engine._h, self._h, first_batch, n_batches,
                                     C.byref(st) if want_stats else None), self.engine._h)
        return st.as_dict() if want_stats else None

    def close(self):
        if self._h:
            lib().a2cid2_plan_destroy(self._h)
        self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Engine:
    """a2cid2_create + a2cid2_bind on buffers allocated through torch (device memory and
    stream only). x, x~ and the gradient buffer are torch tensors of shape [rows, pitch]."""

    def __init__(self, n, d, eta, alpha, alpha_tilde, gamma, storage="f32", n_grad_slots=None, device="cuda:0",
                 stream=None, rows_16B_only=False, momentum=True):
        import torch

        self.torch = torch
        self.n, self.d = int(n), int(d)
        self.storage = storage
        self.dtype_code = A2_BF16 if storage == "bf16" else A2_F32
        self.np_dtype = np.uint16 if storage == "bf16" else np.float32
        self.elem_bytes = 2 if storage == "bf16" else 4
        self.torch_dtype = torch.bfloat16 if storage == "bf16" else torch.float32
        self._h = None
        h = _vp()
        _check(lib().a2cid2_create(self.n, self.d, eta, alpha, alpha_tilde, gamma, self.dtype_code, C.byref(h)))
        self._h = h
        self.momentum = bool(momentum)  # False: the dynamic without x~ (A2_NO_MOMENTUM), no x~ buffer at all
        if not self.momentum:
            _check(lib().a2cid2_set_variant(self._h, A2_NO_MOMENTUM), self._h)
        self.device = torch.device(device)
        # rows start on 32-byte boundaries so that the kernels can use 256-bit accesses
        # (rows_16B_only: start them 16 bytes off instead, which is all the ABI requires)
        q = 32 // self.elem_bytes
        self.pitch = (self.d + q - 1) // q * q
        shift = 16 // self.elem_bytes if rows_16B_only else 0
        self.n_slots = self.n if n_grad_slots is None else int(n_grad_slots)
        with torch.cuda.device(self.device):
            def rows(r):
                flat = torch.zeros(r * self.pitch + shift, dtype=self.torch_dtype, device=self.device)
                return flat[shift:].view(r, self.pitch)

            self.x = rows(self.n)
            self.xt = rows(self.n) if self.momentum else None
            self.g = rows(max(self.n_slots, 1))
            self.stream = torch.cuda.current_stream(self.device) if stream is None else stream
            _check(lib().a2cid2_bind(self._h, self.x.data_ptr(), self.xt.data_ptr() if self.momentum else None,
                                     self.g.data_ptr() if self.n_slots > 0 else None, self.n_slots, self.pitch,
                                     self.stream.cuda_stream), self._h)

    # -- state ---------------------------------------------------------------------------------
    def set_variant(self, variant):
        _check(lib().a2cid2_set_variant(self._h, variant), self._h)

    def set_launch_mode(self, mode):
        _check(lib().a2cid2_set_launch_mode(self._h, mode), self._h)

    def set_rounding(self, mode):
        _check(lib().a2cid2_set_rounding(self._h, mode), self._h)

    def write_state(self, x, x_tilde=None, t=None):
        x = np.ascontiguousarray(x, dtype=self.np_dtype)
        assert x.shape == (self.n, self.d)
        xt = None if x_tilde is None else np.ascontiguousarray(x_tilde, dtype=self.np_dtype)
        tt = None if t is None else _f64(t)
        _check(lib().a2cid2_write_state(self._h, x.ctypes.data, None if xt is None else xt.ctypes.data,
                                        None if tt is None else _ptr(tt, _dp)), self._h)

    def write_grads(self, g, first_slot=0):
        g = np.ascontiguousarray(g, dtype=self.np_dtype)
        assert g.ndim == 2 and g.shape[1] == self.d
        _check(lib().a2cid2_write_grads(self._h, first_slot, g.shape[0], g.ctypes.data), self._h)

    def read_state(self):
        x = np.empty((self.n, self.d), dtype=self.np_dtype)
        xt = np.empty((self.n, self.d), dtype=self.np_dtype) if self.xt is not None else None
        t = np.empty(self.n, dtype=np.float64)
        _check(lib().a2cid2_read_state(self._h, x.ctypes.data, None if xt is None else xt.ctypes.data, _ptr(t, _dp)),
               self._h)
        return x, xt, t

    def times(self):
        t = np.empty(self.n, dtype=np.float64)
        _check(lib().a2cid2_times(self._h, _ptr(t, _dp)), self._h)
        return t

    def set_times(self, t):
        t = _f64(t)
        assert t.shape == (self.n,)
        _check(lib().a2cid2_set_times(self._h, _ptr(t, _dp)), self._h)

    def fill_row(self, which, row, stored):
        """Copy one host row (storage precision: float32, or uint16 bf16 bit patterns) into
        x ('x'), x~ ('xt') or the gradient buffer ('g') through torch: memory plumbing for
        inputs too large to stage as one dense host array."""
        torch = self.torch
        buf = {"x": self.x, "xt": self.xt, "g": self.g}[which]
        src = torch.from_numpy(np.ascontiguousarray(stored))
        if self.storage == "bf16":
            src = src.view(torch.bfloat16)
        buf[row, : self.d].copy_(src, non_blocking=False)

    # -- events --------------------------------------------------------------------------------
    def apply_events(self, times, wi, wj, slot, flags=0, want_stats=False):
        times, wi, wj, slot = _f64(times), _i32(wi), _i32(wj), _i32(slot)
        st = Stats() if want_stats else None
        _check(lib().a2cid2_apply_events(self._h, len(times), _ptr(times, _dp), _ptr(wi, _ip), _ptr(wj, _ip),
                                         _ptr(slot, _ip), flags, C.byref(st) if want_stats else None), self._h)
        return st.as_dict() if want_stats else None

    def plan(self, times, wi, wj, slot, flags=0, t_start=None):
        times, wi, wj, slot = _f64(times), _i32(wi), _i32(wj), _i32(slot)
        ts = None if t_start is None else _f64(t_start)
        p = _vp()
        _check(lib().a2cid2_plan_create(self._h, None if ts is None else _ptr(ts, _dp), len(times), _ptr(times, _dp),
                                        _ptr(wi, _ip), _ptr(wj, _ip), _ptr(slot, _ip), flags, C.byref(p)), self._h)
        return Plan(self, p)

    def flush(self, t_flush):
        _check(lib().a2cid2_flush(self._h, float(t_flush)), self._h)

    def consensus_distance(self, t_eval=None):
        out = C.c_double()
        _check(lib().a2cid2_consensus_distance(self._h, math.nan if t_eval is None else float(t_eval), C.byref(out)),
               self._h)
        return out.value

    def sync(self):
        _check(lib().a2cid2_sync(self._h), self._h)

    def close(self):
        if self._h:
            lib().a2cid2_destroy(self._h)
        self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
