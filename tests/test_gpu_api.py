"""The C ABI on a device: state round trips, checkpoint/resume, plans, error behaviour.
Bad input must come back as an error code with the state untouched; nothing here can fault
the device (every rejection happens on the host before any launch)."""
import ctypes as C
import math

import numpy as np
import pytest

from paper_2306_08289_b200 import binding as B
from paper_2306_08289_b200 import workload as W
from tests import parity as P

pytestmark = pytest.mark.gpu


def _small(storage="f32", d=1234, n_events=800):
    cfg = W.CONFIGS["cfg3"].scaled(d=d, n_events=n_events)
    if storage != cfg.storage:
        cfg = W.WorkloadConfig(**{**cfg.__dict__, "storage": storage})
    return cfg


@pytest.mark.parametrize("storage", ["f32", "bf16"])
def test_state_round_trip_and_padding(storage):
    cfg = _small(storage, d=1001)
    xs, _ = W.x0_matrix(cfg)
    gs, _ = W.grad_matrix(cfg)
    eng = B.Engine(cfg.n, cfg.d, 0.3, 0.5, 1.1, 0.1, storage=storage)
    assert eng.pitch == (1008 if storage == "f32" else 1008)
    eng.write_state(xs)
    x, xt, t = eng.read_state()
    assert np.array_equal(x, xs) and np.array_equal(xt, xs) and np.array_equal(t, np.zeros(cfg.n))
    tt = np.linspace(0.5, 2.0, cfg.n)
    eng.write_state(xs, gs, tt)  # explicit x~ and times
    x, xt, t = eng.read_state()
    assert np.array_equal(x, xs) and np.array_equal(xt, gs) and np.array_equal(t, tt)
    assert np.array_equal(eng.times(), tt)
    eng.close()


def test_checkpoint_and_resume_is_exact():
    cfg = _small()
    ev = W.config_events(cfg)
    xs, _ = W.x0_matrix(cfg)
    gs, _ = W.grad_matrix(cfg)
    par = B.config_params(cfg)
    a = B.Engine(cfg.n, cfg.d, *par, cfg.gamma)
    a.write_state(xs)
    a.write_grads(gs)
    a.apply_events(ev.times, ev.wi, ev.wj, ev.slot)
    want = a.read_state()
    a.close()
    b = B.Engine(cfg.n, cfg.d, *par, cfg.gamma)
    b.write_state(xs)
    b.write_grads(gs)
    h = len(ev) // 2
    b.apply_events(ev.times[:h], ev.wi[:h], ev.wj[:h], ev.slot[:h])
    ckpt = b.read_state()
    b.close()
    c = B.Engine(cfg.n, cfg.d, *par, cfg.gamma)  # a fresh engine restored from the checkpoint
    c.write_state(*ckpt)
    c.write_grads(gs)
    c.apply_events(ev.times[h:], ev.wi[h:], ev.wj[h:], ev.slot[h:])
    got = c.read_state()
    c.close()
    for u, v in zip(want, got):
        assert np.array_equal(u, v)


def test_apply_events_equals_plan_and_reports_stats():
    cfg = _small()
    ev = W.config_events(cfg)
    outs = []
    for mode in ("apply", "apply_per_batch", "apply_slices", "plan", "plan_chunks"):
        eng, _ = P.make_small(cfg)
        if mode.startswith("apply"):
            eng.set_launch_mode({"apply": B.A2_LAUNCH_AUTO, "apply_per_batch": B.A2_LAUNCH_PER_BATCH,
                                 "apply_slices": B.A2_LAUNCH_COLUMN_SLICES}[mode])
            st = eng.apply_events(ev.times, ev.wi, ev.wj, ev.slot, flags=B.A2_SCHED_FUSE, want_stats=True)
            assert st["n_events"] == len(ev) and st["n_batches"] > 0 and st["n_launches"] > 0
            if mode == "apply_per_batch":
                assert st["n_launches"] >= st["n_batches"]
            if mode == "apply_slices":  # a launch holds the items of several batches
                assert st["n_launches"] < st["n_batches"]
            assert st["bytes_moved"] < st["bytes_one_by_one"] and st["descriptor_bytes"] > 0
        else:
            p = eng.plan(ev.times, ev.wi, ev.wj, ev.slot, flags=B.A2_SCHED_FUSE)
            if mode == "plan":
                st = p.run(want_stats=True)
                assert st["n_events"] == len(ev)
            else:
                nb = p.sched.num_batches
                p.run(0, nb // 2)
                p.run(nb // 2, -1)
            p.close()
        outs.append(eng.read_state())
        eng.close()
    for o in outs[1:]:
        assert all(np.array_equal(u, v) for u, v in zip(outs[0], o))


def test_plan_sequencing_errors():
    cfg = _small(n_events=200)
    ev = W.config_events(cfg)
    eng, _ = P.make_small(cfg)
    p = eng.plan(ev.times, ev.wi, ev.wj, ev.slot)
    with pytest.raises(B.A2Error) as e:
        p.run(1, 1)  # batches must be run in order
    assert e.value.code == B.A2_ESTATE
    p.run(0, 2)
    with pytest.raises(B.A2Error) as e:
        p.run(0, 1)  # not twice
    assert e.value.code == B.A2_ESTATE
    with pytest.raises(B.A2Error) as e:
        p.run(2, 10 ** 6)
    assert e.value.code == B.A2_ERANGE
    p.run(2, -1)
    q = eng.plan(ev.times, ev.wi, ev.wj, ev.slot, t_start=np.zeros(cfg.n))  # starts from t = 0, engine is past it
    with pytest.raises(B.A2Error) as e:
        q.run()
    assert e.value.code == B.A2_ESTATE
    p.close()
    q.close()
    eng.close()


def test_rejected_input_leaves_the_state_untouched():
    cfg = _small(n_events=100)
    ev = W.config_events(cfg)
    eng, _ = P.make_small(cfg)
    eng.apply_events(ev.times, ev.wi, ev.wj, ev.slot)
    before = eng.read_state()
    t_last = float(ev.times[-1])
    bad = [
        ([t_last - 1.0], [0], [-1], [0], B.A2_EORDER),       # precedes the worker's last event
        ([t_last + 2, t_last + 1], [0, 1], [-1, -1], [0, 1], B.A2_EORDER),
        ([t_last + 1], [cfg.n], [-1], [0], B.A2_ERANGE),
        ([t_last + 1], [0], [0], [-1], B.A2_ERANGE),
        ([t_last + 1], [0], [-1], [cfg.n], B.A2_ERANGE),
        ([t_last + 1, math.nan], [0, 1], [1, -1], [-1, 1], B.A2_EINVAL),  # bad event after a good one
    ]
    for times, wi, wj, sl, code in bad:
        with pytest.raises(B.A2Error) as e:
            eng.apply_events(times, wi, wj, sl)
        assert e.value.code == code
    with pytest.raises(B.A2Error) as e:
        eng.apply_events([t_last + 1], [0], [1], [-1], flags=128)
    assert e.value.code == B.A2_EINVAL
    with pytest.raises(B.A2Error) as e:
        eng.consensus_distance(t_last - 1.0)  # a common time before a worker's own time
    assert e.value.code == B.A2_EORDER
    with pytest.raises(B.A2Error):
        eng.consensus_distance(math.inf)
    after = eng.read_state()
    assert all(np.array_equal(u, v) for u, v in zip(before, after))
    eng.apply_events([], [], [], [])  # an empty stream is a no-op
    assert all(np.array_equal(u, v) for u, v in zip(before, eng.read_state()))
    eng.close()


def test_bind_rejects_bad_buffers():
    import torch

    L = B.lib()
    h = C.c_void_p()
    assert L.a2cid2_create(4, 100, 0.1, 0.5, 0.5, 0.1, B.A2_F32, C.byref(h)) == B.A2_OK
    buf = torch.zeros(3 * 4 * 104 + 8, dtype=torch.float32, device="cuda:0")
    p = buf.data_ptr()
    x, xt, g = p, p + 4 * 104 * 4, p + 2 * 4 * 104 * 4
    s = torch.cuda.current_stream().cuda_stream
    assert L.a2cid2_bind(h, x, xt, g, 4, 100, s) == B.A2_EINVAL      # pitch not a multiple of 8
    assert L.a2cid2_bind(h, x, xt, g, 4, 96, s) == B.A2_EINVAL       # pitch < d
    assert L.a2cid2_bind(h, x + 4, xt, g, 4, 104, s) == B.A2_EINVAL  # misaligned
    assert L.a2cid2_bind(h, x, x, g, 4, 104, s) == B.A2_EINVAL       # aliased
    assert L.a2cid2_bind(h, x, None, g, 4, 104, s) == B.A2_EINVAL
    assert L.a2cid2_bind(h, x, xt, None, 4, 104, s) == B.A2_EINVAL
    assert L.a2cid2_bind(h, x, xt, None, 0, 104, s) == B.A2_OK       # no gradient buffer: comm events only
    t = np.array([1.0])
    i0, i1, m1 = (np.array([v], dtype=np.int32) for v in (0, 1, -1))
    dp, ip = C.POINTER(C.c_double), C.POINTER(C.c_int32)
    assert L.a2cid2_apply_events(h, 1, t.ctypes.data_as(dp), i0.ctypes.data_as(ip), i1.ctypes.data_as(ip),
                                 m1.ctypes.data_as(ip), 0, None) == B.A2_OK
    assert L.a2cid2_apply_events(h, 1, (t + 1).ctypes.data_as(dp), i0.ctypes.data_as(ip), m1.ctypes.data_as(ip),
                                 i0.ctypes.data_as(ip), 0, None) == B.A2_ERANGE  # gradient event without slots
    assert L.a2cid2_sync(h) == B.A2_OK
    L.a2cid2_destroy(h)


@pytest.mark.parametrize("flags", [B.A2_SCHED_FUSE, B.A2_SCHED_CHAIN])
@pytest.mark.parametrize("storage", ["f32", "bf16"])
def test_rows_aligned_to_16_bytes_only_take_the_128_bit_kernels(storage, flags):
    """Rows on 32-byte boundaries run the 256-bit kernels, rows that are only 16-byte aligned the
    128-bit ones; the arithmetic per element is the same, so the states agree bit for bit."""
    cfg = _small(storage, d=5_003, n_events=600)
    ev = W.config_events(cfg)
    xs, _ = W.x0_matrix(cfg)
    gs, _ = W.grad_matrix(cfg)
    outs = []
    for narrow in (False, True):
        eng = B.Engine(cfg.n, cfg.d, *B.config_params(cfg), cfg.gamma, storage=storage, rows_16B_only=narrow)
        assert (eng.x.data_ptr() % 32 == 16) == narrow
        eng.write_state(xs)
        eng.write_grads(gs)
        eng.apply_events(ev.times, ev.wi, ev.wj, ev.slot, flags=flags)
        t_eval = float(ev.times[-1]) + 0.5
        outs.append((eng.read_state(), eng.consensus_distance(), eng.consensus_distance(t_eval)))
        eng.close()
    (a, ca, cfa), (b, cb, cfb) = outs
    assert all(np.array_equal(u, v) for u, v in zip(a, b))
    assert abs(ca - cb) <= 1e-9 * ca and abs(cfa - cfb) <= 1e-9 * cfa


def test_non_default_stream():
    import torch

    cfg = _small(n_events=300)
    ev = W.config_events(cfg)
    ref_eng, _ = P.make_small(cfg)
    ref_eng.apply_events(ev.times, ev.wi, ev.wj, ev.slot)
    want = ref_eng.read_state()
    ref_eng.close()
    s = torch.cuda.Stream()
    xs, _ = W.x0_matrix(cfg)
    gs, _ = W.grad_matrix(cfg)
    eng = B.Engine(cfg.n, cfg.d, *B.config_params(cfg), cfg.gamma, stream=s)
    torch.cuda.synchronize()
    eng.write_state(xs)
    eng.write_grads(gs)
    eng.apply_events(ev.times, ev.wi, ev.wj, ev.slot)
    got = eng.read_state()
    eng.close()
    assert all(np.array_equal(u, v) for u, v in zip(want, got))


def test_many_items_per_batch_are_split_into_launches():
    """n = 600 workers on a ring: a level holds more items than one launch takes."""
    n, d = 600, 64
    edges = W.ring_edges(n)
    ev = W.poisson_events(n, edges, np.full(len(edges), 1.0), 6000, seed=9)
    rng = np.random.default_rng(1)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    g = rng.standard_normal((n, d)).astype(np.float32)
    eng = B.Engine(n, d, 0.2, 0.5, 1.2, 0.05)
    eng.write_state(x0)
    eng.write_grads(g)
    eng.set_launch_mode(B.A2_LAUNCH_PER_BATCH)
    h = len(ev) // 2
    st = eng.apply_events(ev.times[:h], ev.wi[:h], ev.wj[:h], ev.slot[:h], flags=B.A2_SCHED_FUSE, want_stats=True)
    assert st["n_launches"] > st["n_batches"]
    eng.set_launch_mode(B.A2_LAUNCH_COLUMN_SLICES)  # the caps cut these launches too, anywhere in the item list
    st = eng.apply_events(ev.times[h:], ev.wi[h:], ev.wj[h:], ev.slot[h:], flags=B.A2_SCHED_FUSE, want_stats=True)
    assert st["n_launches"] * 128 >= st["n_items"] and st["n_launches"] > 1
    from oracle.sim import OracleSim

    sim = OracleSim(x0.astype(np.float64), 0.2, 0.5, 1.2, 0.05, grads=g.astype(np.float64))
    sim.apply_stream(ev)
    x, xt, t = eng.read_state()
    assert P.rel_err(x, sim.X) <= 1e-5 and P.rel_err(xt, sim.Xt) <= 1e-5 and np.array_equal(t, sim.t)
    eng.close()


def test_plan_may_outlive_its_engine():
    cfg = _small(n_events=100)
    ev = W.config_events(cfg)
    eng, _ = P.make_small(cfg)
    p = eng.plan(ev.times, ev.wi, ev.wj, ev.slot)
    q = eng.plan(ev.times, ev.wi, ev.wj, ev.slot)
    q.close()
    eng.close()  # p is still alive: it may only be destroyed now
    p.close()


def test_plan_graph_follows_a_change_of_variant():
    """A plan run whole goes out as one CUDA graph recorded when the plan was made; changing what the
    kernels were recorded with (here the variant) must re-record it, not replay the stale one."""
    cfg = _small(n_events=400)
    ev = W.config_events(cfg)
    want_eng, _ = P.make_small(cfg, variant=B.A2_MSG_BEFORE_MIX)
    want_eng.apply_events(ev.times, ev.wi, ev.wj, ev.slot, flags=B.A2_SCHED_FUSE)
    want = want_eng.read_state()
    want_eng.close()
    eng, _ = P.make_small(cfg)
    p = eng.plan(ev.times, ev.wi, ev.wj, ev.slot, flags=B.A2_SCHED_FUSE)  # recorded with the default variant
    assert p.sched.num_batches >= 4
    eng.set_variant(B.A2_MSG_BEFORE_MIX)
    p.run()
    got = eng.read_state()
    p.close()
    eng.close()
    assert all(np.array_equal(u, v) for u, v in zip(want, got))


def test_a_plan_with_four_worker_items_is_refused_by_a_variant_whose_kernels_take_three():
    """Plans are scheduled for the kernels of the variant they were made under; the no-momentum kernels take
    three workers per item, so a four-worker plan must be refused there, before anything is launched."""
    cfg = _small(n_events=600)
    ev = W.config_events(cfg)
    eng, _ = P.make_small(cfg)
    p = eng.plan(ev.times, ev.wi, ev.wj, ev.slot, flags=B.A2_SCHED_CHAIN)
    assert max(len(p.sched.item(k).workers()) for k in range(p.sched.num_items)) == 4
    before = eng.read_state()
    eng.set_variant(B.A2_NO_MOMENTUM)
    with pytest.raises(B.A2Error) as e:
        p.run()
    assert e.value.code == B.A2_ESTATE
    assert all(np.array_equal(u, v) for u, v in zip(before, eng.read_state()))
    # a plan made under the variant holds at most three workers per item and runs
    q = eng.plan(ev.times, ev.wi, ev.wj, ev.slot, flags=B.A2_SCHED_CHAIN)
    assert max(len(q.sched.item(k).workers()) for k in range(q.sched.num_items)) == 3
    q.run()
    eng.sync()
    p.close()
    q.close()
    eng.close()
