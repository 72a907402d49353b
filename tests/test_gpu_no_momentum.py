"""GPU parity of the dynamic without the momentum buffer (Eq. (baselinedynamic), Sec. 3.2; variant
A2_NO_MOMENTUM) against the CPU checker's variant 2, through the C ABI."""
import numpy as np
import pytest

from paper_2306_08289_b200 import binding as B
from paper_2306_08289_b200 import workload as W
from tests import parity as P

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("flags", [0, B.A2_SCHED_FUSE, B.A2_SCHED_CHAIN])
def test_cfg1_full_every_batch(flags):
    cfg = W.CONFIGS["cfg1"]
    eng, chk = P.make_small(cfg, momentum=False)
    worst, nb = P.run_batches_and_check(eng, chk, W.config_events(cfg), flags)
    assert nb > 50
    c_gpu, c_ref = eng.consensus_distance(), chk.plain.consensus()
    assert abs(c_gpu - c_ref) <= 1e-5 * c_ref
    eng.close()


@pytest.mark.parametrize("name,d,n_events", [
    ("cfg2", 20_011, 3000),   # several tiles and a ragged tail (d % 4 == 3)
    ("cfg3", 6_150, 3000),
    ("cfg4", 4_097, 4000),    # one column past a tile of the two-vector kernel
    ("cfg5", 16_389, 4000),   # bf16
])
@pytest.mark.parametrize("flags", [0, B.A2_SCHED_FUSE, B.A2_SCHED_CHAIN])
def test_scaled_configs_every_batch(name, d, n_events, flags):
    cfg = W.CONFIGS[name].scaled(d=d, n_events=n_events)
    eng, chk = P.make_small(cfg, momentum=False)
    worst, nb = P.run_batches_and_check(eng, chk, W.config_events(cfg), flags, every=3)
    print(f"{cfg.name} no momentum flags={flags} batches={nb} worst={worst}")
    eng.close()


@pytest.mark.parametrize("n,d", [(2, 1), (3, 8), (5, 9), (4, 4095), (4, 4097)])
@pytest.mark.parametrize("storage", ["f32", "bf16"])
def test_degenerate_sizes(n, d, storage):
    # bf16: a row is stored at every event here, and 75 stores per worker already cost 2e-2 of its norm
    # (the engine is bit-equal to the storage-modelled checker in these cases), so the stream is kept short
    cfg = W.WorkloadConfig(name=f"tiny{n}x{d}", n=n, graph="ring", d=d, storage=storage,
                           n_events=300 if storage == "f32" else 120,
                           x0_std=1.0, g_std=0.5, gamma=0.05, edge_rate=1.0, fixed_params=(0.7, 0.5, 1.5), seed=78)
    for flags in (0, B.A2_SCHED_FUSE, B.A2_SCHED_CHAIN):
        eng, chk = P.make_small(cfg, momentum=False)
        P.run_batches_and_check(eng, chk, W.config_events(cfg), flags, every=7)
        eng.close()


@pytest.mark.parametrize("name", ["cfg3", "cfg5"])
def test_rows_on_16_byte_boundaries_only(name):
    """Rows that start 16 bytes off a 32-byte boundary take the 128-bit kernels (fp32 and bf16)."""
    cfg = W.CONFIGS[name].scaled(d=9_001, n_events=1500)
    xs, xw = W.x0_matrix(cfg)
    gs, gw = W.grad_matrix(cfg)
    eng = B.Engine(cfg.n, cfg.d, *B.config_params(cfg), cfg.gamma, storage=cfg.storage, n_grad_slots=cfg.n_grad_slots,
                   rows_16B_only=True, momentum=False)
    eng.write_state(xs)
    eng.write_grads(gs)
    chk = P.Checker(xw, P.oracle_params(cfg), cfg.gamma, gw, cfg.storage, variant=B.A2_NO_MOMENTUM)
    P.run_batches_and_check(eng, chk, W.config_events(cfg), B.A2_SCHED_CHAIN, every=9)
    eng.close()


def test_bound_momentum_buffer_is_left_alone_and_the_clock_calls_move_no_rows():
    """With an x~ buffer bound, the variant neither reads nor writes it; a flush only records the time
    and the consensus distance at a common time is that of the stored rows."""
    cfg = W.CONFIGS["cfg2"].scaled(d=2_500, n_events=1500)
    xs, xw = W.x0_matrix(cfg)
    gs, gw = W.grad_matrix(cfg)
    eng = B.Engine(cfg.n, cfg.d, *B.config_params(cfg), cfg.gamma, n_grad_slots=cfg.n_grad_slots)
    marker = np.random.default_rng(4).standard_normal(xs.shape).astype(np.float32)
    eng.write_state(xs, x_tilde=marker)
    eng.write_grads(gs)
    eng.set_variant(B.A2_NO_MOMENTUM)
    ev = W.config_events(cfg)
    st = eng.apply_events(ev.times, ev.wi, ev.wj, ev.slot, flags=B.A2_SCHED_FUSE, want_stats=True)
    chk = P.Checker(xw, P.oracle_params(cfg), cfg.gamma, gw, cfg.storage, variant=B.A2_NO_MOMENTUM)
    chk.plain.apply_stream(ev)
    x, xt, t = eng.read_state()
    assert np.array_equal(xt, marker)
    assert P.rel_err(x, chk.plain.X) <= P.TOL["f32"]
    assert np.array_equal(t, chk.plain.t)
    # the byte counters describe x alone: a communication item 4 rows, a gradient 3
    assert st["bytes_one_by_one"] == (4 * st["n_comm"] + 3 * st["n_grad"]) * cfg.d * 4
    assert st["bytes_moved"] <= st["bytes_one_by_one"]
    t_end = float(ev.times[-1]) + 2.0
    c_stored = eng.consensus_distance()
    assert eng.consensus_distance(t_end) == c_stored
    eng.flush(t_end)
    x2, xt2, t2 = eng.read_state()
    assert np.array_equal(x2, x) and np.array_equal(xt2, marker) and np.all(t2 == t_end)
    eng.close()


def test_whole_plan_as_a_graph_and_the_refusals():
    cfg = W.CONFIGS["cfg1"].scaled(n_events=2000)
    eng, chk = P.make_small(cfg, momentum=False)
    ev = W.config_events(cfg)
    plan = eng.plan(ev.times, ev.wi, ev.wj, ev.slot, flags=B.A2_SCHED_CHAIN)
    assert plan.sched.num_batches >= 4  # long enough to be recorded as a CUDA graph
    plan.run()
    chk.plain.apply_stream(ev)
    x, xt, t = eng.read_state()
    assert xt is None
    assert P.rel_err(x, chk.plain.X) <= P.TOL["f32"]
    plan.close()
    ev2 = W.config_events(cfg.scaled(n_events=50))
    with pytest.raises(B.A2Error) as e:
        eng.apply_events(ev2.times + t.max(), ev2.wi, ev2.wj, ev2.slot, flags=B.A2_SCHED_RESIDENT)
    assert e.value.code == B.A2_EINVAL
    with pytest.raises(B.A2Error) as e:  # leaving the variant needs an x~ buffer
        eng.set_variant(B.A2_MSG_AFTER_MIX)
    assert e.value.code == B.A2_ESTATE
    x3, _, _ = eng.read_state()
    assert np.array_equal(x3, x)  # the refused calls changed nothing
    eng.close()
