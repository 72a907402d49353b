"""GPU parity: the CUDA path, called through the C ABI, against the CPU checker element by
element on the same seeded inputs, after every batch."""
import numpy as np
import pytest

from paper_2306_08289_b200 import binding as B
from paper_2306_08289_b200 import workload as W
from tests import parity as P

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("flags", [0, B.A2_SCHED_FUSE, B.A2_SCHED_CHAIN])
def test_cfg1_full_every_batch(flags):
    cfg = W.CONFIGS["cfg1"]
    eng, chk = P.make_small(cfg)
    worst, nb = P.run_batches_and_check(eng, chk, W.config_events(cfg), flags)
    assert nb > 50
    c_gpu, c_ref = eng.consensus_distance(), chk.plain.consensus()
    assert abs(c_gpu - c_ref) <= 1e-5 * c_ref
    eng.close()


@pytest.mark.parametrize("name,d,n_events", [
    ("cfg2", 20_011, 3000),   # several tiles and a ragged tail (d % 4 == 3)
    ("cfg3", 6_150, 3000),    # d % 4 == 2
    ("cfg4", 4_097, 4000),    # one column past two tiles
    ("cfg5", 16_389, 4000),   # bf16: two tiles + 5 columns
])
@pytest.mark.parametrize("flags", [0, B.A2_SCHED_FUSE, B.A2_SCHED_CHAIN])
def test_scaled_configs_every_batch(name, d, n_events, flags):
    cfg = W.CONFIGS[name].scaled(d=d, n_events=n_events)
    eng, chk = P.make_small(cfg)
    worst, nb = P.run_batches_and_check(eng, chk, W.config_events(cfg), flags)
    print(f"{cfg.name} flags={flags} batches={nb} worst={worst}")
    eng.close()


@pytest.mark.parametrize("n,d", [(2, 1), (2, 3), (3, 8), (5, 9), (4, 2047), (4, 2049)])
@pytest.mark.parametrize("storage", ["f32", "bf16"])
def test_degenerate_sizes(n, d, storage):
    cfg = W.WorkloadConfig(name=f"tiny{n}x{d}", n=n, graph="ring", d=d, storage=storage, n_events=300,
                           x0_std=1.0, g_std=0.5, gamma=0.05, edge_rate=1.0, fixed_params=(0.7, 0.5, 1.5), seed=77)
    for flags in (0, B.A2_SCHED_FUSE, B.A2_SCHED_CHAIN):
        eng, chk = P.make_small(cfg)
        P.run_batches_and_check(eng, chk, W.config_events(cfg), flags, every=7)
        eng.close()


def test_fused_chained_and_unfused_schedules_are_bit_identical():
    """Fusion and chaining only change which rows share a trip through registers, not the arithmetic
    (a communication stored with its two workers swapped gives the same bits: the update is antisymmetric)."""
    cfg = W.CONFIGS["cfg4"].scaled(d=10_003, n_events=3000)
    ev = W.config_events(cfg)
    out = []
    for flags in (0, B.A2_SCHED_FUSE, B.A2_SCHED_CHAIN):
        eng, _ = P.make_small(cfg)
        eng.apply_events(ev.times, ev.wi, ev.wj, ev.slot, flags=flags)
        out.append(eng.read_state())
        eng.close()
    for o in out[1:]:
        assert all(np.array_equal(u, v) for u, v in zip(out[0], o))


@pytest.mark.parametrize("name,d,n_events,pool", [("cfg4", 10_003, 3000, 3), ("cfg3", 6_150, 3000, 8), ("cfg4", 4_097, 2500, 64)])
def test_fresh_gradient_rows_inside_items(name, d, n_events, pool):
    """Every gradient event names its own row (the paper's stochastic gradients are fresh draws, Sec. 3.2):
    fused and chained items then fetch a worker's next row in the middle of the item. Parity after every
    batch, at least one such fetch in the schedule, the fetched rows counted in the bytes moved, and the
    same bits as the schedule with one event per item."""
    from dataclasses import replace

    cfg = replace(W.CONFIGS[name].scaled(d=d, n_events=n_events), grad_pool=pool)
    ev = W.config_events(cfg)
    states = []
    for flags in (0, B.A2_SCHED_FUSE, B.A2_SCHED_CHAIN):
        eng, chk = P.make_small(cfg)
        plan = eng.plan(ev.times, ev.wi, ev.wj, ev.slot, flags=flags)
        reloads = plan.sched.op_reloads(0, plan.sched.num_ops)
        n_fetched = int((reloads >= 0).sum())
        assert (n_fetched > 0) == bool(flags)
        st = plan.sched.stats(cfg.d, 4)
        rows = 0
        for k in range(plan.sched.num_items):
            it = plan.sched.item(k)
            rows += 4 * len(it.workers()) + sum(sl >= 0 for sl in (it.slot_a, it.slot_b, it.slot_c, it.slot_d))
        assert st["bytes_moved"] == (rows + n_fetched) * cfg.d * 4
        plan.close()
        P.run_batches_and_check(eng, chk, ev, flags, every=4)
        states.append(eng.read_state())
        eng.close()
    for o in states[1:]:
        assert all(np.array_equal(u, v) for u, v in zip(states[0], o))


def test_message_before_mix_variant():
    cfg = W.CONFIGS["cfg3"].scaled(d=5_001, n_events=1500)
    eng, chk = P.make_small(cfg, variant=B.A2_MSG_BEFORE_MIX)
    P.run_batches_and_check(eng, chk, W.config_events(cfg), B.A2_SCHED_CHAIN, every=5)
    eng.close()


def test_baseline_parameters_keep_momentum_equal_to_x():
    """eta = 0, alpha = alpha~ = 1/2 (the convergence proposition of Sec. 3.4, non-accelerated): x~ stays a bit-exact copy of x."""
    cfg = W.CONFIGS["cfg2"].scaled(d=3_000, n_events=2000)
    xs, _ = W.x0_matrix(cfg)
    gs, _ = W.grad_matrix(cfg)
    eng = B.Engine(cfg.n, cfg.d, *B.prescribe(1.0, 1.0, accelerated=False), cfg.gamma, n_grad_slots=cfg.n_grad_slots)
    eng.write_state(xs)
    eng.write_grads(gs)
    ev = W.config_events(cfg)
    eng.apply_events(ev.times, ev.wi, ev.wj, ev.slot, flags=B.A2_SCHED_FUSE)
    x, xt, _ = eng.read_state()
    assert np.array_equal(x, xt)
    eng.close()


@pytest.mark.parametrize("name,d", [("cfg1", 10_000), ("cfg2", 50_001), ("cfg5", 30_005)])
def test_consensus_distance_stored_and_at_common_time(name, d):
    cfg = W.CONFIGS[name].scaled(d=d, n_events=1500)
    eng, chk = P.make_small(cfg)
    sim = chk.plain
    ev = W.config_events(cfg)
    c0g, c0r = eng.consensus_distance(), sim.consensus()
    assert abs(c0g - c0r) <= 2e-6 * c0r
    eng.apply_events(ev.times, ev.wi, ev.wj, ev.slot, flags=B.A2_SCHED_FUSE)
    sim.apply_stream(ev)
    x, xt, t = eng.read_state()
    # the reduction itself, on exactly the rows the device holds
    from oracle.sim import OracleSim
    on_dev = OracleSim(P.widen(x, cfg.storage), sim.eta, sim.alpha, sim.alpha_tilde, sim.gamma,
                       xt0=P.widen(xt, cfg.storage), t0=t)
    assert abs(eng.consensus_distance() - on_dev.consensus()) <= 2e-6 * on_dev.consensus()
    t_eval = float(ev.times[-1]) + 0.25
    assert abs(eng.consensus_distance(t_eval) - on_dev.consensus(t_eval)) <= 2e-6 * on_dev.consensus(t_eval)
    # and end to end against the checker's own state
    tol = 1e-4 if cfg.storage == "f32" else 5e-2
    assert abs(eng.consensus_distance() - sim.consensus()) <= tol * sim.consensus()
    assert abs(eng.consensus_distance(t_eval) - sim.consensus(t_eval)) <= tol * sim.consensus(t_eval)
    eng.close()


def test_exact_consensus_is_zero():
    eng = B.Engine(4, 1000, 0.0, 0.5, 0.5, 0.0)
    row = np.random.default_rng(0).standard_normal(1000).astype(np.float32)
    eng.write_state(np.tile(row, (4, 1)))
    assert eng.consensus_distance() == 0.0
    eng.close()


# ---- resident mode: one launch per call, the population's column tile kept in shared memory ----
@pytest.mark.parametrize("name,d,n_events", [
    ("cfg1", 10_000, 2000),  # 4 workers, pool of 16 gradient rows per worker: fits one cache fill
    ("cfg2", 5_003, 6000),   # 16 workers x 128 rows: the cache is refilled chunk by chunk
    ("cfg4", 4_097, 3000),   # 64 workers: one CTA per SM
])
def test_resident_mode_is_bit_identical_to_batches_fp32(name, d, n_events):
    """Same per-element operations in the same per-worker order, so fp32 states agree bit for bit."""
    cfg = W.CONFIGS[name].scaled(d=d, n_events=n_events)
    ev = W.config_events(cfg)
    states = []
    for flags in (B.A2_SCHED_FUSE, B.A2_SCHED_CHAIN, B.A2_SCHED_RESIDENT):
        eng, chk = P.make_small(cfg)
        for lo in range(0, len(ev), 777):  # several calls, so that resident calls chain on stored state
            c = ev.slice(lo, lo + 777)
            st = eng.apply_events(c.times, c.wi, c.wj, c.slot, flags=flags, want_stats=True)
            if flags == B.A2_SCHED_RESIDENT:
                assert st["n_launches"] == 2 and st["n_batches"] == 1
                chk.plain.apply_stream(c)
                x, xt, t = eng.read_state()
                chk.compare(P.widen(x, "f32"), P.widen(xt, "f32"), t, where=f"resident {name} after event {lo + len(c)}")
        states.append(eng.read_state())
        eng.close()
    assert all(np.array_equal(u, v) for u, v in zip(states[0], states[1]))


def test_resident_mode_bf16_storage():
    cfg = W.CONFIGS["cfg5"].scaled(d=6_151, n_events=3000)
    ev = W.config_events(cfg)
    eng, chk = P.make_small(cfg)
    for lo in range(0, len(ev), 500):
        c = ev.slice(lo, lo + 500)
        eng.apply_events(c.times, c.wi, c.wj, c.slot, flags=B.A2_SCHED_RESIDENT)
        chk.plain.apply_stream(c)
        chk.stored.apply_stream(c)  # the tile is held in fp32 during a call and rounded at its end
        chk.stored.round_rows(np.arange(cfg.n))
        x, xt, t = eng.read_state()
        chk.compare(P.widen(x, "bf16"), P.widen(xt, "bf16"), t, where=f"resident bf16 after event {lo + len(c)}")
    eng.close()


def test_resident_mode_plan_variant_and_limits():
    cfg = W.CONFIGS["cfg3"].scaled(d=2_050, n_events=1200)
    ev = W.config_events(cfg)
    eng, chk = P.make_small(cfg, variant=B.A2_MSG_BEFORE_MIX)
    p = eng.plan(ev.times, ev.wi, ev.wj, ev.slot, flags=B.A2_SCHED_RESIDENT)
    assert p.sched.num_batches == 1
    p.run()
    p.close()
    chk.plain.apply_stream(ev)
    x, xt, t = eng.read_state()
    chk.compare(P.widen(x, "f32"), P.widen(xt, "f32"), t, where="resident, message before mix")
    eng.close()
    big = B.Engine(120, 64, 0.1, 0.5, 0.5, 0.1)  # 2 * 120 rows of shared memory are too many
    with pytest.raises(B.A2Error) as e:
        big.apply_events([1.0], [0], [1], [-1], flags=B.A2_SCHED_RESIDENT)
    assert e.value.code == B.A2_EINVAL and "shared memory" in str(e.value)
    big.apply_events([1.0], [0], [1], [-1])  # the batched path takes any n
    big.close()


def test_fifo_pairing_stream_with_ties():
    """The paper's practical event model (availability queue, Sec. 4.1): a gradient completion and
    the pairing it triggers carry the same time stamp, so zero elapsed times occur all the time."""
    from dataclasses import replace

    # ring of 32 at two averagings per gradient; (eta, alpha~) prescribed for exactly these rates
    cfg = replace(W.CONFIGS["cfg3"].scaled(d=4_099, n_events=3000), edge_rate=None, comms_per_grad=2.0)
    ev = W.fifo_pairing_events(cfg.n, cfg.edges(), cfg.comms_per_grad, cfg.n_events, seed=cfg.seed)
    assert np.any(np.diff(ev.times) == 0)
    outs = []
    for flags in (0, B.A2_SCHED_FUSE, B.A2_SCHED_CHAIN, B.A2_SCHED_RESIDENT):
        eng, chk = P.make_small(cfg)
        if flags == B.A2_SCHED_RESIDENT:
            eng.apply_events(ev.times, ev.wi, ev.wj, ev.slot, flags=flags)
            chk.plain.apply_stream(ev)
            x, xt, t = eng.read_state()
            chk.compare(P.widen(x, "f32"), P.widen(xt, "f32"), t, where="fifo stream, resident")
        else:
            P.run_batches_and_check(eng, chk, ev, flags, every=3)
        outs.append(eng.read_state())
        eng.close()
    for o in outs[1:]:
        assert all(np.array_equal(u, v) for u, v in zip(outs[0], o))


def test_consensus_study_reproduces_the_papers_qualitative_claim():
    """Sec. 4.2, the consensus-distance panel of the ImageNet figure: on the 64-worker ring, A2CiD2 at one averaging per gradient brings the
    consensus distance down at least as much as doubling the communication rate does."""
    from paper_2306_08289_b200 import consensus_study as CS

    res = CS.run_study(n=64, d=4_096, T=200.0, pool=16)
    final = {(r["comms_per_grad"], r["accelerated"]): np.mean([v for _, v in r["trace"][-3:]]) for r in res}
    assert final[(2.0, False)] < final[(1.0, False)]          # more communication helps the baseline
    assert final[(1.0, True)] < final[(1.0, False)] * 0.7     # the momentum helps at equal communication
    assert final[(1.0, True)] < final[(2.0, False)] * 1.2     # ... about as much as doubling the rate
    assert final[(2.0, True)] < final[(1.0, True)]


@pytest.mark.parametrize("storage", ["f32", "bf16"])
def test_flush_brings_every_worker_to_a_common_time(storage):
    """a2cid2_flush applies the mixing flow alone; afterwards mean(x) = mean(x~) (Eq. (mean)), which
    does not hold for the lazily stored state."""
    name = "cfg3" if storage == "f32" else "cfg5"
    cfg = W.CONFIGS[name].scaled(d=5_005, n_events=1500)
    ev = W.config_events(cfg)
    eng, chk = P.make_small(cfg)
    eng.apply_events(ev.times, ev.wi, ev.wj, ev.slot, flags=B.A2_SCHED_FUSE)
    chk.plain.apply_stream(ev)
    t_end = float(ev.times[-1]) + 0.75
    with pytest.raises(B.A2Error) as e:
        eng.flush(float(ev.times[-1]) - 1.0)
    assert e.value.code == B.A2_EORDER
    before = eng.read_state()
    eng.flush(t_end)
    chk.plain.flush(t_end)
    x, xt, t = eng.read_state()
    assert np.array_equal(t, np.full(cfg.n, t_end)) and not np.array_equal(before[0], x)
    xw, xtw = P.widen(x, storage), P.widen(xt, storage)
    if storage == "f32":
        assert P.rel_err(xw, chk.plain.X) <= 1e-5 and P.rel_err(xtw, chk.plain.Xt) <= 1e-5
        gap = np.abs(xw.mean(0) - xtw.mean(0)).max() / np.abs(xw.mean(0)).max()
        gap_before = np.abs(before[0].mean(0) - before[1].mean(0)).max() / np.abs(xw.mean(0)).max()
        assert gap < 1e-5 < gap_before
    else:
        assert P.row_norm_err(xw, chk.plain.X) <= 2e-2 and P.row_norm_err(xtw, chk.plain.Xt) <= 2e-2
    # the consensus distance of the flushed state is what consensus_distance(t) reported without writing
    c_now = eng.consensus_distance()
    assert abs(c_now - chk.plain.consensus()) <= (1e-4 if storage == "f32" else 5e-2) * c_now
    eng.flush(t_end)  # already there: nothing to do
    assert all(np.array_equal(u, v) for u, v in zip((x, xt, t), eng.read_state()))
    eng.close()


def _closed_loop_on_the_checker(n, d, graph, comms_per_grad, accelerated, T, gamma, seed, samples):
    """The closed loop of consensus_study.run_closed_loop on the CPU checker: events strictly in time
    order, the gradient of a gradient event computed in fp64 from the worker's stored parameters."""
    from oracle import spectral
    from oracle.sim import OracleSim
    from paper_2306_08289_b200 import consensus_study as CS

    prob, edges, rates, ev = CS.closed_loop_problem(n, d, graph, comms_per_grad, T, seed)
    eta, alpha, alpha_t = spectral.prescribe(n, edges, rates, accelerated=accelerated)[:3]
    sim = OracleSim(np.zeros((n, d)), eta, alpha, alpha_t, gamma, grads=np.zeros((n, d)))
    trace, step = [], max(1, len(ev) // samples)
    for k in range(0, len(ev), step):
        c = ev.slice(k, k + step)
        for e in range(len(c)):
            if c.wj[e] < 0:
                w = int(c.wi[e])
                sim.G[int(c.slot[e])] = prob.a[w] * (sim.X[w] - prob.b[w])
            sim.apply(c.times[e:e + 1], c.wi[e:e + 1], c.wj[e:e + 1], c.slot[e:e + 1])
        t = float(c.times[-1])
        sim.flush(t)
        trace.append((t, float(((sim.X.mean(0) - prob.x_star) ** 2).mean()), sim.consensus() / d))
    return {"trace": trace, "x_final": sim.X.copy()}


def test_closed_loop_quadratic_matches_the_checker_and_shows_the_speed_up():
    """Decentralised SGD on a synthetic quadratic, gradients computed from the current parameters
    (Algorithm 1 in closed loop). The engine and the CPU checker, driven by the same loop, end at the
    same parameters; and with the momentum the consensus distance ends lower at equal communication."""
    from paper_2306_08289_b200 import consensus_study as CS

    kw = dict(n=16, d=300, graph="ring", comms_per_grad=1.0, T=40.0, gamma=0.05, seed=3, samples=4)
    res = {}
    for acc in (False, True):
        g = CS.run_closed_loop(accelerated=acc, **kw)
        o = _closed_loop_on_the_checker(accelerated=acc, **kw)
        assert P.rel_err(g["x_final"], o["x_final"]) <= 1e-4  # the loop feeds rounding back through the gradients
        for (tg, sg, cg), (to, so, co) in zip(g["trace"], o["trace"]):
            assert tg == to and abs(sg - so) <= 1e-3 * so + 1e-9 and abs(cg - co) <= 1e-3 * co
        res[acc] = g["trace"]
    assert res[True][-1][2] < res[False][-1][2]      # consensus distance
    assert res[False][-1][1] < res[False][0][1]      # and the mean does approach the minimiser


@pytest.mark.parametrize("storage,momentum", [("f32", True), ("bf16", True), ("f32", False), ("bf16", False)])
@pytest.mark.parametrize("d", [1, 9, 2_049, 50_003])
def test_launch_modes_give_the_same_bits(storage, momentum, d):
    """One launch per batch, column slices (a launch spans batches; every CTA walks all items over columns of
    its own) and the library's own choice: the same state bit for bit, for every storage type and both
    dynamics, from a single column to slices with a ragged last tile; and that state is the checker's."""
    cfg = W.WorkloadConfig(name=f"modes{d}", n=12, graph="ring", d=d, storage=storage, n_events=900, x0_std=1.0,
                           g_std=0.3, gamma=0.05, edge_rate=1.0, fixed_params=(0.4, 0.5, 1.7), grad_pool=3, seed=91)
    ev = W.config_events(cfg)
    states = []
    for mode in (B.A2_LAUNCH_PER_BATCH, B.A2_LAUNCH_COLUMN_SLICES, B.A2_LAUNCH_AUTO):
        eng, chk = P.make_small(cfg, momentum=momentum)
        eng.set_launch_mode(mode)
        for lo in range(0, len(ev), 300):  # several calls, so that launches start from stored state
            c = ev.slice(lo, lo + 300)
            st = eng.apply_events(c.times, c.wi, c.wj, c.slot, flags=B.A2_SCHED_CHAIN, want_stats=True)
            if mode == B.A2_LAUNCH_COLUMN_SLICES:
                assert st["n_launches"] < st["n_batches"]
        states.append(eng.read_state())
        eng.close()
    for o in states[1:]:
        assert all(u is None and v is None or np.array_equal(u, v) for u, v in zip(states[0], o))
    if storage == "f32":
        eng, chk = P.make_small(cfg, momentum=momentum)
        chk.plain.apply_stream(ev)
        x, xt, t = states[0]
        chk.compare(P.widen(x, "f32"), None if xt is None else P.widen(xt, "f32"), t, where=f"launch modes, d={d}")
        eng.close()


@pytest.mark.parametrize("name,d,n_events", [("cfg4", 4_097, 4000), ("cfg3", 6_150, 3000), ("cfg2", 20_011, 3000)])
def test_round_per_store_parity_every_batch(name, d, n_events):
    """A2_ROUND_PER_STORE: inside an item x is carried as a two-word value and rounded once, when the row is
    stored. Parity with the checker after every batch under the chained schedule; the end state differs from the
    default mode's in the last bits only, and on the 64-worker ring it is closer to the checker."""
    cfg = W.CONFIGS[name].scaled(d=d, n_events=n_events)
    ev = W.config_events(cfg)
    eng, chk = P.make_small(cfg)
    eng.set_rounding(B.A2_ROUND_PER_STORE)
    worst, nb = P.run_batches_and_check(eng, chk, ev, B.A2_SCHED_CHAIN)
    per_store = eng.read_state()
    eng.close()
    base, _ = P.make_small(cfg)
    base.apply_events(ev.times, ev.wi, ev.wj, ev.slot, flags=B.A2_SCHED_CHAIN)
    per_event = base.read_state()
    base.close()
    assert np.array_equal(per_store[2], per_event[2])
    # both are within 1e-5 of the checker, hence within 2e-5 of each other; and they are not the same bits
    assert P.rel_err(per_store[0], per_event[0]) <= 2e-5 and P.rel_err(per_store[1], per_event[1]) <= 2e-5
    assert not np.array_equal(per_store[1], per_event[1])
    err_store = max(P.rel_err(per_store[0], chk.plain.X), P.rel_err(per_store[1], chk.plain.Xt))
    err_event = max(P.rel_err(per_event[0], chk.plain.X), P.rel_err(per_event[1], chk.plain.Xt))
    print(f"{cfg.name}: per store {err_store:.2e}, per event {err_event:.2e}")
    assert err_store <= P.TOL["f32"] and err_event <= P.TOL["f32"]
    if name == "cfg4":  # alpha~ / alpha = 14.5: here the roundings of x dominate, and sparing them shows
        assert err_store < err_event


def test_round_per_store_launch_modes_flush_and_refusals():
    cfg = W.CONFIGS["cfg4"].scaled(d=2_049, n_events=1500)
    ev = W.config_events(cfg)
    states = []
    for mode in (B.A2_LAUNCH_PER_BATCH, B.A2_LAUNCH_COLUMN_SLICES):
        eng, chk = P.make_small(cfg)
        eng.set_rounding(B.A2_ROUND_PER_STORE)
        eng.set_launch_mode(mode)
        eng.apply_events(ev.times, ev.wi, ev.wj, ev.slot, flags=B.A2_SCHED_CHAIN)
        t_end = float(ev.times[-1]) + 0.5
        eng.flush(t_end)
        states.append(eng.read_state())
        if mode == B.A2_LAUNCH_PER_BATCH:
            chk.plain.apply_stream(ev)
            chk.plain.flush(t_end)
            x, xt, t = states[0]
            chk.compare(P.widen(x, "f32"), P.widen(xt, "f32"), t, where="per store, flushed")
            c_ref = chk.plain.consensus()
            assert abs(eng.consensus_distance() - c_ref) <= 1e-4 * c_ref
            # the shared-memory-resident mode rounds at every event: refused, state untouched
            with pytest.raises(B.A2Error) as e:
                eng.apply_events([t_end + 1.0], [0], [1], [-1], flags=B.A2_SCHED_RESIDENT)
            assert e.value.code == B.A2_EINVAL
            assert all(np.array_equal(u, v) for u, v in zip(states[0], eng.read_state()))
        eng.close()
    assert all(np.array_equal(u, v) for u, v in zip(*states))  # the same schedule: the same bits in both launch modes
    # rows that are only 16-byte aligned cannot take the mode: refused before any launch
    odd = B.Engine(cfg.n, cfg.d, *B.config_params(cfg), cfg.gamma, n_grad_slots=cfg.n_grad_slots, rows_16B_only=True)
    odd.set_rounding(B.A2_ROUND_PER_STORE)
    with pytest.raises(B.A2Error) as e:
        odd.apply_events(ev.times[:10], ev.wi[:10], ev.wj[:10], ev.slot[:10])
    assert e.value.code == B.A2_ESTATE and "32-byte" in str(e.value)
    odd.set_rounding(B.A2_ROUND_PER_EVENT)
    odd.apply_events(ev.times[:10], ev.wi[:10], ev.wj[:10], ev.slot[:10])
    odd.close()
    bf = B.Engine(4, 64, 0.1, 0.5, 0.5, 0.1, storage="bf16")
    with pytest.raises(B.A2Error) as e:
        bf.set_rounding(B.A2_ROUND_PER_STORE)
    assert e.value.code == B.A2_EINVAL
    bf.close()
