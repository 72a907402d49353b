"""The host scheduler, without a GPU: its batches replayed through the CPU checker must give
the time-ordered run bit for bit (events on disjoint workers commute: Eq. (dynamic) is local
to the workers an event names), with and without gradient fusion; plus validation."""
import numpy as np
import pytest

from oracle.sim import OracleSim
from paper_2306_08289_b200 import binding as B
from paper_2306_08289_b200 import build as build_mod
from paper_2306_08289_b200 import workload as W


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()


def _replay(cfg, ev, sched, params, x0, G):
    """Advance the checker batch by batch, events sorted by time inside a batch."""
    sim = OracleSim(x0, *params, cfg.gamma, grads=G)
    seen = []
    for b in range(sched.num_batches):
        idx = sched.batch_events(b)
        seen.append(idx)
        idx = idx[np.argsort(ev.times[idx], kind="stable")]
        sim.apply(ev.times[idx], ev.wi[idx], ev.wj[idx], ev.slot[idx])
    return sim, np.concatenate(seen) if seen else np.empty(0, dtype=np.int64)


@pytest.mark.parametrize("name,d,n_events", [("cfg1", 7, 2000), ("cfg2", 5, 3000), ("cfg4", 3, 4000), ("cfg5", 3, 4000)])
@pytest.mark.parametrize("flags", [0, B.A2_SCHED_FUSE, B.A2_SCHED_CHAIN, B.A2_SCHED_FUSE | B.A2_SCHED_ROW_PER_OP,
                                   B.A2_SCHED_CHAIN | B.A2_SCHED_ROW_PER_OP])
def test_batches_replay_to_the_time_ordered_state(name, d, n_events, flags):
    cfg = W.CONFIGS[name].scaled(d=d, n_events=n_events)
    cfg = cfg if cfg.storage == "f32" else W.WorkloadConfig(**{**cfg.__dict__, "storage": "f32"})
    ev = W.config_events(cfg)
    _, x0 = W.x0_matrix(cfg)
    _, G = W.grad_matrix(cfg)
    params = (0.4, 0.5, 1.3)
    ref = OracleSim(x0, *params, cfg.gamma, grads=G)
    ref.apply_stream(ev)
    s = B.Schedule(cfg.n, cfg.n_grad_slots, ev.times, ev.wi, ev.wj, ev.slot, flags=flags)
    sim, seen = _replay(cfg, ev, s, params, x0, G)
    assert np.array_equal(np.sort(seen), np.arange(len(ev)))  # every event exactly once
    assert np.array_equal(sim.X, ref.X) and np.array_equal(sim.Xt, ref.Xt) and np.array_equal(sim.t, ref.t)
    assert np.array_equal(s.t_final(cfg.n), ref.t)
    # structure: items of a batch are worker-disjoint; per-worker event order is kept
    last_pos = {}
    pos = 0
    for b in range(s.num_batches):
        first, cnt = s.batch_items(b)
        used = set()
        for k in range(first, first + cnt):
            it = s.item(k)
            assert it.batch == b and it.n_ops >= 1
            ws = set(it.workers())
            assert len(ws) == len(it.workers()) and not (ws & used)
            assert (it.c < 0 or it.b >= 0) and (it.d < 0 or it.c >= 0) and (flags & B.A2_SCHED_CHAIN or it.c < 0)
            used |= ws
            evs, kinds = s.ops(it.first_op, it.n_ops)
            pairs = {B.A2_OP_COMM: (it.a, it.b), B.A2_OP_COMM_AC: (it.a, it.c), B.A2_OP_COMM_BC: (it.b, it.c),
                     B.A2_OP_COMM_AD: (it.a, it.d), B.A2_OP_COMM_BD: (it.b, it.d), B.A2_OP_COMM_CD: (it.c, it.d)}
            grads = {B.A2_OP_GRAD_A: (it.a, it.slot_a), B.A2_OP_GRAD_B: (it.b, it.slot_b), B.A2_OP_GRAD_C: (it.c, it.slot_c),
                     B.A2_OP_GRAD_D: (it.d, it.slot_d)}
            reloads = s.op_reloads(it.first_op, it.n_ops)
            assert flags & B.A2_SCHED_ROW_PER_OP or np.all(reloads == -1)
            for e, kd, rl in zip(evs, kinds, reloads):
                if kd in pairs:
                    # the pair may be stored the other way round: the update is symmetric in its two workers
                    assert {ev.wi[e], ev.wj[e]} == set(pairs[kd]) and min(pairs[kd]) >= 0
                    touched = pairs[kd]
                else:
                    w, sl = grads[kd]  # sl: the row the worker's gradient registers hold when the operation runs
                    assert ev.wi[e] == w and ev.wj[e] == -1 and ev.slot[e] == sl
                    if rl >= 0:
                        assert rl != sl
                        grads[kd] = (w, int(rl))
                    touched = (w,)
                assert kd not in pairs or rl == -1
                for w in touched:
                    assert last_pos.get(w, -1) < e  # this worker's events come in stream order
                    last_pos[w] = e
                pos += 1
            if not flags:
                assert it.n_ops == 1
    assert pos == len(ev)
    st = s.stats(cfg.d, 4)
    assert st["n_events"] == len(ev) and st["n_comm"] == int((ev.wj >= 0).sum())
    assert st["bytes_one_by_one"] == (8 * st["n_comm"] + 5 * st["n_grad"]) * cfg.d * 4
    if flags:
        assert st["bytes_moved"] < st["bytes_one_by_one"] and s.num_items < len(ev)
        if flags & B.A2_SCHED_ROW_PER_OP:  # never more rows than with items cut at every change of row
            cut = B.Schedule(cfg.n, cfg.n_grad_slots, ev.times, ev.wi, ev.wj, ev.slot, flags=flags & ~B.A2_SCHED_ROW_PER_OP)
            assert st["bytes_moved"] <= cut.stats(cfg.d, 4)["bytes_moved"] and s.num_items <= cut.num_items
            if cfg.grad_pool > 1:
                assert st["bytes_moved"] < cut.stats(cfg.d, 4)["bytes_moved"] and s.num_items < cut.num_items
        if flags == B.A2_SCHED_CHAIN:  # chaining moves fewer rows in fewer batches than gradient fusion alone
            f = B.Schedule(cfg.n, cfg.n_grad_slots, ev.times, ev.wi, ev.wj, ev.slot, flags=B.A2_SCHED_FUSE)
            assert st["bytes_moved"] < f.stats(cfg.d, 4)["bytes_moved"] and s.num_batches < f.num_batches
            two = B.Schedule(cfg.n, cfg.n_grad_slots, ev.times, ev.wi, ev.wj, ev.slot, flags=flags, max_workers_per_item=2)
            three = B.Schedule(cfg.n, cfg.n_grad_slots, ev.times, ev.wi, ev.wj, ev.slot, flags=flags, max_workers_per_item=3)
            assert all(two.item(k).c < 0 for k in range(two.num_items))
            assert all(three.item(k).d < 0 for k in range(three.num_items))
            assert (st["bytes_moved"] <= three.stats(cfg.d, 4)["bytes_moved"] <= two.stats(cfg.d, 4)["bytes_moved"]
                    <= f.stats(cfg.d, 4)["bytes_moved"])
    else:
        assert st["bytes_moved"] == st["bytes_one_by_one"] and s.num_items == len(ev)


def test_greedy_levels_are_as_early_as_possible():
    # 0-1 and 2-3 are independent; 1-2 must wait for both; a gradient on 0 fits beside it
    times = [1.0, 2.0, 3.0, 4.0]
    s = B.Schedule(4, 4, times, [0, 2, 1, 0], [1, 3, 2, -1], [-1, -1, -1, 0])
    assert s.num_batches == 2
    assert sorted(s.batch_events(0)) == [0, 1] and sorted(s.batch_events(1)) == [2, 3]


def test_fusion_folds_pending_gradients_and_respects_caps():
    # gradients on 0,0,1 then comm(0,1), then a trailing gradient on 1
    times = [1.0, 2.0, 3.0, 4.0, 5.0]
    wi, wj, sl = [0, 0, 1, 0, 1], [-1, -1, -1, 1, -1], [0, 0, 1, -1, 1]
    s = B.Schedule(2, 2, times, wi, wj, sl, flags=B.A2_SCHED_FUSE)
    assert s.num_items == 2 and s.num_batches == 2
    it = s.item(0)
    evs, kinds = s.ops(it.first_op, it.n_ops)
    assert (it.a, it.b, it.slot_a, it.slot_b) == (0, 1, 0, 1)
    assert list(evs) == [0, 1, 2, 3] and list(kinds) == [B.A2_OP_GRAD_A, B.A2_OP_GRAD_A, B.A2_OP_GRAD_B, B.A2_OP_COMM]
    tail = s.item(1)
    assert (tail.a, tail.b, tail.n_ops) == (1, -1, 1)
    # a cap of 2 operations per item forces spills; a change of gradient slot too
    s2 = B.Schedule(2, 2, times, wi, wj, sl, flags=B.A2_SCHED_FUSE, max_ops_per_item=2)
    for k in range(s2.num_items):
        assert s2.item(k).n_ops <= 2
    assert sorted(np.concatenate([s2.batch_events(b) for b in range(s2.num_batches)])) == [0, 1, 2, 3, 4]
    s3 = B.Schedule(2, 2, [1.0, 2.0, 3.0], [0, 0, 0], [-1, -1, 1], [0, 1, -1], flags=B.A2_SCHED_FUSE)
    assert s3.num_items == 2 and s3.item(0).slot_a == 0 and s3.item(1).slot_a == 1


def test_chaining_appends_to_the_item_that_holds_the_rows_and_takes_a_third_worker():
    # comm(0,1); gradient on 1; comm(0,1) again -> one item, nothing re-read; then comm(1,2) with 2 free earlier
    # -> worker 2 joins as the third worker; then comm(2,3): 3 is free earlier, but with three workers per item
    # the item is full -> new item
    times = [1.0, 2.0, 3.0, 4.0, 5.0, 6.0]
    wi, wj, sl = [0, 1, 1, 2, 2, 3], [1, -1, 0, 1, 3, -1], [-1, 1, -1, -1, -1, 3]
    s = B.Schedule(4, 4, times, wi, wj, sl, flags=B.A2_SCHED_CHAIN, max_workers_per_item=3)
    assert s.num_items == 2 and s.num_batches == 2
    it = s.item(0)
    evs, kinds = s.ops(it.first_op, it.n_ops)
    assert (it.a, it.b, it.c, it.slot_a, it.slot_b, it.slot_c) == (0, 1, 2, -1, 1, -1)
    assert list(evs) == [0, 1, 2, 3]
    assert list(kinds) == [B.A2_OP_COMM, B.A2_OP_GRAD_B, B.A2_OP_COMM, B.A2_OP_COMM_BC]
    tail = s.item(1)
    evs, kinds = s.ops(tail.first_op, tail.n_ops)
    # the trailing gradient of worker 3 goes into the item that already holds its rows
    assert (tail.a, tail.b, tail.c, tail.slot_b) == (2, 3, -1, 3) and list(evs) == [4, 5]
    assert list(kinds) == [B.A2_OP_COMM, B.A2_OP_GRAD_B]
    assert np.array_equal(s.t_final(4), [3.0, 4.0, 5.0, 6.0])
    # four workers per item (the default): everything fits one item, worker 3 is its fourth
    s4 = B.Schedule(4, 4, times, wi, wj, sl, flags=B.A2_SCHED_CHAIN)
    it4 = s4.item(0)
    evs, kinds = s4.ops(it4.first_op, it4.n_ops)
    assert s4.num_items == 1 and (it4.a, it4.b, it4.c, it4.d, it4.slot_b, it4.slot_d) == (0, 1, 2, 3, 1, 3)
    assert list(evs) == [0, 1, 2, 3, 4, 5]
    assert list(kinds) == [B.A2_OP_COMM, B.A2_OP_GRAD_B, B.A2_OP_COMM, B.A2_OP_COMM_BC, B.A2_OP_COMM_CD, B.A2_OP_GRAD_D]
    # two workers per item at most: the third comm opens a new item
    s2 = B.Schedule(4, 4, times, wi, wj, sl, flags=B.A2_SCHED_CHAIN, max_workers_per_item=2)
    assert s2.num_items == 3 and all(s2.item(k).c < 0 for k in range(3))
    # a gradient row of another slot cannot share the item's single row per worker
    s3 = B.Schedule(2, 2, [1.0, 2.0, 3.0, 4.0], [0, 0, 0, 0], [1, -1, -1, 1], [-1, 0, 1, -1], flags=B.A2_SCHED_CHAIN)
    rows = [(s3.item(k).slot_a, s3.item(k).n_ops) for k in range(s3.num_items)]
    assert rows == [(0, 2), (1, 2)]
    with pytest.raises(B.A2Error):
        B.Schedule(4, 4, times, wi, wj, sl, flags=B.A2_SCHED_CHAIN, max_workers_per_item=5)


def test_empty_stream_and_start_times():
    s = B.Schedule(3, 0, [], [], [], [])
    assert s.num_batches == 0 and s.num_items == 0
    assert np.array_equal(s.t_final(3), np.zeros(3))
    s = B.Schedule(3, 1, [5.0], [2], [-1], [0], t_last=[1.0, 2.0, 3.0])
    assert np.array_equal(s.t_final(3), [1.0, 2.0, 5.0])


@pytest.mark.parametrize("times,wi,wj,sl,t_last,code", [
    ([2.0, 1.0], [0, 1], [-1, -1], [0, 0], None, B.A2_EORDER),            # times decrease
    ([0.5], [0], [-1], [0], [1.0, 0.0, 0.0], B.A2_EORDER),                # before the worker's time
    ([1.5], [1], [0], [-1], [2.0, 0.0, 0.0], B.A2_EORDER),                # before the peer's time
    ([1.0], [3], [-1], [0], None, B.A2_ERANGE),                           # worker out of range
    ([1.0], [0], [0], [-1], None, B.A2_ERANGE),                           # i == j
    ([1.0], [0], [-1], [1], None, B.A2_ERANGE),                           # slot out of range (1 slot)
    ([1.0], [0], [-1], [-1], None, B.A2_ERANGE),                          # neither pair nor slot
    ([1.0], [0], [1], [0], None, B.A2_ERANGE),                            # both pair and slot
    ([1.0], [0], [-2], [-1], None, B.A2_ERANGE),                          # bad peer
    ([float("nan")], [0], [-1], [0], None, B.A2_EINVAL),                  # NaN time
    ([float("inf")], [0], [1], [-1], None, B.A2_EINVAL),
])
def test_malformed_streams_are_rejected(times, wi, wj, sl, t_last, code):
    with pytest.raises(B.A2Error) as e:
        B.Schedule(3, 1, times, wi, wj, sl, t_last=t_last)
    assert e.value.code == code and "event" in str(e.value)


def test_bad_arguments():
    with pytest.raises(B.A2Error) as e:
        B.Schedule(1, 0, [], [], [], [])
    assert e.value.code == B.A2_EINVAL
    with pytest.raises(B.A2Error) as e:
        B.Schedule(3, 0, [], [], [], [], flags=64)
    assert e.value.code == B.A2_EINVAL
    s = B.Schedule(3, 0, [1.0], [0], [1], [-1])
    with pytest.raises(B.A2Error):
        s.batch_items(5)
    with pytest.raises(B.A2Error):
        s.item(9)
    with pytest.raises(B.A2Error):
        s.ops(0, 5)


def test_resident_schedule_is_one_batch_in_stream_order():
    cfg = W.CONFIGS["cfg2"].scaled(d=3, n_events=1500)
    ev = W.config_events(cfg)
    for flags in (B.A2_SCHED_RESIDENT, B.A2_SCHED_RESIDENT | B.A2_SCHED_FUSE):  # the resident flag wins
        s = B.Schedule(cfg.n, cfg.n_grad_slots, ev.times, ev.wi, ev.wj, ev.slot, flags=flags)
        assert s.num_batches == 1 and s.num_items == len(ev) == s.num_ops
        assert np.array_equal(s.batch_events(0), np.arange(len(ev)))
        it = s.item(7)
        assert (it.a, it.n_ops, it.batch) == (ev.wi[7], 1, 0)
    sim = OracleSim(np.zeros((cfg.n, 1)), 0.1, 0.5, 0.5, 0.0, grads=np.zeros((cfg.n_grad_slots, 1)))
    sim.apply_stream(ev)
    assert np.array_equal(s.t_final(cfg.n), sim.t)
    with pytest.raises(B.A2Error):
        B.Schedule(cfg.n, cfg.n_grad_slots, ev.times, ev.wi, ev.wj, ev.slot, flags=16)


def test_fifo_stream_with_ties_replays_exactly():
    n, d = 16, 4
    e = W.ring_edges(n)
    ev = W.fifo_pairing_events(n, e, 2.0, 2500, seed=3)
    rng = np.random.default_rng(0)
    x0, G = rng.standard_normal((n, d)), rng.standard_normal((n, d))
    ref = OracleSim(x0, 0.3, 0.5, 1.1, 0.05, grads=G)
    ref.apply_stream(ev)
    for flags in (0, B.A2_SCHED_FUSE, B.A2_SCHED_CHAIN):
        s = B.Schedule(n, n, ev.times, ev.wi, ev.wj, ev.slot, flags=flags)
        sim = OracleSim(x0, 0.3, 0.5, 1.1, 0.05, grads=G)
        for b in range(s.num_batches):
            idx = np.sort(s.batch_events(b))  # stream order inside the batch (times tie)
            sim.apply(ev.times[idx], ev.wi[idx], ev.wj[idx], ev.slot[idx])
        assert np.array_equal(sim.X, ref.X) and np.array_equal(sim.Xt, ref.Xt) and np.array_equal(sim.t, ref.t)


def test_random_streams_property():
    """Property test over random small streams (ties, bursts on one worker, several gradient rows per
    worker, tight caps): the batches cover every event once, keep workers disjoint inside a batch, and
    replay to the bit-exact state of the time-ordered run."""
    from hypothesis import given, settings, strategies as st

    @st.composite
    def streams(draw):
        n = draw(st.integers(2, 9))
        n_slots = draw(st.integers(1, 2 * n))
        m = draw(st.integers(0, 60))
        gaps = draw(st.lists(st.sampled_from([0.0, 0.0, 0.25, 1.0, 3.5]), min_size=m, max_size=m))
        times = np.cumsum(np.array(gaps, dtype=np.float64)) if m else np.zeros(0)
        wi, wj, sl = [], [], []
        for _ in range(m):
            i = draw(st.integers(0, n - 1))
            if draw(st.booleans()):
                j = draw(st.integers(0, n - 2))
                j = j + 1 if j >= i else j
                wi.append(i); wj.append(j); sl.append(-1)
            else:
                wi.append(i); wj.append(-1); sl.append(draw(st.integers(0, n_slots - 1)))
        flags = draw(st.sampled_from([0, B.A2_SCHED_FUSE, B.A2_SCHED_CHAIN, B.A2_SCHED_CHAIN]))
        if flags and draw(st.booleans()):
            flags |= B.A2_SCHED_ROW_PER_OP
        cap = draw(st.sampled_from([0, 2, 3, 5]))
        kw = draw(st.sampled_from([0, 2, 3, 4]))
        return (n, n_slots, times, np.array(wi, dtype=np.int32), np.array(wj, dtype=np.int32), np.array(sl, dtype=np.int32),
                flags, cap, kw)

    @settings(max_examples=400, deadline=None)
    @given(streams())
    def check(case):
        n, n_slots, times, wi, wj, sl, flags, cap, kw = case
        rng = np.random.default_rng(len(times) * 31 + n)
        x0, G = rng.standard_normal((n, 3)), rng.standard_normal((n_slots, 3))
        ref = OracleSim(x0, 0.4, 0.5, 1.7, 0.1, grads=G)
        ref.apply(times, wi, wj, sl)
        s = B.Schedule(n, n_slots, times, wi, wj, sl, flags=flags, max_ops_per_item=cap, max_workers_per_item=kw)
        sim = OracleSim(x0, 0.4, 0.5, 1.7, 0.1, grads=G)
        seen = []
        for b in range(s.num_batches):
            first, cnt = s.batch_items(b)
            used = set()
            for k in range(first, first + cnt):
                it = s.item(k)
                ws = set(it.workers())
                assert not (ws & used) and (cap == 0 or it.n_ops <= max(cap, 1))
                assert len(ws) <= (kw or 4) and (flags & B.A2_SCHED_CHAIN or len(ws) <= 2)
                used |= ws
                evs, kinds = s.ops(it.first_op, it.n_ops)
                slots = {B.A2_OP_GRAD_A: it.slot_a, B.A2_OP_GRAD_B: it.slot_b, B.A2_OP_GRAD_C: it.slot_c, B.A2_OP_GRAD_D: it.slot_d}
                reloads = s.op_reloads(it.first_op, it.n_ops)
                for x, kd, rl in zip(evs, kinds, reloads):
                    # a gradient operation finds its row in its worker's gradient registers: the item's row for
                    # that worker, or the one fetched after the worker's previous gradient operation
                    assert kd not in slots or sl[x] == slots[kd]
                    if rl >= 0:
                        assert kd in slots and flags & B.A2_SCHED_ROW_PER_OP
                        slots[kd] = int(rl)
                e = evs[np.argsort(times[evs], kind="stable")]
                # inside an item a worker's own events are already in stream order
                for w in ws:
                    mine = [x for x in evs if wi[x] == w or wj[x] == w]
                    assert mine == sorted(mine)
                sim.apply(times[e], wi[e], wj[e], sl[e])
                seen.extend(evs.tolist())
        assert sorted(seen) == list(range(len(times)))
        assert np.array_equal(sim.X, ref.X) and np.array_equal(sim.Xt, ref.Xt) and np.array_equal(sim.t, ref.t)
        assert np.array_equal(s.t_final(n), ref.t)

    check()


def test_storage_model_groups_of_a_schedule_equal_the_item_by_item_loop():
    """The full-size bf16 parity test hands the checker a whole schedule at once (events in item order, a
    rounding point after every item); that must be the item-by-item loop of the batch-wise parity helper."""
    from oracle.sim import OracleSim
    from tests import parity as P
    from tests.test_gpu_fullwidth import _step_groups

    cfg = W.CONFIGS["cfg5"].scaled(d=29, n_events=1500)
    ev = W.config_events(cfg)
    _, xw = W.x0_matrix(cfg)
    _, gw = W.grad_matrix(cfg)
    sched = B.Schedule(cfg.n, cfg.n_grad_slots, ev.times, ev.wi, ev.wj, ev.slot, flags=B.A2_SCHED_CHAIN, max_workers_per_item=3)
    chk = P.Checker(xw, P.oracle_params(cfg), cfg.gamma, gw, "bf16")
    for b in range(sched.num_batches):
        chk.apply_batch(ev, sched, b)
    once = OracleSim(xw, *P.oracle_params(cfg), cfg.gamma, grads=gw)
    once.apply_groups(*_step_groups(ev, sched))
    assert np.array_equal(once.X, chk.stored.X) and np.array_equal(once.Xt, chk.stored.Xt)
    assert np.array_equal(once.t, chk.stored.t) and not np.array_equal(once.X, chk.plain.X)
