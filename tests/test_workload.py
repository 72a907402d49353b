"""The input generator against the paper's model: the Poisson-process assumption of Sec. 3.4 (Poisson clocks), the convergence proposition of Sec. 3.4
(expected counts), App. E.2 (uniform pairing among neighbours), App. E.1 (topologies)."""
import numpy as np
import pytest

from paper_2306_08289_b200 import workload as W


def test_topologies():
    assert len(W.ring_edges(2)) == 1
    assert len(W.ring_edges(64)) == 64
    assert len(W.complete_edges(16)) == 120
    e = W.exponential_edges(64)
    assert len(e) == 352 and np.all(W.degrees(64, e) == 11)
    assert np.all(W.degrees(16, W.exponential_edges(16)) == 7)
    for g in ("ring", "complete", "exponential"):
        ed = W.make_edges(g, 16)
        assert np.all(ed[:, 0] < ed[:, 1]) and len(np.unique(ed, axis=0)) == len(ed)


def test_rate_convention():
    for name, per_worker in [("cfg2", 1.0), ("cfg4", 1.0), ("cfg5", 2.0), ("cfg1", 2.0), ("cfg3", 4.0)]:
        c = W.CONFIGS[name]
        e, r = c.edges(), c.rates()
        part = np.zeros(c.n)
        np.add.at(part, e[:, 0], r)
        np.add.at(part, e[:, 1], r)
        assert np.allclose(part, per_worker)


def test_event_counts_and_pair_histogram():
    n = 16
    e = W.exponential_edges(n)
    rates = W.edge_rates_per_worker(n, e, 2.0)
    ev = W.poisson_events(n, e, rates, 200_000, seed=5)
    T = ev.times[-1]
    n_grad = int((ev.wj < 0).sum())
    n_comm = len(ev) - n_grad
    # n T gradient steps and Tr(Lambda)/2 T communications in expectation
    assert abs(n_grad - n * T) < 5 * np.sqrt(n * T)
    assert abs(n_comm - rates.sum() * T) < 5 * np.sqrt(rates.sum() * T)
    assert np.all(np.diff(ev.times) >= 0) and ev.times[0] > 0
    # gradient events are spread evenly over workers and use their own slot
    g = ev.wi[ev.wj < 0]
    assert np.array_equal(ev.slot[ev.wj < 0], g)
    # with a pool of rows per worker, a worker's gradient events walk its rows round-robin
    ev4 = W.poisson_events(n, e, rates, 5_000, seed=5, grad_pool=4)
    ev1 = W.poisson_events(n, e, rates, 5_000, seed=5)
    assert np.array_equal(ev4.times, ev1.times) and np.array_equal(ev4.wi, ev1.wi) and np.array_equal(ev4.wj, ev1.wj)
    for w in range(n):
        sl = ev4.slot[(ev4.wj < 0) & (ev4.wi == w)]
        assert np.array_equal(sl, w + n * (np.arange(len(sl)) % 4))
    cnt = np.bincount(g, minlength=n)
    assert np.all(np.abs(cnt - n_grad / n) < 5 * np.sqrt(n_grad / n))
    # pairs are proportional to lambda^{ij} and only edges occur
    key = ev.wi[ev.wj >= 0].astype(np.int64) * n + ev.wj[ev.wj >= 0]
    ekey = e[:, 0].astype(np.int64) * n + e[:, 1]
    assert set(np.unique(key)) <= set(ekey)
    hist = np.array([(key == k).sum() for k in ekey])
    assert np.all(np.abs(hist - n_comm / len(e)) < 5 * np.sqrt(n_comm / len(e)))
    # gaps are exponential with the total rate
    gaps = np.diff(np.concatenate([[0.0], ev.times]))
    R = n + rates.sum()
    assert abs(gaps.mean() * R - 1) < 0.02 and abs(gaps.std() * R - 1) < 0.02


def test_streams_are_reproducible_and_rows_independent():
    c = W.CONFIGS["cfg1"]
    a, b = W.config_events(c), W.config_events(c)
    assert np.array_equal(a.times, b.times) and np.array_equal(a.wi, b.wi)
    s0, w0 = W.x0_row(c, 2)
    s1, w1 = W.x0_row(c, 2, cols=np.array([3, 77]))
    assert np.array_equal(s0[[3, 77]], s1) and np.array_equal(w0[[3, 77]], w1)
    assert s0.dtype == np.float32 and w0.dtype == np.float64 and np.array_equal(s0.astype(np.float64), w0)
    assert abs(w0.std() - c.x0_std) < 0.05 * c.x0_std
    assert not np.array_equal(W.x0_row(c, 1)[0], W.grad_row(c, 1)[0])


def test_bf16_rounding_is_nearest_even():
    v = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -8 + 2 ** -20, -0.02, 3.0e-5], dtype=np.float32)
    b = W.bf16_bits_to_f32(W.f32_to_bf16_bits(v))
    assert b[0] == 1.0 and b[1] == 1.0 and b[2] == 1.0 + 2 ** -6 and b[3] == 1.0 + 2 ** -7
    assert np.all(np.abs(b - v) <= np.abs(v) * 2.0 ** -8)
    c = W.CONFIGS["cfg5"].scaled(d=1000)
    s, w = W.x0_row(c, 0)
    assert s.dtype == np.uint16 and np.array_equal(W.bf16_bits_to_f32(s).astype(np.float64), w)


def test_sample_columns_cover_edges():
    cols = W.sample_columns(10_007, 4096, 50, seed=1)
    assert cols[0] == 0 and cols[-1] == 10_006 and 4095 in cols and 4096 in cols and 8192 in cols
    assert np.all(np.diff(cols) > 0)


@pytest.mark.parametrize("graph", ["ring", "exponential", "complete"])
def test_fifo_pairing_model_pairs_neighbours_uniformly(graph):
    """App. E.2: with first-come-first-served pairing among available neighbours, the history of
    communications is close to uniform over the edges (the assumption behind chi_1, chi_2), and
    every worker does about `comms_per_grad` averagings per gradient."""
    n, r = 32, 1.0
    e = W.make_edges(graph, n)
    ev = W.fifo_pairing_events(n, e, r, 60_000, seed=11)
    assert np.all(np.diff(ev.times) >= 0)
    comm = ev.wj >= 0
    n_grad, n_comm = int((~comm).sum()), int(comm.sum())
    assert abs(2 * n_comm / n_grad - r) < 0.05  # an averaging counts for both of its workers
    lo, hi = np.minimum(ev.wi[comm], ev.wj[comm]), np.maximum(ev.wi[comm], ev.wj[comm])
    key = lo.astype(np.int64) * n + hi
    ekey = e[:, 0].astype(np.int64) * n + e[:, 1]
    assert set(np.unique(key)) <= set(ekey)  # only neighbours are paired
    hist = np.array([(key == k).sum() for k in ekey])
    m = hist.mean()
    assert np.all(np.abs(hist - m) < 0.15 * m + 5 * np.sqrt(m))
    part = np.bincount(np.concatenate([lo, hi]), minlength=n)
    grads = np.bincount(ev.wi[~comm], minlength=n)
    assert np.all(np.abs(part / grads - r) < 0.15)
    # a worker is never in two averagings at once: its communications are at least comm_duration apart
    for w in (0, n // 2):
        tw = ev.times[comm & ((ev.wi == w) | (ev.wj == w))]
        assert np.all(np.diff(tw) >= 0.05 - 1e-12)
    # gradient completions of a worker are about one unit apart
    tg = ev.times[(~comm) & (ev.wi == 3)]
    assert abs(np.diff(tg).mean() - 1.0) < 0.05
    ev2 = W.fifo_pairing_events(n, e, r, 60_000, seed=11)
    assert np.array_equal(ev.times, ev2.times) and np.array_equal(ev.wj, ev2.wj)
