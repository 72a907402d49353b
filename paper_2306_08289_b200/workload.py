"""Seeded synthetic inputs: graphs, edge rates, Poisson event streams, x0 and gradient rows.

This module only *draws inputs*. It holds none of the method's arithmetic (no mixing, no
averaging, no spectral quantities) and imports neither the CUDA binding nor the CPU
checker, so both can be fed from it.

What it models, from the paper:
  * the three topologies of the experiments (complete, ring/cycle, exponential), Sec. 4.1
    "Practical implementation" and App. E.1;
  * independent Poisson clocks, rate 1 per worker for gradient events and rate lambda^{ij}
    per edge for pairwise communications (the Poisson-process assumption of Sec. 3.4);
  * "r p2p communications per gradient computation for each worker" with peers picked
    uniformly among neighbours (Sec. 4.1 hyper-parameters, App. E.2): every worker takes
    part in r averagings per unit time, so lambda^{ij} = r / degree on a regular graph.

Random streams are NumPy `Generator(PCG64(SeedSequence([seed, tag, row])))`, one
independent child stream per array row and one for the event stream, so any row can be
regenerated alone (the large configurations are filled row by row).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

TAG_X0 = 1
TAG_G = 2
TAG_EVENTS = 3


# --------------------------------------------------------------------------------------
# graphs
# --------------------------------------------------------------------------------------
def ring_edges(n: int) -> np.ndarray:
    """Cycle 0-1-...-(n-1)-0. n = 2 collapses to a single edge."""
    if n < 2:
        raise ValueError("need n >= 2")
    if n == 2:
        return np.array([[0, 1]], dtype=np.int32)
    e = [(i, (i + 1) % n) for i in range(n)]
    return _canon(e)


def complete_edges(n: int) -> np.ndarray:
    if n < 2:
        raise ValueError("need n >= 2")
    return _canon([(i, j) for i in range(n) for j in range(i + 1, n)])


def exponential_edges(n: int) -> np.ndarray:
    """Undirected circulant with offsets 2^k, k = 0 .. ceil(log2 n) - 1.

    Peers of i are i +- 2^k (mod n); duplicate pairs (the +-n/2 offset) are merged, so for
    n a power of two the degree is 2*log2(n) - 1.
    """
    if n < 2:
        raise ValueError("need n >= 2")
    e = set()
    k = 1
    while k < n:
        for i in range(n):
            j = (i + k) % n
            if i != j:
                e.add((min(i, j), max(i, j)))
        k *= 2
    return _canon(sorted(e))


def _canon(pairs) -> np.ndarray:
    a = np.array([(min(i, j), max(i, j)) for i, j in pairs], dtype=np.int32)
    a = np.unique(a, axis=0)
    return np.ascontiguousarray(a)


def make_edges(graph: str, n: int) -> np.ndarray:
    if graph == "ring":
        return ring_edges(n)
    if graph == "complete":
        return complete_edges(n)
    if graph == "exponential":
        return exponential_edges(n)
    raise ValueError(f"unknown graph {graph!r}")


def degrees(n: int, edges: np.ndarray) -> np.ndarray:
    deg = np.zeros(n, dtype=np.int64)
    np.add.at(deg, edges[:, 0], 1)
    np.add.at(deg, edges[:, 1], 1)
    return deg


def edge_rates_per_worker(n: int, edges: np.ndarray, comms_per_grad: float) -> np.ndarray:
    """lambda^{ij} such that each worker takes part in `comms_per_grad` averagings per unit
    time when peers are chosen uniformly (regular graphs only)."""
    deg = degrees(n, edges)
    if not np.all(deg == deg[0]):
        raise ValueError("per-worker rate convention needs a regular graph")
    return np.full(len(edges), float(comms_per_grad) / float(deg[0]), dtype=np.float64)


# --------------------------------------------------------------------------------------
# configurations
# --------------------------------------------------------------------------------------
@dataclass(frozen=True)
class WorkloadConfig:
    """One synthetic workload. Hyper-parameters that the paper derives from the graph
    (eta, alpha_tilde) are *not* stored here unless the configuration fixes them outright:
    each side computes them from (edges, rates) with its own code."""

    name: str
    n: int
    graph: str
    d: int
    storage: str  # "f32" or "bf16"
    n_events: int
    x0_std: float
    g_std: float
    gamma: float
    edge_rate: float | None = None  # rate per edge, given outright
    comms_per_grad: float | None = None  # else: averagings per worker per unit time
    fixed_params: tuple | None = None  # (eta, alpha, alpha_tilde) if given outright
    consensus_every: int = 0
    grad_pool: int = 1  # gradient rows per worker, used round-robin by its gradient events
    seed: int = 0
    note: str = ""

    @property
    def n_grad_slots(self) -> int:
        return self.n * self.grad_pool

    def edges(self) -> np.ndarray:
        return make_edges(self.graph, self.n)

    def rates(self) -> np.ndarray:
        e = self.edges()
        if self.edge_rate is not None:
            return np.full(len(e), float(self.edge_rate), dtype=np.float64)
        return edge_rates_per_worker(self.n, e, self.comms_per_grad)

    def scaled(self, d: int | None = None, n_events: int | None = None, name: str | None = None):
        """Same recipe at another width / stream length (for parity cases sized for the CPU)."""
        from dataclasses import replace

        return replace(
            self,
            d=self.d if d is None else int(d),
            n_events=self.n_events if n_events is None else int(n_events),
            name=name or f"{self.name}-d{d or self.d}-e{n_events or self.n_events}",
        )


CONFIGS = {
    # n=4 ring, unit rate per edge and per worker, all hyper-parameters given outright.
    "cfg1": WorkloadConfig(
        name="cfg1", n=4, graph="ring", d=10_000, storage="f32", n_events=2_000,
        x0_std=1.0, g_std=1.0, gamma=0.01, edge_rate=1.0, fixed_params=(0.5, 0.5, 0.5), grad_pool=16,
        seed=1001, note="n=4 ring, d=1e4 fp32"),
    # n=16 complete, one averaging per worker per gradient step.
    "cfg2": WorkloadConfig(
        name="cfg2", n=16, graph="complete", d=1_000_000, storage="f32", n_events=50_000,
        x0_std=1.0, g_std=0.1, gamma=0.01, comms_per_grad=1.0, grad_pool=128,
        seed=1002, note="n=16 complete, d=1e6 fp32"),
    # n=32 ring, ResNet-18-sized flat vector, rate 2 per edge.
    "cfg3": WorkloadConfig(
        name="cfg3", n=32, graph="ring", d=11_700_000, storage="f32", n_events=20_000,
        x0_std=0.02, g_std=1e-3, gamma=0.1, edge_rate=2.0,
        seed=1003, note="n=32 ring, d=11.7e6 fp32 (ResNet-18-sized)"),
    # n=64 ring, ResNet-50-sized flat vector, one averaging per worker per gradient step.
    "cfg4": WorkloadConfig(
        name="cfg4", n=64, graph="ring", d=25_600_000, storage="f32", n_events=10_000,
        x0_std=0.02, g_std=1e-3, gamma=0.1, comms_per_grad=1.0, consensus_every=500,
        seed=1004, note="n=64 ring, d=25.6e6 fp32 (ResNet-50-sized)"),
    # n=64 exponential graph, bf16 storage, two averagings per worker per gradient step.
    "cfg5": WorkloadConfig(
        name="cfg5", n=64, graph="exponential", d=25_600_000, storage="bf16", n_events=10_000,
        x0_std=0.02, g_std=1e-3, gamma=0.1, comms_per_grad=2.0,
        seed=1005, note="n=64 exponential, d=25.6e6 bf16 storage"),
}


# --------------------------------------------------------------------------------------
# event stream
# --------------------------------------------------------------------------------------
@dataclass
class EventStream:
    """Time-sorted events. A gradient event has wj = -1 and slot >= 0; a communication
    event has wj >= 0 and slot = -1."""

    times: np.ndarray  # float64, non-decreasing
    wi: np.ndarray  # int32
    wj: np.ndarray  # int32
    slot: np.ndarray  # int32
    meta: dict = field(default_factory=dict)

    def __len__(self) -> int:
        return int(self.times.shape[0])

    def slice(self, a: int, b: int) -> "EventStream":
        return EventStream(self.times[a:b].copy(), self.wi[a:b].copy(), self.wj[a:b].copy(),
                           self.slot[a:b].copy(), dict(self.meta))


def _rng(seed: int, tag: int, row: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(seed), int(tag), int(row)])))


def poisson_events(n: int, edges: np.ndarray, rates: np.ndarray, n_events: int, seed: int,
                   grad_rate: float = 1.0, t0: float = 0.0, stream_id: int = 0, grad_pool: int = 1) -> EventStream:
    """Superposition of independent Poisson clocks (the Poisson-process assumption of Sec. 3.4): one clock of rate
    `grad_rate` per worker and one of rate rates[e] per edge. The superposition is a Poisson
    process of rate R = n*grad_rate + sum(rates); each event belongs to a clock with
    probability rate/R. Worker i owns the gradient rows i, i + n, ..., i + (grad_pool-1) n and
    its k-th gradient event uses row i + n (k mod grad_pool): the paper's stochastic gradients
    are fresh draws at every step (Sec. 3.2), a pool of rows stands in for them."""
    edges = np.asarray(edges, dtype=np.int32).reshape(-1, 2)
    rates = np.asarray(rates, dtype=np.float64)
    if rates.shape[0] != edges.shape[0]:
        raise ValueError("one rate per edge")
    clock_rates = np.concatenate([np.full(n, float(grad_rate)), rates])
    total = float(clock_rates.sum())
    rng = _rng(seed, TAG_EVENTS, stream_id)
    gaps = rng.exponential(1.0 / total, size=n_events)
    times = t0 + np.cumsum(gaps)
    u = rng.random(n_events) * total
    cum = np.cumsum(clock_rates)
    which = np.minimum(np.searchsorted(cum, u, side="right"), len(clock_rates) - 1)
    is_grad = which < n
    wi = np.empty(n_events, dtype=np.int32)
    wj = np.full(n_events, -1, dtype=np.int32)
    slot = np.full(n_events, -1, dtype=np.int32)
    wi[is_grad] = which[is_grad]
    gw = which[is_grad]
    # k-th gradient event of each worker -> k (stable sort groups a worker's events in time order)
    order = np.argsort(gw, kind="stable")
    starts = np.concatenate([[0], np.cumsum(np.bincount(gw, minlength=n))[:-1]])
    kth = np.empty(len(gw), dtype=np.int64)
    kth[order] = np.arange(len(gw)) - starts[gw[order]]
    slot[is_grad] = gw + n * (kth % max(1, int(grad_pool)))
    e_idx = which[~is_grad] - n
    wi[~is_grad] = edges[e_idx, 0]
    wj[~is_grad] = edges[e_idx, 1]
    return EventStream(np.ascontiguousarray(times, dtype=np.float64), wi, wj, slot,
                       {"total_rate": total, "n": n, "seed": seed})


def config_events(cfg: WorkloadConfig, n_events: int | None = None, t0: float = 0.0,
                  stream_id: int = 0) -> EventStream:
    return poisson_events(cfg.n, cfg.edges(), cfg.rates(), cfg.n_events if n_events is None else n_events,
                          cfg.seed, t0=t0, stream_id=stream_id, grad_pool=cfg.grad_pool)


def fifo_pairing_events(n: int, edges: np.ndarray, comms_per_grad: float, n_events: int, seed: int,
                        comm_duration: float = 0.05, jitter: float = 0.1, grad_pool: int = 1,
                        stream_id: int = 0) -> EventStream:
    """The event model of the paper's implementation (Sec. 4.1 "Practical implementation", App. E.2)
    instead of ideal Poisson clocks. Every worker computes gradients back to back; one gradient
    takes a unit of time times a log-normal jitter. After each gradient it draws a Poisson(
    comms_per_grad) number of averagings still to do. A worker is *available* when it is not
    averaging and has averagings left; a coordinator keeps the available workers in a
    first-in-first-out queue and pairs a newly available worker with the longest-waiting available
    neighbour. An averaging occupies both workers for `comm_duration` and counts for both.
    Events are emitted in time order: a gradient event when a gradient completes, a communication
    event at the moment of pairing. Gradient rows as in `poisson_events`."""
    import heapq

    edges = np.asarray(edges, dtype=np.int32).reshape(-1, 2)
    nbr = [set() for _ in range(n)]
    for i, j in edges:
        nbr[int(i)].add(int(j))
        nbr[int(j)].add(int(i))
    rng = _rng(seed, TAG_EVENTS, 1000 + stream_id)
    todo = [0] * n
    busy = [False] * n
    n_grad = [0] * n
    queue: list[int] = []  # available workers, longest-waiting first
    heap: list[tuple[float, int, int, int]] = []  # (time, tie-break, kind, worker); kind 0: gradient done, 1: averaging done
    tick = 0

    def push(t, kind, w):
        nonlocal tick
        heapq.heappush(heap, (t, tick, kind, w))
        tick += 1

    def duration():
        return float(np.exp(jitter * rng.standard_normal() - 0.5 * jitter * jitter))

    for w in range(n):
        push(duration(), 0, w)
    times, wi, wj, slot = [], [], [], []

    def try_enqueue(w, t):
        if todo[w] <= 0 or busy[w] or w in queue:
            return
        for pos, other in enumerate(queue):
            if other in nbr[w]:
                queue.pop(pos)
                times.append(t); wi.append(other); wj.append(w); slot.append(-1)
                for v in (w, other):
                    todo[v] -= 1
                    busy[v] = True
                    push(t + comm_duration, 1, v)
                return
        queue.append(w)

    while len(times) < n_events:
        t, _, kind, w = heapq.heappop(heap)
        if kind == 0:
            times.append(t); wi.append(w); wj.append(-1); slot.append(w + n * (n_grad[w] % max(1, grad_pool)))
            n_grad[w] += 1
            todo[w] += int(rng.poisson(comms_per_grad))
            push(t + duration(), 0, w)
        else:
            busy[w] = False
        try_enqueue(w, t)
    k = n_events
    return EventStream(np.array(times[:k], dtype=np.float64), np.array(wi[:k], dtype=np.int32),
                       np.array(wj[:k], dtype=np.int32), np.array(slot[:k], dtype=np.int32),
                       {"n": n, "seed": seed, "model": "fifo"})


# --------------------------------------------------------------------------------------
# state and gradient rows
# --------------------------------------------------------------------------------------
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bfloat16 bit patterns (uint16). Inputs are finite."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _row(seed: int, tag: int, row: int, d: int, std: float, storage: str,
         cols: np.ndarray | None = None):
    """One row of N(0, std^2) values in the storage precision.

    Returns (stored, widened): `stored` is float32, or uint16 bf16 bit patterns; `widened`
    is the same values as float64, so that every consumer starts from identical numbers."""
    v = _rng(seed, tag, row).standard_normal(d, dtype=np.float32) * np.float32(std)
    if cols is not None:
        v = v[cols]
    if storage == "f32":
        return v, v.astype(np.float64)
    if storage == "bf16":
        b = f32_to_bf16_bits(v)
        return b, bf16_bits_to_f32(b).astype(np.float64)
    raise ValueError(storage)


def x0_row(cfg: WorkloadConfig, row: int, cols: np.ndarray | None = None):
    return _row(cfg.seed, TAG_X0, row, cfg.d, cfg.x0_std, cfg.storage, cols)


def grad_row(cfg: WorkloadConfig, slot: int, cols: np.ndarray | None = None):
    return _row(cfg.seed, TAG_G, slot, cfg.d, cfg.g_std, cfg.storage, cols)


def x0_matrix(cfg: WorkloadConfig):
    """Full [n, d] x0 (stored, widened). Only for configurations that fit host memory."""
    rows = [x0_row(cfg, i) for i in range(cfg.n)]
    return np.stack([r[0] for r in rows]), np.stack([r[1] for r in rows])


def grad_matrix(cfg: WorkloadConfig):
    rows = [grad_row(cfg, i) for i in range(cfg.n_grad_slots)]
    return np.stack([r[0] for r in rows]), np.stack([r[1] for r in rows])


def sample_columns(d: int, tile: int, n_random: int, seed: int) -> np.ndarray:
    """Column indices for spot checks at full size: the first and last vectors, both sides of
    a few tile boundaries, the ragged tail, and random interior columns. Sorted, unique."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(seed), 99])))
    pick = [np.arange(0, min(d, 16)), np.arange(max(0, d - 16), d)]
    n_tiles = (d + tile - 1) // tile
    for tb in sorted(set([1, 2, n_tiles // 2, n_tiles - 1])):
        c = tb * tile
        if 0 < c < d:
            pick.append(np.arange(max(0, c - 8), min(d, c + 8)))
    if n_random > 0:
        pick.append(rng.integers(0, d, size=n_random))
    return np.unique(np.concatenate(pick)).astype(np.int64)
