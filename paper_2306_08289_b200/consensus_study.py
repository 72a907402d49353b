"""Consensus distance with and without the continuous momentum, on synthetic gradients.

The paper tracks the consensus distance between workers during ImageNet training on a ring of 64
workers and finds that adding A2CiD2 at one averaging per gradient step lowers it as much as
doubling the communication rate does (Sec. 4.2 "Consensus improvement", the consensus-distance panel of the ImageNet figure). Neither the
data nor the model are here; this script replays the same comparison with the engine on gradients
that are fresh zero-mean Gaussian draws (a pool of rows per worker), starting from consensus as the
paper does (one All-Reduce before training). It is an experiment, not a parity target.

    python -m paper_2306_08289_b200.consensus_study [--n 64] [--d 262144] [--T 300]
    python -m paper_2306_08289_b200.consensus_study --closed-loop [--d 65536] [--T 150] [--gamma 0.05]

prints, for the baseline (eta = 0, alpha = alpha~ = 1/2) at 1 and 2 averagings per gradient and for
A2CiD2 (the convergence proposition of Sec. 3.4 parameters) at 1 and 2, the consensus distance sum_i |x_i - xbar|^2 / d at ten
common evaluation times. With --closed-loop the gradients are not noise but those of a heterogeneous
quadratic, evaluated at each worker's current parameters, so the run is decentralised SGD proper; it
prints the distance of the workers' mean to the minimiser and the consensus distance.
"""
from __future__ import annotations

import argparse
import json

import numpy as np

from . import binding as B
from . import workload as W


def run_setting(n, d, graph, comms_per_grad, accelerated, T, gamma, g_std, pool, seed, samples=10, device="cuda:0",
                flags=B.A2_SCHED_FUSE):
    edges = W.make_edges(graph, n)
    rates = W.edge_rates_per_worker(n, edges, comms_per_grad)
    chi1, chi2 = B.graph_chi(n, edges, rates)
    eta, alpha, alpha_t = B.prescribe(chi1, chi2, accelerated)
    n_events = int((n + rates.sum()) * T)
    ev = W.poisson_events(n, edges, rates, n_events, seed=seed, grad_pool=pool)
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, 7])))
    x0 = np.tile((rng.standard_normal(d) * 0.02).astype(np.float32), (n, 1))  # consensus at the start
    # the baseline has eta = 0 and alpha~ = alpha: x~ would stay a copy of x, so it runs without the buffer
    eng = B.Engine(n, d, eta, alpha, alpha_t, gamma, n_grad_slots=n * pool, device=device, momentum=bool(accelerated))
    eng.write_state(x0)
    for row in range(n * pool):
        eng.fill_row("g", row, (rng.standard_normal(d) * g_std).astype(np.float32))
    out = []
    step = max(1, n_events // samples)
    for k in range(0, n_events, step):
        c = ev.slice(k, k + step)
        if len(c) == 0:
            break
        eng.apply_events(c.times, c.wi, c.wj, c.slot, flags=flags)
        t_eval = float(c.times[-1])
        out.append((t_eval, eng.consensus_distance(t_eval) / d))  # every worker mixed forward to the same time
    eng.close()
    return {"comms_per_grad": comms_per_grad, "accelerated": bool(accelerated), "eta": eta, "alpha_tilde": alpha_t,
            "chi1": chi1, "chi2": chi2, "events": n_events, "trace": out}


def run_study(n=64, d=262_144, graph="ring", T=300.0, gamma=0.1, g_std=1e-3, pool=64, seed=5, device="cuda:0"):
    settings = [(1.0, False), (2.0, False), (1.0, True), (2.0, True)]
    return [run_setting(n, d, graph, r, acc, T, gamma, g_std, pool, seed, device=device) for r, acc in settings]


# ------------------------------------------------------------------------------------------------
# closed loop: the gradient of every event is computed from the worker's current parameters
# ------------------------------------------------------------------------------------------------
class Quadratic:
    """f_i(x) = 1/2 sum_k a_ik (x_k - b_ik)^2 with a_ik in [0.5, 1.5] (mu = 0.5, L = 1.5) and heterogeneous
    targets b_i ~ N(0, 1). The minimiser of (1/n) sum_i f_i is x*_k = sum_i a_ik b_ik / sum_i a_ik."""

    def __init__(self, n, d, seed):
        rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, 11])))
        self.a = rng.uniform(0.5, 1.5, size=(n, d))
        self.b = rng.standard_normal((n, d))
        self.x_star = (self.a * self.b).sum(0) / self.a.sum(0)


def closed_loop_batches(sched, ev):
    """For every batch of an unfused schedule: its event indices, and the (worker, slot) pairs of its
    gradient events, whose gradient rows have to be produced before the batch runs."""
    out = []
    for b in range(sched.num_batches):
        idx = sched.batch_events(b)
        g = idx[ev.wj[idx] < 0]
        out.append((idx, ev.wi[g].astype(np.int64), ev.slot[g].astype(np.int64)))
    return out


def closed_loop_problem(n, d, graph, comms_per_grad, T, seed):
    """The quadratic, the graph and the event stream of a closed-loop run (shared with the tests)."""
    edges = W.make_edges(graph, n)
    rates = W.edge_rates_per_worker(n, edges, comms_per_grad)
    n_events = int((n + rates.sum()) * T)
    return Quadratic(n, d, seed), edges, rates, W.poisson_events(n, edges, rates, n_events, seed=seed)


def run_closed_loop(n, d, graph, comms_per_grad, accelerated, T, gamma, seed, samples=10, noise_std=0.0,
                    device="cuda:0"):
    """Decentralised SGD on the quadratic with the engine. As in Algorithm 1 the gradient is evaluated
    at the worker's stored parameters when its gradient event fires, then the mixing and the step are
    applied. Gradients are the user's model, not the library's: they are computed here with torch and
    handed over as rows of the gradient buffer, batch by batch."""
    prob, edges, rates, ev = closed_loop_problem(n, d, graph, comms_per_grad, T, seed)
    n_events = len(ev)
    x0 = np.zeros((n, d), dtype=np.float32)
    trace = []
    step = max(1, n_events // samples)
    import torch

    chi1, chi2 = B.graph_chi(n, edges, rates)
    eta, alpha, alpha_t = B.prescribe(chi1, chi2, accelerated)
    eng = B.Engine(n, d, eta, alpha, alpha_t, gamma, n_grad_slots=n, device=device, momentum=bool(accelerated))
    eng.write_state(x0)
    a = torch.from_numpy(prob.a.astype(np.float32)).to(device)
    bt = torch.from_numpy(prob.b.astype(np.float32)).to(device)
    xs = torch.from_numpy(prob.x_star).to(device)
    gen = torch.Generator(device=device).manual_seed(seed)
    for k in range(0, n_events, step):
        c = ev.slice(k, k + step)
        plan = eng.plan(c.times, c.wi, c.wj, c.slot, flags=0)
        for bi, (_, workers, slots) in enumerate(closed_loop_batches(plan.sched, c)):
            if len(workers):
                w = torch.from_numpy(workers).to(device)
                g = a[w] * (eng.x[w, :d] - bt[w])
                if noise_std > 0:
                    g = g + noise_std * torch.randn(g.shape, generator=gen, device=device)
                eng.g[torch.from_numpy(slots).to(device), :d] = g
            plan.run(bi, 1)
        plan.close()
        t = float(c.times[-1])
        eng.flush(t)
        eng.sync()
        xbar = eng.x[:, :d].double().mean(0)
        trace.append((t, float(((xbar - xs) ** 2).mean()), eng.consensus_distance() / d))
    x_final = eng.read_state()[0].astype(np.float64)
    eng.close()
    return {"comms_per_grad": comms_per_grad, "accelerated": bool(accelerated), "events": n_events, "trace": trace,
            "x_final": x_final}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--n", type=int, default=64)
    ap.add_argument("--d", type=int, default=262_144)
    ap.add_argument("--graph", default="ring")
    ap.add_argument("--T", type=float, default=300.0)
    ap.add_argument("--json", action="store_true")
    ap.add_argument("--closed-loop", action="store_true", help="decentralised SGD on a synthetic quadratic instead")
    ap.add_argument("--gamma", type=float, default=0.05)
    a = ap.parse_args()
    if a.closed_loop:
        for r, acc in [(1.0, False), (2.0, False), (1.0, True), (2.0, True)]:
            res = run_closed_loop(a.n, a.d, a.graph, r, acc, a.T, a.gamma, seed=5)
            name = ("A2CiD2  " if acc else "baseline") + f" {r:.0f} com/grad"
            print(f"{name}  |xbar-x*|^2/d: " + " ".join(f"{v:.2e}" for _, v, _ in res["trace"]))
            print(f"{' ' * len(name)}  consensus/d:   " + " ".join(f"{v:.2e}" for _, _, v in res["trace"]))
        return
    res = run_study(n=a.n, d=a.d, graph=a.graph, T=a.T)
    if a.json:
        print(json.dumps(res))
        return
    for r in res:
        name = ("A2CiD2  " if r["accelerated"] else "baseline") + f" {r['comms_per_grad']:.0f} com/grad"
        print(f"{name}  eta={r['eta']:.4f} alpha~={r['alpha_tilde']:.3f}  " +
              " ".join(f"{v:.3e}" for _, v in r["trace"]))


if __name__ == "__main__":
    main()
