"""Consensus distance with and without the continuous momentum, on synthetic gradients.

The paper tracks the consensus distance between workers during ImageNet training on a ring of 64
workers and finds that adding A2CiD2 at one averaging per gradient step lowers it as much as
doubling the communication rate does (Sec. 4.2 "Consensus improvement", the consensus-distance panel of the ImageNet figure). Neither the
data nor the model are here; this script replays the same comparison with the engine on gradients
that are fresh zero-mean Gaussian draws (a pool of rows per worker), starting from consensus as the
paper does (one All-Reduce before training). It is an experiment, not a parity target.

    python -m paper_2306_08289_b200.consensus_study [--n 64] [--d 262144] [--T 300]

prints, for the baseline (eta = 0, alpha = alpha~ = 1/2) at 1 and 2 averagings per gradient and for
A2CiD2 (the convergence proposition of Sec. 3.4 parameters) at 1 and 2, the consensus distance sum_i |x_i - xbar|^2 / d at ten
common evaluation times.
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
    eng = B.Engine(n, d, eta, alpha, alpha_t, gamma, n_grad_slots=n * pool, device=device)
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--n", type=int, default=64)
    ap.add_argument("--d", type=int, default=262_144)
    ap.add_argument("--graph", default="ring")
    ap.add_argument("--T", type=float, default=300.0)
    ap.add_argument("--json", action="store_true")
    a = ap.parse_args()
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
