"""Where the element-wise bound of the bf16 parity tests comes from, measured on the CPU.

The GPU keeps bf16 rows and does fp32 arithmetic between two stores; the checker's storage-modelled run
does fp64 arithmetic between the same stores. Both are correct. This test runs two such implementations
on the CPU -- the fp64 checker with its rows rounded to bf16 after every event, and a NumPy float32
restatement of the same steps (Eq. (dynamic): mixing, gradient jump, pairwise jump) with the same
rounding points -- and records how far apart they end, in bf16 units in the last place. The bounds the
GPU tests apply (tests/parity.py) must contain this figure with the margin stated there."""
import numpy as np

from oracle import spectral
from oracle.sim import OracleSim, round_to_bf16
from paper_2306_08289_b200 import workload as W
from tests import parity as P

f32 = np.float32


def _float32_run_with_bf16_stores(cfg, x0, G, ev, eta, alpha, at):
    X = x0.astype(f32)
    Xt = X.copy()
    G32 = G.astype(f32)
    tl = np.zeros(cfg.n)

    def store(a):
        return round_to_bf16(a.astype(np.float64)).astype(f32)

    def mix(w, t):
        c = f32(-np.expm1(-2.0 * eta * (t - tl[w])) / 2.0)
        dlt = X[w] - Xt[w]
        X[w] = X[w] - c * dlt
        Xt[w] = Xt[w] + c * dlt
        tl[w] = t

    for t, i, j, s in zip(ev.times, ev.wi, ev.wj, ev.slot):
        if j < 0:
            mix(i, t)
            X[i] = store(X[i] - f32(cfg.gamma) * G32[s])
            Xt[i] = store(Xt[i] - f32(cfg.gamma) * G32[s])
        else:
            mix(i, t)
            mix(j, t)
            m = X[i] - X[j]
            X[i], Xt[i] = store(X[i] - f32(alpha) * m), store(Xt[i] - f32(at) * m)
            X[j], Xt[j] = store(X[j] + f32(alpha) * m), store(Xt[j] + f32(at) * m)
    return X, Xt


def test_two_correct_bf16_storage_runs_differ_by_a_few_ulps():
    cfg = W.CONFIGS["cfg5"].scaled(d=2_000, n_events=10_000)
    _, x0 = W.x0_matrix(cfg)
    _, G = W.grad_matrix(cfg)
    ev = W.config_events(cfg)
    eta, alpha, at = spectral.prescribe(cfg.n, cfg.edges(), cfg.rates())[:3]
    ref = OracleSim(x0, eta, alpha, at, cfg.gamma, grads=G)
    for k in range(len(ev)):
        ref.apply_stream(ev.slice(k, k + 1))
        ref.round_rows([ev.wi[k]] + ([ev.wj[k]] if ev.wj[k] >= 0 else []))
    X, Xt = _float32_run_with_bf16_stores(cfg, x0, G, ev, eta, alpha, at)
    u = np.concatenate([P.bf16_ulp_distance(X, ref.X).ravel(), P.bf16_ulp_distance(Xt, ref.Xt).ravel()])
    h = P.ulp_histogram(u)
    print(h)
    # measured: max 3-4 ulps, 98.5 % identical, 99.9 % within one ulp, 5e-5 beyond two
    assert 1.0 <= h["max"] <= 5.0                      # they do differ, by a few ulps
    assert h["eq"] / h["n"] >= 0.975
    assert h["le1"] / h["n"] >= 0.998
    assert h["gt2"] / h["n"] <= 5e-4
    # the GPU tests' bounds contain this with margin for 1e4 times more elements (the tail falls about
    # tenfold per ulp, so four more ulps)
    assert P.BF16_ULP_BOUND >= h["max"] + 3 and P.BF16_MIN_EXACT <= 0.975 and P.BF16_MIN_WITHIN_1 <= 0.998


def test_ulp_helper():
    assert P.ulp_bf16(1.0) == 2.0 ** -7 and P.ulp_bf16(1.99) == 2.0 ** -7 and P.ulp_bf16(2.0) == 2.0 ** -6
    assert P.ulp_bf16(0.02) == 2.0 ** -13
    ref = np.array([[1.0, 1.0, 1e-9, 1.0]])
    gpu = np.array([[1.0, 1.0 + 2.0 ** -7, 1e-9 + 2.0 ** -7, 1.0 - 3 * 2.0 ** -7]])
    u = P.bf16_ulp_distance(gpu, ref)
    # the near-zero element is measured in ulps of the row's rms (0.87 -> 2^-8), not of itself
    np.testing.assert_allclose(u[0], [0.0, 1.0, 2.0, 3.0], rtol=1e-12)
    h = P.ulp_histogram(np.round(u))
    assert h == {"n": 4, "eq": 1, "le1": 2, "le2": 3, "gt2": 1, "max": 3.0}
