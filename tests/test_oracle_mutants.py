"""Do the pins bite? Plausible mistakes are planted in copies of the C checker (on the CPU, in a
temporary directory): a dropped term, a wrong sign, swapped coefficients, a wrong index. For each
mutant at least one of the pins in test_oracle_pins.py must fail."""
import os
import subprocess

import pytest

import oracle.sim as sim_mod
from oracle import build as obuild
from tests import test_oracle_pins as pins

MUTANTS = {
    "mix_sign": ("xt[k] = xt[k] + c * dlt;", "xt[k] = xt[k] - c * dlt;"),
    "mix_rate": ("return -expm1(-2.0 * eta * dt) / 2.0;", "return -expm1(-1.0 * eta * dt) / 2.0;"),
    "mix_no_half": ("return -expm1(-2.0 * eta * dt) / 2.0;", "return -expm1(-2.0 * eta * dt);"),
    "grad_only_x": ("xti[k] = xti[k] - gamma * g[k];", "xti[k] = xti[k];"),
    "grad_sign": ("xi[k] = xi[k] - gamma * g[k];", "xi[k] = xi[k] + gamma * g[k];"),
    "grad_no_mix": ("a2o_mix(xi, xti, d, eta, t - tl[i]);\n            for (int64_t k = 0; k < d; ++k) {\n                xi[k] = xi[k] - gamma",
                    "for (int64_t k = 0; k < d; ++k) {\n                xi[k] = xi[k] - gamma"),
    "comm_j_sign": ("xj[k] = xj[k] + alpha * m;\n                    xtj[k] = xtj[k] + alpha_t * m;\n                }\n            } else {",
                    "xj[k] = xj[k] - alpha * m;\n                    xtj[k] = xtj[k] + alpha_t * m;\n                }\n            } else {"),
    "comm_swapped_coeffs": ("xi[k] = xi[k] - alpha * m;\n                    xti[k] = xti[k] - alpha_t * m;\n                    xj[k] = xj[k] + alpha * m;",
                            "xi[k] = xi[k] - alpha_t * m;\n                    xti[k] = xti[k] - alpha * m;\n                    xj[k] = xj[k] + alpha * m;"),
    "comm_tilde_uses_own_difference": ("const double m = xi[k] - xj[k];\n                    xi[k] = xi[k] - alpha * m;\n                    xti[k] = xti[k] - alpha_t * m;",
                                       "const double m = xi[k] - xj[k];\n                    xi[k] = xi[k] - alpha * m;\n                    xti[k] = xti[k] - alpha_t * (xti[k] - xtj[k]);"),
    "comm_mixes_one_worker": ("a2o_mix(xj, xtj, d, eta, t - tl[j]);\n                for", "for"),
    "comm_forgets_time_j": ("tl[i] = t;\n            tl[j] = t;", "tl[i] = t;"),
    "grad_forgets_time": ("xti[k] = xti[k] - gamma * g[k];\n            }\n            tl[i] = t;", "xti[k] = xti[k] - gamma * g[k];\n            }"),
    "wrong_gradient_row": ("const double* g = G + (size_t)s * ldg;", "const double* g = G + (size_t)i * ldg;"),
    "consensus_not_centred": ("mean /= (double)n;\n        for (int32_t i = 0; i < n; ++i) {\n            const double dev = X[(size_t)i * ld + k] - mean;",
                              "mean /= (double)(n + 1);\n        for (int32_t i = 0; i < n; ++i) {\n            const double dev = X[(size_t)i * ld + k] - mean;"),
    "plain_grad_sign": ("x[k] = x[k] - gamma * g[k];", "x[k] = x[k] + gamma * g[k];"),
    "plain_comm_j_sign": ("y[k] = y[k] + alpha * m;", "y[k] = y[k] - alpha * m;"),
    "plain_comm_message_reversed": ("const double m = x[k] - y[k];", "const double m = y[k] - x[k];"),
    "plain_comm_forgets_time_j": ("a2o_plain_comm(xi, xj, d, alpha);\n                tl[i] = t;\n                tl[j] = t;",
                                  "a2o_plain_comm(xi, xj, d, alpha);\n                tl[i] = t;"),
    "plain_grad_touches_tilde": ("a2o_plain_grad(xi, g, d, gamma);", "a2o_plain_grad(xi, g, d, gamma); a2o_plain_grad(xti, g, d, gamma);"),
    "consensus_at_ignores_flow": ("mean += x - c * (x - xt);", "mean += x;"),
    # the branch that follows Algorithm 1 as printed (message before the mixing line)
    "printed_order_sign_of_mixing_on_j": ("xj[k] = (xj[k] - cj * dj) + alpha * m;", "xj[k] = (xj[k] + cj * dj) + alpha * m;"),
    "printed_order_message_after_mixing": ("const double m = xi[k] - xj[k]; /* from the un-mixed buffers */",
                                           "const double m = (xi[k] - ci * (xi[k] - xti[k])) - (xj[k] - cj * (xj[k] - xtj[k]));"),
    "printed_order_swapped_coeffs": ("xi[k] = (xi[k] - ci * di) - alpha * m;\n                    xti[k] = (xti[k] + ci * di) - alpha_t * m;",
                                     "xi[k] = (xi[k] - ci * di) - alpha_t * m;\n                    xti[k] = (xti[k] + ci * di) - alpha * m;"),
    "printed_order_tilde_mixed_with_wrong_sign": ("xti[k] = (xti[k] + ci * di) - alpha_t * m;", "xti[k] = (xti[k] - ci * di) - alpha_t * m;"),
}

# pins that take the simulator class, and pins that use OracleSim directly
DETECTORS = [
    lambda: pins.test_mixing_keeps_half_sum_and_shrinks_difference(pins.OracleSim),
    lambda: pins.test_mixing_semigroup(pins.OracleSim),
    lambda: pins.test_mixing_matches_series_of_the_generator(),
    lambda: pins.test_comm_keeps_population_sums(pins.OracleSim),
    lambda: pins.test_comm_consensus_drop_identity(0.3),
    lambda: pins.test_two_workers_reach_exact_consensus_in_one_event(pins.OracleSim),
    lambda: pins.test_baseline_equals_textbook_gossip_sgd(pins.OracleSim),
    lambda: pins.test_mean_tracker_identity(),
    lambda: pins.test_brute_force_matrix_exponential(pins.OracleSim, 3, 3, "complete"),
    lambda: pins.test_consensus_at_common_time_matches_flushed_state_and_definition(),
    lambda: pins.test_hand_example(pins.OracleSim),
    lambda: pins.test_plain_dynamic_is_a_product_of_gossip_matrices(pins.OracleSim, 0.3),
    lambda: pins.test_plain_dynamic_is_the_full_one_without_drift(),
    lambda: pins.test_algorithm1_ordering_against_series_exponential(pins.OracleSim, 4, 3, "ring"),
    lambda: pins.test_hand_example_algorithm1_ordering(pins.OracleSim),
]

# mistakes planted in the branch of Algorithm 1's printed ordering must be caught by the pins of that
# branch, which do not consult the NumPy twin
PRINTED_ORDER_DETECTORS = (13, 14)


def _caught():
    failed = []
    for k, det in enumerate(DETECTORS):
        try:
            det()
        except (AssertionError, sim_mod.OracleError):
            failed.append(k)
    return failed


def test_unmutated_checker_passes_every_detector():
    assert _caught() == []


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_planted_mistake_is_caught(name, tmp_path, monkeypatch):
    old, new = MUTANTS[name]
    src = open(obuild.SRC).read()
    assert src.count(old) >= 1, f"mutation site for {name} not found"
    mutated = src.replace(old, new, 1)
    c = tmp_path / "mutant.c"
    so = tmp_path / "mutant.so"
    c.write_text(mutated)
    subprocess.run(["gcc", "-O1", "-std=c99", "-ffp-contract=off", "-fPIC", "-shared", "-o", str(so), str(c), "-lm"],
                   check=True)
    monkeypatch.setattr(sim_mod, "_lib", sim_mod.load(str(so)))
    caught = _caught()
    assert caught, f"no pin noticed the planted mistake '{name}'"
    if name.startswith("printed_order_"):
        assert set(caught) & set(PRINTED_ORDER_DETECTORS), caught
