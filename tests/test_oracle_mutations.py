"""The pins must catch plausible mistakes.  Each case plants ONE mistake in a copy of the oracle
(a dropped term, a wrong sign, a swapped operand) and checks that at least one of the pin tests
then fails.  The mistakes are planted in the oracle's source, on the CPU; the real oracle is
untouched."""
import importlib
import os
import sys
import types

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = open(os.path.join(ROOT, "oracle", "flop_oracle.py")).read()

# (name, text in the oracle, planted replacement, pin tests expected to notice: module.function)
MUTANTS = [
    ("stretch_sign", "s_bar = s * (zeta - gamma) + gamma", "s_bar = s * (zeta - gamma) - gamma",
     ["test_oracle_gates.test_monte_carlo_matches_eq3_and_upper_clamp"]),
    ("temperature_inverted", "+ a) / beta)", "+ a) * beta)",
     ["test_oracle_gates.test_monte_carlo_matches_eq3_and_upper_clamp"]),
    ("eq3_sign", "- beta * np.log(-gamma / zeta))", "+ beta * np.log(-gamma / zeta))",
     ["test_oracle_gates.test_closed_form_values_golden"]),
    ("dz_dalpha_missing_beta", "(zeta - gamma) * s * (1.0 - s) / beta, 0.0)", "(zeta - gamma) * s * (1.0 - s), 0.0)",
     ["test_oracle_gates.test_dz_dalpha_finite_differences"]),
    ("forward_drops_gate", "    Y = Hp @ P.T\n    return H, Hp, Y", "    Y = H @ P.T\n    return H, Hp, Y",
     ["test_oracle_layer.test_sum_of_rank_one_components"]),
    ("forward_transposed_Q", "    H = X @ Q.T\n    Hp = H * z[None, :]\n    Y = Hp @ P.T", "    H = X @ Q[:, ::-1].T\n    Hp = H * z[None, :]\n    Y = Hp @ P.T",
     ["test_oracle_layer.test_sum_of_rank_one_components"]),
    ("dP_uses_ungated_H", "dP = dY.T @ Hp\n", "dP = dY.T @ H\n",
     ["test_oracle_layer.test_backward_matches_central_finite_differences"]),
    ("dz_uses_gated_H", "dP = dY.T @ Hp\n    dz = np.sum(H * dHp, axis=0)", "dP = dY.T @ Hp\n    dz = np.sum(Hp * dHp, axis=0)",
     ["test_oracle_layer.test_three_forms_of_dz_agree"]),
    ("dQ_drops_gate", "dQ = dH.T @ X", "dQ = dHp.T @ X",
     ["test_oracle_layer.test_backward_matches_central_finite_differences"]),
    ("dX_drops_gate", "dX = dH @ Q", "dX = dHp @ Q",
     ["test_oracle_layer.test_backward_matches_central_finite_differences"]),
    ("lagrangian_quadratic_factor", "(lambda1 + 2.0 * lambda2 * diff)", "(lambda1 + lambda2 * diff)",
     ["test_oracle_lagrangian.test_gradient_wrt_alpha_finite_differences"]),
    ("lagrangian_unweighted", "s = np.sum(pi * size_j) / S if S > 0 else 0.0", "s = np.mean(pi) if S > 0 else 0.0",
     ["test_oracle_lagrangian.test_limits_and_equal_sizes"]),
    ("lagrangian_linear_sign", "g = lambda1 * diff + lambda2 * diff * diff", "g = -lambda1 * diff + lambda2 * diff * diff",
     ["test_oracle_lagrangian.test_penalty_is_linear_in_multipliers_and_matches_definition"]),
    ("count_rounds_down", "k = int(np.floor(np.sum(pi) + 0.5))", "k = int(np.floor(np.sum(pi)))",
     ["test_oracle_compact.test_compaction_equals_brute_force_masking", "test_oracle_compact.test_topk_ties_and_edges"]),
    ("keeps_smallest", "key=lambda j: (-a[j], j)", "key=lambda j: (a[j], j)",
     ["test_oracle_compact.test_compaction_equals_brute_force_masking"]),
    ("gate_not_absorbed", "return P[:, idx].copy(), z[idx][:, None] * Q[idx, :]", "return P[:, idx].copy(), Q[idx, :].copy()",
     ["test_oracle_compact.test_compaction_equals_brute_force_masking"]),
    ("compact_gathers_rows_of_P", "return P[:, idx].copy(), z[idx][:, None] * Q[idx, :]",
     "return P[:, np.sort(idx)[::-1]].copy(), z[idx][:, None] * Q[idx, :]",
     ["test_oracle_compact.test_compaction_equals_brute_force_masking"]),
    ("embedding_drops_gate_in_dE", "dE[ids[t]] += dHp[t] * z", "dE[ids[t]] += dHp[t]",
     ["test_oracle_embedding.test_embedding_equals_layer_on_one_hot_inputs"]),
    ("embedding_overwrites_repeated_words", "dE[ids[t]] += dHp[t] * z", "dE[ids[t]] = dHp[t] * z",
     ["test_oracle_embedding.test_embedding_equals_layer_on_one_hot_inputs"]),
    ("agp_prunes_largest", "key=lambda k: (-abs(g[lo + k]), k))", "key=lambda k: (abs(g[lo + k]), k))",
     ["test_oracle_agp.test_magnitude_rule_properties_and_brute_force"]),
    ("agp_tie_order", "key=lambda k: (-abs(g[lo + k]), k))", "key=lambda k: (-abs(g[lo + k]), -k))",
     ["test_oracle_agp.test_ties_and_l1_term"]),
    ("uniform_closed_at_zero", ".astype(np.float64) + 0.5) * 2.0 ** -23", ".astype(np.float64) + 0.0) * 2.0 ** -23",
     ["test_oracle_philox.test_uniform_mapping_open_interval_and_exact_in_fp32"]),
    ("philox_nine_rounds", "for _ in range(10):", "for _ in range(9):",
     ["test_oracle_philox.test_philox_matches_vendor_host_generator"]),
    ("philox_swapped_multipliers", "p0 = _PHILOX_M0 * c0", "p0 = _PHILOX_M1 * c0",
     ["test_oracle_philox.test_philox_matches_vendor_host_generator"]),
    ("philox_key_not_bumped", "k0 = (k0 + _PHILOX_W0) & _MASK32", "k0 = k0 & _MASK32",
     ["test_oracle_philox.test_philox_matches_vendor_host_generator"]),
]


def _mutant_module(old, new):
    assert SRC.count(old) == 1, f"mutation anchor not unique or missing: {old!r}"
    mod = types.ModuleType("flop_oracle_mutant")
    exec(compile(SRC.replace(old, new), "flop_oracle_mutant", "exec"), mod.__dict__)
    return mod


def _pin_fails(test_path, mutant):
    """Run one pin test with its module-level oracle `O` replaced by the mutant."""
    mod_name, fn_name = test_path.split(".")
    tmod = importlib.import_module("tests." + mod_name)
    real = tmod.O
    tmod.O = mutant
    try:
        getattr(tmod, fn_name)()
    except pytest.skip.Exception:
        return None                     # the pin could not run here (e.g. no vendor generator)
    except BaseException:
        return True
    finally:
        tmod.O = real
    return False


@pytest.mark.parametrize("name,old,new,pins", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(name, old, new, pins):
    if ROOT not in sys.path:
        sys.path.insert(0, ROOT)
    mutant = _mutant_module(old, new)
    results = [_pin_fails(p, mutant) for p in pins]
    if all(r is None for r in results):
        pytest.skip("the only pins for this mistake need a library that is not present")
    assert any(r is True for r in results), f"mistake {name!r} passed {pins}"


def test_the_unmutated_oracle_passes_the_same_pins():
    clean = _mutant_module("for _ in range(10):", "for _ in range(10):")
    for _, _, _, pins in MUTANTS:
        for p in pins:
            assert _pin_fails(p, clean) in (False, None), p
