"""The pins must be able to fail: plant one plausible mistake at a time in a copy of the
oracle's C source (CPU only), compile it, and check that at least one pin rejects it."""
import ctypes
import os
import subprocess

import pytest

import oracle
import test_oracle_pins as pins
import test_oracle_sample_pins as spins
import test_oracle_mcns_pins as npins
import test_oracle_edge_pins as epins

SRC = os.path.join(os.path.dirname(oracle.__file__), "mcsd_oracle.c")

# (name, text to find, replacement, pins expected to catch it)
MUTANTS = [
    ("residual_sign", "double d = p[x] - q[x];", "double d = q[x] - p[x];",
     [lambda: pins.test_output_token_is_distributed_as_p(4, 3, 0)]),
    ("accept_inequality", "if (r[i] <= rho) return i;", "if (r[i] >= rho) return i;",
     [pins.test_k1_is_textbook_speculative_sampling]),
    ("residual_not_normalised", "p[x] = (d > 0.0 ? d : 0.0) / s;", "p[x] = (d > 0.0 ? d : 0.0);",
     [lambda: pins.test_output_token_is_distributed_as_p(4, 3, 0)]),
    ("alg2_q_not_zeroed", "            q[xt] = 0.0;\n            double w = 0.0;", "            double w = 0.0;",
     [lambda: pins.test_output_token_is_distributed_as_p(4, 3, 1)]),
    ("alg2_q_not_renormalised", "for (int32_t x = 0; x < V; ++x) q[x] /= w;", ";",
     [lambda: pins.test_output_token_is_distributed_as_p(4, 3, 1)]),
    ("alg2_applied_to_alg1", "if (mode == 1 && valid && q[xt] > 0.0) {", "if (mode == 0 && valid && q[xt] > 0.0) {",
     [lambda: pins.test_rejection_probability_is_the_normaliser_and_rejected_tokens_stay_zero(0)]),
    ("zero_q_accepted", "if (qx > 0.0) {", "if (qx >= 0.0) {",
     [pins.test_forced_rejection_on_zero_draft_probability]),
    ("invcdf_non_strict", "if (cum > target) return x;", "if (cum >= target) return x;",
     [pins.test_invcdf_brute_force_exact_fractions]),
    ("invcdf_off_by_one", "if (cum > target) return x;", "if (cum > target) return x + 1 < V ? x + 1 : x;",
     [pins.test_invcdf_never_returns_zero_mass_and_clamps]),
    ("temperature_inverted", "- m) / T);", "- m) * T);",
     [lambda: pins.test_softmax_matches_library_routine(0.7)]),
    ("softmax_no_max", "if (l > m) m = l;\n    }\n    double Z", "if (l > m) m = 0;\n    }\n    double Z",
     [pins.test_softmax_handles_minus_inf_and_large_logits]),
    ("argmax_highest_index", "if (l > m) { m = l; a = x; }", "if (l >= m) { m = l; a = x; }",
     [pins.test_argmax_lowest_index_on_ties]),
    ("wrong_uniform_slot", "r[i] = (double)unif_b[2 * (first + i)];", "r[i] = (double)unif_b[2 * (first + i) + 1];",
     [pins.test_chain_tree_is_standard_speculative_decoding]),
    ("uniform_of_parent", "r[i] = (double)unif_b[2 * (first + i)];", "r[i] = (double)unif_b[2 * n];",
     [pins.test_chain_tree_is_standard_speculative_decoding]),
    ("candidates_reversed", "cands[i] = cand_b[first + i];", "cands[i] = cand_b[first + k - 1 - i];",
     [pins.test_temperature_zero_is_greedy_matching, pins.test_output_marginal_through_verify_on_uniform_grid]),
    ("bonus_from_root", "tok[len] = bon[n];", "tok[len] = bon[0];",
     [lambda: pins.test_all_node_form_equals_sequential_walk([2, 2], 0)]),
    ("draft_row_of_wrong_node", "mcsd_oracle_softmax(draft_b + (size_t)n * V, V, T, qbuf);",
     "mcsd_oracle_softmax(draft_b, V, T, qbuf);",
     [pins.test_chain_tree_is_standard_speculative_decoding]),
    ("leaf_bonus_from_wrong_uniform", "*bonus = mcsd_oracle_invcdf(residual, V, (double)unif_b[2 * n + 1]);\n        if (*bonus < 0) *status |= ORACLE_STATUS_NO_MASS;\n        return -1;\n    }\n    mcsd",
     "*bonus = mcsd_oracle_invcdf(residual, V, (double)unif_b[2 * n]);\n        return -1;\n    }\n    mcsd",
     [pins.test_output_marginal_through_verify_on_uniform_grid]),
    ("t0_accepts_any_candidate", "int32_t match = cand_b[first + i] == a;", "int32_t match = 1;",
     [pins.test_temperature_zero_is_greedy_matching]),
    ("eq1_drawn_token_not_removed", "if (mode == 1) q[x] = 0.0;", ";",
     [spins.test_hand_computed_draws_without_replacement]),
    ("eq1_removal_applied_with_replacement", "if (mode == 1) q[x] = 0.0;", "q[x] = 0.0;",
     [spins.test_draws_with_replacement_reproduce_q]),
    ("draw_uses_wrong_uniform", "int32_t x = mcsd_oracle_invcdf(q, V, u[i]);", "int32_t x = mcsd_oracle_invcdf(q, V, u[0]);",
     [spins.test_hand_computed_draws_without_replacement]),
    ("topk_ascending", "(double)logits[x] > (double)logits[best]) best = x;", "(double)logits[x] < (double)logits[best]) best = x;",
     [spins.test_temperature_zero_is_top_k_with_lowest_index_on_ties]),
    ("topk_highest_index_on_ties", "(double)logits[x] > (double)logits[best]) best = x;", "(double)logits[x] >= (double)logits[best]) best = x;",
     [spins.test_temperature_zero_is_top_k_with_lowest_index_on_ties]),
    ("naive_draw_uses_acceptance_uniform", "int32_t x = mcsd_oracle_invcdf(residual, V, (double)unif_b[2 * n + 1]);\n        if (x < 0) { *status",
     "int32_t x = mcsd_oracle_invcdf(residual, V, (double)unif_b[2 * n]);\n        if (x < 0) { *status",
     [npins.test_emitted_token_is_a_draw_from_p_and_accepted_iff_a_candidate_carries_it]),
    ("naive_match_inverted", "int32_t match = cand_b[first + i] == x;", "int32_t match = cand_b[first + i] != x;",
     [npins.test_emitted_token_is_a_draw_from_p_and_accepted_iff_a_candidate_carries_it]),
    ("naive_endpoint_not_the_draw", "        *bonus = x;\n        return -1;", "        *bonus = cand_b[first];\n        return -1;",
     [npins.test_walk_over_levels_and_leaf_endpoint]),
    ("sample_children_of_wrong_node", "const float *d = draft + ((size_t)b * n_internal + n) * V;", "const float *d = draft + ((size_t)b * n_internal) * V;",
     [lambda: spins.test_tree_level_routine_is_the_node_routine_in_child_order(1, 0.7)]),
    ("zero_mass_residual_overwritten", "} else {\n            *status |= ORACLE_STATUS_DEGENERATE;",
     "} else {\n            for (int32_t x = 0; x < V; ++x) p[x] = 0.0;\n            *status |= ORACLE_STATUS_DEGENERATE;",
     [lambda: epins.test_zero_residual_mass_keeps_p_and_later_candidates_see_it(0)]),
    ("zero_mass_not_reported", "} else {\n            *status |= ORACLE_STATUS_DEGENERATE;\n        }", "}",
     [lambda: epins.test_zero_residual_mass_after_a_candidate_of_probability_zero(1)]),
    ("zero_mass_divided_anyway", "if (s > 0.0) {", "if (s >= 0.0) {",
     [lambda: epins.test_all_candidates_rejected_on_zero_mass_draws_from_the_kept_p(0)]),
    ("no_mass_not_reported", "if (*bonus < 0) *status |= ORACLE_STATUS_NO_MASS;", ";",
     [lambda: epins.test_target_row_without_mass_at_the_root("nan", 0), epins.test_leaf_without_mass_ends_the_walk_with_no_token]),
    ("no_mass_returns_a_token", "    return last;\n}", "    return last < 0 ? 0 : last;\n}",
     [lambda: epins.test_target_row_without_mass_at_the_root("all_minus_inf", 1)]),
    ("naive_no_mass_not_reported", "if (x < 0) { *status |= ORACLE_STATUS_NO_MASS; *bonus = -1; return -1; }",
     "if (x < 0) { *bonus = -1; return -1; }",
     [lambda: epins.test_target_row_without_mass_at_the_root("plus_inf", 2)]),
    ("uniform_cap_missing", "if (!(r[i] < 1.0)) r[i] = 1.0;", ";",
     [epins.test_uniform_not_below_one_counts_as_one]),
    ("alg2_renormalises_when_nothing_was_removed", "if (mode == 1 && valid && q[xt] > 0.0) {", "if (mode == 1) { if (!valid) xt = 0;",
     [lambda: epins.test_zero_residual_mass_on_a_long_row_whose_sum_is_not_exactly_one(1)]),
]


@pytest.mark.parametrize("name,find,repl,catchers", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(name, find, repl, catchers, tmp_path, monkeypatch):
    text = open(SRC).read()
    assert text.count(find) >= 1, f"mutation site for {name} not found"
    mutated = text.replace(find, repl)
    c_path = tmp_path / "mutant.c"
    so_path = tmp_path / f"libmutant_{name}.so"
    c_path.write_text(mutated)
    subprocess.run(["gcc", "-O1", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-w", "-o", str(so_path),
                    str(c_path), "-lm"], check=True)
    monkeypatch.setattr(oracle, "_lib", oracle._bind(ctypes.CDLL(str(so_path))))
    caught = False
    for pin in catchers:
        try:
            pin()
        except (AssertionError, ValueError, ZeroDivisionError, IndexError, FloatingPointError):
            caught = True
            break
    assert caught, f"no pin noticed the planted mistake {name!r}"
