"""How strong are the oracle's pins?  Each case plants ONE plausible mistake in a copy of the oracle's C source
(on the CPU, in a temporary directory; the real oracle is untouched), builds it, and runs the pin tests of
test_oracle_pins.py against the mutant: at least one pin must fail.  A mistake that no pin notices would mean
the GPU path could share it unnoticed.
"""
import importlib.util
import os
import shutil

import pytest

import test_oracle_pins as pins
import test_thinning_oracle_pins as thin_pins
import test_weighted_oracle_pins as w_pins

ORACLE_DIR = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "oracle")

# (name, text in pcg_oracle.c, replacement, which occurrence)
MUTATIONS = [
    ("dropped_degree_in_coarse_graining", "s += weights ? p[t] * weights[k] : p[t] / (double)tok_degree[t];",
     "s += weights ? p[t] * weights[k] : p[t];", 0),
    ("inverted_acceptance_ratio", "double ratio = Q[g] > 0.0 ? P[g] / Q[g] : INFINITY;",
     "double ratio = P[g] > 0.0 ? Q[g] / P[g] : INFINITY;", 0),
    ("residual_with_wrong_sign", "R[g] = P[g] > Q[g] ? P[g] - Q[g] : 0.0;", "R[g] = Q[g] > P[g] ? Q[g] - P[g] : 0.0;", 0),
    ("within_group_draw_ignores_degree", "w[k] = weights ? p[t] * weights[lo + k] : p[t] / (double)tok_degree[t];",
     "w[k] = weights ? p[t] * weights[lo + k] : p[t];", 0),
    ("within_group_draw_uses_draft", "w[k] = weights ? p[t] * weights[lo + k] : p[t] / (double)tok_degree[t];",
     "w[k] = weights ? q[t] * weights[lo + k] : q[t] / (double)tok_degree[t];", 0),
    ("accept_draw_uses_label_uniform", "((double)u[2 * i + 1] < ratio + accept_bias)",
     "((double)u[2 * i] < ratio + accept_bias)", 0),
    ("label_index_off_by_one", "j = (int)floor(uj);", "j = (int)ceil(uj);", 0),
    ("temperature_ignored", "p[t] = load_logit(logits, dtype, off + t) / T;", "p[t] = load_logit(logits, dtype, off + t);", 0),
    ("bonus_token_from_last_drafted_row", "softmax_row(target_logits, dtype, b * (int64_t)(K + 1) + K, V, T, p);",
     "softmax_row(target_logits, dtype, b * (int64_t)(K + 1) + K - 1, V, T, p);", 0),
    ("terminal_group_uses_token_uniform", "gs = inverse_cdf(R, M, (double)u[2 * K], NULL,",
     "gs = inverse_cdf(R, M, (double)u[2 * K + 1], NULL,", 0),
    ("residual_not_clamped", "R[g] = P[g] > Q[g] ? P[g] - Q[g] : 0.0;", "R[g] = fabs(P[g] - Q[g]);", 0),
    ("accepted_position_emits_group_representative", "tok_out[i] = x; /*", "tok_out[i] = group_tok[group_ptr[g]]; /*", 0),
    ("first_rejection_does_not_stop_the_loop", "            n = i;\n            have_Q = 1;\n            break;",
     "            if (n == K) n = i;\n            have_Q = 1;", 0),
]

PIN_CALLS = (
    [lambda o: pins.test_hand_worked_example(o), lambda o: pins.test_group_probs_special_cases(o),
     lambda o: pins.test_singleton_groups_equal_textbook_speculative_sampling(o),
     lambda o: pins.test_partition_groups_equal_textbook_sampling_on_lumped_distributions(o)]
    + [lambda o, T=T: pins.test_softmax_matches_library_routine(o, T) for T in (0.8, 2.5)]
    + [lambda o, n=n: pins.test_group_probs_sum_to_one_and_match_dense_matrix(o, n) for n in ("C1", "C4")]
    + [lambda o, s=s: pins.test_label_coupling_and_acceptance_probability(o, s) for s in (11, 12)]
    + [lambda o, s=s: pins.test_residual_group_law_and_emitted_group_is_target_coarse(o, s) for s in (11, 13)]
    + [lambda o, s=s: pins.test_within_group_and_bonus_token_law(o, s) for s in (11, 14)]
    + [lambda o, n=n: pins.test_emission_structure_on_workloads(o, n) for n in ("C1",)]
)


# planted mistakes in the thinning sampler, checked against the thinning pins
THIN_MUTATIONS = [
    ("thinning_ratio_inverted", "double a = P[k] > 0.0 ? 1.0 - Q[k] / P[k] : 0.0;",
     "double a = Q[k] > 0.0 ? 1.0 - P[k] / Q[k] : 0.0;", 0),
    ("thinning_candidate_from_draft", "pm[t] = p[cand_order ? cand_order[t] : t];",
     "pm[t] = (have_Q ? q : p)[cand_order ? cand_order[t] : t];", 0),
    ("thinning_candidate_not_mapped_back_through_the_order", "if (cand_order) y = cand_order[y];", "", 0),
    ("thinning_masses_not_taken_in_the_given_order", "pm[t] = p[cand_order ? cand_order[t] : t];", "pm[t] = p[t];", 0),
    ("thinning_keep_uses_label_uniform", "keep = (double)tu[3 * r + 2] < a;", "keep = (double)tu[3 * r + 1] < a;", 0),
    ("thinning_label_uses_token_uniform", "draw_label(y, (double)tu[3 * r + 1], weights,", "draw_label(y, (double)tu[3 * r], weights,", 0),
    ("thinning_bonus_is_thinned_too", "if (have_Q) { /* thinning probability", "if (1) { /* thinning probability", 0),
    ("thinning_keeps_with_complement", "keep = (double)tu[3 * r + 2] < a;", "keep = (double)tu[3 * r + 2] >= a;", 0),
    ("thinning_token_from_draft_conditional", "w[k] = weights ? p[t] * weights[lo + k] : p[t] / (double)tok_degree[t];",
     "w[k] = weights ? q[t] * weights[lo + k] : q[t] / (double)tok_degree[t];", 0),
]

THIN_PIN_CALLS = (
    [lambda o, s=s, r=r: thin_pins.test_thinning_group_law_trials_and_token_law(o, s, r) for s, r in ((11, None), (13, 102))]
    + [lambda o, s=s: thin_pins.test_thinning_bonus_is_one_candidate_from_the_target(o, s, None) for s in (11,)]
    + [lambda o: thin_pins.test_thinning_with_singleton_groups_is_token_level_residual_sampling(o, None),
       lambda o: thin_pins.test_thinning_exhaustion_falls_back_to_the_enumerated_draw(o),
       lambda o: thin_pins.test_thinning_never_reads_trials_it_does_not_reach(o),
       lambda o: thin_pins.test_thinning_candidate_walks_the_tokens_in_the_given_order(o)]
)


# planted mistakes in the general-weights branches and the acceptance bias, checked against the weighted pins
WEIGHT_MUTATIONS = [
    ("label_weights_read_without_the_pair_index", "wx[e] = weights[rev_nz[rev_ptr[x] + e]];", "wx[e] = weights[rev_ptr[x] + e];", 0),
    ("label_draw_ignores_weights", "    if (!weights) {\n        double uj = u * (double)N;", "    if (1) {\n        double uj = u * (double)N;", 0),
    ("within_group_weights_not_offset_by_the_group", "w[k] = weights ? p[t] * weights[lo + k]", "w[k] = weights ? p[t] * weights[k]", 0),
    ("within_group_draw_ignores_weights", "w[k] = weights ? p[t] * weights[lo + k] : p[t] / (double)tok_degree[t];",
     "w[k] = p[t] / (double)tok_degree[t];", 0),
    ("coarse_graining_weights_not_offset_by_the_group", "s += weights ? p[t] * weights[k]", "s += weights ? p[t] * weights[k - group_ptr[g]]", 0),
    ("coarse_graining_ignores_weights", "s += weights ? p[t] * weights[k] : p[t] / (double)tok_degree[t];",
     "s += p[t] / (double)tok_degree[t];", 0),
    ("bias_multiplies_the_ratio", "((double)u[2 * i + 1] < ratio + accept_bias)", "((double)u[2 * i + 1] < ratio * (1.0 + accept_bias))", 0),
    ("bias_subtracted", "((double)u[2 * i + 1] < ratio + accept_bias)", "((double)u[2 * i + 1] < ratio - accept_bias)", 0),
    ("bias_ignored", "((double)u[2 * i + 1] < ratio + accept_bias)", "((double)u[2 * i + 1] < ratio)", 0),
    ("bias_added_to_the_target_mass", "double ratio = Q[g] > 0.0 ? P[g] / Q[g] : INFINITY;",
     "double ratio = Q[g] > 0.0 ? (P[g] + accept_bias) / Q[g] - accept_bias : INFINITY;", 0),
]

WEIGHT_PIN_CALLS = (
    [lambda o: w_pins.test_weighted_group_probs_exact_rationals(o), lambda o: w_pins.test_weighted_label_draw_hand_cases(o),
     lambda o: w_pins.test_weighted_label_law_and_acceptance_law(o),
     lambda o: w_pins.test_weighted_emitted_group_is_target_coarse(o),
     lambda o: w_pins.test_weighted_within_group_and_bonus_token_law(o)]
    + [lambda o, b=b: w_pins.test_acceptance_bias_law(o, b) for b in (0.3, 0.05)]
)


def _mutant(tmp_path, name, old, new, occurrence):
    src = open(os.path.join(ORACLE_DIR, "pcg_oracle.c")).read()
    parts = src.split(old)
    assert len(parts) > occurrence + 1, f"mutation target not found in the oracle source: {old!r}"
    mutated = old.join(parts[:occurrence + 1]) + new + old.join(parts[occurrence + 1:])
    d = tmp_path / name
    d.mkdir()
    (d / "pcg_oracle.c").write_text(mutated)
    shutil.copy(os.path.join(ORACLE_DIR, "pcg_oracle.py"), d / "pcg_oracle.py")
    spec = importlib.util.spec_from_file_location(f"oracle_mutant_{name}", d / "pcg_oracle.py")
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)  # its paths point at the copy: it compiles and loads the mutated source
    return mod


@pytest.mark.parametrize("name,old,new,occurrence", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_every_planted_mistake_is_caught_by_a_pin(tmp_path, name, old, new, occurrence):
    mutant = _mutant(tmp_path, name, old, new, occurrence)
    caught = []
    for i, call in enumerate(PIN_CALLS):
        try:
            call(mutant)
        except AssertionError:
            caught.append(i)
    assert caught, f"no pin noticed the planted mistake '{name}'"


@pytest.mark.parametrize("name,old,new,occurrence", THIN_MUTATIONS, ids=[m[0] for m in THIN_MUTATIONS])
def test_every_planted_thinning_mistake_is_caught_by_a_pin(tmp_path, name, old, new, occurrence):
    mutant = _mutant(tmp_path, name, old, new, occurrence)
    caught = []
    for i, call in enumerate(THIN_PIN_CALLS):
        try:
            call(mutant)
        except AssertionError:
            caught.append(i)
    assert caught, f"no pin noticed the planted mistake '{name}'"


@pytest.mark.parametrize("name,old,new,occurrence", WEIGHT_MUTATIONS, ids=[m[0] for m in WEIGHT_MUTATIONS])
def test_every_planted_weights_or_bias_mistake_is_caught_by_a_pin(tmp_path, name, old, new, occurrence):
    mutant = _mutant(tmp_path, name, old, new, occurrence)
    caught = []
    for i, call in enumerate(WEIGHT_PIN_CALLS):
        try:
            call(mutant)
        except AssertionError:
            caught.append(i)
    assert caught, f"no pin noticed the planted mistake '{name}'"


def test_the_unmodified_copy_passes_every_pin(tmp_path):
    """Control: the same machinery with no mistake planted must pass, so a failure above means the mistake."""
    clean = _mutant(tmp_path, "clean", "double ratio", "double ratio", 0)
    for call in PIN_CALLS + THIN_PIN_CALLS + WEIGHT_PIN_CALLS:
        call(clean)
