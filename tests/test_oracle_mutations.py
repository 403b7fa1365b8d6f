"""Do the pins bite?  Each case plants ONE plausible mistake in a copy of the oracle's C
source (on the CPU, in a temporary directory), builds it, swaps it in for the real oracle and
runs the pin battery: at least one pin must fail.  A mutation that no pin notices would mean
that part of the oracle is unpinned."""
import ctypes
import os
import subprocess

import pytest

import oracle
import test_oracle_pins as pins

SRC = os.path.join(os.path.dirname(oracle.__file__), "gnnco_oracle.c")

MUTATIONS = {
    "aggregation drops the node's own features":
        ("for (int32_t f = 0; f < fi; ++f) m[f] = Hp[(size_t)i * fi + f];", "for (int32_t f = 0; f < fi; ++f) m[f] = 0.0;"),
    "normaliser is |N(i)|+2": ("double inv = 1.0 / (double)(rp[i + 1] - rp[i] + 1);", "double inv = 1.0 / (double)(rp[i + 1] - rp[i] + 2);"),
    "size term has the wrong sign": ("alpha * edge_term - beta * node_term", "alpha * edge_term + beta * node_term"),
    "every edge counted twice in the loss": ("if (ci[k] > i) edge_term += p[i] * p[ci[k]];", "edge_term += p[i] * p[ci[k]];"),
    "penalty term dropped from the loss": ("+ lambda * pen_term;", "+ 0.0 * pen_term;"),
    "sigmoid of -z": ("p[i] = 1.0 / (1.0 + exp(-z));", "p[i] = 1.0 / (1.0 + exp(z));"),
    "edge gradient halved": ("double dp = alpha * nb - beta", "double dp = 0.5 * alpha * nb - beta"),
    "penalty missing from the gradient": ("+ (pen ? lambda * pen[i] : 0.0);", "+ 0.0;"),
    "transposed aggregation not normalised": ("dm[f] = acc / (double)(rp[i + 1] - rp[i] + 1);", "dm[f] = acc;"),
    "transposed aggregation forgets the node itself":
        ("for (int32_t f = 0; f < fi; ++f) dH[(size_t)i * fi + f] += dm[f];", ";"),
    "ReLU derivative ignored": ("if (!(Z[l - 1][q] > 0.0)) dH[q] = 0.0;", ";"),
    "input gradient uses W instead of W^T":
        ("acc += dZ[(size_t)i * fo + h] * Wl[(size_t)f * fo + h];", "acc += dZ[(size_t)i * fo + h] * Wl[((size_t)h * fi + f) % ((size_t)fi * fo)];"),
    "Adam without bias correction of m": ("W[q] -= lr * (m[q] / c1)", "W[q] -= lr * (m[q])"),
    "Adam eps inside the root": ("/ (sqrt(v[q] / c2) + eps);", "/ sqrt(v[q] / c2 + eps);"),
    "Adam second moment uses g instead of g^2": ("(1.0 - b2) * g[q] * g[q];", "(1.0 - b2) * g[q];"),
    "threshold uses > instead of >=": ("x[i] = p[i] >= threshold ? 1 : 0;", "x[i] = p[i] > threshold ? 1 : 0;"),
    "intra conflicts counted from both ends": ("if (colidx[k] > i && x[i] && x[colidx[k]]) ++intra;", "if (x[i] && x[colidx[k]]) ++intra;"),
    "per-subgraph count misses the second endpoint": ("per_part[node_part[bnd_v[e]]]++;", ";"),
    "boundary edge stored as (u, v) instead of (min, max)":
        ("bpairs[2 * E_b] = a < b ? a : b;\n      bpairs[2 * E_b + 1] = a < b ? b : a;", "bpairs[2 * E_b] = a;\n      bpairs[2 * E_b + 1] = b;"),
    "new ids ignore the original order inside a part":
        ("int32_t id = fill[part[i]]++;", "int32_t id = part_ptr[part[i] + 1] - 1 - (fill[part[i]]++ - part_ptr[part[i]]);"),
    "base action picks u on equal probabilities": ("action[c] = p[u] < p[v] ? 0 : 1;", "action[c] = p[u] <= p[v] ? 0 : 1;"),
    "actions mark the wrong endpoint's subgraph": ("active[node_part[node]] = 1;", "active[node_part[bnd_u[conflict_idx[c]]]] = 1;"),
    "conflict list keeps non-violated edges": ("if (viol[e]) conflict_idx[c++] = (int32_t)e;", "conflict_idx[c++] = (int32_t)e;"),
    "repair clears the nodes that were NOT chosen": ("if (pen[i] != 0.0f && x[i]) {", "if (pen[i] == 0.0f && x[i]) {"),
    "repair counts chosen nodes that were not selected": ("if (pen[i] != 0.0f && x[i]) {", "if (pen[i] != 0.0f) {"),
    "modularity counts internal edges once": ("q += 2.0 * (double)in_edges[s] / two_m - share * share;", "q += (double)in_edges[s] / two_m - share * share;"),
    "degree sum misses the second endpoint": ("    tot[a] += 1;\n    tot[b] += 1;", "    tot[a] += 1;"),
    "bf16 storage truncates instead of rounding to nearest": ("u += 0x7FFFu + ((u >> 16) & 1u);", ";"),
    "bf16 storage rounds ties away from zero": ("u += 0x7FFFu + ((u >> 16) & 1u);", "u += 0x8000u;"),
    "bf16 storage rounds the double directly (one rounding)":
        ("  float f = (float)x;\n  uint32_t u;\n  memcpy(&u, &f, 4);\n  if ((u & 0x7F800000u) == 0x7F800000u) return (double)f;",
         "  float f = (float)x;\n  uint32_t u;\n  memcpy(&u, &f, 4);\n  if ((u & 0x7F800000u) == 0x7F800000u) return (double)f;\n"
         "  if ((u & 0xFFFFu) == 0x8000u && (double)f != x) u += (fabs(x) > fabs((double)f)) ? 1u : 0xFFFFFFFFu;"),
    "bf16 storage leaves the aggregated input unrounded":
        ("if (store_bf16 && l < L)\n        for (int32_t f = 0; f < fi; ++f) m[f] = round_bf16(m[f]);", ";"),
    "bf16 storage also rounds the output layer's aggregate": ("if (store_bf16 && l < L)", "if (store_bf16)"),
    "bf16 storage leaves the activation unrounded":
        ("if (store_bf16)\n          for (int32_t h = 0; h < fo; ++h) hr[h] = round_bf16(hr[h]);", ";"),
    "Louvain: ties go to the highest community id":
        ("if (sc > best_score || (sc == best_score && best != own && c < best))", "if (sc > best_score || (sc == best_score && best != own && c > best))"),
    "Louvain: two single nodes may swap": (" && !(size[own] == 1 && size[best] == 1 && best > own)) {\n      next[a] = best;", ") {\n      next[a] = best;"),
    "Louvain: the node's own degree stays in its community's total":
        ("const int64_t own_score = two_m * kin[own] - (tot[own] - k[a]) * k[a];", "const int64_t own_score = two_m * kin[own] - tot[own] * k[a];"),
    "Louvain: gain without the factor 2m": ("int64_t sc = two_m * kin[c] - tot[c] * k[a];", "int64_t sc = kin[c] - tot[c] * k[a];"),
    "Louvain: a sweep that lowers Q is kept": ("if (q_new <= qnum) break;", "if (q_new <= qnum && 0) break;"),
    "Louvain: internal weight counted once in Q": ("in2[comm[a]] += 2 * g->loop[a];", "in2[comm[a]] += g->loop[a];"),
    "inv_deg without the +1": ("inv_deg[i] = 1.0f / (float)(hi - lo + 1);", "inv_deg[i] = 1.0f / (float)(hi - lo > 0 ? hi - lo : 1);"),
}

BATTERY = [
    lambda: pins.test_bookkeeping_brute_force(40, 0.2, 5, 2),
    lambda: pins.test_bookkeeping_brute_force(25, 0.3, 9, 5),
    lambda: pins.test_forward_and_loss_match_dense_definition([6, 4, 1], False),
    lambda: pins.test_forward_and_loss_match_dense_definition([7, 5, 3, 1], True),
    pins.test_aggregation_preserves_constant_features_and_isolated_nodes,
    pins.test_zero_weights_closed_forms,
    pins.test_single_node_subgraph_by_hand,
    pins.test_loss_on_binary_probabilities_is_the_qubo_value,
    lambda: pins.test_gradients_match_central_finite_differences([5, 4, 1], False),
    lambda: pins.test_gradients_match_central_finite_differences([6, 5, 4, 1], False),
    pins.test_sigmoid_chain_identity_for_one_layer,
    pins.test_adam_two_steps_against_exact_rational_arithmetic,
    pins.test_adam_first_step_is_sign_step_and_zero_gradient_stays,
    lambda: pins.test_decode_brute_force(1),
    lambda: pins.test_decode_brute_force(2),
    lambda: pins.test_conflict_list_base_action_and_penalty_brute_force(1),
    lambda: pins.test_conflict_list_base_action_and_penalty_brute_force(2),
    lambda: pins.test_repair_removes_exactly_the_chosen_nodes_brute_force(1),
    lambda: pins.test_partition_quality_matches_networkx_and_the_pairwise_definition(30, 0.2, 4, 1),
    lambda: pins.test_louvain_sweep_picks_the_brute_force_best_community(12, 0.3, 2),
    lambda: pins.test_louvain_sweep_picks_the_brute_force_best_community(11, 0.5, 3),
    pins.test_eq2_gain_is_what_the_sweep_compares,
    lambda: pins.test_louvain_level_keeps_a_sweep_only_if_exact_modularity_rises(8, 0.3, 5),
    lambda: pins.test_louvain_level_keeps_a_sweep_only_if_exact_modularity_rises(12, 0.3, 7),
    pins.test_louvain_recovers_planted_blocks_and_reports_their_exact_modularity,
    pins.test_louvain_small_cases_by_hand,
    pins.test_round_bf16_is_exact_round_to_nearest_even,
    lambda: pins.test_bf16_storage_forward_matches_dense_definition_with_rounding_written_out([7, 5, 3, 1], False),
    pins.test_bf16_storage_hidden_preactivations_and_output_layer_keep_full_precision,
    pins.test_bf16_storage_mode_is_a_no_op_when_every_stored_value_is_a_bf16_number,
    pins.test_bf16_storage_gradients_are_those_of_the_rounded_forward_values,
]


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_a_pin_fails_when_the_oracle_is_mutated(name, tmp_path, monkeypatch):
    old, new = MUTATIONS[name]
    text = open(SRC).read()
    assert text.count(old) == 1, "mutation target not found exactly once: %r" % old
    src = tmp_path / "mutant.c"
    src.write_text(text.replace(old, new))
    lib_path = str(tmp_path / "libmutant.so")
    subprocess.check_call(["gcc", "-O1", "-fopenmp", "-shared", "-fPIC", "-o", lib_path, str(src), "-lm"])
    real = oracle._native()
    mutant = ctypes.CDLL(lib_path)
    for fn in ("oracle_bookkeeping", "oracle_subgraph_step", "oracle_train_step", "oracle_adam", "oracle_decode",
               "oracle_conflict_list", "oracle_base_action", "oracle_apply_actions", "oracle_repair", "oracle_partition_quality",
               "oracle_round_bf16", "oracle_louvain", "oracle_louvain_sweep"):
        getattr(mutant, fn).argtypes = getattr(real, fn).argtypes
        getattr(mutant, fn).restype = getattr(real, fn).restype
    monkeypatch.setattr(oracle, "_lib", mutant)
    caught = 0
    for check in BATTERY:
        try:
            check()
        except (AssertionError, oracle.OracleError, ValueError, IndexError, KeyError):
            caught += 1
    assert caught >= 1, "no pin noticed: " + name


# The Gumbel-softmax oracle is numpy, not C: the same game on its Python source.
PY_MUTATIONS = {
    "Gumbel noise subtracted": ("a = a + (-np.log(-np.log(", "a = a - (-np.log(-np.log("),
    "noise with a single logarithm": ("(-np.log(-np.log(np.asarray(U, dtype=np.float64))))", "(-np.log(np.asarray(U, dtype=np.float64)))"),
    "temperature multiplies": ("a = a / float(tau)", "a = a * float(tau)"),
    "normalised over nodes instead of features": ("e / e.sum(axis=1, keepdims=True)", "e / e.sum(axis=0, keepdims=True)"),
    "softmax without the exponential": ("e = np.exp(a)", "e = a - a.min() + 1.0"),
}

PY_BATTERY = [
    pins.test_gumbel_softmax_without_noise_is_the_library_softmax,
    pins.test_gumbel_softmax_two_features_closed_form,
    pins.test_gumbel_softmax_invariants_and_temperature_limits,
    pins.test_gumbel_max_trick_reproduces_the_softmax_distribution,
]


@pytest.mark.parametrize("name", sorted(PY_MUTATIONS))
def test_a_pin_fails_when_the_gumbel_softmax_oracle_is_mutated(name, monkeypatch):
    import inspect
    import numpy as np
    old, new = PY_MUTATIONS[name]
    text = inspect.getsource(oracle.gumbel_softmax)
    assert text.count(old) == 1, "mutation target not found exactly once: %r" % old
    scope = {"np": np, "Optional": __import__("typing").Optional}
    exec(text.replace(old, new), scope)
    monkeypatch.setattr(oracle, "gumbel_softmax", scope["gumbel_softmax"])
    caught = 0
    for check in PY_BATTERY:
        try:
            check()
        except (AssertionError, ValueError, FloatingPointError):
            caught += 1
    assert caught >= 1, "no pin noticed: " + name
