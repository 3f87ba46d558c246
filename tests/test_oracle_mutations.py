"""Do the pins bite?  Each case plants ONE plausible mistake in a copy of the CPU
oracle (a dropped term, a wrong sign or index, a transposed operand, a wrong
rounding mode) and checks that at least one pin of tests/test_oracle_pins.py or
tests/test_oracle_algorithm.py then fails.  The mistakes are planted in the
oracle's source text, on the CPU; the CUDA library is not involved."""
import os
import sys
import types

import pytest

import test_oracle_algorithm as algo_pins
import test_oracle_pins as pins

ORACLE_PATH = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "oracle", "muloco_oracle.py")

# (name, text in the oracle, what a mistaken author might have written, pins expected to catch it)
MUTATIONS = [
    ("ns: Gram of the wrong side", "A = X @ X.T", "A = X.T @ X", ["test_ns_matches_svd_closed_form"]),
    ("ns: cubic term dropped", "B = b * A + c * (A @ A)", "B = c * (A @ A)", ["test_ns_matches_svd_closed_form"]),
    ("ns: sign of b", "B = b * A + c * (A @ A)", "B = -b * A + c * (A @ A)", ["test_ns_scalar_iterates_golden"]),
    ("ns: quintic term applied to A, not A^2", "B = b * A + c * (A @ A)", "B = b * A + c * A", ["test_ns_scalar_iterates_golden"]),
    ("ns: no normalisation", "X = X / (np.linalg.norm(X) + float(eps))", "X = X / 1.0", ["test_ns_matches_svd_closed_form"]),
    ("ns: spectral instead of Frobenius norm", "X = X / (np.linalg.norm(X) + float(eps))",
     "X = X / (np.linalg.norm(X, 2) + float(eps))", ["test_ns_matches_svd_closed_form"]),
    ("ns: tall matrix not transposed back", "    if transposed:\n        X = X.T\n    return X", "    return X",
     ["test_ns_equivariance_and_transpose", "test_ns_matches_svd_closed_form"]),
    ("muon: dampened momentum", "m_new = float(beta) * M.astype(np.float64) + g",
     "m_new = float(beta) * M.astype(np.float64) + (1.0 - float(beta)) * g", ["test_muon_momentum_and_nesterov_input"]),
    ("muon: Nesterov uses the old momentum", "Uin = g + float(beta) * m_st if nesterov else m_st",
     "Uin = g + float(beta) * M0 if nesterov else m_st", ["test_muon_momentum_and_nesterov_input"]),
    ("muon: lr scale inverted", "return math.sqrt(cols / rows)", "return math.sqrt(rows / cols)",
     ["test_muon_lr_mult_is_sqrt_cols_over_rows", "test_muon_rank1_closed_form"]),
    ("muon: weight decay dropped", "W[...] = (w - eta * O - eta_wd * float(wd) * float(wd_mult) * w).astype(np.float32)",
     "W[...] = (w - eta * O).astype(np.float32)", ["test_muon_rank1_closed_form", "test_muon_weight_decay_scaling_flag"]),
    ("muon: update added instead of subtracted",
     "W[...] = (w - eta * O - eta_wd * float(wd) * float(wd_mult) * w).astype(np.float32)",
     "W[...] = (w + eta * O - eta_wd * float(wd) * float(wd_mult) * w).astype(np.float32)", ["test_muon_rank1_closed_form"]),
    ("adamw: second moment without the square", "(1.0 - b2) * g64 * g64", "(1.0 - b2) * g64",
     ["test_adamw_against_textbook_loop", "test_adamw_first_step_closed_form"]),
    ("adamw: eps inside the square root", "step = mh / (np.sqrt(vh) + float(eps))", "step = mh / np.sqrt(vh + float(eps))",
     ["test_adamw_first_step_closed_form", "test_adamw_against_textbook_loop"]),
    ("adamw: coupled (L2) decay", "+ float(wd) * float(wd_mult) * th\n", "+ 0.0 * th\n",
     ["test_adamw_first_step_closed_form", "test_adamw_against_textbook_loop"]),
    ("adamw: bias correction with t-1", "mh = mh / (1.0 - b1 ** t)", "mh = mh / (1.0 - b1 ** max(t - 1, 1))",
     ["test_adamw_constant_gradient_and_no_bias_correction", "test_adamw_against_textbook_loop"]),
    ("outer: pseudogradient sign", "acc += tg - th.astype(np.float64)", "acc += th.astype(np.float64) - tg",
     ["test_pseudogradient_definitions"]),
    ("outer: sum instead of mean", "return acc / len(thetas)", "return acc", ["test_pseudogradient_definitions"]),
    ("outer: old momentum in the parameter update", "- mu * u_new - eta * p)", "- (u_new - eta * p) - eta * p)",
     ["test_outer_step_closed_forms"]),
    ("outer: plain momentum (no Nesterov look-ahead)", "- mu * u_new - eta * p)", "- u_new)", ["test_outer_step_closed_forms"]),
    ("quantiser: truncation instead of round-to-nearest-even", "q = np.rint((xb * inv[:, None]).astype(np.float32))",
     "q = np.trunc((xb * inv[:, None]).astype(np.float32))",
     ["test_quantiser_round_half_to_even_and_brute_force", "test_quantiser_properties"]),
    ("quantiser: asymmetric range", "qmax = np.float32((1 << (bits - 1)) - 1)", "qmax = np.float32(1 << (bits - 1))",
     ["test_quantiser_properties", "test_quantiser_round_half_to_even_and_brute_force"]),
    ("quantiser: one scale per tensor", "amax = np.max(np.abs(xb), axis=1).astype(np.float32)          # [rows]",
     "amax = np.full(xb.shape[0], np.max(np.abs(x)), dtype=np.float32)",
     ["test_quantiser_blocks_do_not_span_rows_and_vectors_are_one_row", "test_quantiser_properties"]),
    ("schedule: fragments all due together", "if t % H == (j * H // J) % H", "if t % H == 0",
     ["test_fragments_due_schedule"]),
    ("two-stage: second quantisation skipped", "    _, _, psi = quantize_blocks(mean, bits, block)\n    return psi.reshape(tg.shape)",
     "    return mean", ["test_two_stage_compression_collapses_for_one_worker", "test_error_feedback_changes_nothing_when_nothing_is_lost"]),
    ("error feedback: accumulator keeps what was sent", "ef[i][...] = (e - c.reshape(e.shape)).astype(np.float32)",
     "ef[i][...] = e", ["test_error_feedback_conserves_what_was_not_sent"]),
    ("error feedback: delta not added", "e = ((beta * ef[i]).astype(np.float32) + delta).astype(np.float32)",
     "e = (beta * ef[i]).astype(np.float32) + np.float32(0) * delta", ["test_error_feedback_conserves_what_was_not_sent"]),
    ("top-k: smallest magnitudes kept", "tau = np.sort(flat)[n - kk]\n    return np.where(np.abs(a) >= tau, a, np.float32(0)).astype(np.float32)",
     "tau = np.sort(flat)[kk - 1]\n    return np.where(np.abs(a) <= tau, a, np.float32(0)).astype(np.float32)",
     ["test_topk_matches_brute_force_selection"]),
    ("top-k: selection on signed values", "tau = np.sort(flat)[n - kk]\n    return np.where(np.abs(a) >= tau, a,",
     "tau = np.sort(a.reshape(-1))[n - kk]\n    return np.where(a >= tau, a,", ["test_topk_matches_brute_force_selection"]),
    ("top-k: one entry too many", "tau = np.sort(flat)[n - kk]", "tau = np.sort(flat)[max(n - kk - 1, 0)]",
     ["test_topk_matches_brute_force_selection", "test_topk_is_the_best_k_term_approximation"]),
    ("top-k: selection per row", "    flat = np.abs(a).reshape(-1)\n    n = flat.size\n    if n == 0:\n        return a.copy()\n",
     "    if a.ndim == 2 and a.shape[0] > 1:\n        return np.stack([topk_sparsify(r, fraction) for r in a])\n"
     "    flat = np.abs(a).reshape(-1)\n    n = flat.size\n    if n == 0:\n        return a.copy()\n",
     ["test_topk_ties_counts_and_degenerate_inputs", "test_topk_matches_brute_force_selection"]),
    ("top-k: count rounded up", "max(1, math.floor(float(np.float32(fraction)) * n))", "max(1, math.ceil(float(np.float32(fraction)) * n))",
     ["test_topk_ties_counts_and_degenerate_inputs", "test_topk_matches_brute_force_selection"]),
    ("top-k: mean sparsified instead of the workers' deltas", "            c = topk_sparsify(delta, fraction)\n        acc = (acc + c).astype(np.float32)\n    return (acc * np.float32(1.0 / K)).astype(np.float32)",
     "            c = delta\n        acc = (acc + c).astype(np.float32)\n    return topk_sparsify((acc * np.float32(1.0 / K)).astype(np.float32), fraction)",
     ["test_sparsified_pseudogradient_definitions_and_error_feedback"]),
    ("top-k error feedback: sent part left in the accumulator", "ef[i][...] = (e - c).astype(np.float32)", "ef[i][...] = e",
     ["test_sparsified_pseudogradient_definitions_and_error_feedback"]),
    ("sync: replicas not reset", "self.theta_k[k][i][...] = self.theta_g[i]", "pass",
     ["test_j1_equals_non_streaming_and_state_is_kept_across_syncs", "test_streaming_touches_each_fragment_once_per_period",
      "test_k1_outer_identity_reproduces_plain_muon"]),
]


def _mutant(old: str, new: str) -> types.ModuleType:
    src = open(ORACLE_PATH).read()
    assert src.count(old) >= 1, f"mutation target not found in the oracle: {old!r}"
    src = src.replace(old, new, 1)
    if "M0" in new:                                   # helper name for the 'old momentum' mistake
        src = src.replace("    g = np.asarray(G, dtype=np.float64)\n    m_new =",
                          "    g = np.asarray(G, dtype=np.float64)\n    M0 = M.astype(np.float64)\n    m_new =", 1)
    mod = types.ModuleType("oracle_mutant")
    mod.__file__ = ORACLE_PATH
    sys.modules["oracle_mutant"] = mod                # dataclasses look their module up by name
    exec(compile(src, ORACLE_PATH, "exec"), mod.__dict__)
    return mod


def _run_pin(module, name, mutant) -> bool:
    """Runs one pin (all its parametrisations) against the mutant; True if it failed."""
    fn = getattr(module, name)
    saved = module.O
    module.O = mutant
    try:
        cases = [{}]
        for mark in getattr(fn, "pytestmark", []):
            if mark.name == "parametrize":
                names = [n.strip() for n in mark.args[0].split(",")]
                vals = [v if len(names) > 1 else (v,) for v in mark.args[1]]
                cases = [dict(c, **dict(zip(names, v))) for c in cases for v in vals]
        for kwargs in cases:
            try:
                fn(**kwargs)
            except Exception:                          # an assertion, or the mistake breaking the code outright
                return True
        return False
    finally:
        module.O = saved


def _find(name):
    return pins if hasattr(pins, name) else algo_pins


@pytest.mark.parametrize("label,old,new,expected", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(label, old, new, expected):
    mutant = _mutant(old, new)
    caught = [name for name in expected if _run_pin(_find(name), name, mutant)]
    assert caught, f"no pin noticed: {label}"


def test_unmodified_oracle_passes_the_same_harness():
    # the harness itself must not produce failures: an identity 'mutation' passes every pin used above
    clean = _mutant("A = X @ X.T", "A = X @ X.T")
    for name in sorted({n for m in MUTATIONS for n in m[3]}):
        assert not _run_pin(_find(name), name, clean), name
