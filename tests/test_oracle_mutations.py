"""Are the oracle's pins sharp?  Each case below plants one plausible mistake in a copy of the
oracle's C source (a dropped term, a wrong sign or index, a swapped operand, the other ordering),
builds it, and runs a battery of the pins against the mutant.  The battery is ordered: hand
examples, closed forms, library routines and invariants first, the brute-force re-evaluation
last.  Every mutant must be caught by the pin named beside it -- none may get as far as the
brute force, which is the test's own restatement of the algorithm."""
import ctypes
import os
import subprocess

import pytest

import oracle
import test_oracle_pins as pins

SRC = os.path.join(os.path.dirname(oracle.__file__), "desloc_oracle.c")

MUTANTS = {
    "adam_u_not_dampened": ("un[m] = c->beta1 * up + (1.0 - c->beta1) * gh;\n                vn[m] = c->beta2",
                            "un[m] = c->beta1 * up + gh;\n                vn[m] = c->beta2"),
    "adam_v_without_square": ("un[m] = c->beta1 * up + (1.0 - c->beta1) * gh;\n                vn[m] = c->beta2 * vp + (1.0 - c->beta2) * gh * gh;",
                              "un[m] = c->beta1 * up + (1.0 - c->beta1) * gh;\n                vn[m] = c->beta2 * vp + (1.0 - c->beta2) * gh;"),
    "adam_v_decays_with_beta1": ("un[m] = c->beta1 * up + (1.0 - c->beta1) * gh;\n                vn[m] = c->beta2 * vp",
                                 "un[m] = c->beta1 * up + (1.0 - c->beta1) * gh;\n                vn[m] = c->beta1 * vp"),
    "adam_eps_outside_the_root": ("d = lr / sqrt(vn[m] + c->eps * c->eps) * un[m];",
                                  "d = lr / (sqrt(vn[m]) + c->eps) * un[m];"),
    "step_sign": ("xn[m] = xp * (1.0 - lr * c->weight_decay) - d;", "xn[m] = xp * (1.0 - lr * c->weight_decay) + d;"),
    "weight_decay_without_lr": ("xp * (1.0 - lr * c->weight_decay)", "xp * (1.0 - c->weight_decay)"),
    "average_after_by_default": ("const int post = (c->flags & DESLOC_ORACLE_POST_AVERAGE) != 0;",
                                 "const int post = 1;"),
    "adopt_divides_by_new_v": ("double vold = (double)v[k];", "double vold = vn[m];"),
    "adopt_divides_by_mean_v": ("if ((c->flags & DESLOC_ORACLE_ADOPT_AVG_NORMALISER) && !post &&", "if (!post &&"),
    "adopt_clip_lower_bound_missing": ("if (r < -clip_bound) r = -clip_bound;", ";"),
    "adopt_momentum_takes_raw_gradient": ("un[m] = c->beta1 * up + (1.0 - c->beta1) * r;",
                                          "un[m] = c->beta1 * up + (1.0 - c->beta1) * gh;"),
    "sync_one_step_late": ("if (Kx > 0 && t % Kx == 0) mask |= ORACLE_SYNC_X;",
                           "if (Kx > 0 && (t + Kx - 1) % Kx == 0) mask |= ORACLE_SYNC_X;"),
    "sgdm_keeps_v_bit": ("if (opt != ORACLE_SGDM && Kv > 0 && t % Kv == 0)", "if (Kv > 0 && t % Kv == 0)"),
    "mean_divides_by_m_minus_1": ("return acc / (double)M;\n}", "return acc / (double)(M > 1 ? M - 1 : 1);\n}"),
    "u_sync_takes_x_mean": ("const double up = (!post && (mask & ORACLE_SYNC_U)) ? ubar : (double)u[k];",
                            "const double up = (!post && (mask & ORACLE_SYNC_U)) ? xbar : (double)u[k];"),
    "x_sync_ignored": ("const double xp = (!post && (mask & ORACLE_SYNC_X)) ? xbar : (double)x[k];",
                       "const double xp = (double)x[k];"),
    "clip_off": ("if (a > rho) a = rho;", ";"),
    "clip_loses_sign": ("return g < 0.0 ? -a : a;", "return a;"),
    "norm_clip_squares_the_norm": ("scales_out[m] = (nrm > max_norm) ? max_norm / nrm : 1.0;",
                                   "scales_out[m] = (nrm > max_norm) ? max_norm / (nrm * nrm) : 1.0;"),
    "norm_clip_after_coordinate_clip": ("clip_coord((double)g[k] * gs, c->clip_rho)", "clip_coord((double)g[k], c->clip_rho) * gs"),
    "rel_change_normalised_by_now": ("den += b * b;", "den += a * a;"),
    "d_without_learning_rate": ("if (d_out) d_out[k] = d;", "if (d_out) d_out[k] = d / lr;"),
    "d_includes_the_decay_term": ("if (d_out) d_out[k] = d;", "if (d_out) d_out[k] = xp - xn[m];"),
    "d_of_the_wrong_worker": ("if (d_out) d_out[k] = d;", "if (d_out) d_out[(int64_t)(M - 1 - m) * stride + i] = d;"),
    "tensor_norm_without_root": ("out[(int64_t)m * num_tensors + k] = sqrt(acc);", "out[(int64_t)m * num_tensors + k] = acc;"),
    "tensor_norm_reads_the_padding": ("const double e = a[(int64_t)m * stride + offs[k] + i];",
                                      "const double e = a[(int64_t)m * stride + offs[k] + i - (k > 0)];"),
    "total_norm_adds_norms_not_squares": ("all += acc;", "all += sqrt(acc);"),
    "post_average_steps_with_local_states": ("            if (mask & ORACLE_SYNC_U) {\n                double acc = 0.0;\n                for (int m = 0; m < M; ++m) acc += un[m];\n                acc /= (double)M;\n                for (int m = 0; m < M; ++m) un[m] = acc;\n            }",
                                             "            ;"),
}


BATTERY = [
    ("hand_sgdm", pins.test_hand_example_sgdm_exact_rationals),
    ("hand_adam", pins.test_hand_example_adam),
    ("hand_adopt", pins.test_hand_example_adopt),
    ("schedule", pins.test_schedule_is_t_mod_k_from_zero),
    ("clip_definition", pins.test_coordinate_clip_definition),
    ("adam_root_closed_form", pins.test_adam_stability_term_sits_inside_the_root),
    ("adopt_clip_closed_form", pins.test_adopt_normalised_gradient_clip_is_two_sided),
    ("mean_preserved", pins.test_averaging_step_preserves_the_mean_of_the_averaged_array),
    ("norm_clip_closed_forms", pins.test_norm_clip_closed_forms),
    ("rel_change_closed_forms", pins.test_rel_change_closed_forms),
    ("worker_mean_closed_forms", pins.test_worker_mean_closed_forms_and_doubling_keeps_the_mean),
    ("d_hand_examples", pins.test_update_d_matches_hand_examples),
    ("d_closed_forms", pins.test_update_d_one_step_closed_forms),
    ("d_torch_adamw", pins.test_update_d_is_the_parameter_change_of_torch_adamw_without_the_decay_term),
    ("tensor_norms", pins.test_tensor_norms_closed_forms_and_library),
    ("torch_adamw", lambda: pins.test_m1_is_plain_adam((3, 5, 7), 0.1)),
    ("torch_sgd", lambda: pins.test_m1_is_plain_sgdm((4, 2, 0))),
    ("sgdm_mean_iterate", lambda: pins.test_sgdm_mean_iterate_is_centralized_sgdm((2, 3))),
    ("schedule_independent_means", lambda: pins.test_state_means_do_not_depend_on_schedule_exact(2)),
    ("post_full_sync_minibatch_sgdm",
     pins.test_post_average_full_sync_makes_replicas_equal_and_k1_is_minibatch_sgdm),
    ("post_is_pre_shifted", lambda: pins.test_post_average_equals_pre_average_shifted_by_one_step(oracle.SGDM)),
    ("brute_force", lambda: [pins.test_brute_force_small(3, opt, False)
                             for opt in (oracle.ADAM, oracle.ADOPT, oracle.SGDM)]
     + [pins.test_brute_force_small(2, oracle.ADAM, True)]),
]

# The pin that catches each planted mistake first.
CAUGHT_BY = {
    "adam_eps_outside_the_root": "adam_root_closed_form",
    "adam_u_not_dampened": "hand_adam",
    "adam_v_decays_with_beta1": "d_torch_adamw",
    "adam_v_without_square": "hand_adam",
    "adopt_clip_lower_bound_missing": "adopt_clip_closed_form",
    "adopt_divides_by_mean_v": "hand_adopt",
    "adopt_divides_by_new_v": "hand_adopt",
    "adopt_momentum_takes_raw_gradient": "hand_adopt",
    "average_after_by_default": "hand_sgdm",
    "clip_loses_sign": "clip_definition",
    "clip_off": "clip_definition",
    "d_includes_the_decay_term": "d_closed_forms",
    "d_of_the_wrong_worker": "d_hand_examples",
    "d_without_learning_rate": "d_hand_examples",
    "mean_divides_by_m_minus_1": "hand_sgdm",
    "norm_clip_after_coordinate_clip": "norm_clip_closed_forms",
    "norm_clip_squares_the_norm": "norm_clip_closed_forms",
    "post_average_steps_with_local_states": "post_full_sync_minibatch_sgdm",
    "rel_change_normalised_by_now": "rel_change_closed_forms",
    "sgdm_keeps_v_bit": "schedule",
    "step_sign": "hand_sgdm",
    "sync_one_step_late": "hand_sgdm",
    "tensor_norm_reads_the_padding": "tensor_norms",
    "tensor_norm_without_root": "tensor_norms",
    "total_norm_adds_norms_not_squares": "tensor_norms",
    "u_sync_takes_x_mean": "hand_sgdm",
    "weight_decay_without_lr": "d_closed_forms",
    "x_sync_ignored": "hand_sgdm",
}


def first_failing_pin():
    """Runs the battery in order; returns the name of the first pin that fails, or None."""
    for name, pin in BATTERY:
        try:
            pin()
        except AssertionError:
            return name
    return None


def test_battery_passes_on_the_real_oracle():
    assert first_failing_pin() is None


def test_every_mutant_has_a_named_catcher():
    assert sorted(CAUGHT_BY) == sorted(MUTANTS)
    assert "brute_force" not in CAUGHT_BY.values()


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_planted_mistake_is_caught(name, tmp_path, monkeypatch):
    old, new = MUTANTS[name]
    src = open(SRC).read()
    assert src.count(old) >= 1, f"mutation site for {name} not found: the oracle source changed"
    mutated = src.replace(old, new, 1)
    c_file, so_file = tmp_path / "mutant.c", tmp_path / "mutant.so"
    c_file.write_text(mutated)
    subprocess.check_call(["gcc", "-O1", "-std=c99", "-ffp-contract=off", "-shared", "-fPIC", "-o",
                           str(so_file), str(c_file), "-lm"])
    monkeypatch.setattr(oracle, "_lib", oracle.configure(ctypes.CDLL(str(so_file))))
    caught = first_failing_pin()
    assert caught == CAUGHT_BY[name], f"{name}: caught by {caught}, expected {CAUGHT_BY[name]}"
