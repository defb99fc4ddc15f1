"""The pins have teeth: a mistake planted in a copy of the reference makes at least one fail.

Each mutant is the reference's C source with one line changed (a flipped sign, a dropped
term, a wrong index, another reading of the staleness).  It is built in a temporary folder
and the pin tests are re-run against it; every mutant must be caught.
"""
import json
import os
import shutil
import subprocess

import pytest

from oracle import reference as R
from tests import test_oracle_arrivals as TA
from tests import test_oracle_update as TU

ORACLE_DIR = os.path.dirname(os.path.abspath(R.__file__))

MUTANTS = {
    "decay_sign": ("update_rule.inc", "REAL t = acc + dk * w[k];", "REAL t = acc - dk * w[k];"),
    "descent_sign": ("update_rule.inc", "w[k] = w[k] - v[k];", "w[k] = w[k] + v[k];"),
    "momentum_dropped": ("update_rule.inc", "v[k] = m * v[k] + t;", "v[k] = t;"),
    "decay_dropped": ("update_rule.inc", "REAL t = acc + dk * w[k];", "REAL t = acc;"),
    "no_averaging": ("update_rule.inc", "((double)c * (double)sigma[l])", "((double)sigma[l])"),
    "wrong_gradient_index": ("update_rule.inc", "acc = acc + s[l] * grads[l][k];", "acc = acc + s[l] * grads[0][k];"),
    "wrong_scale_index": ("update_rule.inc", "acc = acc + s[l] * grads[l][k];", "acc = acc + s[0] * grads[l][k];"),
    "decay_unmodulated": ("update_rule.inc", "const REAL d = ROUND_SCALE(wd * S);", "const REAL d = ROUND_SCALE(wd * alpha0[0]);"),
    "rate_at_apply_time": ("softsync_oracle.c", "alpha0[l] = ps->pending[order[l]].alpha0;", "alpha0[l] = ps->alpha0;"),
    "barrier_lets_stale_in": ("softsync_oracle.c", "if (tau != 0) return -3;", "if (tau > 1) return -3;"),
    "regrouped_sum": ("update_rule.inc", "v[k] = m * v[k] + t;", "v[k] = (m * v[k] + acc) + (t - acc);"),
    "penalty_linear_in_staleness": ("update_rule.inc", "pow(rho, (double)tau[l])", "(1.0 - (1.0 - rho) * (double)tau[l])"),
    "penalty_not_averaged": ("update_rule.inc", "pow(rho, (double)tau[l]) / (double)c", "pow(rho, (double)tau[l])"),
    "penalty_counts_one_more": ("update_rule.inc", "pow(rho, (double)tau[l])", "pow(rho, (double)tau[l] + 1.0)"),
    "multipliers_swapped": ("update_rule.inc", "if (dm) dk = (REAL)dm[k] * d;", "if (dm) dk = (REAL)lm[k] * d;"),
    "rate_multiplier_skips_decay": ("update_rule.inc", "if (lm) t = (REAL)lm[k] * t;", "if (lm) t = (REAL)lm[k] * acc + dk * w[k];"),
    "decay_multiplier_dropped": ("update_rule.inc", "if (dm) dk = (REAL)dm[k] * d;", ""),
    "layer_bound_off_by_one": ("softsync_oracle.c", "for (int64_t k = bounds[q]; k < bounds[q + 1]; ++k) {", "for (int64_t k = bounds[q] + (q > 0); k < bounds[q + 1] + (q + 1 < nseg); ++k) {"),
    "staleness_plus_one": ("softsync_oracle.c", "sigma = tau > 0 ? tau : 1;", "sigma = tau + 1;"),
    "staleness_ignored": ("softsync_oracle.c", "sigma = tau > 0 ? tau : 1;", "sigma = 1;"),
    "clock_jumps": ("softsync_oracle.c", "ps->ts += 1;", "ps->ts += ps->c;"),
    "arrival_order_sum": ("softsync_oracle.c", "if (a->learner != b->learner) return a->learner < b->learner;\n    return a->push_index < b->push_index;", "(void)a; (void)b; return 0;"),
    "group_one_short": ("softsync_oracle.c", "if (ps->npending == ps->c) { apply_pending(ps); return 1; }",
                        "if (ps->npending == ps->c || (ps->c > 1 && ps->npending == ps->c - 1)) { ps->c = ps->npending; apply_pending(ps); return 1; }"),
    "stale_pull": ("softsync_oracle.c", "ps->pulled_ts[learner] = ps->ts;", "ps->pulled_ts[learner] = ps->ts > 0 ? ps->ts - 1 : 0;"),
}


def _pins():
    examples = json.load(open(TU.GOLDEN))["examples"]
    pins = [lambda e=e, p=p: TU.test_hand_worked_examples_exact(e, p) for e in examples for p in (32, 64)]
    pins += [
        TU.test_single_learner_is_sequential_momentum_sgd_bit_for_bit,
        TU.test_single_learner_matches_library_sgd_optimizer,
        lambda: TU.test_one_softsync_with_barrier_is_synchronous_averaged_sgd(4),
        TU.test_downpour_case_is_per_push_sgd,
        TU.test_fp32_rounding_order_is_the_documented_one,
        TU.test_hardsync_protocol_is_eq_1_and_enforces_the_barrier,
        TU.test_step_schedule_without_momentum_is_library_sgd_with_a_changing_rate,
        TU.test_rate_in_force_at_arrival_enters_the_geometric_sum,
        lambda: TU.test_plain_rule_is_a_weighted_sum_of_gradients("exp", 12, 3),
        lambda: TU.test_exponential_penalty_is_a_weighted_sum_with_geometric_weights(0.8),
        TU.test_layer_multipliers_are_per_layer_rates_and_decays_of_library_sgd,
        TU.test_layer_multipliers_of_one_change_nothing_and_zero_rate_freezes_a_layer,
        TU.test_layer_multipliers_fp32_rounding_order,
        TU.test_momentum_is_a_geometric_sum_of_past_steps,
        TU.test_decay_and_momentum_follow_the_linear_recurrence_in_matrix_form,
        TU.test_arrival_order_inside_a_group_does_not_change_the_bits,
        lambda: TA.test_clock_and_staleness_against_brute_force_recount("uniform", 18, 4),
        lambda: TA.test_homogeneous_learners_match_measured_staleness(1, 0.8, 1.2),
    ]
    return pins


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_planted_mistake_is_caught(name, tmp_path):
    fname, old, new = MUTANTS[name]
    for f in ("softsync_oracle.c", "arrival_sim.c", "update_rule.inc"):
        shutil.copy(os.path.join(ORACLE_DIR, f), tmp_path / f)
    src = (tmp_path / fname).read_text()
    assert src.count(old) == 1, "mutation site must exist exactly once"
    (tmp_path / fname).write_text(src.replace(old, new))
    so = str(tmp_path / ("mutant_%s.so" % name))
    subprocess.run(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fPIC", "-shared", "-o", so,
                    "softsync_oracle.c", "arrival_sim.c", "-lm"], check=True, cwd=tmp_path)
    caught = 0
    with R.use_library(so):
        for pin in _pins():
            try:
                pin()
            except (AssertionError, ValueError, pytest.fail.Exception):
                caught += 1
    assert caught >= 1, "no pin noticed the planted mistake %r" % name


def test_unmutated_reference_passes_the_same_pins():
    for pin in _pins():
        pin()
