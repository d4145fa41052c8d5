"""Do the pins bite?  Each case plants one plausible mistake in a copy of the oracle's C source (a dropped term,
a wrong sign, a swapped operand or index, a wrong divisor), builds it, and requires that at least one of the
pins in test_oracle_pins.py fails against it.  The mistakes live on the CPU, in the copy only.

Also checked: the unmodified source passes the same pins through the same machinery (so a failure below is
caused by the planted mistake, not by the harness), and mistakes in the Python part of the oracle (selection,
scores, schedule sizing) are caught the same way.
"""

import os
import subprocess

import pytest

import test_oracle_pins as pins
from oracle import build as obuild
from oracle import reference as orc

# (name, text in cocodc_oracle.c, replacement)
C_MUTATIONS = [
    ("pseudo-gradient sign", "double delta_m = (double)snap[(size_t)m * snap_stride + i] - thg;",
     "double delta_m = thg - (double)snap[(size_t)m * snap_stride + i];"),
    ("mean not divided by M", "Delta = sum / (double)M;", "Delta = sum;"),
    ("mean divided by M+1", "Delta = sum / (double)M;", "Delta = sum / (double)(M + 1);"),
    ("pseudo-gradient from current instead of recorded parameters",
     "double delta_m = (double)snap[(size_t)m * snap_stride + i] - thg;",
     "double delta_m = (double)now[(size_t)m * now_stride + i] - thg;"),
    ("momentum without the old buffer", "double u_new = mu * (double)u[i] + Delta;", "double u_new = Delta;"),
    ("plain instead of Nesterov momentum", "double G = thg + eta * (Delta + mu * u_new);", "double G = thg + eta * u_new;"),
    ("learning rate dropped", "double G = thg + eta * (Delta + mu * u_new);", "double G = thg + (Delta + mu * u_new);"),
    ("global update subtracted", "double G = thg + eta * (Delta + mu * u_new);", "double G = thg - eta * (Delta + mu * u_new);"),
    ("rate not divided by tau", "double g = sgn4 * (a - b) / (double)tau;", "double g = sgn4 * (a - b);"),
    ("forward and printed readings swapped", "double sgn4 = (sign_mode == SIGN_FORWARD) ? 1.0 : -1.0;",
     "double sgn4 = (sign_mode == SIGN_FORWARD) ? -1.0 : 1.0;"),
    ("descent reading not flipped", "double sgn7 = (sign_mode == SIGN_DESCENT) ? -1.0 : 1.0;", "double sgn7 = 1.0;"),
    ("divergence from current instead of recorded parameters", "double D = G - b;", "double D = G - a;"),
    ("divergence sign", "double D = G - b;", "double D = b - G;"),
    ("second-order term linear in g", "double gcorr = g + lambda * g * g * (D / (double)H);",
     "double gcorr = g + lambda * g * (D / (double)H);"),
    ("second-order term without 1/H", "double gcorr = g + lambda * g * g * (D / (double)H);",
     "double gcorr = g + lambda * g * g * D;"),
    ("second-order term without lambda", "double gcorr = g + lambda * g * g * (D / (double)H);",
     "double gcorr = g + g * g * (D / (double)H);"),
    ("H and tau swapped in Eq. 6", "double gcorr = g + lambda * g * g * (D / (double)H);",
     "double gcorr = g + lambda * g * g * (D / (double)tau);"),
    ("target without the tau steps", "target = G + sgn7 * gcorr * (double)tau;", "target = G + sgn7 * gcorr;"),
    ("target starts from the old global state", "target = G + sgn7 * gcorr * (double)tau;",
     "target = b + sgn7 * gcorr * (double)tau;"),
    ("blend weights swapped", "return (1.0 - alpha) * a + alpha * target;", "return alpha * a + (1.0 - alpha) * target;"),
    ("blend keeps the local value", "return (1.0 - alpha) * a + alpha * target;", "return (1.0 - alpha) * a + target;"),
    ("norm of Delta not squared", "sumsq += (long double)Delta * (long double)Delta;", "sumsq += fabsl((long double)Delta);"),
    ("sum of squares sums plain values", "s += (long double)x[i] * (long double)x[i];", "s += (long double)x[i];"),
    ("worker rows transposed in the merge", "double a = (double)now[(size_t)m * now_stride + i];\n                double b = (double)snap[(size_t)m * snap_stride + i];\n                now_out[(size_t)m * n + i] =",
     "double a = (double)now[(size_t)(M - 1 - m) * now_stride + i];\n                double b = (double)snap[(size_t)m * snap_stride + i];\n                now_out[(size_t)m * n + i] ="),
    ("received sum divided by the local worker count", "Delta = total / (double)M_total;",
     "Delta = total / (double)M;"),
    ("only the first device's partial sum is used", "for (int r = 0; r < n_recv; ++r)", "for (int r = 0; r < 1; ++r)"),
    ("per-device sum skips the last worker", "for (int m = 0; m < M; ++m)\n            sum += (double)snap[(size_t)m * snap_stride + i] - thg;",
     "for (int m = 0; m + 1 < M || m == 0; ++m)\n            sum += (double)snap[(size_t)m * snap_stride + i] - thg;"),
]

# the pins that exercise the C part (each a zero-argument callable)
def _c_pins():
    out = []
    for name in ("test_mean_is_identity_for_one_worker", "test_identical_workers_and_permutation",
                 "test_plain_averaging_when_lr_one_no_momentum", "test_plain_sgd_when_no_momentum",
                 "test_outer_update_matches_torch_nesterov_sgd", "test_lambda_zero_is_linear_in_local_change",
                 "test_compensation_term_scaling_laws", "test_self_sync_is_a_no_op_for_forward_and_descent",
                 "test_alpha_zero_keeps_local_parameters", "test_reduces_to_streaming_diloco", "test_reduces_to_diloco",
                 "test_unprocessed_fragments_are_not_reported_and_layouts_agree", "test_norm_closed_forms",
                 "test_step_norm_is_norm_of_delta", "test_received_sum_mode_equals_stacked_workers"):
        out.append(getattr(pins, name))
    for row in pins.rows("nesterov_worked.txt"):
        out.append(lambda row=row: pins.test_nesterov_golden(row))
    for row in pins.rows("delay_compensation_worked.txt"):
        out.append(lambda row=row: pins.test_delay_compensation_golden(row))
    for sign in (orc.SIGN_FORWARD, orc.SIGN_PRINTED, orc.SIGN_DESCENT):
        out.append(lambda sign=sign: pins.test_zero_delay_gives_global_state(sign, 0.5, 4))
    return out


def _failures(checks):
    failed = 0
    for check in checks:
        try:
            check()
        except (AssertionError, ValueError, ZeroDivisionError, FloatingPointError):
            failed += 1
    return failed


@pytest.fixture()
def swap_library(tmp_path, monkeypatch):
    def swap(source_text):
        src = tmp_path / "mutant.c"
        lib = tmp_path / "libmutant.so"
        src.write_text(source_text)
        subprocess.run(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-o", str(lib), str(src), "-lm"],
                       check=True)
        monkeypatch.setattr(orc, "_lib", orc.load_library(str(lib)))
    return swap


def test_unmodified_source_passes_through_the_same_machinery(swap_library):
    swap_library(open(obuild.SOURCE).read())
    assert _failures(_c_pins()) == 0


@pytest.mark.parametrize("name,old,new", C_MUTATIONS, ids=[m[0] for m in C_MUTATIONS])
def test_planted_mistake_in_the_arithmetic_is_caught(swap_library, name, old, new):
    text = open(obuild.SOURCE).read()
    assert text.count(old) >= 1, f"mutation target not found: {name}"
    swap_library(text.replace(old, new, 1))
    assert _failures(_c_pins()) >= 1, f"no pin noticed: {name}"


# ---- the Python part: selection, scores, schedule sizing ------------------------------------------------

def _py_pins():
    out = [pins.test_sync_budget_never_below_K, pins.test_budget_one_is_algorithm_2,
           pins.test_never_synced_fragments_go_first_in_index_order, pins.test_count_budget_brute_force,
           pins.test_params_budget_brute_force, pins.test_selection_is_deterministic_and_rejects_nan,
           pins.test_norm_closed_forms, pins.test_unprocessed_fragments_are_not_reported_and_layouts_agree,
           pins.test_exact_budget_matches_the_textbook_knapsack_table,
           pins.test_exact_budget_forced_fragments_ties_and_head]
    for row in pins.rows("schedule_sizing.txt"):
        out.append(lambda row=row: pins.test_sync_budget_golden(row))
    return out


PY_MUTATIONS = [
    ("floor replaced by rounding up in Eq. 8", "sync_budget",
     lambda f: (lambda K, H, gamma, Tc, Ts: (max(K, -int(-gamma * H * Tc // Ts)), max(1, H // max(K, -int(-gamma * H * Tc // Ts)))))),
    ("Eq. 8 without the max with K", "sync_budget",
     lambda f: (lambda K, H, gamma, Tc, Ts: (max(1, int(gamma * H * Tc / Ts)), max(1, H // max(1, int(gamma * H * Tc / Ts)))))),
    ("selection ignores staleness", "select_fragments",
     lambda f: (lambda scores, last_sync, sizes, t_now, H, kind, budget, ineligible=None:
                f(scores, last_sync, sizes, t_now, 10 ** 9, kind, budget, ineligible))),
    ("selection takes the smallest score", "select_fragments",
     lambda f: (lambda scores, last_sync, sizes, t_now, H, kind, budget, ineligible=None:
                f([-float(s) for s in scores], last_sync, sizes, t_now, H, kind, budget, ineligible))),
    ("selection ignores the ineligible mask", "select_fragments",
     lambda f: (lambda scores, last_sync, sizes, t_now, H, kind, budget, ineligible=None:
                f(scores, last_sync, sizes, t_now, H, kind, budget, None))),
    ("parameter budget counted in fragments", "select_fragments",
     lambda f: (lambda scores, last_sync, sizes, t_now, H, kind, budget, ineligible=None:
                f(scores, last_sync, [1] * len(sizes), t_now, H, kind, budget, ineligible))),
    ("exact budget falls back to the greedy walk", "select_fragments",
     lambda f: (lambda scores, last_sync, sizes, t_now, H, kind, budget, ineligible=None:
                f(scores, last_sync, sizes, t_now, H, min(kind, 1), budget, ineligible))),
    ("score not divided by the interval", "fragment_scores",
     lambda f: (lambda fragments, delta_g, interval=None: f(fragments, delta_g, None))),
]


def test_python_pins_pass_unmodified():
    assert _failures(_py_pins()) == 0


@pytest.mark.parametrize("name,attr,wrap", PY_MUTATIONS, ids=[m[0] for m in PY_MUTATIONS])
def test_planted_mistake_in_the_decisions_is_caught(monkeypatch, name, attr, wrap):
    monkeypatch.setattr(orc, attr, wrap(getattr(orc, attr)))
    assert _failures(_py_pins()) >= 1, f"no pin noticed: {name}"
