"""Do the pins bite?  Plausible mistakes are planted in copies of the oracle's C source (on the CPU,
never in the GPU path); every mutant must make at least one pin of test_oracle_pins.py fail."""
import ctypes
import os
import subprocess

import pytest

import oracle
import test_oracle_pins as pins

SRC = os.path.join(os.path.dirname(oracle.__file__), "sgdb_oracle.c")

# (name, text in the source, replacement)
MUTANTS = [
    ("divide_by_all_workers", "mean[i] = sum / (double)N;", "mean[i] = sum / (double)(N + 0 * ld + 1);"),
    ("stale_gradients_kept", "if (tags[w] != t) continue;", "if (tags[w] > t) continue;"),
    ("future_gradients_kept", "if (tags[w] != t) continue;", "if (tags[w] < t) continue;"),
    ("infinite_arrivals_kept", "if (!isfinite(arrival[w])) continue;", "if (isnan(arrival[w])) continue;"),
    ("ties_by_higher_id", "return a < b;", "return a > b;"),
    ("latest_first", "if (arrival[a] < arrival[b]) return 1;\n  if (arrival[a] > arrival[b]) return 0;",
     "if (arrival[a] > arrival[b]) return 1;\n  if (arrival[a] < arrival[b]) return 0;"),
    ("keeps_one_too_few", "for (int32_t k = 0; k < N; ++k) { /* the server stops waiting at |G| = N */",
     "for (int32_t k = 0; k + 1 < N; ++k) {"),
    ("row_major_transposed", "(int64_t)order[k] * ld + i", "(int64_t)i * N + order[k]"),
    ("sums_first_n_rows", "grad_at(grad, dtype, (int64_t)order[k] * ld + i)", "grad_at(grad, dtype, (int64_t)k * ld + i)"),
    ("bf16_low_half", "((uint32_t)bits) << 16", "((uint32_t)bits)"),
    ("sgd_sign", "theta[i] = theta[i] - opt->lr * g;", "theta[i] = theta[i] + opt->lr * g;"),
    ("momentum_scaled_gradient", "s0[i] = opt->momentum * s0[i] + g;", "s0[i] = opt->momentum * s0[i] + (1.0 - opt->momentum) * g;"),
    ("rmsprop_eps_outside", "sqrt(s0[i] + opt->eps)", "(sqrt(s0[i]) + opt->eps)"),
    ("rmsprop_no_decay_complement", "(1.0 - opt->decay) * g * g", "g * g"),
    ("rmsprop_lr_outside_momentum", "s1[i] = opt->momentum * s1[i] + opt->lr * g / sqrt(s0[i] + opt->eps);\n        theta[i] = theta[i] - s1[i];",
     "s1[i] = opt->momentum * s1[i] + g / sqrt(s0[i] + opt->eps);\n        theta[i] = theta[i] - opt->lr * s1[i];"),
    ("adam_no_bias_correction", "double m_hat = s0[i] / (1.0 - pow(opt->beta1, (double)opt->step));", "double m_hat = s0[i];"),
    ("adam_eps_inside", "(sqrt(v_hat) + opt->eps)", "sqrt(v_hat + opt->eps)"),
    ("adam_moments_swapped", "s1[i] = opt->beta2 * s1[i] + (1.0 - opt->beta2) * g * g;", "s1[i] = opt->beta1 * s1[i] + (1.0 - opt->beta1) * g * g;"),
    ("adagrad_decays", "s0[i] = s0[i] + g * g;", "s0[i] = 0.9 * s0[i] + g * g;"),
    ("adagrad_eps_inside", "theta[i] = theta[i] - opt->lr * g / (sqrt(s0[i]) + opt->eps);", "theta[i] = theta[i] - opt->lr * g / sqrt(s0[i] + opt->eps);"),
    ("ema_weights_swapped", "avg[i] = alpha * avg[i] + (1.0 - alpha) * theta[i];", "avg[i] = (1.0 - alpha) * avg[i] + alpha * theta[i];"),
    ("ema_of_updated_parameters", "if (rc == ORACLE_OK) oracle_ema(avg, theta_t, P, alpha);", "if (rc == ORACLE_OK) oracle_ema(avg, theta, P, alpha);"),
    ("ema_moves_without_update", "if (rc == ORACLE_OK) oracle_ema(avg, theta_t, P, alpha);", "oracle_ema(avg, theta_t, P, alpha);"),
    ("schedule_without_the_half", "(double)t * (double)N / (2.0 * T)", "(double)t * (double)N / T"),
    ("schedule_ignores_workers", "(double)t * (double)N / (2.0 * T)", "(double)t / (2.0 * T)"),
    ("deadline_strict", "if (!(arrival[w] <= deadline)) continue;", "if (!(arrival[w] < deadline)) continue;"),
    ("deadline_ignored", "if (!(arrival[w] <= deadline)) continue;", ""),
    ("deadline_drops_last_kept", "rc = oracle_aggregate(grad, dtype, P, ld, *n_kept, order, mean); /* divisor: the number kept */",
     "rc = oracle_aggregate(grad, dtype, P, ld, (*n_kept > 1 ? *n_kept - 1 : 1), order, mean);"),
    ("arrival_average_moves_every_time", "if (rc == ORACLE_OK && *outcome == 2 && avg != NULL) oracle_ema(avg, theta_t, P, alpha);",
     "if (rc == ORACLE_OK && *outcome >= 1 && avg != NULL) oracle_ema(avg, theta_t, P, alpha);"),
    ("arrival_average_of_updated", "if (rc == ORACLE_OK && *outcome == 2 && avg != NULL) oracle_ema(avg, theta_t, P, alpha);",
     "if (rc == ORACLE_OK && *outcome == 2 && avg != NULL) oracle_ema(avg, theta, P, alpha);"),
    ("arrival_counts_stale", "if (row_tag != t || t < state[2] || state[0] >= N) {", "if (t < state[2] || state[0] >= N) {"),
    ("arrival_never_closes", "state[2] = t + 1;", "state[2] = state[2];"),
    ("arrival_divides_late", "for (int64_t i = 0; i < P; ++i) acc[i] = acc[i] / (double)N;", "for (int64_t i = 0; i < P; ++i) acc[i] = acc[i] / (double)(N + 1);"),
    ("machine_sends_at_its_first_worker", "if (members == 0 || arrival[w] > latest) latest = arrival[w];",
     "if (members == 0 || arrival[w] < latest) latest = arrival[w];"),
    ("machine_with_a_stale_worker_counts", "if (tags[w] != t || !isfinite(arrival[w])) counts = 0;",
     "if (!isfinite(arrival[w])) counts = 0;"),
    ("machine_with_a_missing_worker_counts", "if (tags[w] != t || !isfinite(arrival[w])) counts = 0;",
     "if (tags[w] != t) counts = 0;"),
    ("machine_messages_are_sums", "total += message / (double)members;", "total += message;"),
    ("machine_mean_divides_by_workers", "mean[i] = total / (double)N;", "mean[i] = total / (double)(*n_rows);"),
    ("machine_without_workers_sends", "if (members == 0 || !counts) continue;", "if (!counts) continue;"),
    ("machine_rows_in_id_order", "while (pos > first && arrives_before(arrival, w, order[pos - 1])) {", "while (0) {"),
    ("machine_message_skips_a_worker", "message += grad_at(grad, dtype, (int64_t)w * ld + i);\n        ++members;",
     "if (members > 0) message += grad_at(grad, dtype, (int64_t)w * ld + i);\n        ++members;"),
    ("arrival_deadline_strict", "|| !isfinite(row_arrival) || !(row_arrival <= deadline)) {", "|| !isfinite(row_arrival) || !(row_arrival < deadline)) {"),
    ("arrival_deadline_ignored", "|| !isfinite(row_arrival) || !(row_arrival <= deadline)) {", "|| !isfinite(row_arrival)) {"),
    ("arrival_deadline_counts_stale", "if (row_tag != t || t < state[2] || !isfinite(row_arrival)", "if (t < state[2] || !isfinite(row_arrival)"),
    ("close_divides_by_n_min", "for (int64_t i = 0; i < P; ++i) acc[i] = acc[i] / (double)state[0];", "for (int64_t i = 0; i < P; ++i) acc[i] = acc[i] / (double)n_min;"),
    ("close_ignores_n_min", "if (state[0] < n_min) return ORACLE_INSUFFICIENT;", "if (state[0] < 1) return ORACLE_INSUFFICIENT;"),
    ("close_leaves_iteration_open", "state[0] = 0;\n  state[2] = t + 1;\n  *outcome = 2;\n  return ORACLE_OK;\n}\n", "state[0] = 0;\n  *outcome = 2;\n  return ORACLE_OK;\n}\n"),
    ("close_averages_updated_parameters", "if (avg != NULL) oracle_ema(avg, theta, P, alpha); /* theta is still theta(t) here */\n  for (int64_t i = 0; i < P; ++i) acc[i] = acc[i] / (double)state[0];\n  int rc = oracle_update(theta, s0, s1, acc, P, opt);\n  if (rc != ORACLE_OK) return rc;",
     "for (int64_t i = 0; i < P; ++i) acc[i] = acc[i] / (double)state[0];\n  int rc = oracle_update(theta, s0, s1, acc, P, opt);\n  if (rc != ORACLE_OK) return rc;\n  if (avg != NULL) oracle_ema(avg, theta, P, alpha);"),
    ("arrival_keeps_old_sum", "if (state[0] == 0)\n    for (int64_t i = 0; i < P; ++i) acc[i] = 0.0; /* G = {} */", ""),
]

PIN_TESTS = [getattr(pins, n) for n in dir(pins) if n.startswith("test_")]


def _run_pin(fn):
    marks = [m for m in getattr(fn, "pytestmark", []) if m.name == "parametrize"]
    if not marks:
        fn()
        return
    names = [n.strip() for n in marks[0].args[0].split(",")]
    for values in marks[0].args[1]:
        values = values if isinstance(values, (tuple, list)) else (values,)
        fn(**dict(zip(names, values)))


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_mutant_is_caught_by_a_pin(tmp_path, name, old, new):
    text = open(SRC).read()
    assert text.count(old) >= 1, "mutation site not found: the oracle changed, update this list"
    mutated = text.replace(old, new, 1)
    c_path, so_path = tmp_path / "mutant.c", tmp_path / "mutant.so"
    c_path.write_text(mutated)
    subprocess.run(["gcc", "-O1", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-o", str(so_path), str(c_path), "-lm"],
                   check=True)
    lib = ctypes.CDLL(str(so_path))
    for fn_name in ("oracle_select", "oracle_aggregate", "oracle_update", "oracle_step", "oracle_accumulate_arrival",
                    "oracle_step_ema", "oracle_select_deadline", "oracle_step_deadline", "oracle_accumulate_arrival_ema",
                    "oracle_select_grouped", "oracle_step_grouped", "oracle_accumulate_arrival_deadline", "oracle_accumulate_close"):
        getattr(lib, fn_name).restype = ctypes.c_int
    lib.oracle_ema.restype = None
    lib.oracle_learning_rate.restype = ctypes.c_double
    oracle._load()
    saved = oracle._lib
    oracle._lib = lib
    caught = []
    try:
        for fn in PIN_TESTS:
            try:
                _run_pin(fn)
            except AssertionError:
                caught.append(fn.__name__)
            except Exception as e:  # a crash of the mutant inside a pin also exposes it
                caught.append(fn.__name__ + ":" + type(e).__name__)
    finally:
        oracle._lib = saved
    assert caught, "no pin noticed the planted mistake '%s'" % name


def test_unmutated_oracle_passes_every_pin_through_the_same_driver():
    for fn in PIN_TESTS:
        _run_pin(fn)
