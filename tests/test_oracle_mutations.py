"""The pins must have teeth: plant one plausible mistake at a time in a copy of the oracle's source
(on the CPU, in a temporary directory) and check that at least one pin fails for it."""

import ctypes
import subprocess
from pathlib import Path

import numpy as np
import pytest

import test_oracle_allocate as t_alloc
import test_oracle_fit as t_fit
import test_oracle_gains as t_gains
import test_oracle_normalise as t_norm
import test_oracle_warm_start as t_warm

SRC = Path(__file__).resolve().parent.parent / "oracle" / "slaq_oracle.cpp"

# (what is planted, text to replace, replacement)
MUTATIONS = [
    ("reduction with the wrong sign", "const double delta = loss[i - 1] - loss[i];",
     "const double delta = loss[i] - loss[i - 1];"),
    ("family I Jacobian: wrong sign of d/db", "J[1] = dq * x;", "J[1] = -dq * x;"),
    ("family II Jacobian: wrong sign of d/dbeta", "J[1] = -x * e;", "J[1] = x * e;"),
    ("family I: c dropped from the denominator", "const double q = p[0] * x * x + p[1] * x + p[2];",
     "const double q = p[0] * x * x + p[1] * x;"),
    ("weights in the wrong order", "D.w[i] = std::pow(gamma, (double)(H - 1 - i));",
     "D.w[i] = std::pow(gamma, (double)i);"),
    ("weight dropped from the gradient", "accg[a] += w * (long double)J[a] * r;", "accg[a] += (long double)J[a] * r;"),
    ("normal matrix transposed into a lower-triangular copy only", "A[a][b] = A[b][a] = (double)accA[a][b];",
     "A[a][b] = (double)accA[a][b];"),
    ("acceptance test inverted", "if (S_trial < S) {", "if (S_trial > S) {"),
    ("window coordinate not centred on the newest point", "D.x[i] = (double)(i - (H - 1)) / D.span;",
     "D.x[i] = (double)i / D.span;"),
    ("step in window coordinates uses s instead of w", "const double dX = T * w / (fit.span * den * den_prev);\n"
     "            const double q_now", "const double dX = T * s / (fit.span * den * den_prev);\n            const double q_now"),
    ("iterations per epoch without the serial part", "const double den = s * (double)n + w;",
     "const double den = w;"),
    ("exponential gain without the decay factor", "gain = std::exp(alpha - beta * X_prev) * (-std::expm1(-beta * dX));",
     "gain = -std::expm1(-beta * dX);"),
    ("ties go to the highest job id", "return l.job > r.job;", "return l.job < r.job;"),
    ("greedy picks the smallest gain", "if (l.gain != r.gain) return l.gain < r.gain;",
     "if (l.gain != r.gain) return l.gain > r.gain;"),
    ("no one-core floor", "alloc[j] = 1;\n                ++handed;", "alloc[j] = 0;"),
    ("time law: slope and intercept mixed up", "const double ss = (st - ww * su) / cnt;",
     "const double ss = (st + ww * su) / cnt;"),
    ("warm start: family I carried without the shift of the origin", "out[1] = (2.0 * a * t + b) * r / sigma;",
     "out[1] = b * r / sigma;"),
    ("warm start: family II carried without the change of scale", "out[0] = p[0] - p[1] * t + std::log(sigma);",
     "out[0] = p[0] - p[1] * t;"),
    ("warm start: stretch of the window inverted", "const double r = D.span / warm->span;",
     "const double r = warm->span / D.span;"),
    ("warm start: an unusable carried point is kept", "startedI = rI.ok;", "startedI = true;"),
    ("envelope: chord test inverted", "<= (R[n] - R[b]) * (double)(b - a)) hull.pop_back();",
     ">= (R[n] - R[b]) * (double)(b - a)) hull.pop_back();"),
    ("target hint: every gain capped by the whole allowance", "const double left = reduction_cap - before;",
     "const double left = reduction_cap;"),
    ("fallback: mean change without the weights", "num += (long double)D.w[i] * dnorm;", "num += (long double)dnorm;"),
    ("fallback: no cap at the newest level", "out.r_cap = D.y[H - 1] > 0.0 ? D.y[H - 1] : kInf;", "out.r_cap = kInf;"),
    ("fallback: a window of four points or more without a fit predicts nothing",
     "out.status = (H >= cfg.min_fit_points) ? ST_FIT_FAILED : ST_SHORT;",
     "out.status = (H >= cfg.min_fit_points) ? ST_FLAT : ST_SHORT;"),
]

PINS = [
    lambda m: t_norm.test_hand_worked_example(m),
    lambda m: t_norm.test_changes_fall_from_one(m),
    lambda m: t_fit.test_solver_on_a_line_is_weighted_linear_regression(m),
    lambda m: [t_fit.test_jacobians_match_central_differences(m, f, p)
               for f, p in ((0, [0.7, 1.3, 2.1, -0.2]), (1, [-0.5, 1.7, 0.2, 0.0]))],
    lambda m: t_fit.test_fit_never_raises_the_objective_and_ends_at_a_local_minimum(m),
    lambda m: t_fit.test_exact_recovery_of_noise_free_curves(m),
    lambda m: t_gains.test_gains_telescope_to_the_curve_drop(m),
    lambda m: t_gains.test_time_model_recovered_from_samples(m),
    lambda m: t_alloc.test_greedy_equals_brute_force_on_tiny_clusters(m),
    lambda m: t_alloc.test_capacity_and_floor(m),
    lambda m: t_alloc.test_ties_go_to_the_lowest_job_id(m),
    lambda m: [t_warm.test_carried_parameters_describe_the_same_curve(m, f) for f in (0, 1)],
    lambda m: t_warm.test_the_solver_never_ends_above_its_carried_starting_point(m),
    lambda m: t_warm.test_an_unusable_carried_point_falls_back_to_the_first_guess(m),
    lambda m: t_fit.test_windows_on_which_no_family_can_start_use_the_mean_normalised_change(m),
    lambda m: t_fit.test_the_cap_of_the_fallback_is_the_newest_normalised_level(m),
    lambda m: t_gains.test_concave_envelope_equals_its_definition(m),
    lambda m: t_gains.test_target_loss_hint_caps_the_predicted_reduction(m),
]


@pytest.fixture(scope="module")
def pristine_source():
    return SRC.read_text()


@pytest.mark.parametrize("what,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_a_planted_mistake_is_caught(oracle_mod, pristine_source, tmp_path, what, old, new):
    assert pristine_source.count(old) == 1, f"mutation site not found exactly once: {old!r}"
    src = tmp_path / "mutant.cpp"
    lib_path = tmp_path / "libmutant.so"
    src.write_text(pristine_source.replace(old, new))
    subprocess.run(["g++", "-std=c++17", "-O1", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared", "-o",
                    str(lib_path), str(src)], check=True)
    mutant = oracle_mod._bind(ctypes.CDLL(str(lib_path)))
    good = oracle_mod._load()
    caught = []
    oracle_mod._lib = mutant
    try:
        for i, pin in enumerate(PINS):
            try:
                with np.errstate(all="ignore"):
                    pin(oracle_mod)
            except Exception:   # an assertion, or the mutant broke so badly that the pin could not even run
                caught.append(i)
                break
    finally:
        oracle_mod._lib = good
    assert caught, f"no pin noticed: {what}"


def test_the_pristine_oracle_passes_the_same_pins(oracle_mod):
    for pin in PINS:
        pin(oracle_mod)
