"""Do the pins have teeth?  Each entry below plants one plausible mistake in a copy of the oracle's
source (a dropped term, a wrong sign, a wrong index, a swapped operand), compiles it on the CPU and
runs the pins against it: at least one pin must fail for every mutant.  Nothing here touches a GPU or
the CUDA library; the mistakes exist only in a temporary file."""
import ctypes as C
import os
import subprocess
import tempfile

import pytest

import oracle
import test_oracle_dn as dn
import test_oracle_misc as misc
import test_oracle_variants as var

SRC = os.path.join(os.path.dirname(os.path.abspath(oracle.__file__)), "alsgd_oracle.cpp")

DN_PINS = [dn.test_hand_trace_c0_eight_elements, dn.test_hand_trace_c_quarter_eight_elements,
           dn.test_eq5_four_identical_arrivals_with_N1, dn.test_eq4_single_nesterov_step_random,
           dn.test_beta_zero_is_plain_outer_sgd, dn.test_buffer_holds_sum_and_resets_every_Nth,
           dn.test_momentum_weights_sum_to_beta_over_a_cycle,
           lambda: dn.test_matches_exact_unrolled_sums(3, 0.25), lambda: dn.test_matches_exact_unrolled_sums(4, 0.0),
           dn.test_one_cycle_equals_synchronous_diloco_with_nesterov, dn.test_current_mode_uses_running_theta,
           dn.test_server_bookkeeping_ticks_boundaries_staleness, dn.test_pg_norm_and_nonfinite_flag,
           dn.test_pg_norm_in_current_mode_is_taken_against_the_running_theta]
ADAM_PINS = [misc.test_adamw_hand_case, misc.test_adamw_first_step_is_sign_step_without_eps_and_decay,
             misc.test_adamw_constant_gradient_keeps_sign_stepping, misc.test_adamw_zero_gradient_is_pure_decoupled_decay,
             misc.test_adamw_against_library_adamw_in_double]
BF16_PINS = [misc.test_bf16_named_values, misc.test_bf16_every_high_half_at_the_critical_low_halves, misc.test_reseed_copies_and_casts]
HOST_PINS = [misc.test_shard_sampling_eq2, misc.test_dylu_values, misc.test_lr_schedule_endpoints_and_clamps, misc.test_poly_weight,
             misc.test_schedule_grace_window_timeline, misc.test_schedule_equal_speeds_behave_synchronously,
             misc.test_schedule_zero_grace_distinct_times_gives_singletons_in_time_order,
             misc.test_schedule_stops_at_t_max_local_updates, misc.test_schedule_invariants_on_random_timelines]
VAR_PINS = [var.test_buffered_hand_trace, var.test_buffered_with_N1_is_plain_nesterov_and_matches_dn_at_cycle_ends,
            var.test_delay_compensation_hand_case_and_zero_drift, var.test_weighted_arrival_hand_case_and_homogeneity,
            var.test_poly_weights_and_threshold_bookkeeping, var.test_delay_compensation_comes_before_the_staleness_weight,
            var.test_sgd_momentum_outer_step_hand_trace, var.test_sgd_momentum_outer_step_properties]

# (name, text to find, replacement, which occurrence (None = all), pins that must catch it)
MUTANTS = [
    ("boundary one arrival early", "((t + 1) % (uint64_t)N == 0)", "(t % (uint64_t)N == 0)", None, DN_PINS),
    ("pseudo-gradient sign", "float g = start - p[i];", "float g = p[i] - start;", 0, DN_PINS),
    ("buffer does not accumulate", "const float d = Delta[i] + g;", "const float d = g;", None, DN_PINS),
    ("momentum takes Delta, not Delta/N", "const float mn = (beta * m[i]) + (d * invN);          // m_{t+1}", "const float mn = (beta * m[i]) + d;          // m_{t+1}", None, DN_PINS),
    ("boundary step uses the old momentum", "const float u = (cb * mn) + gn;", "const float u = (cb * m[i]) + gn;", None, DN_PINS),
    ("ascent instead of descent", "theta[i] = theta[i] - (eps * u);", "theta[i] = theta[i] + (eps * u);", None, DN_PINS),
    ("buffer never reset", "m[i] = mn;\n            Delta[i] = 0.0f;", "m[i] = mn;\n            Delta[i] = d;", None, DN_PINS),
    ("boundary weight without + c", "(1.0 - (double)c * (double)N + (double)c)", "(1.0 - (double)c * (double)N)", None, DN_PINS),
    ("momentum activation ignored between boundaries", "(c == 0.0f) ? gn : ((cn * m[i]) + gn)", "gn", None, DN_PINS),
    ("g instead of g/N", "const float gn = g * invN;", "const float gn = g;", None, DN_PINS),
    ("momentum written between boundaries", "theta[i] = theta[i] - (eps * u);\n            Delta[i] = d;", "theta[i] = theta[i] - (eps * u);\n            m[i] = d;\n            Delta[i] = d;", None, DN_PINS),
    ("current mode ignored", "const float start = pg_current ? theta[i] : base[i];\n        float g", "const float start = base[i];\n        float g", None, DN_PINS),
    ("second moment of g, not g^2", "(omb2 * (gi * gi))", "(omb2 * gi)", None, ADAM_PINS),
    ("no first bias correction", "const float mh = mi / bc1;", "const float mh = mi;", None, ADAM_PINS),
    ("no second bias correction", "const float vh = vi / bc2;", "const float vh = vi;", None, ADAM_PINS),
    ("bias corrections swapped", "std::pow((double)b1, (double)step)", "std::pow((double)b2, (double)step)", None, ADAM_PINS),
    ("decay not scaled by the parameter", "(wd * pi)", "wd", None, ADAM_PINS),
    ("decay sign", "(r + (wd * pi))", "(r - (wd * pi))", None, ADAM_PINS),
    ("decay applied everywhere", "if (decay && decay[i]) {", "if (true) {", None, ADAM_PINS),
    ("first moment without (1 - b1)", "(omb1 * gi)", "gi", None, ADAM_PINS),
    ("round half up", "if (rest > 0x8000u) {", "if (rest >= 0x8000u) {", None, BF16_PINS),
    ("ties to odd", "if (keep & 1u) rounded", "if (!(keep & 1u)) rounded", None, BF16_PINS),
    ("truncation", "rounded = keep + 1u;                    // above the midpoint: up", "rounded = keep;", None, BF16_PINS),
    ("DyLU rounds instead of flooring", "std::floor((speeds[w] / vmax) * (double)H)", "std::round((speeds[w] / vmax) * (double)H)", None, HOST_PINS),
    ("DyLU may give zero steps", "x < 1.0 ? 1u", "x < 1.0 ? 0u", None, HOST_PINS),
    ("cosine sign", "(1.0 + std::cos(ratio * pi))", "(1.0 - std::cos(ratio * pi))", None, HOST_PINS),
    ("ratio not clamped", "if (ratio > 1.0) ratio = 1.0;", "", None, HOST_PINS),
    ("warm-up ignores eta_max", "(double)t * eta_max / (double)t_warmup", "(double)t / (double)t_warmup", None, HOST_PINS),
    ("ties to the higher id", "completed_time[u] < completed_time[w]) w = u;", "completed_time[u] <= completed_time[w]) w = u;", None, HOST_PINS),
    ("grace test strict", "completed_time[w] - tau_sync <= tau_grace", "completed_time[w] - tau_sync < tau_grace", None, HOST_PINS),
    ("restart without the grace period", "const double restart = tau_sync + tau_grace;", "const double restart = tau_sync;", None, HOST_PINS),
    ("t_local not counted", "t_local += local_updates[w];", "t_local += 0;", None, HOST_PINS),
    ("workers of a window restart at their own completion, not together",
     "completed_time[u] = restart + durations[(uint64_t)u * n_rounds + round[u]];",
     "completed_time[u] = completed_time[u] + tau_grace + durations[(uint64_t)u * n_rounds + round[u]];", None, HOST_PINS),
    ("window opened by the latest pending completion", "completed_time[u] < completed_time[w]) w = u;", "completed_time[u] > completed_time[w]) w = u;", None, HOST_PINS),
    ("shard gap sign", "const double gap = size_share - learned_share;", "const double gap = learned_share - size_share;", None, HOST_PINS),
    ("shard gap not clipped at zero", "probs[i] = gap > 0.0 ? gap : 0.0;", "probs[i] = gap > 0.0 ? gap : -gap;", None, HOST_PINS),
    ("shard probabilities not normalised", "probs[i] = norm > 0.0 ? probs[i] / norm : sizes[i] / total_size;", "probs[i] = norm > 0.0 ? probs[i] : sizes[i] / total_size;", None, HOST_PINS),
    ("Poly exponent", "std::pow(1.0 + (double)staleness, -0.5)", "std::pow(1.0 + (double)staleness, -1.0)", None, VAR_PINS + HOST_PINS),
    ("delay compensation drift sign", "const float drift = theta[i] - start;", "const float drift = start - theta[i];", None, VAR_PINS),
    ("delay compensation with g, not g*g", "(dc_lambda * (g * g))", "(dc_lambda * g)", None, VAR_PINS),
    ("buffered step with beta, not beta^2", "((beta * beta) * m[i])", "(beta * m[i])", None, VAR_PINS),
    ("buffered theta moves between boundaries", "} else {\n                Delta[i] = d;\n            }\n            continue;", "} else {\n                theta[i] = theta[i] - (eps * gn);\n                Delta[i] = d;\n            }\n            continue;", None, VAR_PINS),
    ("weight ignored", "if (weight != 1.0f) g = weight * g;", "", None, VAR_PINS),
    ("current mode ignored in the norm", "const float start = pg_current ? theta[i] : base[i];\n        const float g", "const float start = base[i];\n        const float g", None, DN_PINS),
    ("norm of the sum, not sum of squares", "acc += (double)g * (double)g;", "acc += (double)g;", None, DN_PINS),
    ("non-finite test misses infinities", "if (!std::isfinite(g)) bad = 1;", "if (std::isnan(g)) bad = 1;", None, DN_PINS),
    ("SGD momentum step with beta^2", "u = (beta * m[i]) + mean;", "u = ((beta * beta) * m[i]) + mean;", None, VAR_PINS),
    ("SGD momentum step with gradient weight 1 + beta", "u = (beta * m[i]) + mean;", "u = (beta * m[i]) + ((1.0f + beta) * mean);", None, VAR_PINS),
    ("SGD momentum mode falls through to Nesterov", "if (buffered == 2) {", "if (buffered == 3) {", None, VAR_PINS),
    ("weight applied before delay compensation",
     "            g = g + ((dc_lambda * (g * g)) * drift);\n        }\n        if (weight != 1.0f) g = weight * g;",
     "            const float gw = weight * g;\n            g = gw + ((dc_lambda * (gw * gw)) * drift);\n        } else if (weight != 1.0f) g = weight * g;",
     None, VAR_PINS),
]


def build_mutant(text, workdir, tag):
    src = os.path.join(workdir, f"m{tag}.cpp")
    lib = os.path.join(workdir, f"m{tag}.so")
    with open(src, "w") as f:
        f.write(text)
    subprocess.check_call(["g++", "-O1", "-std=c++17", "-ffp-contract=off", "-fPIC", "-shared", "-o", lib, src])
    return lib


@pytest.fixture(scope="module")
def workdir():
    with tempfile.TemporaryDirectory() as d:
        yield d


def test_pins_pass_on_the_unmodified_oracle():
    for pin in DN_PINS + ADAM_PINS + BF16_PINS + HOST_PINS + VAR_PINS:
        pin()


@pytest.mark.parametrize("idx", range(len(MUTANTS)), ids=[m[0] for m in MUTANTS])
def test_every_planted_mistake_is_caught(idx, workdir, monkeypatch):
    name, find, repl, which, pins = MUTANTS[idx]
    text = open(SRC).read()
    assert find in text, f"mutation site for '{name}' not found: the oracle source changed"
    if which is None:
        mutated = text.replace(find, repl)
    else:
        pos = -1
        for _ in range(which + 1):
            pos = text.index(find, pos + 1)
        mutated = text[:pos] + repl + text[pos + len(find):]
    assert mutated != text
    lib = oracle._configure(C.CDLL(build_mutant(mutated, workdir, idx)))
    monkeypatch.setattr(oracle, "_lib", lib)
    caught = []
    for pin in pins:
        try:
            pin()
        except AssertionError:
            caught.append(pin)
            break
    assert caught, f"no pin notices: {name}"
