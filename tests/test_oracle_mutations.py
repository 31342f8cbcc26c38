"""Do the oracle's pins notice a mistake?  (CPU only.)

Each case below plants ONE plausible error in a copy of oracle/ref_oracle.c -- a dropped term, a wrong sign,
a transposed operand, a missing normalisation -- builds the copy with the oracle's own compiler flags, and runs
tests/test_oracle_pins.py against it in a child process (tests/oracle_mutation_runner.py; the oracle front end
loads the library named by REF_ORACLE_LIB instead of building its own).  The pins must FAIL for every planted
error and pass for an unaltered copy.  The errors live in the CPU oracle only; nothing here touches the CUDA
library.
"""
import json
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "ref_oracle.c")
CFLAGS = ["-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared", "-fPIC"]

# (name, text in ref_oracle.c, replacement, which occurrence when the text appears more than once)
MUTATIONS = [
    # Eq. 2: the weights
    ("weights_plain_mean", "lambda[k] = (double)b[k] / (double)S;", "lambda[k] = 1.0 / (double)K;", 0),
    ("weights_not_normalised", "lambda[k] = (double)b[k] / (double)S;", "lambda[k] = (double)b[k] / (double)K;", 0),
    # Eq. 3 with momentum
    ("extra_one_over_K", "p[j] = p[j] - lr * v[j];", "p[j] = p[j] - lr * v[j] / (double)K;", 0),
    ("momentum_subtracts_gradient", "v[j] = mu * v[j] + g;", "v[j] = mu * v[j] - g;", 0),
    ("step_along_gradient_not_velocity", "p[j] = p[j] - lr * v[j];", "p[j] = p[j] - lr * g;", 0),
    ("step_ascends", "p[j] = p[j] - lr * v[j];", "p[j] = p[j] + lr * v[j];", 0),
    ("parameters_before_velocity", "v[j] = mu * v[j] + g;\n        p[j] = p[j] - lr * v[j];",
     "p[j] = p[j] - lr * v[j];\n        v[j] = mu * v[j] + g;", 0),
    ("dampened_momentum", "v[j] = mu * v[j] + g;", "v[j] = mu * v[j] + (1.0 - mu) * g;", 0),
    ("norm_not_squared", "sq += g * g;", "sq += fabs(g);", 0),
    ("zero_batch_worker_still_read", "if (b[k] == 0) continue;\n            g += lambda[k] * grad_at(grads[k], grad_dtype, j);\n        }\n        v[j]",
     "g += lambda[k] * grad_at(grads[k], grad_dtype, j);\n        }\n        v[j]", 0),
    ("bf16_read_as_low_half", "((uint32_t)h) << 16", "((uint32_t)h) << 15", 0),
    # Adam
    ("adam_second_moment_not_squared", "(1.0 - beta2) * g * g;", "(1.0 - beta2) * g;", 0),
    ("adam_no_bias_correction_m", "double mhat = m[j] / c1;", "double mhat = m[j];", 0),
    ("adam_no_bias_correction_u", "double uhat = u[j] / c2;", "double uhat = u[j];", 0),
    ("adam_eps_inside_root", "(sqrt(uhat) + eps)", "sqrt(uhat + eps)", 0),
    ("adam_step_counted_from_zero", "pow(beta1, (double)t)", "pow(beta1, (double)(t - 1) + 0.5)", 0),
    ("adam_norm_not_squared", "sq += g * g;", "sq += fabs(g);", 1),
    # linear-softmax gradient
    ("no_one_hot_subtraction", "z[y[i]] -= 1.0;", "", 0),
    ("gradient_sum_not_mean", "G[(size_t)d * C + c] = s / (double)n;", "G[(size_t)d * C + c] = s;", 0),
    ("W_transposed", "(double)W[(size_t)d * C + c]", "(double)W[(size_t)c * D + d]", 0),
    ("gradient_transposed", "G[(size_t)d * C + c] = s / (double)n;", "G[(size_t)c * D + d] = s / (double)n;", 0),
    ("softmax_without_denominator", "z[c] = exp(z[c] - zmax) / den;", "z[c] = exp(z[c] - zmax);", 0),
    ("loss_sign", "total += -((z[y[i]] - zmax) - log(den));", "total += ((z[y[i]] - zmax) - log(den));", 0),
    ("loss_sum_not_mean", "*loss = total / (double)n;", "*loss = total;", 0),
    # Eq. 4-5
    ("tbar_sum_not_mean", "double tbar = tsum / (double)K;", "double tbar = tsum;", 0),
    ("delta_sign", "double delta = -X[k] * (t - tbar);", "double delta = X[k] * (t - tbar);", 0),
    ("delta_without_throughput", "double delta = -X[k] * (t - tbar);", "double delta = -(t - tbar);", 0),
    ("gain_ignored", "q[k] = (double)b[k] + kp * delta;", "q[k] = (double)b[k] + delta;", 0),
    ("global_batch_not_restored", "q[k] = q[k] * (double)S / btsum;", "q[k] = q[k];", 0),
    # integers
    ("ties_to_the_highest_index", "if (best < 0 || gap > best_gap) { best = k; best_gap = gap; }",
     "if (best < 0 || gap >= best_gap) { best = k; best_gap = gap; }", 0),
    ("missing_units_to_smallest_remainder", "double gap = q[k] - (double)f[k];", "double gap = (double)f[k] - q[k];", 0),
    ("default_lower_bound_zero", "lo ? lo[k] : 1", "lo ? lo[k] : 0", None),
    ("upper_bound_ignored_when_filling", "if (f[k] >= h) continue;", "", 0),
    ("nearest_integer_start", "double fl = floor(q[k]);", "double fl = floor(q[k] + 0.5);", 0),
    ("lower_bound_ignored_when_trimming", "if (f[k] <= l) continue;", "", 0),
    ("surplus_from_smallest_excess", "double gap = (double)f[k] - q[k];", "double gap = q[k] - (double)f[k];", 0),
    ("start_not_clamped_to_upper_bound", "if (x > h) x = h;", "", 0),
    ("start_not_clamped_to_lower_bound", "if (x < l) x = l;", "", 0),
    # static allocation
    ("static_sums_to_b0", "q[k] = (double)S * X[k] / xsum;", "q[k] = (double)b0 * X[k] / xsum;", 0),
    # stabilised controller
    ("ewma_weights_swapped", "alpha * t[k] + (1.0 - alpha) * ewma[k]", "(1.0 - alpha) * t[k] + alpha * ewma[k]", 0),
    ("ewma_not_restarted", "*n_since = 0;\n", "\n", 0),
    ("dead_band_signed", "fabs((double)nb[k] - (double)b[k]) / (double)b[k]", "((double)nb[k] - (double)b[k]) / (double)b[k]", 0),
    ("dead_band_relative_to_new", "fabs((double)nb[k] - (double)b[k]) / (double)b[k]", "fabs((double)nb[k] - (double)b[k]) / (double)nb[k]", 0),
    ("dead_band_not_strict", "if (worst > dmin) {", "if (worst >= dmin) {", 0),
    ("dead_band_on_the_mean", "if (rel > worst) worst = rel;", "worst += rel / (double)K;", 0),
    ("learnt_bound_is_the_raised_batch", "learnt_max[k] = prev_b[k];", "learnt_max[k] = b[k];", 0),
    ("learnt_bound_on_a_gain", "X[k] < prev_X[k]", "X[k] > prev_X[k]", 0),
    ("learnt_bound_without_a_raise", "prev_X[k] > 0.0 && b[k] > prev_b[k] && X[k] < prev_X[k]", "prev_X[k] > 0.0 && X[k] < prev_X[k]", 0),
    ("learnt_bound_never_lowered", "learnt_max[k] == 0 || prev_b[k] < learnt_max[k]", "learnt_max[k] == 0", 0),
    ("no_fallback_to_user_bounds", "if (rc == REF_ERR_INFEASIBLE) {", "if (!use_learnt) {", 0),
    ("previous_state_is_the_new_batch", "prev_b[k] = b[k]; prev_X[k] = X[k];", "prev_b[k] = nb[k]; prev_X[k] = X[k];", 0),
    ("throughput_from_raw_time", "X[k] = (double)b[k] / ewma[k];", "X[k] = (double)b[k] / t[k];", 0),
]


def _mutate(text, old, new, which):
    n = text.count(old)
    assert n >= 1, f"text to alter not found in ref_oracle.c: {old!r}"
    if which is None:
        return text.replace(old, new)
    assert which < n, (old, n)
    if which == 0 and n == 1:
        return text.replace(old, new)
    pos = -1
    for _ in range(which + 1):
        pos = text.index(old, pos + 1)
    return text[:pos] + new + text[pos + len(old):]


def _build(args):
    name, old, new, which, workdir, source = args
    c = os.path.join(workdir, name + ".c")
    so = os.path.join(workdir, name + ".so")
    with open(c, "w") as f:
        f.write(source if old is None else _mutate(source, old, new, which))
    subprocess.run(["gcc", *CFLAGS, "-o", so, c, "-lm"], check=True)
    return name, so


def _run_group(pairs):
    """One child process runs the pin file against each library of the group in turn."""
    env = dict(os.environ, OMP_NUM_THREADS="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "oracle_mutation_runner.py"),
                        *[f"{n}={so}" for n, so in pairs]], cwd=ROOT, env=env, capture_output=True, text=True,
                       timeout=1200)
    rows = [json.loads(line) for line in r.stdout.splitlines() if line.startswith("{")]
    assert r.returncode == 0 and len(rows) == len(pairs), (r.returncode, r.stdout[-1500:], r.stderr[-1500:])
    return rows


def test_every_planted_mistake_fails_a_pin(tmp_path):
    source = open(SRC).read()
    jobs = [("unaltered", None, None, None, str(tmp_path), source)]
    jobs += [(n, o, w, i, str(tmp_path), source) for n, o, w, i in MUTATIONS]
    workers = min(4, os.cpu_count() or 1)
    with ThreadPoolExecutor(max_workers=workers) as pool:
        built = list(pool.map(_build, jobs))
        groups = [built[g::workers] for g in range(workers)]
        rows = [row for rows in pool.map(_run_group, groups) for row in rows]
    by_name = {row["name"]: row for row in rows}
    assert by_name["unaltered"]["rc"] == 0, "the pins do not pass on an unaltered copy of the oracle"
    # pytest exits 1 when tests ran and some failed; anything else (collection error, crash) is not a catch
    survived = [n for n, _, _, _ in MUTATIONS if by_name[n]["rc"] == 0]
    broken = [by_name[n] for n, _, _, _ in MUTATIONS if by_name[n]["rc"] not in (0, 1)]
    assert not broken, broken
    assert not survived, f"no pin notices: {survived}"
    assert all(by_name[n]["first"] for n, _, _, _ in MUTATIONS), by_name
    with open(os.path.join(str(tmp_path), "caught_by.txt"), "w") as f:
        for n, _, _, _ in MUTATIONS:
            f.write(f"{n}\t{by_name[n]['first']}\n")


def test_mutations_are_distinct_and_apply():
    source = open(SRC).read()
    names = [m[0] for m in MUTATIONS]
    assert len(set(names)) == len(names)
    for name, old, new, which in MUTATIONS:
        assert _mutate(source, old, new, which) != source, name
