"""Would the GPU parity tests notice a wrong result?  (The errors are planted in the CPU oracle.)

A parity test proves something only if its tolerance is tight enough to separate a correct kernel from a
wrong formula.  Each case builds a copy of oracle/ref_oracle.c with ONE error -- some gross (Eq. 1's plain
mean for Eq. 2's weights), some small (a weight off by one part in 10^4, ten times the fp32 tolerance) --
and runs a GPU parity file against that copy in a child process: the CUDA library is untouched and correct,
the oracle is wrong, so the comparison must FAIL.  The same selection run against an unaltered copy passes.
"""
import os
import subprocess
import sys

import pytest

from test_oracle_mutations import CFLAGS, ROOT, SRC, _mutate

pytestmark = pytest.mark.gpu

AGG = ["tests/test_gpu_aggregate.py", "-k", "worker_counts or config_small or norm_flag or sizes_and_ragged"]
ADAM = ["tests/test_gpu_adam.py", "-k", "teacher_forced"]
GRAD = ["tests/test_gpu_worker_grad.py", "-k", "shapes_including or grouped_matches"]
HOST = ["tests/test_gpu_host_pipeline.py"]
MULTI = ["tests/test_gpu_multi_tensor.py"]

CASES = [
    # (name, text in ref_oracle.c, replacement, occurrence, parity selection that must fail)
    ("weights_plain_mean", "lambda[k] = (double)b[k] / (double)S;", "lambda[k] = 1.0 / (double)K;", 0, AGG),
    ("one_weight_off_by_1e-4", "for (int32_t k = 0; k < K; ++k) lambda[k] = (double)b[k] / (double)S;",
     "for (int32_t k = 0; k < K; ++k) lambda[k] = (double)b[k] / (double)S;\n    lambda[0] *= 1.0001;", 0, AGG),
    ("extra_one_over_K", "p[j] = p[j] - lr * v[j];", "p[j] = p[j] - lr * v[j] / (double)K;", 0, AGG),
    ("dampened_momentum", "v[j] = mu * v[j] + g;", "v[j] = mu * v[j] + (1.0 - mu) * g;", 0, AGG),
    ("momentum_off_by_1e-4", "v[j] = mu * v[j] + g;", "v[j] = 1.0001 * mu * v[j] + g;", 0, AGG),
    ("norm_misses_the_last_element", "sq += g * g;", "if (j + 1 < N) sq += g * g;", 0, AGG),
    ("weights_plain_mean_host_pipeline", "lambda[k] = (double)b[k] / (double)S;", "lambda[k] = 1.0 / (double)K;", 0, HOST),
    ("weights_plain_mean_tensor_list", "lambda[k] = (double)b[k] / (double)S;", "lambda[k] = 1.0 / (double)K;", 0, MULTI),
    ("adam_eps_inside_root", "(sqrt(uhat) + eps)", "sqrt(uhat + eps)", 0, ADAM),
    ("adam_no_bias_correction_u", "double uhat = u[j] / c2;", "double uhat = u[j];", 0, ADAM),
    ("adam_beta2_off_by_1e-4", "u[j] = beta2 * u[j] + (1.0 - beta2) * g * g;",
     "u[j] = beta2 * u[j] + (1.0 - beta2) * 1.0002 * g * g;", 0, ADAM),
    ("gradient_sum_not_mean", "G[(size_t)d * C + c] = s / (double)n;", "G[(size_t)d * C + c] = s;", 0, GRAD),
    ("no_one_hot_subtraction", "z[y[i]] -= 1.0;", "", 0, GRAD),
    ("logits_off_by_1e-3", "z[c] = s;", "z[c] = 1.001 * s;", 0, GRAD),
    ("loss_sum_not_mean", "*loss = total / (double)n;", "*loss = total;", 0, GRAD),
]


def _build(workdir, name, old, new, which):
    source = open(SRC).read()
    c = os.path.join(workdir, name + ".c")
    so = os.path.join(workdir, name + ".so")
    with open(c, "w") as f:
        f.write(source if old is None else _mutate(source, old, new, which))
    subprocess.run(["gcc", *CFLAGS, "-o", so, c, "-lm"], check=True)
    return so


def _run(selection, lib_path):
    env = dict(os.environ, REF_ORACLE_LIB=lib_path)
    r = subprocess.run([sys.executable, "-m", "pytest", *selection, "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
                        "--no-header"], cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    return r.returncode, r.stdout[-2000:]


def test_unaltered_copy_passes_every_selection(tmp_path):
    so = _build(str(tmp_path), "unaltered", None, None, None)
    for sel in (AGG, ADAM, GRAD, HOST, MULTI):
        rc, tail = _run(sel, so)
        assert rc == 0, tail


@pytest.mark.parametrize("name,old,new,which,selection", CASES, ids=[c[0] for c in CASES])
def test_a_wrong_oracle_fails_the_gpu_parity_tests(tmp_path, name, old, new, which, selection):
    so = _build(str(tmp_path), name, old, new, which)
    rc, tail = _run(selection, so)
    # 1 = tests ran and at least one failed; 0 would mean the tolerance hides the error, anything else a crash
    assert rc == 1, f"exit {rc}\n{tail}"
    assert "AssertionError" in tail or "assert" in tail
