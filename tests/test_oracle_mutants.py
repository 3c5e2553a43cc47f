"""The pins must be able to fail: each plausible mistake planted in a copy of the oracle (a different tie rule,
a transposed operand, a wrong clamp bound, a dropped term, ...) has to be caught by tests/test_oracle_pins.py.
The mistakes are planted in the CPU oracle only; nothing here touches the GPU."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "q8_oracle.c")

MUTANTS = {
    "ties_away_from_zero": ("float r = rintf(p);              /* nearest integer, halves to even */", "float r = roundf(p);"),
    "product_in_double": ("float p = x * S;                 /* one fp32 multiply (no contraction) */\n    if (isnan(p)) return 0;\n    float r = rintf(p);",
                          "double p = (double)x * (double)S;\n    if (isnan(p)) return 0;\n    float r = (float)rint(p);"),
    "clamp_at_128": ("return ((int64_t)1 << (b - 1)) - 1;", "return ((int64_t)1 << (b - 1));"),
    "weight_transposed": ("s += (int64_t)xq[m * K + k] * (int64_t)wq[n * K + k];", "s += (int64_t)xq[m * K + k] * (int64_t)wq[k * N + n];"),
    "ema_wrong_sign": ("*ema = *ema + step;", "*ema = *ema - step;"),
    "ema_zero_init": ("    if (*n == 0 || decay == 0.0f) {\n        *ema = batch_absmax;\n    } else {", "    if (0) {\n        *ema = batch_absmax;\n    } else {"),
    "bias_ties_away": ("double r = (double)rintf(p);", "double r = (double)roundf(p);"),
    "bias_product_in_double": ("float S_out = S_x * S_w;\n    double M32", "double S_out = (double)S_x * (double)S_w;\n    double M32"),
    "bias_add_drops_overflow_count": ("            if (s > INT32_MAX || s < INT32_MIN) bad += 1;\n            acc[m * N + n] = (int32_t)(uint32_t)(uint64_t)s;",
                                      "            acc[m * N + n] = (int32_t)(uint32_t)(uint64_t)s;"),
    "bias_add_saturates": ("            acc[m * N + n] = (int32_t)(uint32_t)(uint64_t)s;",
                           "            acc[m * N + n] = s > INT32_MAX ? INT32_MAX : (s < INT32_MIN ? INT32_MIN : (int32_t)s);"),
    "ema_decay_zero_uses_update_formula": ("if (*n == 0 || decay == 0.0f) {", "if (*n == 0) {"),
    "empty_batch_counts_as_zero_maximum": ("if (numel <= 0) return *n == 0 ? 1.0f : q8o_scale_from_absmax(*ema, flag);", ""),
    "bias_without_weight_scale": ("float S_out = S_x * S_w;\n    double M32", "float S_out = S_x;\n    double M32"),
    "dequant_by_sum_of_scales": ("double denom = (double)S_x * (double)S_w;", "double denom = (double)S_x + (double)S_w;"),
    "gelu_without_half": ("y[i] = 0.5 * y[i] * (1.0 + erf(y[i] * inv_sqrt2));", "y[i] = y[i] * (1.0 + erf(y[i] * inv_sqrt2));"),
    "scale_uses_128": ("return (float)q8o_M(8) / absmax;", "return 128.0f / absmax;"),
    "layernorm_unbiased_variance": ("var /= (double)H;", "var /= (double)(H - 1);"),
    "attention_no_scale": ("double scale = 1.0 / sqrt((double)d);", "double scale = 1.0;"),
    "embedding_wrong_row": ("int8_t q = Eq[id * H + h];", "int8_t q = Eq[(id + 1 < V ? id + 1 : id) * H + h];"),
}


def _run_pins(env_extra):
    env = dict(os.environ, PYTHONPATH=ROOT, **env_extra)
    return subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                           os.path.join("tests", "test_oracle_pins.py")], cwd=ROOT, env=env, capture_output=True, text=True)


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_pins_catch_planted_mistake(name, tmp_path):
    old, new = MUTANTS[name]
    text = open(SRC).read()
    assert text.count(old) == 1, f"mutation site for {name} not found exactly once"
    src = tmp_path / "mutant.c"
    src.write_text(text.replace(old, new))
    so = tmp_path / "libmutant.so"
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
                           str(src), "-lm", "-o", str(so)])
    r = _run_pins({"Q8_ORACLE_SO": str(so)})
    assert r.returncode != 0, f"no pin noticed the planted mistake '{name}'"
    assert "failed" in r.stdout


def test_unmutated_oracle_passes_the_same_run():
    r = _run_pins({})
    assert r.returncode == 0, r.stdout[-2000:]
