"""The pins must have teeth: plant one plausible mistake at a time in a COPY of the oracle
source, rebuild it, and require that the pin suite fails.  CPU only; the mistakes live in
the oracle copy, never in the CUDA path."""
import os
import subprocess
import sys
import tempfile

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "local_adaalter_oracle.cpp")

MUTATIONS = {
    # name: (old, new)
    "fresh_accumulator_in_denominator": ("      float d = Bs[j] + q;\n      float r = et / std::sqrt(d);\n      double dd", "      float d = B2[(size_t)0 * n + j] + q;\n      float r = et / std::sqrt(d);\n      double dd"),
    "shadow_fresh_accumulator": ("double dd = Bsd[j] + (double)tp * eps2d;", "double dd = B2d[j] + (double)tp * eps2d;"),
    "placeholder_without_t_prime": ("float q = (float)tp * eps2;", "float q = eps2;"),
    "shadow_placeholder_without_t_prime": ("Bsd[j] + (double)tp * eps2d", "Bsd[j] + eps2d"),
    "ascent_instead_of_descent": ("X[ix] = std::fmaf(-r, g, X[ix]);", "X[ix] = std::fmaf(r, g, X[ix]);"),
    "accumulate_g_not_g_squared": ("B2[ix] = std::fmaf(g, g, B2[ix]);", "B2[ix] = B2[ix] + g;"),
    "shadow_accumulate_abs": ("B2d[ix] = B2d[ix] + gd * gd;", "B2d[ix] = B2d[ix] + std::fabs(gd);"),
    "no_sqrt_in_update": ("      float r = et / std::sqrt(d);\n      double dd", "      float r = et / d;\n      double dd"),
    "stale_not_refreshed_at_sync": ("      Bs[j] = bm;\n", "\n"),
    "t_prime_not_reset": ("      Bsd[j] = bmd;\n    }\n    tp = 0;\n", "      Bsd[j] = bmd;\n    }\n"),
    "sum_instead_of_mean": ("float xm = tree_sum(vx) / (float)W;\n      float bm", "float xm = tree_sum(vx);\n      float bm"),
    "b2_not_averaged": ("        B2[(size_t)i * n + j] = bm;\n", ""),
    "gradient_at_worker0_iterate": ("float dlt = X[ix] - c[j];", "float dlt = X[j] - c[j];"),
    "sync_one_step_late": ("if (rule != kRuleAdaGrad && tp == H) sync();", "if (rule != kRuleAdaGrad && tp == H + 1) sync();"),
    "cos_sin_swapped": ("return (j & 1) ? b : a;", "return (j & 1) ? a : b;"),
    "u1_can_be_zero_offset": ("uint32_t k = (uint32_t)(z >> 40) + 1u;\n  uint32_t q = (uint32_t)(z >> 8) & 0xFFFFFFu;\n  float R",
                              "uint32_t k = (uint32_t)(z >> 39 & 0xFFFFFF) + 1u;\n  uint32_t q = (uint32_t)(z >> 8) & 0xFFFFFFu;\n  float R"),
    "octant_sign_error": ("case 2: c = -sn; s = cs;  break;", "case 2: c = sn; s = cs;  break;"),
    "missing_factor_two_in_log": ("0x1.62e430p+0f /* fl32(2 ln 2) */", "0x1.62e430p-1f"),
    "bf16_truncates": ("u += 0x7FFFu + ((u >> 16) & 1u);", ""),
    "warmup_ignored": ("return eta * std::fmin(1.0f, ratio);", "return eta;"),
    "adagrad_stale_denominator": ("float d = b + eps2;", "float d = B2[j] + eps2;"),
    "adagrad_shadow_stale_denominator": ("std::sqrt(bd + eps2d)", "std::sqrt(B2d[j] + eps2d)"),
    "adagrad_no_gradient_averaging": ("float gm = tree_sum(vg) / (float)W;", "float gm = vg[0];"),
    "local_sgd_ascent": ("X[ix] = std::fmaf(-et, g, X[ix]);", "X[ix] = std::fmaf(et, g, X[ix]);"),
    "local_sgd_sum_not_mean": ("float xm = tree_sum(vx) / (float)W;\n      double xs", "float xm = tree_sum(vx);\n      double xs"),
    "worker_key_ignores_worker": ("return mix64(kt + kGamma * (uint64_t)(worker + 1));", "return mix64(kt + kGamma);"),
}


def _has_fma():
    with open("/proc/cpuinfo") as f:
        return " fma " in f.read().replace("\n", " ")


def _run_one(name):
    old, new = MUTATIONS[name]
    src = open(SRC).read()
    if src.count(old) != 1:
        return name, None, f"mutation anchor for {name} not unique/present"
    with tempfile.TemporaryDirectory() as d:
        cpp, so = os.path.join(d, "m.cpp"), os.path.join(d, "m.so")
        with open(cpp, "w") as f:
            f.write(src.replace(old, new))
        cmd = ["g++", "-std=c++17", "-O1", "-ffp-contract=off", "-shared", "-fPIC", "-o", so, cpp]
        if _has_fma():
            cmd.insert(3, "-mfma")
        subprocess.run(cmd, check=True)
        env = dict(os.environ, LA_ORACLE_SO=so)
        r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                            os.path.join(ROOT, "tests", "test_oracle_alg3.py"),
                            os.path.join(ROOT, "tests", "test_oracle_baselines.py"),
                            os.path.join(ROOT, "tests", "test_oracle_noise.py")],
                           env=env, cwd=ROOT, capture_output=True, text=True)
        return name, r.returncode, r.stdout[-2000:]


@pytest.fixture(scope="module")
def mutation_results():
    """All mutants are built and evaluated concurrently (one pytest child each)."""
    from concurrent.futures import ThreadPoolExecutor
    with ThreadPoolExecutor(max_workers=max(2, (os.cpu_count() or 2))) as ex:
        return {name: (rc, out) for name, rc, out in ex.map(_run_one, sorted(MUTATIONS))}


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_pins_catch_mutation(name, mutation_results):
    rc, out = mutation_results[name]
    assert rc is not None, out
    assert rc != 0, f"no pin noticed the planted mistake '{name}'"
    assert "failed" in out, out
