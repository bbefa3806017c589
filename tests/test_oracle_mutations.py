"""Do the pins bite?  Plant one plausible mistake at a time in a COPY of the oracle (a dropped term, a
wrong sign or index, a swapped operand), rebuild it on the CPU, and check that the pin suite fails.

Each case names the pin file that has to notice.  Nothing here touches the GPU path or the real oracle.
"""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "tq_oracle.c")

MUTATIONS = [
    # (name, text in tq_oracle.c, replacement, pin file that must fail)
    ("philox multiplier", "(uint64_t)0xD2511F53u * (uint64_t)c0", "(uint64_t)0xD2511F55u * (uint64_t)c0", "test_oracle_philox.py"),
    ("philox key schedule", "k1 += 0xBB67AE85u;", "k1 += 0xBB67AE86u;", "test_oracle_philox.py"),
    ("slot halves swapped", "(slot & 1u) ? (word >> 16) : (word & 0xFFFFu)", "(slot & 1u) ? (word & 0xFFFFu) : (word >> 16)", "test_oracle_philox.py"),
    ("truncation sign", "fminf(fmaxf(g, -alpha), alpha)", "fminf(fmaxf(g, alpha), alpha)", "test_oracle_quantizer.py"),
    ("probability sign", "p = x - (float)k;", "p = (float)k + 1.0f - x;", "test_oracle_quantizer.py"),
    ("interval boundary", "if (q->levels[j] <= t) k = j;", "if (q->levels[j] < t) k = j;", "test_oracle_quantizer.py"),
    ("threshold scale", "float scaled = p * 65536.0f;", "float scaled = p * 32768.0f;", "test_oracle_quantizer.py"),
    ("threshold comparison", "(r16 < up_threshold(p))", "(r16 <= up_threshold(p))", "test_oracle_quantizer.py"),
    ("bit order", "packed[bit >> 5] |= (uint32_t)1u << (bit & 31u);", "packed[bit >> 5] |= (uint32_t)1u << (31u - (bit & 31u));", "test_oracle_pack_aggregate.py"),
    ("mean divisor", "acc / (float)n_workers", "acc / (float)(n_workers + 1)", "test_oracle_pack_aggregate.py"),
    ("worker order", "for (uint32_t i = 0; i < n_workers; ++i) {\n            const uint32_t *pw", "for (uint32_t i = n_workers; i-- > 0;) {\n            const uint32_t *pw", "test_oracle_pack_aggregate.py"),
    ("sum of squares", "sum_sq += (double)a * (double)a;", "sum_sq += (double)a;", "test_oracle_params.py"),
    ("tail comparison", "if (a > g_min) {", "if (a >= g_min * 0.5f) {", "test_oracle_params.py"),
    ("log of ratio", "log((double)a / (double)g_min)", "log((double)a)", "test_oracle_params.py"),
    ("two-sided rho", "(double)st->n_tail / (2.0 * (double)st->d)", "(double)st->n_tail / ((double)st->d)", "test_oracle_params.py"),
    ("alpha exponent", "pow(2.0 * m->rho * s * s / (m->gamma - 2.0), 1.0 / (m->gamma - 1.0))", "pow(2.0 * m->rho * s * s / (m->gamma - 2.0), 1.0 / m->gamma)", "test_oracle_params.py"),
    ("fixed-point exponent", "((m->gamma - 2.0) * Q), 1.0 / (m->gamma - 1.0))", "((m->gamma - 2.0) * Q), 1.0 / (m->gamma - 2.0))", "test_oracle_params.py"),
    ("bias denominator", "/ ((m->gamma - 2.0) * (m->gamma - 3.0));", "/ ((m->gamma - 1.0) * (m->gamma - 2.0));", "test_oracle_params.py"),
    ("level placement", "(2.0 * (double)k / (double)s - 1.0) * Ha", "((double)k / (double)s) * Ha", "test_oracle_params.py"),
    ("biscaled exponent", "cbrt(outer) * pow(1.0 - k, 2.0 / 3.0)", "cbrt(outer) * pow(1.0 - k, 1.0 / 3.0)", "test_oracle_biscaled.py"),
    ("biscaled density split", "double denom = 2.0 * c2 * (1.0 - k) * alpha + 2.0 * c1 * k * alpha;", "double denom = 2.0 * c2 * k * alpha + 2.0 * c1 * (1.0 - k) * alpha;", "test_oracle_biscaled.py"),
    ("biscaled level offset", "double c = (double)k - 0.5 * (double)s;", "double c = (double)k - 0.5 * (double)(s + 1);", "test_oracle_biscaled.py"),
    ("biscaled inner mass", "double p1 = orc_model_QU(m, beta) / (2.0 * beta);", "double p1 = orc_model_QU(m, beta) / beta;", "test_oracle_biscaled.py"),
    ("update sign", "theta[j] = theta[j] - step;", "theta[j] = theta[j] + step;", "test_oracle_pack_aggregate.py"),
    ("momentum order", "float m = carried + g;", "float m = carried + lr * g;", "test_oracle_pack_aggregate.py"),
    ("power of two rounded up", "return ldexpf(0.5f, e);", "return ldexpf(1.0f, e);", "test_oracle_params.py"),
    ("power-of-two floor keeps subnormals", "if (!(x >= FLT_MIN)) return 0.0f;", "if (!(x > 0.0f)) return 0.0f;", "test_oracle_params.py"),
    ("bf16 widening shift", "uint32_t bits = (uint32_t)in[i] << 16;", "uint32_t bits = (uint32_t)in[i] << 15;", "test_oracle_load_window.py"),
    ("window index off by one", "orc_code_at(q, g[i], seed, worker, j0 + i);", "orc_code_at(q, g[i], seed, worker, j0 + i + 1);", "test_oracle_load_window.py"),
    ("cube root dropped", "double cb = cbrt((1.0 - 2.0 * m->rho) / (2.0 * m->g_min));\n    if (x <= m->g_min) return cb * x;", "double cb = (1.0 - 2.0 * m->rho) / (2.0 * m->g_min);\n    if (x <= m->g_min) return cb * x;", "test_oracle_params.py"),
]


@pytest.mark.parametrize("name,old,new,pin", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(tmp_path, name, old, new, pin):
    text = open(SRC).read()
    assert text.count(old) == 1, f"mutation site for '{name}' not found exactly once"
    src = tmp_path / "tq_oracle_mutant.c"
    lib = tmp_path / "libtq_oracle_mutant.so"
    src.write_text(text.replace(old, new))
    subprocess.run(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
                    "-o", str(lib), str(src), "-lm"], check=True, capture_output=True)
    env = dict(os.environ, TQ_ORACLE_LIB=str(lib))
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", pin), "-x", "-q", "-p", "no:cacheprovider"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode != 0, f"the pins in {pin} did not notice: {name}"
    assert "failed" in r.stdout or "error" in r.stdout.lower()


def test_unmutated_copy_passes(tmp_path):
    """Control: the same machinery on an unchanged copy is green (so a failure above is the mistake's)."""
    lib = tmp_path / "libtq_oracle_copy.so"
    subprocess.run(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
                    "-o", str(lib), SRC, "-lm"], check=True, capture_output=True)
    env = dict(os.environ, TQ_ORACLE_LIB=str(lib))
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_oracle_pack_aggregate.py"), "-x", "-q",
                        "-p", "no:cacheprovider"], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-500:]
