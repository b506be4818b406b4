"""Do the pins hold the oracle in place?  Each case plants one plausible mistake in a private copy of the
oracle (a dropped term, a wrong sign or index, a transposed operand, an off-by-one comparison), runs the pins
that are meant to notice it against that copy, and requires them to fail.  The mistakes live only in the
temporary copies, on the CPU; the oracle in the repository is run once unchanged as the control."""
import os
import shutil
import subprocess
import sys
import tempfile
from concurrent.futures import ThreadPoolExecutor

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
C, FILTERED, SEEDS = "difr_oracle.c", "filtered.py", "seed_expansion.py"

# (name, file, text to replace, replacement, test file, -k expression)
MISTAKES = [
    ("philox multipliers swapped", C, "mul_a = 0xD2511F53u, mul_b = 0xCD9E8D57u", "mul_a = 0xCD9E8D57u, mul_b = 0xD2511F53u",
     "test_oracle_philox.py", "curand_host_generator"),
    ("philox key schedule uses one constant twice", C, "kb += weyl_b;", "kb += weyl_a;",
     "test_oracle_philox.py", "curand_host_generator"),
    ("philox mixes the wrong high halves", C, "uint32_t n0 = (uint32_t)(pb >> 32) ^ x1 ^ ka;",
     "uint32_t n0 = (uint32_t)(pa >> 32) ^ x1 ^ ka;", "test_oracle_philox.py", "curand_host_generator"),
    ("counter words in the wrong order", C, "{id >> 2, position, tag, 0u}", "{position, id >> 2, tag, 0u}",
     "test_oracle_philox.py", "ro_word_layout"),
    ("wrong output word for an id", C, "return out[id & 3u];", "return out[3u - (id & 3u)];",
     "test_oracle_philox.py", "ro_word_layout"),
    ("uniform not at the midpoint", C, "((double)(word >> 9) + 0.5) * (1.0 / 8388608.0)",
     "((double)(word >> 9) + 1.0) * (1.0 / 8388608.0)", "test_oracle_philox.py", "midpoint"),
    ("Gumbel sign", C, "return -log(-log(oracle_uniform23(word)));", "return log(-log(oracle_uniform23(word)));",
     "test_oracle_philox.py", "gumbel_matches"),
    ("dot product over a transposed W", C, "acc += hd[k] * bf16_to_double(w[k]);",
     "acc += hd[k] * bf16_to_double(W[k * V + v]);", "test_oracle_scores.py", "library_matmul"),
    ("temperature dropped from the noisy logit", C, "y[v] = logit[v] + temperature * G;", "y[v] = logit[v] + G;",
     "test_oracle_scores.py", "draws_from_the_temperature_softmax"),
    ("competitor is always the argmax", C, "int64_t c = (t == i1) ? i2 : i1; /* strongest competitor */",
     "int64_t c = i1;", "test_oracle_scores.py", "numpy_replay"),
    ("ties go to the highest id", C, "if (i1 < 0 || y[v] > y[i1]) {\n      i2 = i1;\n      i1 = v;\n    } else if (i2 < 0 || y[v] > y[i2]) {\n      i2 = v;\n    }\n  }\n  int in_range",
     "if (i1 < 0 || y[v] >= y[i1]) {\n      i2 = i1;\n      i1 = v;\n    } else if (i2 < 0 || y[v] >= y[i2]) {\n      i2 = v;\n    }\n  }\n  int in_range",
     "test_oracle_scores.py", "exact_ties"),
    ("margin with the wrong sign", C, "A = y[t] - y[c];\n    if (A == 0.0", "A = y[c] - y[t];\n    if (A == 0.0",
     "test_oracle_scores.py", "nonnegative_margin"),
    ("closed form without the square root of two", C, "return std_normal_cdf(A / (sigma * sqrt(2.0)));",
     "return std_normal_cdf(A / sigma);", "test_oracle_scores.py", "sampling_loop_of_the_algorithm"),
    ("log-sum-exp ignores the temperature", C,
     "out->lse[r] = temperature > 0.0 ? log_sum_exp_scaled(logit, V, 1.0 / temperature) : NAN;",
     "out->lse[r] = temperature > 0.0 ? log_sum_exp_scaled(logit, V, 1.0) : NAN;",
     "test_oracle_scores.py", "numpy_replay or library_matmul"),
    ("IPT interval starts after the claimed id", C, "for (int64_t v = 0; v < t; ++v) a += p[v];",
     "for (int64_t v = 0; v <= t; ++v) a += p[v];", "test_oracle_scores.py", "brute_force_cdf"),
    ("IPT interval centred on minus mu", C, "normal_interval_mass((a - mu) / sigma, (b - mu) / sigma)",
     "normal_interval_mass((a + mu) / sigma, (b + mu) / sigma)", "test_oracle_scores.py", "brute_force_cdf"),
    ("interval mass: wrong sign in the straddling case", C,
     "return 1.0 - 0.5 * erfc(zb / r2) - 0.5 * erfc(-za / r2);",
     "return 1.0 - 0.5 * erfc(zb / r2) + 0.5 * erfc(-za / r2);", "test_oracle_scores.py", "telescope or cancellation"),
    ("IPT softmax without the temperature", C, "p[v] = exp(logit[v] * inv_temp - lse);", "p[v] = exp(logit[v] - lse);",
     "test_oracle_scores.py", "brute_force_cdf or follow_the_softmax"),
    ("raw-logit rank counts the claim itself", C, "rank += (logit[v] > logit[t]);", "rank += (logit[v] >= logit[t]);",
     "test_oracle_scores.py", "numpy_replay"),
    ("suspicious class one id too large", C, "ranks[r] >= rank_cutoff", "ranks[r] > rank_cutoff",
     "test_oracle_risk.py", "three_classes or rank_cutoff_counts"),
    ("suspicious bits in nats", C, "b = log2((double)rank_cutoff);", "b = log((double)rank_cutoff);",
     "test_oracle_risk.py", "exfiltratable"),
    ("admissible set: the sample is its own competitor", C, "int64_t c = (i == i1) ? i2 : i1;", "int64_t c = i1;",
     "test_oracle_risk.py", "rescoring_every_id"),
    ("B_i with the wrong sign", FILTERED, "    B = cutoff - logits[S]\n\n    def integrand", "    B = cutoff + logits[S]\n\n    def integrand",
     "test_oracle_filtered.py", "simulated_event or monte_carlo_loop"),
    ("nucleus measured before the top-k is applied", FILTERED, "z = logits[kept] / temperature\n            p = np.exp(z - z.max())\n            c = np.cumsum(p) / p.sum()",
     "z = logits[kept] / temperature\n            p = np.exp(z - z.max())\n            c = np.cumsum(p) / np.exp(logits / temperature - z.max()).sum()",
     "test_oracle_filtered.py", "hand_worked"),
    ("context hash forgets the place of a token", SEEDS, "[place & 0xFFFFFFFF, token & 0xFFFFFFFF, 0, 1]",
     "[0, token & 0xFFFFFFFF, 0, 1]", "test_oracle_seed_expansion.py", "place_of_a_token"),
    ("context includes the row's own token", SEEDS,
     "            out[r] = c\n            c = (c + element_word(r - seq_offsets[q], tokens[r])) & MASK64",
     "            c = (c + element_word(r - seq_offsets[q], tokens[r])) & MASK64\n            out[r] = c",
     "test_oracle_seed_expansion.py", "changed_token or equal_histories"),
]


def _mirror(tmp, file=None, old=None, new=None):
    """A private tree: oracle/ (source only, optionally with one replacement), tests/ and workloads/."""
    shutil.copytree(os.path.join(ROOT, "oracle"), os.path.join(tmp, "oracle"),
                    ignore=shutil.ignore_patterns("*.so", "__pycache__"))
    shutil.copytree(os.path.join(ROOT, "workloads"), os.path.join(tmp, "workloads"),
                    ignore=shutil.ignore_patterns("__pycache__"))
    os.makedirs(os.path.join(tmp, "tests"))
    for name in os.listdir(os.path.join(ROOT, "tests")):
        if name == "conftest.py" or name.startswith("test_oracle_"):
            shutil.copy(os.path.join(ROOT, "tests", name), os.path.join(tmp, "tests", name))
    shutil.copytree(os.path.join(ROOT, "tests", "golden"), os.path.join(tmp, "tests", "golden"),
                    ignore=shutil.ignore_patterns("full_*.npz"))  # stored full-size values: GPU tests only
    if file is not None:
        path = os.path.join(tmp, "oracle", file)
        text = open(path).read()
        assert text.count(old) >= 1, f"mutation site not found in {file}: {old!r}"
        open(path, "w").write(text.replace(old, new, 1))
        # the changed file must still build: a pin that "fails" on a syntax error has noticed nothing
        if file.endswith(".c"):
            subprocess.check_call(["gcc", "-fsyntax-only", "-fopenmp", path])
        else:
            subprocess.check_call([sys.executable, "-m", "py_compile", path])


def _run_pins(tmp, test_file, expr):
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider", os.path.join("tests", test_file)]
    if expr:
        cmd += ["-k", expr]
    env = dict(os.environ, OMP_NUM_THREADS="2", PYTHONDONTWRITEBYTECODE="1")
    env.pop("PYTHONPATH", None)
    r = subprocess.run(cmd, cwd=tmp, env=env, capture_output=True, text=True, timeout=600)
    return r.returncode, r.stdout[-2000:] + r.stderr[-2000:]


def _one(case):
    name, file, old, new, test_file, expr = case
    with tempfile.TemporaryDirectory() as tmp:
        _mirror(tmp, file, old, new)
        rc, log = _run_pins(tmp, test_file, expr)
    return name, rc, log


def test_the_unchanged_oracle_passes_in_the_private_tree():
    """Control: the harness itself (copy, compile, run) does not make pins fail."""
    with tempfile.TemporaryDirectory() as tmp:
        _mirror(tmp)
        rc, log = _run_pins(tmp, "test_oracle_philox.py", "known_answer or ro_word_layout or midpoint")
        assert rc == 0, log
        rc, log = _run_pins(tmp, "test_oracle_seed_expansion.py", "place_of_a_token")
        assert rc == 0, log


def test_every_planted_mistake_is_caught():
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        results = list(pool.map(_one, MISTAKES))
    # pytest exit code 1 = tests ran and some failed; anything else (0: not noticed, 2..5: the run itself broke)
    # is a failure of this test
    missed = [(name, rc, log) for name, rc, log in results if rc != 1]
    assert not missed, "\n\n".join(f"--- {name}: pytest exit code {rc}\n{log}" for name, rc, log in missed)
