"""Do the pins bite?  Plausible mistakes are planted, one at a time, in COPIES of the oracle's
C source (a dropped term, a wrong sign, index or comparison, a transposed operand, a rule of
Algorithm 1 read differently); each copy is compiled and the pin suite
(tests/test_oracle_pins.py) is run against it in a child process.  Every mutant must fail at
least one pin.  Nothing here touches the CUDA path or the oracle that the other tests use.
"""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "ead_oracle.c")

# (name, text in ead_oracle.c, what the mistaken version says instead)
MUTANTS = [
    ("logits_transposed_operand",
     "acc += bf16_to_f64(w[j]) * hd[j];", "acc += bf16_to_f64(W[j * V + i]) * hd[j];"),
    ("entropy_wrong_sign",
     "if (p > 0.0) H -= p * log(p);", "if (p > 0.0) H += p * log(p);"),
    ("softmax_not_normalised",
     "double p = exp(z[i] - m) / Z;", "double p = exp(z[i] - m);"),
    ("entropy_drops_log_Z",
     "if (p > 0.0) H -= p * log(p);", "if (p > 0.0) H -= p * (z[i] - m);"),
    ("bits_conversion_inverted",
     "if (unit == 1) H /= log(2.0);", "if (unit == 1) H *= log(2.0);"),
    ("zero_times_log_zero_not_guarded",
     "if (p > 0.0) H -= p * log(p);", "H -= p * log(p);"),
    ("arg_max_keeps_last_of_equal_maxima",
     "if (z[i] > z[best]) best = i;", "if (z[i] >= z[best]) best = i;"),
    ("window_is_the_whole_history",
     "int64_t cnt = (*n < (int64_t)w) ? *n : (int64_t)w;", "int64_t cnt = *n;"),
    ("mean_divides_by_w_during_warm_up",
     "double Hbar = sum / (double)cnt;", "double Hbar = sum / (double)w;"),
    ("switch_up_not_strict",
     "if (*model == 0 && Hbar > tau) {", "if (*model == 0 && Hbar >= tau) {"),
    ("switch_down_strict",
     "} else if (*model == 1 && Hbar <= tau) {", "} else if (*model == 1 && Hbar < tau) {"),
    ("dwell_off_by_one",
     "if (*c >= d_min) {", "if (*c > d_min) {"),
    ("counter_not_reset_at_a_switch",
     "            *model = 1;\n            *c = 0;", "            *model = 1;"),
    ("counter_reset_at_every_test",
     "    if (*c >= d_min) {\n", "    if (*c >= d_min) {\n        if (*model == 0 && Hbar <= tau) *c = 0;\n"),
    ("window_cleared_at_a_switch",
     "            *model = 0;\n            *c = 0;", "            *model = 0;\n            *c = 0;\n            *n = 0;"),
    ("temperature_multiplies",
     "double lp = z[i] / T;", "double lp = z[i] * T;"),
    ("gumbel_wrong_sign",
     "double g = -log(-log(oracle_uniform(seed, row, step, i)));",
     "double g = log(-log(oracle_uniform(seed, row, step, i)));"),
    ("uniform_ignores_the_word_index",
     "uint32_t k = out[i & 3] >> 9;", "uint32_t k = out[0] >> 9;"),
    ("philox_round_count",
     "for (int r = 0; r < 10; ++r) {", "for (int r = 0; r < 7; ++r) {"),
    ("parameter_ratio_shares_swapped",
     "double alpha = 1.0 - usage_large, beta = usage_large;",
     "double alpha = usage_large, beta = 1.0 - usage_large;"),
    ("run_reads_another_rows_hidden_state",
     "oracle_logits(W_large, Vm, H_large, h_large + (t * B + b) * H_large, z);",
     "oracle_logits(W_large, Vm, H_large, h_large + (t * B + 0) * H_large, z);"),
    ("run_entropy_of_the_idle_model",
     "int64_t Vm = model == 0 ? V : V_large;\n            if (model == 0)",
     "int64_t Vm = model == 0 ? V : V_large;\n            if (model == 0 && V != V_large)"),
    ("end_of_sequence_stops_the_row_one_token_early",
     "if (eos_token >= 0 && tk == eos_token) done = 1;",
     "if (eos_token >= 0 && tk == eos_token) { done = 1; if (tok) tok[o] = -1; }"),
    ("usage_counts_steps_after_the_sequence_ended",
     "if (tok && tok[t] < 0) continue;", "if (tok && tok[t] < -1) continue;"),
    ("switch_count_counts_the_steps_without_a_switch",
     "if (next[t] != used[t]) sw += 1;", "if (next[t] == used[t]) sw += 1;"),
]


def _run_mutant(args):
    name, old, new, workdir = args
    src = open(SRC).read()
    if src.count(old) != 1:
        return name, "stale", f"the text to replace occurs {src.count(old)} times in ead_oracle.c"
    c_path = os.path.join(workdir, name + ".c")
    so_path = os.path.join(workdir, name + ".so")
    with open(c_path, "w") as f:
        f.write(src.replace(old, new))
    cc = subprocess.run(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
                         "-o", so_path, c_path, "-lm"], capture_output=True, text=True)
    if cc.returncode != 0:
        return name, "stale", cc.stderr[-400:]
    env = dict(os.environ, EAD_ORACLE_LIB=so_path, OMP_NUM_THREADS="2")
    res = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_oracle_pins.py"),
                          "-x", "-q", "-p", "no:cacheprovider"], capture_output=True, text=True, env=env, cwd=ROOT)
    tail = (res.stdout + res.stderr)[-600:]
    if res.returncode == 1:
        return name, "caught", tail
    if res.returncode == 0:
        return name, "survived", tail
    return name, "broken", f"pytest exit code {res.returncode}: {tail}"


@pytest.fixture(scope="module")
def verdicts(tmp_path_factory):
    workdir = str(tmp_path_factory.mktemp("oracle_mutants"))
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        out = list(pool.map(_run_mutant, [(n, o, r, workdir) for n, o, r in MUTANTS]))
    return {name: (verdict, detail) for name, verdict, detail in out}


def test_the_unchanged_source_passes_through_the_same_route(tmp_path):
    """The harness itself: a copy without a mistake must pass every pin."""
    name, verdict, detail = _run_mutant(("unchanged", "/* bf16 is the upper half", "/* bf16 is the upper half",
                                        str(tmp_path)))
    assert verdict == "survived", detail


@pytest.mark.parametrize("name", [m[0] for m in MUTANTS])
def test_a_planted_mistake_fails_a_pin(verdicts, name):
    verdict, detail = verdicts[name]
    assert verdict == "caught", f"{name}: {verdict}\n{detail}"
