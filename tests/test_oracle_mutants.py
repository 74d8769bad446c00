"""Do the pins have teeth?  Each case plants one plausible mistake in a copy of the CPU oracle
(a dropped term, a wrong sign or index, a transposed operand), builds it, and checks that at least
one pin of tests/test_oracle_pins.py fails against the mutant.  CPU only; the mistakes live in
copies of the oracle, never in the product."""
import ctypes
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "sp_oracle.c")

# (name, text to find, replacement, pins expected to notice)
MUTANTS = [
    ("harmonic_mean_as_arithmetic", "S = n_nonempty ? (double)n_nonempty / inv : 0.0;",
     "{ double sum = 0.0; for (int i = 0; i < N; ++i) sum += L[i]; S = n_nonempty ? sum / n_nonempty : 0.0; }",
     "positions"),
    ("doc_step_inverted", "double step = (scheme == 0) ? (L[i] > 0 ? S / (double)L[i] : 0.0) : 1.0;",
     "double step = (scheme == 0) ? (L[i] > 0 ? (double)L[i] / S : 0.0) : 1.0;", "positions"),
    ("rope_sign_flipped", "v[ia] = (float)(a * c - b * s);", "v[ia] = (float)(a * c + b * s);", "rope"),
    ("rope_exponent_dropped_factor", "pow(base, -2.0 * (double)m / (double)rot_dim)",
     "pow(base, -1.0 * (double)m / (double)rot_dim)", "rope"),
    ("prefill_forgets_preamble", "for (int64_t j = 0; j < P; ++j, ++c) {\n                        const int64_t kr = (int64_t)pre_start[b] + j;\n                        kp[c] = k + (kr * Hkv + hk) * D; vp[c] = v + (kr * Hkv + hk) * D;\n                    }\n                    for (int64_t j = 0; j <= ri.off; ++j, ++c) {",
     "for (int64_t j = 0; j < 0; ++j, ++c) {\n                        const int64_t kr = (int64_t)pre_start[b] + j;\n                        kp[c] = k + (kr * Hkv + hk) * D; vp[c] = v + (kr * Hkv + hk) * D;\n                    }\n                    for (int64_t j = 0; j <= ri.off; ++j, ++c) {",
     "prefill"),
    ("prefill_causal_off_by_one", "for (int64_t j = 0; j <= ri.off; ++j, ++c) {\n                        const int64_t kr = (int64_t)path_start[ri.path] + j;",
     "for (int64_t j = 0; j < ri.off + (ri.off == 0); ++j, ++c) {\n                        const int64_t kr = (int64_t)path_start[ri.path] + j;", "prefill"),
    ("attention_value_from_key", "acc_o[d] += p * (double)vv[d];", "acc_o[d] += p * (double)kptr[j][d];", "prefill or decode"),
    ("softmax_without_max_in_lse", "const double l = m + log(denom);", "const double l = log(denom);", "prefill or decode"),
    ("gqa_head_map_transposed", "const int hk = h / group;\n                int64_t c = 0;", "const int hk = h % Hkv;\n                int64_t c = 0;", "prefill"),
    ("score_drops_weight", "scores[i] = (float)(w * sum + pr);", "scores[i] = (float)(sum + pr);", "path_scores"),
    ("score_logsumexp_sign", "const double lp = (double)row[y] - (m + log(denom));", "const double lp = (double)row[y] - (m - log(denom));", "path_scores"),
    ("score_counts_ignored_rows", "if (y == -1) { if (row_logp) row_logp[t] = 0.0f; continue; }", "if (y == -1) { if (row_logp) row_logp[t] = 0.0f; sum += -1.0; continue; }", "path_scores"),
    ("topk_keeps_smallest", "if (s[a] != s[b]) return s[a] > s[b];", "if (s[a] != s[b]) return s[a] < s[b];", "topk"),
    ("topk_ties_to_higher_index", "if (s[a] != s[b]) return s[a] > s[b];\n    return a < b;", "if (s[a] != s[b]) return s[a] > s[b];\n    return a > b;", "topk"),
    ("alibi_sign_flipped", "bias[cc] = -(double)slopes[h] * fabs((double)pos[r] - (double)pos[kr]);",
     "bias[cc] = (double)slopes[h] * fabs((double)pos[r] - (double)pos[kr]);", "alibi"),
    ("alibi_position_of_wrong_key", "bias[cc] = -(double)slopes[h] * fabs((double)pos[r] - (double)pos[kr]);",
     "bias[cc] = -(double)slopes[h] * fabs((double)pos[r] - (double)pos[cc]);", "alibi"),
    ("alibi_signed_distance", "bias[cc] = -(double)slopes[h] * fabs((double)pos[r] - (double)pos[kr]);",
     "bias[cc] = -(double)slopes[h] * ((double)pos[kr] - (double)pos[r]);", "alibi"),
    ("alibi_decode_tail_position_from_cache", "const double pk = cc < n_cache ? (double)cache_pos[kr] : (double)tail_pos[kr];",
     "const double pk = (double)cache_pos[kr];", "alibi"),
    ("decode_forgets_tail", "for (int j = 0; j < tl; ++j, ++c) {", "for (int j = 0; j < 0; ++j, ++c) {", "decode"),
    ("decode_keeps_only_first_path", "for (int jj = 0; jj < k; ++jj) {\n                const int i = kept_idx[b * k + jj];\n                if (i < ppo[b] || i >= ppo[b + 1]) continue;",
     "for (int jj = 0; jj < (k > 1 ? 1 : k); ++jj) {\n                const int i = kept_idx[b * k + jj];\n                if (i < ppo[b] || i >= ppo[b + 1]) continue;", "decode"),
]


@pytest.mark.parametrize("name,old,new,which", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_pins_catch_planted_mistake(tmp_path, name, old, new, which):
    text = open(SRC).read()
    assert text.count(old) >= 1, f"mutation anchor for {name} not found in the oracle"
    mutated = text.replace(old, new, 1)
    csrc = tmp_path / "sp_oracle_mutant.c"
    csrc.write_text(mutated)
    lib = tmp_path / "libsp_oracle_mutant.so"
    subprocess.check_call(["gcc", "-O1", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", str(lib), str(csrc), "-lm"])
    # run the relevant pins in a child process whose oracle package loads the mutant library
    code = (
        "import sys, ctypes; sys.path.insert(0, %r); sys.path.insert(0, %r)\n"
        "import oracle\n"
        "oracle._lib = ctypes.CDLL(%r); oracle._lib.spo_num_threads.restype = ctypes.c_int\n"
        "import pytest\n"
        "sys.exit(pytest.main(['-q', '-x', '-p', 'no:cacheprovider', %r, '-k', %r]))\n"
        % (ROOT, os.path.join(ROOT, "tests"), str(lib), os.path.join(ROOT, "tests", "test_oracle_pins.py"), which)
    )
    r = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=600)
    assert r.returncode != 0, f"no pin noticed the planted mistake '{name}':\n{r.stdout[-800:]}"
    assert "failed" in r.stdout or "error" in r.stdout.lower()
