"""Do the pins bite?  Each case plants one plausible mistake in a copy of the oracle's C source (a dropped
scale, a wrong head mapping, a rotated slot, a transposed operand, ...), builds it, and runs the pin suite
against it in a child process: the suite has to fail.  The mistakes live only in temporary copies."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "rollart_oracle.c")

MUTANTS = {
    "dropped_scale": ("double sj = scale * dot;", "double sj = dot;"),
    "wrong_head_mapping": ("int32_t h = hq / g;", "int32_t h = hq % Hkv;"),
    "no_max_subtraction": ("double wj = exp(s[j - j0] - m);", "double wj = exp(s[j - j0]);"),
    "rotated_slot_in_k": ("const uint16_t *kp = k_pool + (((int64_t)pg * Hkv + h) * P + j % P) * D;",
                          "const uint16_t *kp = k_pool + (((int64_t)pg * Hkv + h) * P + (j + 1) % P) * D;"),
    "v_read_from_k_pool": ("const uint16_t *vp = v_pool + (((int64_t)pg", "const uint16_t *vp = k_pool + (((int64_t)pg"),
    "last_key_dropped": ("for (int32_t j = j0; j < c; ++j) {\n                int32_t pg = page_table[(int64_t)t * max_pages + j / P];\n                const uint16_t *vp",
                         "for (int32_t j = j0; j < c - 1; ++j) {\n                int32_t pg = page_table[(int64_t)t * max_pages + j / P];\n                const uint16_t *vp"),
    "not_normalised": ("o[d] = acc[d] / Z;", "o[d] = acc[d];"),
    "wrong_sign_in_lse": ("lse[r * Hq + hq] = m + log(Z);", "lse[r * Hq + hq] = m - log(Z);"),
    "append_off_by_one": ("int64_t pos = (int64_t)len + r;", "int64_t pos = (int64_t)len + r + 1;"),
    "append_v_gets_k": ("memcpy(v_pool + dst, v_new + src,", "memcpy(v_pool + dst, k_new + src,"),
    "gather_rotated_slot": ("int64_t src = (((int64_t)pg * Hkv + h) * P + r % P) * D;",
                            "int64_t src = (((int64_t)pg * Hkv + h) * P + (r + 1) % P) * D;"),
    "combine_inverted_weight": ("double a = exp(parts_lse[s] - M);", "double a = exp(M - parts_lse[s]);"),
    "reserve_rounds_down": ("int64_t want = ((int64_t)seq_lens[t] + new_tokens[i] + P - 1) / P;\n        for (int64_t lp = have;",
                            "int64_t want = ((int64_t)seq_lens[t] + new_tokens[i]) / P;\n        for (int64_t lp = have;"),
    "release_keeps_length": ("        seq_lens[t] = 0;\n", "        seq_lens[t] = seq_lens[t];\n"),
    "evict_includes_the_boundary_version": ("(int64_t)start_version[t] < (int64_t)current_version - (int64_t)alpha)",
                                             "(int64_t)start_version[t] <= (int64_t)current_version - (int64_t)alpha)"),
    "evict_takes_empty_rows": ("if (seq_lens[t] > 0 && (int64_t)start_version[t]", "if (seq_lens[t] >= 0 && (int64_t)start_version[t]"),
    "e4m3_wrong_bias": ("else v = ldexp(1.0 + (double)m / 8.0, e - 7);", "else v = ldexp(1.0 + (double)m / 8.0, e - 8);"),
    "e4m3_subnormals_as_normals": ("else if (e == 0) v = ldexp((double)m / 8.0, -6);",
                                   "else if (e == 0) v = ldexp(1.0 + (double)m / 8.0, -7);"),
    "e4m3_truncates": ("int m = (int)nearbyint((2.0 * fr - 1.0) * 8.0);", "int m = (int)floor((2.0 * fr - 1.0) * 8.0);"),
    "e4m3_ties_away": ("int m = (int)nearbyint((2.0 * fr - 1.0) * 8.0);", "int m = (int)round((2.0 * fr - 1.0) * 8.0);"),
    "e4m3_subnormal_step": ("mag = (uint8_t)nearbyint(ldexp(a, 9));", "mag = (uint8_t)nearbyint(ldexp(a, 8));"),
}


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_pins_catch_planted_mistake(name, tmp_path):
    old, new = MUTANTS[name]
    text = open(SRC).read()
    assert text.count(old) == 1, f"mutation site for {name} not found exactly once"
    c_file, so_file = tmp_path / "mutant.c", tmp_path / "mutant.so"
    c_file.write_text(text.replace(old, new))
    subprocess.run(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", str(so_file), str(c_file), "-lm"], check=True)
    env = dict(os.environ, ROLLART_ORACLE_LIB=str(so_file))
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                        os.path.join(ROOT, "tests", "test_oracle_pins.py"), os.path.join(ROOT, "tests", "test_oracle_pages.py"),
                        os.path.join(ROOT, "tests", "test_oracle_fp8.py")],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode != 0, f"the pins did not notice the planted mistake '{name}'"
    assert "failed" in r.stdout or "error" in r.stdout.lower(), r.stdout[-400:]
