"""Plants single mistakes in a copy of the CPU checker and verifies that the pin
suites (tests/test_oracle_pins.py, tests/test_oracle_minmax_pins.py, tests/test_oracle_l2_pins.py,
tests/test_oracle_onebit_pins.py) reject every one of them.  Everything here runs
on the CPU; the planted copies are compiled into a temporary directory."""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "mqg_oracle.c")

# (name, text in the source, replacement)
MUTANTS = [
    ("dropped_half_L", "float t = fmaf(x[i], inv, halfL);", "float t = fmaf(x[i], inv, 0.0f);"),
    ("unfused_encode", "float t = fmaf(x[i], inv, halfL);", "float t = x[i] * inv + halfL;"),
    ("wrong_sign_x", "float t = fmaf(x[i], inv, halfL);", "float t = fmaf(-x[i], inv, halfL);"),
    ("scale_not_doubled", "float two_s = 2.0f * s;", "float two_s = s;"),
    ("uncentred_draw", "((float)h[i] + 0.5f) * (1.0f / 65536.0f)", "((float)h[i]) * (1.0f / 65536.0f)"),
    ("round_down_always", "(u < r) ? 1 : 0", "0"),
    ("inverted_compare", "(u < r) ? 1 : 0", "(u > r) ? 1 : 0"),
    ("pack_msb_first", "if ((q[i] >> j) & 1u) {", "if ((q[i] >> (bits - 1 - j)) & 1u) {"),
    ("pack_word_bit_reversed", "words[pos >> 5] |= (uint32_t)1u << (pos & 31u);",
     "words[pos >> 5] |= (uint32_t)0x80000000u >> (pos & 31u);"),
    ("levels_2_pow_k", "const int L = (1 << bits) - 1;", "const int L = (1 << bits);"),
    ("dequant_missing_factor_2", "(float)(2 * (int)q[i] - L)", "(float)((int)q[i] - L)"),
    ("dequant_double_rounding", "xhat[i] = level * hstep;", "xhat[i] = (level * s) / Lf;"),
    ("apply_unfused", "params[i] = fmaf(-lr, acc[i], params[i]);", "params[i] = params[i] - lr * acc[i];"),
    ("apply_wrong_sign", "params[i] = fmaf(-lr, acc[i], params[i]);", "params[i] = fmaf(lr, acc[i], params[i]);"),
    ("philox_constants_swapped", "(uint64_t)0xD2511F53u * (uint64_t)c0", "(uint64_t)0xCD9E8D57u * (uint64_t)c0"),
    ("philox_nine_rounds", "round < 10", "round < 9"),
    ("philox_key_not_bumped", "k1 += 0xBB67AE85u;", ""),
    ("draw_wrong_half", "(16u * (e & 1u))", "(16u * ((e & 1u) ^ 1u))"),
    ("draw_worker_step_swapped", "(uint32_t)(blk >> 32), worker, step }", "(uint32_t)(blk >> 32), step, worker }"),
    ("scale_signed_max", "float a = fabsf(x[i]);", "float a = x[i];"),
    ("flush_threshold", "ldexpf(1.0f, -96)", "ldexpf(1.0f, -90)"),
    ("bf16_low_half", "(uint32_t)in[i] << 16", "(uint32_t)in[i]"),
    ("sum_skips_last_worker", "for (int w = 0; w < W; ++w) {\n        mqo_unpack", "for (int w = 0; w < W - (W > 2); ++w) {\n        mqo_unpack"),
    ("requantize_skips_mean", "g[i] = g[i] * mean_scale;", "g[i] = g[i];"),
    ("zero_bucket_minus_zero", "if (s == 0.0f) { xhat[i] = 0.0f; continue; }", "if (s == 0.0f) { xhat[i] = -0.0f; continue; }"),
]


# mistakes planted in the (min, max) nearest-rounding variant, caught by tests/test_oracle_minmax_pins.py
MUTANTS_MINMAX = [
    ("mm_dropped_half", "float t = fmaf(d, inv, 0.5f);", "float t = fmaf(d, inv, 0.0f);"),
    ("mm_unfused", "float t = fmaf(d, inv, 0.5f);", "float t = d * inv + 0.5f;"),
    ("mm_levels_2_pow_k", "        float inv = Lf / r;                               /* one rounding */",
     "        float inv = (Lf + 1.0f) / r;"),
    ("mm_offset_from_hi", "float d = x[i] - lo;", "float d = hi - x[i];"),
    ("mm_no_clamp", "if (code > L) code = L;", ""),
    ("mm_range_uses_abs", "if (x[i] < lo) lo = x[i];", "if (fabsf(x[i]) < lo) lo = x[i];"),
    ("mm_keeps_minus_zero", "ranges[2 * k] = lo + 0.0f;", "ranges[2 * k] = lo;"),
    ("mm_hi_lo_swapped", "ranges[2 * k + 1] = hi + 0.0f;\n", "ranges[2 * k + 1] = ranges[2 * k]; ranges[2 * k] = hi + 0.0f;\n"),
    ("mm_decode_unfused", "xhat[i] = fmaf((float)q[i], step, lo);", "xhat[i] = (float)q[i] * step + lo;"),
    ("mm_decode_from_hi", "xhat[i] = fmaf((float)q[i], step, lo);", "xhat[i] = fmaf(-(float)q[i], step, hi);"),
    ("mm_decode_step_per_2_pow_k", "float step = r / Lf;", "float step = r / (Lf + 1.0f);"),
    ("mm_constant_decodes_to_zero", "if (r < tiny) { xhat[i] = lo; continue; }", "if (r < tiny) { xhat[i] = 0.0f; continue; }"),
    ("mm_flush_threshold", "        if (r < tiny) { q[i] = 0; continue; }", "        if (r < 1e-20f) { q[i] = 0; continue; }"),
    ("mm_sum_skips_last_worker", "for (int w = 0; w < W; ++w) {\n        mqo_unpack(codes[w], n, bits, q);\n        mqo_dequantize_minmax",
     "for (int w = 0; w < W - (W > 2); ++w) {\n        mqo_unpack(codes[w], n, bits, q);\n        mqo_dequantize_minmax"),
]

# mistakes planted in the L2-norm scale variant, caught by tests/test_oracle_l2_pins.py
MUTANTS_L2 = [
    ("l2_rows_summed_in_sequence",
     "for (uint64_t width = padded; width > 1; width /= 2)  /* N2: one tree level per pass */\n"
     "        for (uint64_t j = 0; j < width / 2; ++j)\n"
     "            node[j] = node[2 * j] + node[2 * j + 1];",
     "for (uint64_t j = 1; j < padded; ++j) node[0] = node[0] + node[j];"),
    ("l2_pairs_half_a_level_apart", "node[j] = node[2 * j] + node[2 * j + 1];", "node[j] = node[j] + node[j + width / 2];"),
    ("l2_unfused_square", "a = fmaf(x[j], x[j], a);", "a = x[j] * x[j] + a;"),
    ("l2_chain_right_to_left", "for (uint64_t j = j0; j < j1; ++j) a = fmaf(x[j], x[j], a);",
     "for (uint64_t j = j1; j-- > j0; ) a = fmaf(x[j], x[j], a);"),
    ("l2_short_last_row_dropped", "uint64_t rows = (len + 31) / 32;", "uint64_t rows = len >= 32 ? len / 32 : 1;"),
    ("l2_rows_of_16", "uint64_t j0 = 32 * r, j1 = j0 + 32;", "uint64_t j0 = 32 * r, j1 = j0 + 16;"),
    ("l2_no_root", "scales[k] = (S < tiny) ? 0.0f : sqrtf(S);", "scales[k] = (S < tiny) ? 0.0f : S;"),
    ("l2_flush_decided_on_root", "scales[k] = (S < tiny) ? 0.0f : sqrtf(S);", "scales[k] = (sqrtf(S) < tiny) ? 0.0f : sqrtf(S);"),
    ("l2_sum_of_magnitudes", "a = fmaf(x[j], x[j], a);", "a = fabsf(x[j]) + a;"),
    ("l2_scale_is_max_abs", "mqo_bucket_norms(x, n, bucket, scales);\n    mqo_draw_h", "mqo_bucket_scales(x, n, bucket, scales);\n    mqo_draw_h"),
]

# mistakes planted in the 1-bit error-feedback variant, caught by tests/test_oracle_onebit_pins.py
MUTANTS_ONEBIT = [
    ("ob_old_residual_ignored", "v[i] = v[i] + residual[i];", "v[i] = v[i];"),
    ("ob_zero_counts_as_negative", "q[i] = (v[i] >= 0.0f) ? 1 : 0;", "q[i] = (v[i] > 0.0f) ? 1 : 0;"),
    ("ob_residual_against_ideal_mean", "float xhat = (r < tiny) ? neg : fmaf((float)q[i], r, neg);",
     "float xhat = (r < tiny) ? neg : (q[i] ? pos : neg);"),
    ("ob_residual_sign", "residual[i] = v[i] - xhat;", "residual[i] = xhat - v[i];"),
    ("ob_mean_over_whole_bucket", "float pos = c1 ? S1 / (float)c1 : 0.0f;", "float pos = c1 ? S1 / (float)(b1 - b0) : 0.0f;"),
    ("ob_ranges_swapped", "ranges[2 * k] = neg;\n        ranges[2 * k + 1] = pos;",
     "ranges[2 * k] = pos;\n        ranges[2 * k + 1] = neg;"),
    ("ob_rows_summed_in_sequence",
     "        node[r] = a;\n    }\n    for (uint64_t width = padded; width > 1; width /= 2)\n"
     "        for (uint64_t j = 0; j < width / 2; ++j)\n            node[j] = node[2 * j] + node[2 * j + 1];\n    float S = node[0];\n    free(node);\n    return S;\n}\n\n/* E1..E5",
     "        node[r] = a;\n    }\n    for (uint64_t j = 1; j < padded; ++j) node[0] = node[0] + node[j];\n"
     "    float S = node[0];\n    free(node);\n    return S;\n}\n\n/* E1..E5"),
    ("ob_class_sum_takes_every_element", "if ((v[j] >= 0.0f ? 1 : 0) == cls) a = a + v[j];", "a = a + v[j];"),
    ("ob_constant_bucket_keeps_codes", "if (r < tiny) q[i] = 0;", ""),
]


def _run(args):
    name, old, new, tmpdir = args
    text = open(SRC).read()
    assert text.count(old) >= 1, name
    mutated = text.replace(old, new, 1)
    c = os.path.join(tmpdir, name + ".c")
    so = os.path.join(tmpdir, name + ".so")
    with open(c, "w") as f:
        f.write(mutated)
    subprocess.run(["gcc", "-O2", "-std=c99", "-ffp-contract=off", "-fno-fast-math", "-fPIC",
                    "-shared", "-o", so, c, "-lm"], check=True)
    env = dict(os.environ, MQG_ORACLE_LIB=so)
    pins = ("test_oracle_minmax_pins.py" if name.startswith("mm_")
            else "test_oracle_l2_pins.py" if name.startswith("l2_")
            else "test_oracle_onebit_pins.py" if name.startswith("ob_") else "test_oracle_pins.py")
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                        os.path.join(ROOT, "tests", pins)],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    return name, r.returncode, r.stdout[-400:]


def test_every_planted_mistake_is_caught(tmp_path):
    jobs = [(n, o, w, str(tmp_path)) for n, o, w in MUTANTS + MUTANTS_MINMAX + MUTANTS_L2 + MUTANTS_ONEBIT]
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 2)) as ex:
        results = list(ex.map(_run, jobs))
    survivors = [name for name, rc, _ in results if rc == 0]
    assert not survivors, "pins do not catch: %s" % survivors
    crashed = [(name, out) for name, rc, out in results if rc not in (0, 1)]
    assert not crashed, crashed
