"""Do the pins pin?  Each case plants one plausible mistake in a COPY of the oracle's C source (a
dropped term, a wrong sign, a swapped operand, a wrong index), builds it and runs the pin suite
against that library in a process of its own: the suite must fail.  A mutant that survives means
some line of the oracle is checked by nothing but itself."""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "swiftprune_oracle.c")

# (name, text in the source, replacement, which occurrence)
MUTANTS = [
    # statistics (Algorithm 1, step 1)
    ("colsq_not_squared", "colsq[q] += v * v;", "colsq[q] += v;", 0),
    ("colsq_wrong_channel", "double v = (double)spo_decode(row[q], dtype);",
     "double v = (double)spo_decode(row[q1 - 1 - (q - q0)], dtype);", 0),
    ("total_drops_last", "for (int64_t q = 0; q < n; ++q)\n        S += colsq[q];",
     "for (int64_t q = 0; q + 1 < n; ++q)\n        S += colsq[q];", 0),
    # decoders
    ("half_exponent_bias", "((expo + 112u) << 23)", "((expo + 111u) << 23)", 0),
    ("half_subnormal_scale", "(1.0f / 16777216.0f)", "(1.0f / 8388608.0f)", 0),
    ("bf16_shift", "(uint32_t)h << 16", "(uint32_t)h << 15", 0),
    # Eq. 8
    ("score32_half_dropped", "float c = 0.5f / den;", "float c = 1.0f / den;", 0),
    ("score32_sign_of_u", "float den = 1.0f - u;\n    float c", "float den = 1.0f + u;\n    float c", 0),
    ("score32_w_not_squared", "float w2 = w * w;\n    return w2 * c;", "float w2 = fabsf(w);\n    return w2 * c;", 0),
    ("score64_inverted_ratio", "(1.0 - xq2 / S)", "(1.0 - S / xq2)", 0),
    ("factor_half_dropped", "c[q] = 0.5f / den;", "c[q] = 1.0f / den;", 0),
    # Algorithm 1 / Table 2, binary32
    ("ewma32_test_reversed", "if (L < thr) {", "if (L > thr) {", 0),
    ("ewma32_threshold_sign", "float thr = est - la_dev;", "float thr = est + la_dev;", 0),
    ("ewma32_est_not_initialised", "if (i == 0)\n                est = L;\n            float la_dev",
     "float la_dev", 0),
    ("ewma32_dev_from_old_est",
     "est = keep_part + new_part;\n            float diff = fabsf(est - L);",
     "float diff = fabsf(est - L);\n            est = keep_part + new_part;", 0),
    ("ewma32_alpha_beta_swapped", "float new_part = alpha * L;", "float new_part = beta * L;", 0),
    ("ewma32_dev_keeps_alpha", "const float one_minus_beta = 1.0f - beta;",
     "const float one_minus_beta = 1.0f - alpha;", 0),
    ("ewma32_dev_gain_is_alpha", "float dnew = beta * diff;", "float dnew = alpha * diff;", 0),
    ("ewma32_S_never_updated", "S = S - w2;", "S = S;", 0),
    ("ewma32_S_grows", "S = S - w2;", "S = S + w2;", 0),
    ("ewma32_x2_reading_takes_w2", "S = S - colsq32[i];", "S = S - w * w;", 0),
    ("ewma32_pruned_weight_kept", "bits = 0; /* w_i = 0 */", "/* w_i = 0 */", 0),
    # Algorithm 1, binary64
    ("ewma64_test_reversed", "if (L < thr) {", "if (L > thr) {", 1),
    ("ewma64_dev_from_old_est",
     "est = (1.0 - alpha) * est + alpha * L;\n            dev = (1.0 - beta) * dev + beta * fabs(est - L);",
     "dev = (1.0 - beta) * dev + beta * fabs(est - L);\n            est = (1.0 - alpha) * est + alpha * L;", 0),
    ("ewma64_alpha_beta_swapped", "est = (1.0 - alpha) * est + alpha * L;",
     "est = (1.0 - alpha) * est + beta * L;", 0),
    ("ewma64_threshold_sign", "double thr = est - la * dev;", "double thr = est + la * dev;", 0),
    ("ewma64_S_never_updated", "S = S - w * w;", "S = S;", 0),
    # mask layout
    ("mask_bit_order", "(uint32_t)1u << (i & 31)", "(uint32_t)1u << (31 - (i & 31))", 0),
    # Section 3.3
    ("nm_keeps_the_small_ones", "for (int k = 0; k < M - N; ++k) {", "for (int k = 0; k < N; ++k) {", 0),
    ("nm_prunes_the_largest", "spo_less32(L[j], L[best])", "spo_less32(L[best], L[j])", 0),
    ("nm_tie_prunes_higher_column", "if (best < 0 || spo_less32(L[j], L[best]))",
     "if (best < 0 || !spo_less32(L[best], L[j]))", 0),
    ("nm_nan_ranks_lowest", "if (isnan(a))\n        return 0;\n    if (isnan(b))\n        return 1;",
     "if (isnan(a))\n        return 1;\n    if (isnan(b))\n        return 0;", 0),
    ("nm_groups_offset", "L[j] = spo_score32(spo_decode(W[r * ldw + g + j], dtype), colsq32[g + j], S32);",
     "L[j] = spo_score32(spo_decode(W[r * ldw + g + j], dtype), colsq32[g + (j + 1) % M], S32);", 0),
    # write-back
    ("apply_mask_inverted", "Wout[r * ldo + i] = keep ? W[r * ldw + i] : (uint16_t)0;",
     "Wout[r * ldo + i] = keep ? (uint16_t)0 : W[r * ldw + i];", 0),
]


def _mutate(text, old, new, which):
    pos = -1
    for _ in range(which + 1):
        pos = text.find(old, pos + 1)
        assert pos >= 0, "mutation site not found: %r" % old
    return text[:pos] + new + text[pos + len(old):]


def _pins_fail_with(name, old, new, which, tmp):
    with open(SRC) as f:
        text = _mutate(f.read(), old, new, which)
    c_path = os.path.join(tmp, name + ".c")
    so_path = os.path.join(tmp, "lib" + name + ".so")
    with open(c_path, "w") as f:
        f.write(text)
    subprocess.run(["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared",
                    "-fPIC", "-o", so_path, c_path, "-lm"], check=True)
    env = dict(os.environ, SWIFTPRUNE_ORACLE_LIBRARY=so_path, OMP_NUM_THREADS="1")
    proc = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_oracle_pins.py"),
                           "-x", "-q", "-p", "no:cacheprovider"], cwd=ROOT, env=env,
                          capture_output=True, text=True, timeout=600)
    return proc.returncode != 0, proc.stdout[-400:]


def test_unmutated_source_is_what_the_pins_accept(tmp_path):
    # the harness itself: the same build of the unchanged source passes
    with open(SRC) as f:
        text = f.read()
    failed, tail = _pins_fail_with("identity", text[:40], text[:40], 0, str(tmp_path))
    assert not failed, tail


def test_every_planted_mistake_fails_a_pin(tmp_path):
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        futures = {m[0]: pool.submit(_pins_fail_with, *m, str(tmp_path)) for m in MUTANTS}
        survivors = [name for name, f in futures.items() if not f.result()[0]]
    assert not survivors, "no pin noticed: " + ", ".join(survivors)
