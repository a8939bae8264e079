"""The pins must notice plausible mistakes.  Each case plants one mistake in a copy of the oracle's
C source (on the CPU, nothing here touches a GPU), builds it, and runs the pin tests against it in
a subprocess: they have to fail."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "granq_oracle.c")

MUTATIONS = {
    "wrong_sign_of_zero_point_in_eq1": ("float u = t + zk;", "float u = t - zk;"),
    "ties_away_from_zero": ("float r = rintf(u);", "float r = floorf(u + 0.5f);"),
    "scale_divided_by_2_pow_b": ("float s = (hi - lo) / qmax;", "float s = (hi - lo) / (qmax + 1.0f);"),
    "no_upper_clamp": ("if (q > qmax) q = qmax;", ""),
    "mask_excludes_code_zero": ("int inside = (r >= 0.0f) && (r <= qmax);", "int inside = (r > 0.0f) && (r <= qmax);"),
    "dequantize_without_zero_point": ("float yv = sk * d;", "float yv = sk * q;"),
    "zero_point_from_plus_lo": ("float z = rintf((-lo) / s);", "float z = rintf(lo / s);"),
    "max_taken_as_min": ("if (v > hi[k]) hi[k] = v;", "if (v < hi[k]) hi[k] = v;"),
    "sample_channel_groups_collapsed": ("return o * g->C + c;", "return c;"),
    "bf16_ties_away": ("u += 0x7FFFu + lsb;", "u += 0x8000u;"),
    "no_degenerate_floor": ("if (!(s >= 1e-8f)) s = 1e-8f;", "if (!(s > 0.0f)) s = 1.0f;"),
    "gradient_not_masked": ("inside ? gv : 0.0f", "gv"),
    "packed_mask_most_significant_bit_first": ("(1u << (e % 8))", "(0x80u >> (e % 8))"),
    "packed_backward_reads_bits_in_reverse": ("(packed[e / 8] >> (e % 8)) & 1", "(packed[e / 8] >> (7 - e % 8)) & 1"),
    "packed_backward_ignores_mask": ("bit ? gv : 0.0f", "gv"),
    "distortion_error_not_squared_difference": ("sdd += d * d;", "sdd += d;"),
    "distortion_cosine_without_norm_of_q": ("double den = sqrt(sums[0]) * sqrt(sums[1]);", "double den = sums[0];"),
    "distortion_relative_error_not_rooted": ("sqrt(sums[3]) / sqrt(sums[0])", "sums[3] / sums[0]"),
    "packed_codes_most_significant_bit_first": ("if ((codes[e] >> j) & 1) packed[k / 8]",
                                                "if ((codes[e] >> (bits - 1 - j)) & 1) packed[k / 8]"),
    "packed_codes_stride_of_8_bits": ("int64_t k = e * bits + j;\n            if ((codes[e] >> j) & 1)",
                                      "int64_t k = e * 8 + j;\n            if ((codes[e] >> j) & 1)"),
    "dequant_packed_adds_zero_point": ("float d = (float)code - z[grp];", "float d = (float)code + z[grp];"),
    "accumulate_without_zero_point": ("float d = (float)code - z[c];\n                    float a = s[c] * d;", "float d = (float)code;\n                    float a = s[c] * d;"),
    "accumulate_weight_indexed_transposed": ("acc += (double)w[o * C + c] * (double)a;", "acc += (double)w[c * O + o] * (double)a;"),
    "accumulate_inloop_scale_of_the_output_channel": ("acc += (double)w[o * C + c] * (double)s[c] * ((double)code - (double)z[c]);",
                                                      "acc += (double)w[o * C + c] * (double)s[o % C] * ((double)code - (double)z[c]);"),
    "accumulate_skips_the_last_channel": ("for (int64_t c = 0; c < C; ++c) {\n                    const uint8_t code = channels_last ? codes[(n * P + p) * C + c] : codes[(n * C + c) * P + p];\n                    float d",
                                          "for (int64_t c = 0; c + 1 < C; ++c) {\n                    const uint8_t code = channels_last ? codes[(n * P + p) * C + c] : codes[(n * C + c) * P + p];\n                    float d"),
    "packed_mask_last_byte_not_cleared": ("for (int64_t b = 0; b < (E + 7) / 8; ++b) packed[b] = 0;",
                                          "for (int64_t b = 0; b < E / 8; ++b) packed[b] = 0;"),
}


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_pins_catch_planted_mistake(name, tmp_path):
    old, new = MUTATIONS[name]
    text = open(SRC).read()
    assert text.count(old) == 1, f"mutation target not found exactly once: {old!r}"
    src = tmp_path / "granq_oracle.c"
    src.write_text(text.replace(old, new))
    (tmp_path / "granq_oracle.h").write_text(open(os.path.join(ROOT, "oracle", "granq_oracle.h")).read())
    lib = tmp_path / "libmutant.so"
    subprocess.check_call(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
                           "-o", str(lib), str(src), "-lm"])
    env = dict(os.environ, GRANQ_ORACLE_LIB_OVERRIDE=str(lib))
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_oracle_pins.py"), "-x", "-q",
                        "-p", "no:cacheprovider"], env=env, cwd=ROOT, capture_output=True, text=True)
    assert r.returncode != 0, f"the pins did not notice: {name}\n{r.stdout[-800:]}"
