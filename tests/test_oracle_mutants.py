"""Do the pins bite?  Each case plants one plausible mistake in a copy of the oracle's C source,
builds it, swaps it in for the real oracle, and demands that a named pin test fails."""
import os
import subprocess

import pytest

import oracle
from tests import test_oracle_algorithm as t_alg
from tests import test_oracle_operators as t_ops
from tests import test_oracle_primitives as t_prim
from tests import test_oracle_whole_vector as t_whole

SRC = os.path.join(os.path.dirname(oracle.__file__), "dsq_oracle.c")

MUTANTS = [
    # (name, text to replace, replacement, pin that must fail)
    ("running sum instead of pairwise",
     "  float left = pairwise_sum(a, half);\n  float right = pairwise_sum(a + half, half);\n  float s = left + right;\n  return s;",
     "  float s = 0.0f; for (size_t i = 0; i < len; ++i) s = s + a[i];\n  return s;",
     lambda: [t_prim.test_pairwise_sum_hand_derived(e, i) for e, i in t_prim._cases()]),
    ("sign scale divides by the nominal chunk length",
     "s = l1 / (float)len;", "s = l1 / (float)L;",
     t_ops.test_sign1_short_last_chunk_divides_by_true_length),
    ("l2 sign scale divides by the length instead of its root",
     "s = l2 / root_len;", "s = l2 / (float)len;",
     lambda: t_ops.test_sign1_l2_scale_is_rms_and_keeps_the_l2_magnitude(10000, 4096)),
    ("l2 sign scale sums |v| instead of v*v",
     "float e2 = e * e;\n        term[t] = e2;", "float e2 = fabsf(e);\n        term[t] = e2;",
     lambda: t_ops.test_sign1_l2_scale_is_rms_and_keeps_the_l2_magnitude(10000, 4096)),
    ("clipping keeps one bit too many",
     "uint32_t kept = u >> b;       /* the high 32 - b bits */", "uint32_t kept = (u >> (b - 1)) << 1 >> 1;",
     t_ops.test_clip_worked_binary_cases),
    ("clipping rounds to nearest instead of clearing bits",
     "uint32_t kept = u >> b;       /* the high 32 - b bits */", "uint32_t kept = (u + (1u << (b - 1))) >> b;",
     t_ops.test_clip_worked_binary_cases),
    ("sparsifier scales by S - 1",
     "const float factor = scaled ? (float)S : 1.0f;", "const float factor = scaled ? (float)(S - 1) : 1.0f;",
     t_ops.test_rsparse_keeps_each_entry_with_probability_one_in_S_and_scaled_form_is_unbiased),
    ("sparsifier draws from the second Philox word",
     "uint32_t o = rnd[0] % S;", "uint32_t o = rnd[1] % S;",
     lambda: t_ops.test_rsparse_structure_of_what_is_sent(1)),
    ("sparsifier keeps offsets o and o + 1",
     "if (t % S == o) {", "if (t % S == o || t % S == (o + 1) % S) {",
     lambda: t_ops.test_rsparse_structure_of_what_is_sent(0)),
    ("sign bit is v > 0",
     "int nonneg = v[j] >= 0.0f;\n      if (nonneg) bits[j / 32]", "int nonneg = v[j] > 0.0f;\n      if (nonneg) bits[j / 32]",
     lambda: t_ops.test_sign1_scale_is_l1_mean_per_chunk_and_bits_are_signs(10000, 4096)),
    ("top-k ties go to the higher index",
     "if (a->idx != b->idx) return a->idx < b->idx ? -1 : 1;", "if (a->idx != b->idx) return a->idx > b->idx ? -1 : 1;",
     t_ops.test_topk_all_equal_takes_lowest_indices_and_matches_partition),
    ("top-k compares signed values",
     "order[j].key = f32_bits(v[j]) & 0x7FFFFFFFu;", "order[j].key = f32_bits(v[j]) ^ 0x80000000u;",
     lambda: t_ops.test_topk_matches_brute_force_with_ties(200, 13)),
    ("quantiser rounds up with probability 1 - frac",
     "uint32_t level = (uint32_t)f + (u < p ? 1u : 0u);", "uint32_t level = (uint32_t)f + (u < 1.0f - p ? 1u : 0u);",
     t_ops.test_qsgd_unbiased_and_variance_by_monte_carlo),
    ("quantiser uses the next Philox word",
     "uint32_t w = rnd[t % 4];", "uint32_t w = rnd[(t + 1) % 4];",
     t_ops.test_qsgd_levels_bracket_the_value_and_decode_roundtrip),
    ("Philox swaps its multipliers",
     "uint64_t p0 = mult0 * (uint64_t)c0;\n    uint64_t p1 = mult1 * (uint64_t)c2;",
     "uint64_t p0 = mult1 * (uint64_t)c0;\n    uint64_t p1 = mult0 * (uint64_t)c2;",
     t_prim.test_philox_matches_independent_library),
    ("server adds its error before scaling",
     "float mean = acc * inv_n;\n    float s = mean + delta_s[j];", "float mean = acc + delta_s[j];\n    float s = mean * inv_n;",
     t_prim.test_server_mean_special_cases),
    ("residual has the wrong sign",
     "float r = v[j] - C[j];", "float r = C[j] - v[j];",
     lambda: t_alg.test_telescoping_identity_of_the_global_update_rule("sign1", "sign1")),
    ("update adds instead of subtracting",
     "float r = x[j] - t;", "float r = x[j] + t;",
     t_alg.test_identity_reduces_to_parallel_sgd_bitwise),
    ("whole-vector factor divides by the padded length",
     "s = l1 / (float)d;", "s = l1 / (float)next_pow2_u64(d);",
     t_whole.test_whole_vector_sign_short_vector_divides_by_its_true_length),
    ("padded sum forgets a partly filled right half",
     "float right = pairwise_sum_padded(a + half, len > half ? len - half : 0, half);",
     "float right = len >= L ? pairwise_sum_padded(a + half, half, half) : 0.0f;",
     lambda: t_whole.test_padded_pairwise_sum_equals_the_sum_over_the_written_out_padding(1025, 2048)),
    ("ternary keeps an entry with probability 1 - |e|/|m|",
     "kept = u < p;", "kept = u < 1.0f - p;",
     t_whole.test_ternary_is_unbiased_before_scaling_and_keeps_the_largest_entry_always),
    ("ternary factor divides by the length instead of the non-zero count",
     "if (count > 0) s = l1 / (float)count;", "if (count > 0) s = l1 / (float)d;",
     t_whole.test_ternary_structure_scale_and_the_documented_philox_word),
    ("ternary takes the largest signed value as m",
     "if (a > m) m = a;", "if (v[j] > m) m = v[j];",
     t_whole.test_ternary_degenerate_vectors),
    ("ternary draws from the quantiser's counter",
     "uint32_t ctr[4] = {(uint32_t)(j / 4), 0xFFFFFFFEu, wid, step};", "uint32_t ctr[4] = {(uint32_t)(j / 4), 0u, wid, step};",
     t_whole.test_ternary_structure_scale_and_the_documented_philox_word),
    ("uncompensated server forgets the 1/n",
     "float mean = acc * inv_n;\n    v[j] = mean;", "float mean = acc;\n    v[j] = mean;",
     lambda: t_whole.test_without_compensation_the_model_follows_plain_compressed_sgd("sign1", "topk")),
]


@pytest.mark.parametrize("name,old,new,pin", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(tmp_path, name, old, new, pin):
    text = open(SRC).read()
    assert text.count(old) == 1, f"mutation site for '{name}' not found exactly once"
    mutant_c = tmp_path / "mutant.c"
    mutant_c.write_text(text.replace(old, new))
    mutant_so = tmp_path / "mutant.so"
    subprocess.run(["gcc", "-std=c11", "-O2", "-fPIC", "-shared", "-ffp-contract=off", "-o", str(mutant_so), str(mutant_c),
                    "-lm"], check=True)
    real = oracle.lib()
    oracle._lib = oracle.load(str(mutant_so))
    try:
        with pytest.raises((AssertionError, ValueError)):
            pin()
    finally:
        oracle._lib = real
    pin()   # and the real oracle passes the same pin
