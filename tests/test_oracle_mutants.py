"""Each plausible mistake, planted in a private copy of the oracle's source, must
trip at least one pin.  The mistakes are planted on the CPU only."""
import subprocess

import pytest

from oracle import dlion_oracle as orc
from tests import oracle_pins

MUTANTS = {
    "delta_uses_beta2": ("const float a1 = beta1 * mo;", "const float a1 = beta2 * mo;"),
    "delta_uses_om2": ("const float b1 = om1 * gf;", "const float b1 = om2 * gf;"),
    "delta_uses_new_momentum": ("const float a1 = beta1 * mo;",
                                "const float a1 = beta1 * (beta2 * mo + om2 * gf);"),
    "delta_negated": ("word |= sign_bit(c) << b;", "word |= sign_bit(-c) << b;"),
    "sign_of_zero_negative": ("return (v >= 0.0f) ? 1u : 0u;", "return (v > 0.0f) ? 1u : 0u;"),
    "bit_order_reversed": ("word |= sign_bit(c) << b;", "word |= sign_bit(c) << (31 - b);"),
    "momentum_uses_beta1": ("store_state(m, mdtype, idx, a2 + b2);", "store_state(m, mdtype, idx, a1 + b1);"),
    "momentum_drops_gradient": ("store_state(m, mdtype, idx, a2 + b2);", "store_state(m, mdtype, idx, a2);"),
    "one_minus_beta_dropped": ("const float om2 = 1.0f - beta2;", "const float om2 = 1.0f;"),
    "tie_goes_negative": ("Delta = (S >= 0) ? 1.0f : -1.0f;", "Delta = (S > 0) ? 1.0f : -1.0f;"),
    "sum_is_count": ("const int32_t S = 2 * P - N;", "const int32_t S = P;"),
    "average_without_division": ("Delta = static_cast<float>(S) / static_cast<float>(N);",
                                 "Delta = static_cast<float>(S);"),
    "weight_decay_sign": ("const float t2 = Delta + t1;", "const float t2 = Delta - t1;"),
    "weight_decay_dropped": ("const float t1 = weight_decay * xo;", "const float t1 = 0.0f * xo;"),
    "update_sign": ("x[j] = xo - t3;", "x[j] = xo + t3;"),
    "lr_outside_decay": ("const float t3 = lr * t2;", "const float t3 = lr * Delta + t1;"),
    "only_first_worker_counted": ("P += static_cast<int32_t>((packed[static_cast<size_t>(i) * W",
                                  "P += static_cast<int32_t>((packed[static_cast<size_t>(0) * W"),
    "padding_written": ("if (j < lo || j >= hi) continue;            // padding bit stays 0",
                        "if (j >= d_pad) continue;"),
    "wire_planes_reversed": ("delta_wire[p * W + w] |= ((P >> p) & 1u) << b;",
                             "delta_wire[p * W + w] |= ((P >> (K - 1 - p)) & 1u) << b;"),
    "wire_majority_bit_inverted": ("Delta = ((delta_wire[j / 32] >> (j % 32)) & 1u) ? 1.0f : -1.0f;",
                                   "Delta = ((delta_wire[j / 32] >> (j % 32)) & 1u) ? -1.0f : 1.0f;"),
    "wire_decode_without_doubling": ("Delta = static_cast<float>(2 * P - N) / static_cast<float>(N);",
                                     "Delta = static_cast<float>(P - N) / static_cast<float>(N);"),
    "wire_apply_sign": ("x[j] = xo - u3;", "x[j] = xo + u3;"),
    "wire_tie_negative": ("static_cast<int64_t>(n_workers) >= 0) delta_wire[w] |= 1u << b;",
                          "static_cast<int64_t>(n_workers) > 0) delta_wire[w] |= 1u << b;"),
    "bf16_store_truncates": ("u += 0x7FFFu + lsb;", "u += 0u;"),
    "bf16_store_rounds_half_up": ("u += 0x7FFFu + lsb;", "u += 0x8000u;"),
    "betas_of_worker_zero": ("const float beta1 = beta1s[i], beta2 = beta2s[i];",
                             "const float beta1 = beta1s[0], beta2 = beta2s[0];"),
    "global_blend_uses_beta2": ("const float p1 = beta1 * mo;", "const float p1 = beta2 * mo;"),
    "global_blend_uses_new_momentum": ("const float p1 = beta1 * mo;", "const float p1 = beta1 * (beta2 * mo + w2 * gf);"),
    "global_votes_instead_of_mean": ("total = (i == 0) ? mt : total + mt;",
                                     "total = (i == 0 ? 0.0f : total) + ((mt >= 0.0f) ? 1.0f : -1.0f);"),
    "global_only_first_worker": ("total = (i == 0) ? mt : total + mt;", "total = (i == 0) ? mt : total;"),
    "global_one_minus_beta_dropped": ("const float w1 = 1.0f - beta1;                               // R1: (1-beta) in binary32",
                                      "const float w1 = 1.0f;"),
    "global_sign_negated": ("const float Delta = (G >= 0.0f) ? 1.0f : -1.0f;",
                            "const float Delta = (G >= 0.0f) ? -1.0f : 1.0f;"),
    "global_momentum_not_updated": ("m[idx] = p2 + q2;", "m[idx] = mo;"),
    "global_momentum_uses_beta1": ("m[idx] = p2 + q2;", "m[idx] = p1 + q1;"),
    "global_weight_decay_sign": ("const float v2 = Delta + v1;", "const float v2 = Delta - v1;"),
    "global_update_sign": ("x[j] = xo - v3;", "x[j] = xo + v3;"),
    "global_sums_gradients_only": ("const float mt = p1 + q1;                    // the blend each worker would send",
                                   "const float mt = gf;"),
    "counts16_last_worker_skipped": ("for (uint32_t worker = 0; worker < n_workers; ++worker) {",
                                     "for (uint32_t worker = 0; worker + 1 < n_workers; ++worker) {"),
    "counts16_bit_order": ("votes += (packed[worker * words + j / 32] >> (j % 32)) & 1u;",
                           "votes += (packed[worker * words + j / 32] >> (31 - j % 32)) & 1u;"),
    "counts16_truncated_to_a_byte": ("count16[j] = static_cast<uint16_t>(votes);",
                                     "count16[j] = static_cast<uint16_t>(votes & 0xFFu);"),
    "ternary_tie_goes_positive": ("Delta = (S > 0) ? 1.0f : ((S < 0) ? -1.0f : 0.0f);",
                                  "Delta = (S > 0) ? 1.0f : ((S < 0) ? -1.0f : 1.0f);"),
    "ternary_strict_sign_flipped": ("Delta = (S > 0) ? 1.0f : ((S < 0) ? -1.0f : 0.0f);",
                                    "Delta = (S > 0) ? -1.0f : ((S < 0) ? 1.0f : 0.0f);"),
    "ternary_message_planes_swapped": ("delta_wire[w] |= (code & 1u) << b;\n                    delta_wire[W + w] |= (code >> 1) << b;",
                                       "delta_wire[W + w] |= (code & 1u) << b;\n                    delta_wire[w] |= (code >> 1) << b;"),
    "ternary_message_tie_as_plus": ("const uint32_t code = (S3 > 0) ? 2u : ((S3 < 0) ? 0u : 1u);",
                                    "const uint32_t code = (S3 >= 0) ? 2u : 0u;"),
    "ternary_decode_without_offset": ("Delta = static_cast<float>(static_cast<int32_t>(low + 2u * high) - 1);",
                                      "Delta = static_cast<float>(static_cast<int32_t>(low + 2u * high));"),
    "ternary_one_plane": ("if (mode == DLION_ORACLE_MAJORITY_TERNARY) return 2;", "if (mode == DLION_ORACLE_MAJORITY_TERNARY) return 1;"),
    "average_down_bits_floor_log": ("while ((1ull << bits) < static_cast<uint64_t>(n_workers) + 1ull) ++bits;",
                                    "while ((2ull << bits) <= static_cast<uint64_t>(n_workers)) ++bits;"),
}


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_mutant_is_caught(name, tmp_path, oracle):
    old, new = MUTANTS[name]
    src = open(orc._SRC).read()
    assert src.count(old) == 1, f"mutation site for {name} not found exactly once"
    msrc = tmp_path / "mutant.cpp"
    msrc.write_text(src.replace(old, new))
    out = tmp_path / "libmutant.so"
    subprocess.run(["g++", *orc.CXXFLAGS, "-o", str(out), str(msrc)], check=True)
    lib = orc.load(str(out))
    caught = []
    for check in oracle_pins.ALL_CHECKS:
        try:
            check(lib)
        except (AssertionError, ValueError):
            caught.append(check.__name__)
    assert caught, f"no pin notices the planted mistake '{name}'"
