"""Mutation check of the pins: plant one plausible mistake at a time in a *copy* of the
oracle's C source (a wrong sign, index, transposition, dropped term), build it on the CPU,
and require that at least one pin fails.  The committed oracle is never modified."""
import os
import subprocess

import pytest

from oracle import ref
import test_oracle_pins as pins
import test_oracle_g1 as g1pins

SRC = os.path.join(os.path.dirname(ref.__file__), "cmoe_oracle.c")

MUTANTS = [
    ("nibble sign", "if (code >= 8) code -= 16;", "if (code >= 8) code -= 15;"),
    ("nibble order", "(idx % 2 == 0) ? (byte & 0xF) : (byte >> 4)", "(idx % 2 == 1) ? (byte & 0xF) : (byte >> 4)"),
    ("scale group", "s[idx / 32]", "s[idx / 16]"),
    ("half rebias", "(expo + 112u)", "(expo + 111u)"),
    ("cluster argmin", "if (z[g] > z[gs]) gs = g;", "if (z[g] < z[gs]) gs = g;"),
    ("C transposed", "D->C[(size_t)j * G + g]", "D->C[(size_t)g * d + j]"),
    ("R cluster stride", "D->R[((size_t)gs * d + j) * K + i]", "D->R[((size_t)gs * K + i) * d + j]"),
    ("cluster bias dropped", "if (D->b_c) acc += (double)D->b_c[g];", ""),
    ("expert bias index", "D->b_e[(size_t)gs * K + i]", "D->b_e[(size_t)i]"),
    ("topk ascending", "l[i] > l[best]", "l[i] < l[best]"),
    ("gate not renormalised", "/ denom);", ");"),
    ("gate sign", "exp((double)l[sel[s]] - lmax) / denom", "exp(lmax - (double)l[sel[s]]) / denom"),
    ("U index transposed", "((int64_t)e * r + p) * din + a", "((int64_t)e * din + a) * r + p"),
    ("V index transposed", "((int64_t)e * dout + b) * r + p", "((int64_t)e * r + p) * dout + b"),
    ("residual dropped", "acc[b] += u * (double)Vd[p * dout + b];", ";"),
    ("residual sign", "acc[b] += u * (double)Vd[p * dout + b];", "acc[b] -= u * (double)Vd[p * dout + b];"),
    ("base of wrong cluster", "g = e / K, r = D->r;", "g = e % D->G, r = D->r;"),
    ("gelu tanh-less", "(1.0 + erf((double)u / sqrt(2.0)))", "(1.0 + erf((double)u))"),
    ("gelu half dropped", "0.5 * (double)u *", "(double)u *"),
    ("W1 transposed read", "const float* w = W1 + (size_t)j * d_ff;", "const float* w = W1 + (size_t)j;"),
    ("gate dropped in combine", "(double)gate[(size_t)n * k + s] *", ""),
    ("only first slot combined", "for (int s = 0; s < k; ++s)\n        acc += (double)gate", "for (int s = 0; s < 1; ++s)\n        acc += (double)gate"),
    ("param count", "(int64_t)D->E * 2 * D->r", "(int64_t)D->E * D->r"),
    ("bf16 read as the low half", "uint32_t bits = (uint32_t)h << 16;", "uint32_t bits = (uint32_t)h;"),
    ("bf16 flag ignored", "D->base_is_bf16 ? cmoe_ref_bf16_to_float(B[a * dout + b]) : cmoe_ref_half_to_float(B[a * dout + b])",
     "cmoe_ref_half_to_float(B[a * dout + b])"),
    ("loads count the first kept expert only", "for (int s = 0; s < k; ++s) loads[slot[(size_t)t * k + s]] += 1;",
     "for (int s = 0; s < 1; ++s) loads[slot[(size_t)t * k + s]] += 1;"),
    ("mean over all tokens", "sum[j] / (double)loads[e] : 0.0;", "sum[j] / (double)T : 0.0;"),
    ("EMA weights swapped", "(1.0 - (double)beta) * (double)mu[(size_t)e * d + j] + (double)beta * mean",
     "(double)beta * (double)mu[(size_t)e * d + j] + (1.0 - (double)beta) * mean"),
    ("EMA applied without tokens", "if (mu && loads[e] > 0)", "if (mu)"),
    ("sample variance", "sqrt(var / (double)E) / mean", "sqrt(var / (double)(E - 1)) / mean"),
    ("variance instead of deviation", "sqrt(var / (double)E) / mean", "(var / (double)E) / mean"),
    ("g1: least probable clusters", "z[g] > z[best]", "z[g] < z[best]"),
    ("g1: a cluster may be kept twice", "gone[best] = 1;", ";"),
    ("g1: cluster weights not renormalised", "const double pg = exp((double)z[gs] - (double)z[gsel[0]]) / zden;",
     "const double pg = exp((double)z[gs] - (double)z[gsel[0]]);"),
    ("g1: cluster weights dropped", "(float)(pg * (exp((double)l[sel[s]] - lmax) / denom))", "(float)((exp((double)l[sel[s]] - lmax) / denom))"),
    ("g1: only the last expert's output kept", "ysum[(size_t)n * d + c] += (double)gate[(size_t)n * kk + s] *",
     "ysum[(size_t)n * d + c] = (double)gate[(size_t)n * kk + s] *"),
    ("g1: expert bias of the first kept cluster", "if (D->b_e) acc += (double)D->b_e[(size_t)gs * K + i];\n        l[i] = (float)acc;\n      }\n      char taken[64];",
     "if (D->b_e) acc += (double)D->b_e[(size_t)gsel[0] * K + i];\n        l[i] = (float)acc;\n      }\n      char taken[64];"),
]

PINS = [
    pins.test_half_decode_all_bit_patterns,
    pins.test_int4_every_byte_both_positions,
    pins.test_int4_hand_written_vector,
    pins.test_parameter_ratio_closed_form,
    pins.test_hand_worked_layer,
    lambda: pins.test_rank_zero_is_dense_ffn_per_cluster(0),
    lambda: pins.test_one_expert_per_cluster_is_top1_moe(0),
    lambda: pins.test_routes_by_enumeration(dict(E=12, G=3, k=3)),
    lambda: pins.test_explicit_weights_match_factored_form("tiny", 0),
    pins.test_residual_only_layer,
    pins.test_formed_weights_orientation,
    pins.test_invariants,
    pins.test_bf16_decode_all_bit_patterns,
    pins.test_bf16_bases_are_decoded_as_bf16,
    pins.test_expert_stats_hand_counted,
    pins.test_expert_stats_conservation_and_numpy_counts,
    g1pins.test_one_cluster_is_the_pinned_routing_and_forward,
    lambda: g1pins.test_routes_by_enumeration(dict(E=12, G=3, k=2), 2),
    g1pins.test_forward_against_a_dense_evaluation,
    g1pins.test_all_clusters_and_all_experts_is_the_full_soft_mixture,
    g1pins.test_hand_worked_token,
    g1pins.test_ties_and_bad_arguments,
]


@pytest.mark.parametrize("label,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_mutant_is_caught(tmp_path, monkeypatch, label, old, new):
    text = open(SRC).read()
    assert text.count(old) >= 1, f"mutation site for '{label}' not found in the oracle source"
    c_file = tmp_path / "mutant.c"
    c_file.write_text(text.replace(old, new, 1))
    so = tmp_path / "libmutant.so"
    subprocess.run(["gcc", "-O1", "-fopenmp", "-shared", "-fPIC", "-w", "-I", os.path.dirname(SRC),
                    "-o", str(so), str(c_file), "-lm"], check=True)
    monkeypatch.setattr(ref, "_lib", ref.load(str(so)))
    caught = False
    for pin in PINS:
        try:
            pin()
        except (AssertionError, ValueError, FloatingPointError):
            caught = True
            break
    assert caught, f"no pin noticed the planted mistake: {label}"
