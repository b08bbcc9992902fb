"""Do the pins bite?  Each case plants ONE plausible mistake in a copy of the oracle's C source (a dropped
factor, a flipped sign, a transposed index, a strict instead of a non-strict comparison, ...), builds that copy
on the CPU and runs the pins of tests/test_oracle_pins.py against it: at least one of the named pins must fail.
The real oracle is untouched; nothing here runs on a GPU.
"""
import importlib.util
import os
import subprocess

import pytest

from tests import test_oracle_pins as pins

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "clada_oracle.c")
FRONT = os.path.join(ROOT, "oracle", "clada_oracle.py")

# (name, text in the source, replacement, which occurrence (None = all), pins that must notice)
MUTATIONS = [
    ("silu_sign", "return g / (1.0 + exp(-g));", "return g / (1.0 + exp(g));", None,
     [(pins.test_dense_ffn_matches_matrix_formulation, dict(dtype="f32"))]),
    ("gate_without_up", "return silu(g) * u;", "return silu(g);", None,
     [(pins.test_dense_ffn_matches_matrix_formulation, dict(dtype="f32")),
      (pins.test_scores_against_explicit_matrix_norms, {})]),
    ("gelu_constant", "0.044715 * g * g * g", "0.44715 * g * g * g", None,
     [(pins.test_gelu_form_scalar_values, {})]),
    ("relu_keeps_negative", "return g > 0.0 ? g : 0.0;", "return g;", None,
     [(pins.test_relu_form_worked_example, {})]),
    ("norm_of_row_not_column", "double w = elem(W_out, dtype, (size_t)i * d_ff + j);",
     "double w = elem(W_out, dtype, (size_t)j * d_model + i);", 0,
     [(pins.test_scores_against_explicit_matrix_norms, {})]),
    ("select_strict", "int keep = !(scores[j] < tau);", "int keep = (scores[j] > tau);", None,
     [(pins.test_select_brute_force_tiny, {})]),
    ("ffn_mask_strict", "keep[j] = (uint8_t)!(scores[j] < tau);", "keep[j] = (uint8_t)(scores[j] > tau);", None,
     [(pins.test_zero_sparsity_is_dense_bit_for_bit, {})]),
    ("entropy_sign", "H -= exp(logp) * logp;", "H += exp(logp) * logp;", None,
     [(pins.test_entropy_uniform_is_ln_V, dict(V=4096))]),
    ("surprisal_sign", "*surprisal = -(elem(logits, dtype, (size_t)token) - m - logZ);",
     "*surprisal = (elem(logits, dtype, (size_t)token) - m - logZ);", None,
     [(pins.test_two_level_closed_form, dict(a=5.0, V=4096))]),
    ("lambda_gamma_swapped", "mult = mult + lambda[l];", "mult = mult + gamma[l];", None,
     [(pins.test_adjust_four_cases, {})]),
    ("ffn_output_weights_transposed", "acc += h[j] * elem(W_out, dtype, (size_t)i * d_ff + j);",
     "acc += h[j] * elem(W_out, dtype, (size_t)j * d_model + i);", None,
     [(pins.test_sparse_ffn_is_masked_matrix_product, {})]),
    ("nested_counts_strict", "c += !(scores[j] < taus[k]);", "c += (scores[j] > taus[k]);", None,
     [(pins.test_nested_lists_equal_the_masks, {})]),
    ("nested_order_ascending", "if (p->a > q->a) return -1;", "if (p->a > q->a) return 2;", None,
     [(pins.test_nested_lists_equal_the_masks, {})]),
    ("level_bits_swapped", "return (surprisal > tau_s ? 1 : 0) + (entropy > tau_H ? 2 : 0);",
     "return (surprisal > tau_s ? 2 : 0) + (entropy > tau_H ? 1 : 0);", None,
     [(pins.test_load_level_indexes_the_four_thresholds, {})]),
    ("round_down_not_nearest", "nearbyint(v / quantum)", "floor(v / quantum)", None,
     [(pins.test_round_storage_matches_library_casts, {})]),
    ("down_proj_transposed", "acc += Z[(size_t)t * d_ff + j] * elem(W_out, dtype, (size_t)i * d_ff + j);",
     "acc += Z[(size_t)t * d_ff + j] * elem(W_out, dtype, (size_t)j * d_model + i);", None,
     [(pins.test_down_proj_worked_example, {})]),
    ("cett_cut_order_descending", "if (x->a < y->a) return -1;\n    if (x->a > y->a) return 1;",
     "if (x->a < y->a) return 1;\n    if (x->a > y->a) return -1;", None,
     [(pins.test_cett_curve_matches_definition, {})]),
    ("half_exponent_bias", "ldexp(1.0 + (double)frac / 1024.0, ex - 15)", "ldexp(1.0 + (double)frac / 1024.0, ex - 16)", None,
     [(pins.test_fp16_and_bf16_widening_every_bit_pattern, {})]),
]


def _build_mutant(tmp_path, name, old, new, which):
    src = open(SRC).read()
    assert src.count(old) >= 1, f"mutation {name}: the text to replace is not in the oracle any more"
    if which is None:
        mutated = src.replace(old, new)
    else:
        parts = src.split(old)
        mutated = old.join(parts[:which + 1]) + new + old.join(parts[which + 1:])
    c_path = os.path.join(tmp_path, f"oracle_{name}.c")
    so_path = os.path.join(tmp_path, f"liboracle_{name}.so")
    with open(c_path, "w") as f:
        f.write(mutated)
    subprocess.run(["gcc", "-O1", "-std=c99", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
                    c_path, "-o", so_path, "-lm"], check=True)
    spec = importlib.util.spec_from_file_location(f"clada_oracle_mutant_{name}", FRONT)
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    mod._SRC, mod._LIB, mod._lib = c_path, so_path, None     # the front end loads the mutant instead
    return mod


@pytest.mark.parametrize("name,old,new,which,watchers", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_a_planted_mistake_fails_a_pin(tmp_path, name, old, new, which, watchers):
    mutant = _build_mutant(str(tmp_path), name, old, new, which)
    caught = []
    for pin, kwargs in watchers:
        try:
            pin(mutant, **kwargs)
        except AssertionError:
            caught.append(pin.__name__)
    assert caught, f"no pin noticed the planted mistake '{name}'"


def test_the_unmutated_copy_passes_the_same_pins(tmp_path):
    """The harness itself: a copy without a mistake passes every pin used above."""
    clean = _build_mutant(str(tmp_path), "clean", "return silu(g) * u;", "return silu(g) * u;", None)
    seen = set()
    for _, _, _, _, watchers in MUTATIONS:
        for pin, kwargs in watchers:
            key = (pin.__name__, tuple(sorted(kwargs.items())))
            if key in seen:
                continue
            seen.add(key)
            pin(clean, **kwargs)
