"""Planted mistakes: each mutant of the oracle source must be caught by at least one pin.

The mistake is planted in a temporary copy of the oracle's C source, on the CPU; the
pins of test_oracle_pins.py are then re-run against the mutant library."""
import ctypes
import os
import subprocess

import pytest

import oracle
import test_oracle_pins as pins

MUTANTS = {
    "scale_dropped": ("s[j] = scale * acc;", "s[j] = acc;"),
    "not_normalised": ("REAL p = s[j] / denom;", "REAL p = s[j];"),
    "value_dims_reversed": ("out[d] += p * widen(V[(size_t)j * hd + d]);",
                            "out[d] += p * widen(V[(size_t)j * hd + (hd - 1 - d)]);"),
    "query_dims_reversed": ("acc += widen(q[d]) *", "acc += widen(q[hd - 1 - d]) *"),
    "key_used_as_value": ("out[d] += p * widen(V[", "out[d] += p * widen(K["),
    "causal_excludes_self": ("Kb, Vb, t + 1, hd", "Kb, Vb, t, hd"),
    "causal_sees_one_ahead": ("Kb, Vb, t + 1, hd", "Kb, Vb, (t + 2 > T ? T : t + 2), hd"),
    "decode_drops_last_row": ("int n = len[b];", "int n = len[b] - 1;"),
    "decode_reads_one_past": ("int n = len[b];", "int n = len[b] + 1;"),
    "token_excludes_itself": ("int n = appended ? len_old + i + 1 : len_old - n_q + i + 1;",
                              "int n = appended ? len_old + i : len_old - n_q + i + 1;"),
    "attend_only_not_causal": ("int n = appended ? len_old + i + 1 : len_old - n_q + i + 1;",
                               "int n = appended ? len_old + i + 1 : len_old;"),
    "attend_only_counts_from_the_start": ("int n = appended ? len_old + i + 1 : len_old - n_q + i + 1;",
                                          "int n = appended ? len_old + i + 1 : i + 1;"),
    "linear_weight_transposed": ("widen(W[(size_t)o * K + k])", "widen(W[((size_t)k * N + o) % ((size_t)N * K)])"),
    "linear_bias_dropped": ("REAL acc = bias ? widen(bias[o]) : (REAL)0;", "REAL acc = 0;"),
    "linear_bias_of_wrong_feature": ("REAL acc = bias ? widen(bias[o]) : (REAL)0;", "REAL acc = bias ? widen(bias[(o + 1) % N]) : (REAL)0;"),
    "rounding_truncates": ("double q = nearbyint(ldexp(a, 7 - e));", "double q = floor(ldexp(a, 7 - e));"),
    "rounding_ties_away": ("double q = nearbyint(ldexp(a, 7 - e));", "double q = floor(ldexp(a, 7 - e) + 0.5);"),
    "projection_k_and_v_swapped": ("k_new[o] = round_to_bf16(row[D + h * hd + d]);\n                    v_new[o] = round_to_bf16(row[2 * D + h * hd + d]);",
                                   "k_new[o] = round_to_bf16(row[2 * D + h * hd + d]);\n                    v_new[o] = round_to_bf16(row[D + h * hd + d]);"),
    "projection_q_not_grouped_by_head": ("size_t o = ((((size_t)b * H + h) * n) + i) * hd + d;   /* [B][H][n][hd] */",
                                         "size_t o = ((((size_t)b * n + i) * H) + h) * hd + d;"),
    "projection_takes_k_for_q": ("q_out[o] = row[h * hd + d];", "q_out[o] = row[D + h * hd + d];"),
    "projection_reset_ignored": ("if (reset_mask ? (reset_mask[b] != 0) : (reset_first != 0)) len[b] = 0;\n    FN(bto_kv_append)", ";\n    FN(bto_kv_append)"),
    "projection_rows_of_wrong_token": ("const REAL* row = y + ((size_t)b * n + i) * 3 * D;", "const REAL* row = y + ((size_t)b * n + (n - 1 - i)) * 3 * D;"),
    "token_reset_ignored": ("if (do_reset) len[b] = 0;", ";"),
    "append_ignores_length": ("* cap + (size_t)(len[b] + i)) * hd;", "* cap + (size_t)(i)) * hd;"),
    "append_no_length_update": ("        len[b] += n_new;", "        ;"),
    "prefill_ignores_stride": ("(size_t)bh * (size_t)kv_seq_stride * hd;", "(size_t)bh * (size_t)T * hd;"),
    "heads_swapped_in_decode": ("attend_rows(q + bh * hd, kc + bh * cap * hd,",
                                "attend_rows(q + ((size_t)b * H + (H - 1 - h)) * hd, kc + bh * cap * hd,"),
}

PIN_FUNCS = [
    pins.test_single_row_returns_its_value_exactly,
    pins.test_equal_keys_give_mean_of_values,
    pins.test_two_rows_is_a_logistic_blend,
    pins.test_handmade_scores_one_two_three,
    pins.test_dominant_key_selects_its_value,
    lambda: pins.test_probabilities_sum_to_one_and_hull(5),
    lambda: pins.test_brute_force_tiny(6, 8),
    pins.test_prefill_matches_library_causal_attention,
    pins.test_prefill_honours_kv_stride,
    pins.test_cached_decode_equals_full_recompute,
    pins.test_block_length_one_is_vanilla_causal_attention,
    pins.test_ragged_lengths_and_rows_past_len_are_ignored,
    pins.test_spike_row_at_the_length_boundary,
    pins.test_append_overflow_and_empty_cache,
    lambda: pins.test_token_decoder_never_crosses_a_block_boundary(4, 2),
    pins.test_token_step_equals_attention_over_prefix_plus_same_block_tokens,
    pins.test_token_attend_only_and_masked_reset,
    pins.test_attend_only_over_the_last_rows_equals_the_appending_step,
    pins.test_round_to_bf16_is_nearest_even,
    pins.test_linear_identity_one_hot_zero_input_and_library_product,
    pins.test_prefix_projection_layout,
    pins.test_qkv_projection_with_identity_blocks_caches_the_input_rows,
    pins.test_project_then_append_equals_append_of_projected_rows,
    pins.test_qkv_projection_reset_is_the_block_boundary_reset,
    pins.test_projected_step_equals_appending_step_on_projected_rows,
]


def build_mutant(tmp_path, name, old, new):
    src = open(os.path.join(os.path.dirname(oracle.__file__), "bt_oracle.c")).read()
    assert src.count(old) >= 1, f"mutation site for {name} not found"
    mutated = src.replace(old, new)
    c = tmp_path / f"{name}.c"
    c.write_text(mutated)
    objs = []
    for real, sfx in (("double", ""), ("float", "_f32")):
        o = tmp_path / f"{name}{sfx}.o"
        subprocess.check_call(["gcc", "-O1", "-fopenmp", "-fPIC", "-std=c11", f"-DREAL={real}",
                               f"-DSUFFIX={sfx}", "-c", str(c), "-o", str(o)])
        objs.append(str(o))
    so = tmp_path / f"lib{name}.so"
    subprocess.check_call(["gcc", "-shared", "-fopenmp", "-o", str(so)] + objs + ["-lm"])
    return ctypes.CDLL(str(so))


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_mutant_is_caught(name, tmp_path, monkeypatch):
    old, new = MUTANTS[name]
    oracle.lib()  # make sure the real one is built first
    monkeypatch.setattr(oracle, "_lib", build_mutant(tmp_path, name, old, new))
    caught = []
    for f in PIN_FUNCS:
        try:
            f()
        except AssertionError:
            caught.append(getattr(f, "__name__", "pin"))
    assert caught, f"no pin noticed the planted mistake '{name}'"


def test_unmutated_source_passes_the_same_pins():
    for f in PIN_FUNCS:
        f()


# The densified block-decoder step is written in the oracle's Python layer (append, then one plain decode
# per query over a growing prefix): its planted mistakes are edits of that source, run against the pins
# that compare it with dense causal attention.
PY_MUTANTS = {
    "multi_query_sees_one_row_less": ("before + i + 1, before)", "before + i, before)"),
    "multi_query_sees_one_row_more": ("before + i + 1, before)", "np.minimum(before + i + 2, after), before)"),
    "multi_query_not_causal": ("before + i + 1, before)", "after, before)"),
    "multi_query_outputs_shifted": ("out[:, :, i] = block_decode_attn(c, np.ascontiguousarray(q[:, :, i])",
                                    "out[:, :, i] = block_decode_attn(c, np.ascontiguousarray(q[:, :, (i + 1) % m])"),
    "multi_query_rows_not_appended": ("    kv_append(c, k_new, v_new)\n    after = c.len.copy()", "    after = c.len.copy()"),
}


@pytest.mark.parametrize("name", sorted(PY_MUTANTS))
def test_python_layer_mutant_is_caught(name, monkeypatch):
    old, new = PY_MUTANTS[name]
    path = oracle.__file__
    src = open(path).read()
    assert src.count(old) == 1, f"mutation site for {name} not found"
    ns = {"__name__": "oracle", "__file__": path, "__package__": "oracle"}
    exec(compile(src.replace(old, new), path, "exec"), ns)
    monkeypatch.setattr(oracle, "block_decode_step_multi", ns["block_decode_step_multi"])
    caught = []
    for f in (pins.test_densified_step_is_the_matching_rows_of_dense_causal_attention,
              pins.test_densified_step_without_room_appends_nothing):
        try:
            f()
        except AssertionError:
            caught.append(f.__name__)
    assert caught, f"no pin noticed the planted mistake '{name}'"
