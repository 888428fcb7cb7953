"""Each plausible mistake, planted in a copy of the oracle on the CPU, must trip a pin.

The copies are made by editing the oracle's C text, compiled to a temporary shared
object and run through the same pins as the real oracle.  A mutant that survives
means the pins would not have noticed that mistake in the real oracle either.
"""
import os

import pytest

import oracle
import oracle_pins
from oracle import liec_oracle as wrapper

MUTANTS = {
    "sign_of_zero_negative": ("int neg = xs[j] < 0.0f;", "int neg = xs[j] <= 0.0f;"),
    "bit_order_reversed": ("(uint32_t)1 << (j % 32)", "(uint32_t)1 << (31 - j % 32)"),
    "segment_word_offset_dropped": ("words[woff + j / 32] |=", "words[j / 32] |="),
    "scale_not_divided": ("double mean = S / (double)n;", "double mean = S;"),
    "scale_without_abs": ("if (a < 0.0f) a = -a;", ""),
    "scale_summed_in_binary32": ("double left = tree_node", "float left = tree_node"),
    "scale_running_sum": ("double left = tree_node(x, n, lo, len / 2);\n    double right = tree_node(x, n, lo + len / 2, len / 2);\n    return left + right;",
                          "double s = 0.0; for (int64_t q = lo; q < lo + len && q < n; ++q) s += (double)(x[q] < 0 ? -x[q] : x[q]);\n    return s;"),
    "decoded_sign_flipped": ("dec[off[t] + j] = neg ? -s : s;", "dec[off[t] + j] = neg ? s : -s;"),
    "topk_smallest_first": ("return p->key > q->key ? -1 : 1;", "return p->key > q->key ? 1 : -1;"),
    "topk_tie_higher_index": ("return p->pos < q->pos ? -1 : 1;", "return p->pos < q->pos ? 1 : -1;"),
    "topk_signed_key": ("& 0x7fffffffu", "& 0xffffffffu"),
    "topk_segment_relative_index": ("idx[out] = (uint32_t)(off[t] + j);", "idx[out] = (uint32_t)j;"),
    "mean_not_divided": ("float mean = acc / (float)N;", "float mean = acc;"),
    "global_error_not_added": ("v[j] = e[j] + mean;", "v[j] = mean;"),
    "global_error_subtracted": ("v[j] = e[j] + mean;", "v[j] = e[j] - mean;"),
    "workers_summed_backwards": ("acc = acc + P[(size_t)i * d + j];", "acc = acc + P[(size_t)(N - 1 - i) * d + j];"),
    "downlink_compresses_error": ("rc = compress(down, v, d, T, off, k, down_set,", "rc = compress(down, e, d, T, off, k, down_set,"),
    "error_update_sign": ("e[j] = v[j] - p[j];", "e[j] = p[j] - v[j];"),
    "compensation_sign": ("float diff = p[j] - pi[j];", "float diff = pi[j] - p[j];"),
    "compensation_dropped": ("const float *pi = P + (size_t)i * d;", "const float *pi = g;"),
    "gradient_subtracted": ("float u = diff + g[j];", "float u = diff - g[j];"),
    "learning_rate_dropped": ("float step = lr * u;", "float step = u;"),
    "averaging_keeps_local_model": ("x[j] = xbar[j] - scaled;", "x[j] = x[j] - scaled;"),
    "averaging_forgets_error": ("v[j] = e[j] + gmean;", "v[j] = gmean;"),
    "averaging_keeps_error": ("e[j] = v[j] - v[j];", "e[j] = e[j];"),
    "mean_model_not_divided": ("xbar[j] = acc / (float)N;", "xbar[j] = acc;"),
    "sumsq_running_sum": ("double left = tree_sq_node(x, n, lo, len / 2);\n    double right = tree_sq_node(x, n, lo + len / 2, len / 2);\n    return left + right;",
                          "double s = 0.0; for (int64_t q = lo; q < lo + len && q < n; ++q) s += (double)x[q] * (double)x[q];\n    return s;"),
    "sumsq_summed_in_binary32": ("double left = tree_sq_node", "float left = tree_sq_node"),
    "bf16_widened_into_low_half": ("uint32_t u = (uint32_t)in[j] << 16;", "uint32_t u = (uint32_t)in[j];"),
    "sumsq_not_squared": ("return a * a;                  /* exact: 24-bit significands */", "return a < 0 ? -a : a;"),
    "randk_value_from_slot_not_index": ("val[q] = x[j];", "val[q] = x[q];"),
    "randk_segment_check_dropped": ("if (j < off[t] || j >= off[t + 1]) return -3;", ""),
    "randk_order_check_dropped": ("if (r > 0 && set[q - 1] >= set[q]) return -3;", ""),
    "randk_every_worker_uses_first_subset": ("up_sets ? up_sets + (size_t)i * K : NULL", "up_sets"),
    "randk_downlink_uses_uplink_subset": ("rc = compress(down, v, d, T, off, k, down_set,", "rc = compress(down, v, d, T, off, k, up_sets,"),
    "philox_nine_rounds": ("for (int r = 0; r < 10; ++r) {", "for (int r = 0; r < 9; ++r) {"),
    "philox_multipliers_swapped": ("const uint64_t p0 = (uint64_t)0xD2511F53u * c[0];\n    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c[2];",
                                   "const uint64_t p0 = (uint64_t)0xCD9E8D57u * c[0];\n    const uint64_t p1 = (uint64_t)0xD2511F53u * c[2];"),
    "philox_key_bumped_before_first_round": ("if (r > 0) { k[0] += 0x9E3779B9u; k[1] += 0xBB67AE85u; }", "{ k[0] += 0x9E3779B9u; k[1] += 0xBB67AE85u; }"),
    "philox_halves_not_crossed": ("const uint32_t n0 = hi1 ^ c[1] ^ k[0];\n    const uint32_t n2 = hi0 ^ c[3] ^ k[1];",
                                  "const uint32_t n0 = hi0 ^ c[1] ^ k[0];\n    const uint32_t n2 = hi1 ^ c[3] ^ k[1];"),
    "subset_words_in_reverse_order": ("scores[j] = out[j % 4] >> 2;", "scores[j] = out[3 - j % 4] >> 2;"),
    "subset_score_keeps_31_bits": ("scores[j] = out[j % 4] >> 2;", "scores[j] = out[j % 4] >> 1;"),
    "subset_row_and_epoch_swapped": ("const uint32_t ctr[4] = { (uint32_t)(j / 4), t, row, epoch };", "const uint32_t ctr[4] = { (uint32_t)(j / 4), t, epoch, row };"),
    "subset_one_block_per_element": ("const uint32_t ctr[4] = { (uint32_t)(j / 4), t, row, epoch };", "const uint32_t ctr[4] = { (uint32_t)j, t, row, epoch };"),
    "subset_seed_high_half_ignored": ("(uint32_t)(seed >> 32) };", "0u };"),
    "subset_lowest_scores": ("return p->score > q->score ? -1 : 1;", "return p->score > q->score ? 1 : -1;"),
    "subset_tie_higher_index": ("return p->pos > q->pos ? 1 : -1;", "return p->pos > q->pos ? -1 : 1;"),
    "subset_not_sorted": ("qsort(subset, (size_t)k, sizeof(uint32_t), by_value);", ""),
    "subset_indices_segment_relative": ("for (int64_t r = 0; r < k[t]; ++r) dst[r] += (uint32_t)off[t];   /* flat index */", ""),
    "subset_same_for_every_row": ("liec_oracle_subset_scores(seed, epoch, (uint32_t)row, (uint32_t)t, n, scores);", "liec_oracle_subset_scores(seed, epoch, 0u, (uint32_t)t, n, scores);"),
    "ascent_instead_of_descent": ("x[j] = x[j] - step;", "x[j] = x[j] + step;"),
}


def _failures(L):
    failed = []
    for pin in oracle_pins.ALL_PINS:
        try:
            pin(L)
        except AssertionError:
            failed.append(pin.__name__)
    return failed


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_mutant_is_caught(name, tmp_path):
    old, new = MUTANTS[name]
    with open(wrapper._SRC) as fh:
        text = fh.read()
    assert text.count(old) == 1, f"mutation site for {name} not found exactly once"
    src = tmp_path / "mutant.c"
    src.write_text(text.replace(old, new))
    out = str(tmp_path / "libmutant.so")
    import subprocess
    subprocess.run(["gcc", *wrapper.CFLAGS, "-w", str(src), "-o", out], check=True)
    failed = _failures(oracle.lib(out))
    assert failed, f"mutant {name} passed every pin"


def test_real_oracle_passes_every_pin():
    assert _failures(oracle.lib()) == []
