"""Each planted mistake in a *copy* of the oracle's source must trip at least one pin.

The mistakes are planted on the CPU, in a temporary copy of the oracle's C file; the
committed oracle is never touched.  This shows that the pins in test_oracle_pins.py are
sharp enough to catch the plausible errors (dropped scale, wrong GQA map, off-by-one
causal limit, wrong span edge, wrong page arithmetic, steer sign, missing normalisation).
"""
import ctypes
import os
import subprocess

import pytest

from oracle import oracle
from oracle.build import SRC
from tests import test_oracle_pins as pins

MUTATIONS = {
    "dropped_scale": ("p[t] = scale * dot;", "p[t] = dot;"),
    "gqa_map_modulo": ("const int g = h / group;", "const int g = h % num_kv_heads;"),
    "causal_sees_one_more": ("const int pos = seq_lens[s] - n_s + i;",
                             "const int pos = seq_lens[s] - n_s + i + 1 < seq_lens[s] ? seq_lens[s] - n_s + i + 1 : seq_lens[s] - 1;"),
    "causal_top_left": ("const int pos = seq_lens[s] - n_s + i;", "const int pos = i;"),
    "span_hi_edge": ("if (hi > pos + 1) hi = pos + 1;", "if (hi > pos) hi = pos;"),
    "span_lo_edge": ("for (int t = lo; t < hi; ++t) acc += p[t];",
                     "for (int t = lo + 1; t < hi; ++t) acc += p[t];"),
    "page_slot_shifted": ("const uint16_t *vrow = v_cache + page * kv_block_stride\n"
                          "                                       + (int64_t)(t % page_size) * kv_token_stride",
                          "const uint16_t *vrow = v_cache + page * kv_block_stride\n"
                          "                                       + (int64_t)((t + 1) % page_size) * kv_token_stride"),
    "steer_sign": ("o[d] += (double)alpha[h]", "o[d] -= (double)alpha[h]"),
    "no_normalisation": ("for (int t = 0; t <= pos; ++t) p[t] /= z;", ""),
    "exponent_doubled": ("p[t] = exp(p[t] - mx);", "p[t] = exp(2.0 * (p[t] - mx));"),
}

PIN_FUNCS = [
    lambda: pins.test_brute_force_materialised_matrix(dict(seq_lens=(37, 48, 5), q_lens=(37, 9, 1), Hq=4, Hkv=2, D=8)),
    pins.test_identical_keys_give_uniform_attention,
    pins.test_first_row_returns_first_value_plus_steer,
    pins.test_two_keys_sigmoid,
    pins.test_partition_sums_to_one_and_additivity,
    pins.test_alpha_zero_is_identity_and_steer_is_additive,
    pins.test_decode_equals_last_prefill_row_and_chunk_equals_rows,
    pins.test_scale_is_applied_to_the_logits,
    lambda: pins.test_hooks_off_matches_scaled_dot_product_attention(8, 2, 64),
]


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(name, tmp_path, monkeypatch):
    old, new = MUTATIONS[name]
    src = open(SRC).read()
    assert src.count(old) >= 1, f"mutation anchor for {name} not found in the oracle source"
    mutated = tmp_path / "mutant.c"
    mutated.write_text(src.replace(old, new, 1))
    lib_path = tmp_path / "libmutant.so"
    subprocess.run(["gcc", "-O1", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", str(lib_path),
                    str(mutated), "-lm"], check=True)
    lib = ctypes.CDLL(str(lib_path))
    lib.hook_attn_oracle.restype = ctypes.c_int
    lib.hook_attn_oracle_threads.restype = ctypes.c_int
    oracle._load()
    monkeypatch.setattr(oracle, "_lib", lib)
    caught = 0
    for f in PIN_FUNCS:
        try:
            f()
        except (AssertionError, ValueError):
            caught += 1
    assert caught >= 1, f"no pin noticed the planted mistake '{name}'"
