"""Do the pins bite?  Each case plants one plausible mistake in a COPY of the oracle's C source
(on the CPU, in a temporary directory), builds it, points the oracle's Python wrapper at the mutant
and runs the pins: at least one of them must fail.  The real oracle is untouched."""
import ctypes as C
import os
import subprocess

import pytest

from oracle import spd_oracle as orc
from tests import test_oracle_pins as pins

SRC = os.path.join(os.path.dirname(orc.__file__), "spd_oracle.c")

# (name, text to find, replacement, how many occurrences to replace: 0 = all)
MUTANTS = [
    ("scale dropped", "out[t] = s->sm_scale * acc;", "out[t] = acc;", 0),
    ("head map interleaved", "int kvh = h / (s->num_q_heads / s->num_kv_heads);", "int kvh = h % s->num_kv_heads;", 0),
    ("head map in V fetch", "int kvh = h / g;", "int kvh = h % s->num_kv_heads;", 0),
    ("page and slot swapped", "kv->page_indptr[u] + t / P]", "kv->page_indptr[u] + t % P]", 0),
    ("slot ignored", "* P + t % P) * D", "* P) * D", 0),
    ("kv-head stride lost", "(page * s->num_kv_heads + kvh)", "(page + kvh)", 0),
    ("bf16 widened one bit short", ") << 16;", ") << 15;", 0),
    ("V read from K", "widen(kv->v_pool, ro + d, s->dtype)", "widen(kv->k_pool, ro + d, s->dtype)", 0),
    ("partitions swapped in full", "const oracle_kv *kv = i < n_in ? priv : pub;", "const oracle_kv *kv = i < n_in ? pub : priv;", 0),
    ("partial denominator off", "l[idx] = den;", "l[idx] = den + 1.0;", 0),
    ("partial keeps a stale max", "m[idx] = mx;", "m[idx] = mx + 0.5;", 0),
    ("merge weight inverted", "exp(mc - M)", "exp(M - mc)", 0),
    ("merge forgets the weight on l", "L += w * parts_l[c * rows + r];", "L += parts_l[c * rows + r];", 0),
    ("merge forgets the weight on O", "o_out[r * D + d] += w * parts_o", "o_out[r * D + d] += parts_o", 0),
    ("alpha applied the wrong way", "(l_in[r] + alpha * l_out[r])", "(l_in[r] + l_out[r] / alpha)", 0),
    ("prefill: first token sees nothing", "n = i - first + 1;", "n = i - first;", 0),
    ("prefill: user boundary off by one", "tok_indptr[u + 1] <= i) ++u;", "tok_indptr[u + 1] < i) ++u;", 0),
    ("prefill: scale dropped", "sc[j] = s->sm_scale * acc;", "sc[j] = acc;", 0),
    ("prefill: values in reverse order", "widen(v, ((first + j) * Hkv + kvh) * D + d, s->dtype);", "widen(v, ((first + n - 1 - j) * Hkv + kvh) * D + d, s->dtype);", 0),
    ("range lower bound ignored", "for (int64_t t = tok_lo; t < hi; ++t) {\n                double p", "for (int64_t t = 0; t < hi; ++t) {\n                double p", 0),
]

BATTERY = [
    pins.test_golden_hand_example,
    lambda: pins.test_brute_force_tiny(4, 2, 8),
    pins.test_split_point_identity_every_split,
    pins.test_nway_and_nested_merge,
    pins.test_alpha_form_matches_max_form,
    pins.test_uniform_scores_give_mean_of_v,
    pins.test_single_key_returns_its_value,
    pins.test_matches_dense_numpy_and_torch_sdpa,
    pins.test_gqa_head_map_is_contiguous_groups,
    pins.test_indexing_probe_one_hot_query,
    pins.test_bf16_bits_are_widened_exactly_and_page_shuffle_is_invisible,
    pins.test_prefill_is_causal_softmax_and_hands_over_to_decode,
]


def _pins_pass() -> bool:
    for check in BATTERY:
        try:
            check()
        except (AssertionError, FloatingPointError, ValueError, IndexError, ZeroDivisionError):
            return False
    return True


def test_unmutated_source_passes_the_battery():
    orc._load()
    assert _pins_pass()


@pytest.mark.parametrize("name,find,repl,_n", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(tmp_path, monkeypatch, name, find, repl, _n):
    text = open(SRC).read()
    assert find in text, f"mutation target vanished from the oracle source: {find!r}"
    mutant_c = tmp_path / "mutant.c"
    mutant_c.write_text(text.replace(find, repl))
    mutant_so = tmp_path / "libmutant.so"
    subprocess.check_call(["gcc", "-O1", "-fopenmp", "-shared", "-fPIC", "-o", str(mutant_so), str(mutant_c), "-lm"])
    lib = C.CDLL(str(mutant_so))
    lib.spd_oracle_num_threads.restype = C.c_int
    orc._load()
    monkeypatch.setattr(orc, "_lib", lib)
    import numpy as np
    with np.errstate(all="ignore"):
        assert not _pins_pass(), f"no pin noticed: {name}"
