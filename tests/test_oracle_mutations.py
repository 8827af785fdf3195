"""Are the oracle's pins sharp?  Plant plausible mistakes in a copy of the oracle's C source
(on the CPU, never in the CUDA path), build it, and check that at least one pin fails for
every one of them, while the unmodified source passes them all."""
import ctypes
import os
import subprocess

import pytest

import oracle
import test_oracle_mask as pins_mask
import test_oracle_round as pins_round

SRC = os.path.join(os.path.dirname(oracle.__file__), "saps_oracle.c")

PINS = [
    pins_mask.test_golden_mix, pins_mask.test_golden_round_key, pins_mask.test_golden_hash,
    pins_mask.test_golden_threshold, pins_mask.test_golden_first_and_last_columns,
    pins_mask.test_mask_matches_hash_and_threshold, pins_mask.test_threshold_comparison_is_strict,
    lambda: pins_mask.test_density_within_binomial_5_sigma(1 << 20, 0.25),
    pins_round.test_worked_example, pins_round.test_full_mask_no_gradient_is_dense_product_with_W,
    pins_round.test_empty_mask_is_axpy, pins_round.test_unmasked_coordinates_untouched_bit_for_bit,
    pins_round.test_pair_sum_preserved_to_one_rounding, pins_round.test_lemma_1_mask_and_gossip_commute,
    lambda: pins_round.test_hypercube_consensus(8), pins_round.test_pack_definition,
    pins_round.test_unfused_wire_path_equals_the_round, pins_round.test_eq7_order_is_the_matrix_form,
    pins_round.test_eq7_order_reductions, pins_round.test_unpack_avg_is_the_receiving_side_of_the_round,
    pins_round.test_consensus_distance_closed_forms,
]

# (what the mistake is, text to replace, replacement)
MUTATIONS = [
    ("merge replaces instead of averaging", "float v = 0.5f * s;", "float v = a[(size_t)j * N + k];"),
    ("factor 1/2 dropped", "float v = 0.5f * s;", "float v = s;"),
    ("difference instead of sum in the average", "float s = a[(size_t)i * N + k] + a[(size_t)j * N + k];",
     "float s = a[(size_t)i * N + k] - a[(size_t)j * N + k];"),
    ("SGD step with the wrong sign", "x[(size_t)i * N + k] = x[(size_t)i * N + k] - step;",
     "x[(size_t)i * N + k] = x[(size_t)i * N + k] + step;"),
    ("only one peer of a pair is updated", "            a[(size_t)j * N + k] = v;\n", ""),
    ("mask inverted", "if (!m[k])\n                continue;\n            float s", "if (m[k])\n                continue;\n            float s"),
    ("hash: second multiplier replaced by the first", "    v *= ORC_M2;\n    v ^= k1;", "    v *= ORC_M1;\n    v ^= k1;"),
    ("hash: round key k1 not mixed in", "    v ^= k1;\n", ""),
    ("hash: wrong shift", "    v ^= k1;\n    v ^= v >> 16;", "    v ^= k1;\n    v ^= v >> 17;"),
    ("key: high word of t ignored", "    a = orc_mix(a ^ (uint32_t)(t >> 32));", "    a = orc_mix(a);"),
    ("threshold compare off by one", "(uint64_t)orc_hash((uint32_t)k, k0, k1) < thr", "(uint64_t)orc_hash((uint32_t)k, k0, k1) <= thr"),
    ("threshold rounds up", "double s = floor(keep_frac * 4294967296.0);", "double s = ceil(keep_frac * 4294967296.0);"),
    ("pack stores the column after the kept one", "idx[r] = (uint32_t)k;", "idx[r] = (uint32_t)k + 1;"),
    ("pack transposes worker and slot", "vals[(size_t)i * cap + r] = a[(size_t)i * N + k];",
     "vals[(size_t)r * n + i] = a[(size_t)i * N + k];"),
    ("pack drops kept zeros", "        if (!m[k])\n            continue;\n        if (r < cap) {",
     "        if (!m[k] || a[k] == 0.0f)\n            continue;\n        if (r < cap) {"),
    ("Eq. 7 order applies the gradient first", "    orc_pair_average(n, N, x, pairs, m);\n    orc_sgd(n, N, x, g, lr);",
     "    orc_sgd(n, N, x, g, lr);\n    orc_pair_average(n, N, x, pairs, m);"),
    ("unpack adds without halving", "x[(size_t)i * N + idx[r]] = 0.5f * s;", "x[(size_t)i * N + idx[r]] = s;"),
    ("consensus distance divides by n - 1", "mean /= (double)n;", "mean /= (double)(n - 1);"),
]


def _build(source: str, path) -> ctypes.CDLL:
    c = path / "mutant.c"
    so = path / f"mutant_{abs(hash(source)) % 10 ** 9}.so"
    c.write_text(source)
    subprocess.run(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-o", str(so), str(c), "-lm"],
                   check=True)
    return oracle._bind(ctypes.CDLL(str(so)))


def _failures(lib, monkeypatch) -> int:
    monkeypatch.setattr(oracle, "_lib", lib)
    failed = 0
    for pin in PINS:
        try:
            pin()
        except AssertionError:
            failed += 1
    return failed


def test_unmodified_source_passes_every_pin(tmp_path, monkeypatch):
    assert _failures(_build(open(SRC).read(), tmp_path), monkeypatch) == 0


@pytest.mark.parametrize("what,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(what, old, new, tmp_path, monkeypatch):
    source = open(SRC).read()
    assert source.count(old) >= 1, f"mutation target not found: {what}"
    mutated = source.replace(old, new, 1)
    assert _failures(_build(mutated, tmp_path), monkeypatch) >= 1, f"no pin noticed: {what}"
