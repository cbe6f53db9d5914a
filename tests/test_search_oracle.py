"""Pins of the search oracle, and proof that they catch plausible mistakes planted in temporary
copies of its source (CPU only; the committed oracle is untouched)."""
import os
import subprocess

import pytest

import oracle
import search_pins

HERE = os.path.dirname(oracle.__file__)
SRC = os.path.join(HERE, "moc_search_oracle.c")
SRC_EVAL = os.path.join(HERE, "moc_oracle.c")


def test_search_pins():
    lib = oracle._load()
    search_pins.run_all(lambda n, e, w, m, C: oracle.OracleGraph(n, e, w, m, C, lib=lib), lib)


MUTANTS = {
    "philox_multipliers_swapped": ("const uint64_t p0 = M0 * c0, p1 = M1 * c2;", "const uint64_t p0 = M1 * c0, p1 = M0 * c2;"),
    "philox_nine_rounds": ("round < 10", "round < 9"),
    "philox_key_not_advanced": ("k0 += W0;", ";"),
    "philox_words_transposed": ("c0 = n0; c1 = n1; c2 = n2; c3 = n3;", "c0 = n2; c1 = n1; c2 = n0; c3 = n3;"),
    "insert_after_instead_of_before": ("child[j] = seq[q];\n        for (int32_t t = j; t < T; ++t) child[t + 1] = seq[t];",
                                       "child[j] = seq[j < T ? j : q]; child[j + (j < T)] = seq[q];\n        for (int32_t t = j + 1; t < T; ++t) child[t + 1] = seq[t];"),
    "insert_range_T": ("(r2 % ((uint32_t)T + 1u))", "(r2 % (uint32_t)T)"),
    "move_range_short": ("(int32_t)(r2 % (uint32_t)T); /* T = len + 1 insertion points */", "(int32_t)(r2 % (uint32_t)(T > 1 ? T - 1 : 1));"),
    "kinds_mask_ignored": ("const uint32_t op = enabled[r0 % k];", "const uint32_t op = r0 % 3u;"),
    "ops_permuted": ("if (op == 1) return len;", "if (op == 2) return len;"),
    "accept_strict": ("return dur_c <= dur_p;", "return dur_c < dur_p;"),
    "accept_ignores_budget": ("const int64_t a = peak_c > M ? peak_c : M, b = peak_p > M ? peak_p : M;\n    if (a != b) return a < b;\n    return dur_c",
                              "const int64_t a = peak_c, b = peak_p;\n    if (a != b) return a < b;\n    return dur_c"),
    "accept_invalid_child": ("if (st_c < 0) return 0;", "if (st_c < -1) return 0;"),
    "counter_transposed": ("{gen, chain0 + (uint32_t)c, e, 0u}", "{chain0 + (uint32_t)c, gen, e, 0u}"),
    "chain_offset_ignored": ("{gen, chain0 + (uint32_t)c, e, 0u}", "{gen, (uint32_t)c, e, 0u}"),
    "sample_not_in_counter": ("{gen, chain0 + (uint32_t)c, e, 0u}", "{gen, chain0 + (uint32_t)c, 0u, e}"),
    "last_sample_wins_ties": ("                              !moc_oracle_accept(cand_pk, cand_du, cand_st, pk, du, st, M))) {", "                              1)) {"),
    "first_valid_sample_taken": ("if (!have || (moc_oracle_accept(pk, du, st, cand_pk, cand_du, cand_st, M) &&", "if (!have || (0 &&"),
    "key_halves_swapped": ("{(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)}", "{(uint32_t)(seed >> 32), (uint32_t)(seed & 0xFFFFFFFFu)}"),
    "fitness_not_updated": ("dur[c] = cand_du;\n", ""),
    "best_last_of_equals": ("(a == b && dur[c] < dur[best])", "(a == b && dur[c] <= dur[best])"),
}


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_search_mutant_is_caught(name, tmp_path):
    old, new = MUTANTS[name]
    src = open(SRC).read()
    assert src.count(old) == 1, f"mutation site for {name} not found exactly once"
    c = tmp_path / "mutant.c"
    so = tmp_path / "mutant.so"
    c.write_text(src.replace(old, new))
    subprocess.run(["gcc", "-O1", "-std=c11", "-shared", "-fPIC", "-pthread", "-I", os.path.dirname(SRC), "-o", str(so), str(c), SRC_EVAL], check=True)
    lib = oracle.load_library(str(so))
    with pytest.raises(AssertionError):
        search_pins.run_all(lambda n, e, w, m, C: oracle.OracleGraph(n, e, w, m, C, lib=lib), lib)
