"""Pins of the interval-form oracle, and proof that they catch plausible mistakes planted in temporary
copies of its source (CPU only; the committed oracle is untouched)."""
import os
import subprocess

import pytest

import oracle
import interval_pins

HERE = os.path.dirname(oracle.__file__)
SRC = os.path.join(HERE, "moc_interval_oracle.c")
SRC_EVAL = os.path.join(HERE, "moc_oracle.c")


def test_interval_pins():
    interval_pins.run_all(lambda n, e, w, m, C: oracle.OracleGraph(n, e, w, m, C))


MUTANTS = {
    "eq5_not_strict": ("s[u * C + j] + 1 <= s[v * C + i]", "s[u * C + j] <= s[v * C + i]"),
    "eq5_end_exclusive": ("s[v * C + i] <= e[u * C + j]) found = 1;", "s[v * C + i] < e[u * C + j]) found = 1;"),
    "eq5_inactive_producer": ("if (a[u * C + j] && s[u * C + j] + 1", "if (s[u * C + j] + 1"),
    "eq5_inactive_consumer": ("                if (!a[v * C + i]) continue;\n                int found", "                int found"),
    "eq4_end_exclusive": ("s[v * C + i] <= t && t <= e[v * C + i]) use", "s[v * C + i] <= t && t < e[v * C + i]) use"),
    "eq4_counts_inactive": ("if (a[v * C + i] && s[v * C + i] <= t", "if (s[v * C + i] <= t"),
    "eq4_strict_budget": ("if (peak > M) mask", "if (peak >= M) mask"),
    "eq3_wrong_neighbour": ("e[v * C + i] > s[v * C + i + 1]", "s[v * C + i] > s[v * C + i + 1]"),
    "eq2_active_only": ("if (s[v * C + i] > e[v * C + i]) mask", "if (a[v * C + i] && s[v * C + i] > e[v * C + i]) mask"),
    "eq6_same_node_too": ("for (int32_t u = v + 1; u < n; ++u)", "for (int32_t u = v; u < n; ++u)"),
    "eq6_active_only": ("if (s[v * C + i] == s[u * C + j]) mask", "if (a[v * C + i] && a[u * C + j] && s[v * C + i] == s[u * C + j]) mask"),
    "eq7_any_slot": ("if (a[v * C] != 1) mask", "if (a[v * C] != 1 && a[v * C + 1] != 1) mask"),
    "dur_counts_inactive": ("if (a[v * C + i]) dur += g->w[v];", "dur += g->w[v];"),
    "dur_uses_m": ("if (a[v * C + i]) dur += g->w[v];", "if (a[v * C + i]) dur += g->m[v];"),
    "stage_offset": ("j * (j - 1) / 2 + k) ok = 1;", "j * (j + 1) / 2 + k) ok = 1;"),
    "stage_first_free": ("if (s[v * C] != k * (k + 1) / 2) mask |= BIT_STAGE;", ";"),
    "domain_zero_allowed": ("k < n * C; ++k)\n        if (s[k] < 1 ||", "k < n * C; ++k)\n        if (s[k] < 0 ||"),
    "sequence_by_node_order": ("for (int64_t t = 1; t <= D; ++t) {\n        int32_t here = 0;", "for (int64_t t = D; t >= 1; --t) {\n        int32_t here = 0;"),
}


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_interval_mutant_is_caught(name, tmp_path):
    old, new = MUTANTS[name]
    src = open(SRC).read()
    assert src.count(old) == 1, f"mutation site for {name} not found exactly once"
    c = tmp_path / "mutant.c"
    so = tmp_path / "mutant.so"
    c.write_text(src.replace(old, new))
    subprocess.run(["gcc", "-O1", "-std=c11", "-shared", "-fPIC", "-pthread", "-I", HERE, "-o", str(so), str(c), SRC_EVAL],
                   check=True)
    lib = oracle.load_library(str(so))
    with pytest.raises(AssertionError):
        interval_pins.run_all(lambda n, e, w, m, C: oracle.OracleGraph(n, e, w, m, C, lib=lib))
