"""Shows that the pin suite catches plausible mistakes: each case below alters one expression in a
temporary copy of the oracle's C source, builds it, and expects the pin suite to fail on it.
Mistakes are planted only in these CPU copies; the committed oracle is untouched."""
import os
import subprocess

import pytest

import pins
import oracle

SRC = os.path.join(os.path.dirname(oracle.__file__), "moc_oracle.c")

MUTANTS = {
    # interval end exclusive instead of inclusive (Eq. 4)
    "free_exclusive": ("delta[fr[p] + 1] -= g->m[seq[p]];", "delta[fr[p]] -= g->m[seq[p]];"),
    # sink released with its own step
    "sink_not_kept": ("if (!g->has_succ[v]) fr[last[v]] = T - 1;", ";"),
    # every step charged to the FIRST copy of the predecessor instead of the newest
    "oldest_copy": ("last[v] = t;\n    }", "if (last[v] < 0) last[v] = t;\n    }"),
    # predecessor/successor transposed when building the lists
    "transposed_edges": ("g->pred_start[edges[2 * e + 1] + 1]++;", "g->pred_start[edges[2 * e] + 1]++;"),
    # duration counts each node once
    "dur_no_recompute": ("for (int32_t t = 0; t < T; ++t) dur += g->w[seq[t]];",
                         "for (int32_t v = 0; v < n; ++v) dur += g->w[v];"),
    # budget test strict
    "budget_strict": ("(peak <= M) ? 1 : 0", "(peak < M) ? 1 : 0"),
    # free step never extended (dropped term)
    "no_extension": ("else if (fr[last[u]] < t) fr[last[u]] = t;", "else {}"),
    # missing predecessor not detected
    "no_violation": ("if (last[u] < 0) violated = 1;", "if (last[u] < 0) {}"),
    # allocation one step late
    "alloc_late": ("delta[p] += g->m[seq[p]];", "delta[p + 1] += g->m[seq[p]];"),
    # copy-count cap ignored
    "no_cap": ("if (count[v] < 1 || count[v] > (g->cap ? g->cap[v] : g->C)) ok = 0;", "if (count[v] < 1) ok = 0;"),
    # per-node caps ignored
    "node_caps_ignored": ("count[v] > (g->cap ? g->cap[v] : g->C)", "count[v] > g->C"),
    # wrong weight array in the profile
    "w_for_m": ("delta[p] += g->m[seq[p]];\n        delta[fr[p] + 1] -= g->m[seq[p]];",
                "delta[p] += g->w[seq[p]];\n        delta[fr[p] + 1] -= g->w[seq[p]];"),
}


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_mutant_is_caught(name, tmp_path):
    old, new = MUTANTS[name]
    src = open(SRC).read()
    assert src.count(old) == 1, f"mutation site for {name} not found exactly once"
    if name == "transposed_edges":
        # transpose consistently: swap the roles of the two endpoints everywhere in the builder
        mutated = src.replace("int32_t u = edges[2 * e], v = edges[2 * e + 1];\n        g->pred[fill[v]++] = u;",
                              "int32_t v = edges[2 * e], u = edges[2 * e + 1];\n        g->pred[fill[v]++] = u;")
        mutated = mutated.replace(old, new)
    else:
        mutated = src.replace(old, new)
    assert mutated != src
    c = tmp_path / "mutant.c"
    so = tmp_path / "mutant.so"
    c.write_text(mutated)
    subprocess.run(["gcc", "-O1", "-std=c11", "-shared", "-fPIC", "-pthread", "-I", os.path.dirname(SRC), "-o", str(so), str(c)], check=True)
    lib = oracle.load_library(str(so))

    def make_graph(n, edges, w, m, C):
        return oracle.OracleGraph(n, edges, w, m, C, lib=lib)

    with pytest.raises(AssertionError):
        pins.run_all(make_graph)
