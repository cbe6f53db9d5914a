"""The pin suite for an oracle implementation: ``run_all(make_graph)`` raises AssertionError when
the implementation disagrees with the paper's worked example, a closed form, the independent
definitions of tests/defs.py or an invariant.  ``make_graph(n, edges, w, m, C)`` must return an
object with ``eval(seq, M) -> dict(peak, dur, status, profile, free)``.

The suite is a function (not only pytest tests) so that deliberately broken variants of the oracle
can be run through it, which shows that each plausible mistake is caught (test_oracle_mutants.py).
"""
from __future__ import annotations

import itertools
import os
import random

import numpy as np

import defs

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
BIG = 1 << 60


def read_golden(name):
    out = {}
    for line in open(os.path.join(GOLDEN, name)):
        line = line.split("#")[0].strip()
        if not line:
            continue
        k, v = line.split(":", 1)
        out[k.strip()] = v.strip()
    return out


def ints(s):
    return [int(x) for x in s.split()]


# ---------------------------------------------------------------- worked example of the paper
def pin_paper_example(make_graph):
    g = read_golden("paper_fig2_worked_example.txt")
    n = int(g["n"])
    e = ints(g["edges"])
    edges = list(zip(e[0::2], e[1::2]))
    m = ints(g["m"])
    seq = ints(g["seq"])
    events = ints(g["filled_events"])
    G = make_graph(n, edges, [2, 3, 4, 5], m, 2)
    r = G.eval(seq, BIG)
    assert r["status"] == 1
    assert r["peak"] == int(g["peak"])
    assert int(np.argmax(r["profile"])) == int(g["peak_step"])
    # usage sets printed in the text: event -> resident node outputs
    for key, val in g.items():
        if key.startswith("usage_event_"):
            step = events.index(int(key.rsplit("_", 1)[1]))
            assert r["profile"][step] == sum(m[v] for v in ints(val))
    assert r["free"][0] == int(g["free_of_step_0"])
    assert list(r["profile"]) == [1, 2, 2, 2, 3]
    assert list(r["free"]) == [1, 2, 4, 4, 4]
    assert r["dur"] == 2 + 3 + 4 + 2 + 5
    # same graph, distinguishable sizes: remat lowers 12 -> 9, and 9 <= M = floor(.8*12) is feasible
    G2 = make_graph(n, edges, [1, 1, 1, 1], [5, 4, 3, 1], 2)
    a = G2.eval([0, 1, 2, 3], 9)
    b = G2.eval(seq, 9)
    assert list(a["profile"]) == [5, 9, 12, 9] and a["peak"] == 12 and a["status"] == 0
    assert list(a["free"]) == [3, 2, 3, 3]
    assert list(b["profile"]) == [5, 9, 7, 8, 9] and b["peak"] == 9 and b["status"] == 1
    assert G2.eval(seq, 8)["status"] == 0


# ---------------------------------------------------------------- closed forms
def pin_chain(make_graph):
    """Line graph (Section 1.1): usage(t) = m[t-1] + m[t]; recomputation cannot lower the peak."""
    rnd = random.Random(5)
    for n in (2, 3, 5, 9):
        m = [rnd.randint(1, 50) for _ in range(n)]
        w = [rnd.randint(1, 9) for _ in range(n)]
        edges = [(i, i + 1) for i in range(n - 1)]
        G = make_graph(n, edges, w, m, 2)
        r = G.eval(list(range(n)), BIG)
        expect = [m[0]] + [m[t - 1] + m[t] for t in range(1, n)]
        assert list(r["profile"]) == expect and r["peak"] == max(expect) and r["dur"] == sum(w)
    n, m = 4, [3, 9, 2, 7]
    G = make_graph(n, [(i, i + 1) for i in range(n - 1)], [1] * n, m, 2)
    base = G.eval(list(range(n)), BIG)["peak"]
    for T in range(n, 2 * n + 1):
        for seq in itertools.product(range(n), repeat=T):
            r = G.eval(list(seq), BIG)
            if r["status"] >= 0:
                assert r["peak"] >= base


def pin_small_cases(make_graph):
    # diamond
    E = [(0, 1), (0, 2), (1, 3), (2, 3)]
    G = make_graph(4, E, [1, 2, 3, 4], [4, 2, 3, 1], 2)
    r = G.eval([0, 1, 2, 3], BIG)
    assert list(r["profile"]) == [4, 6, 9, 6] and r["dur"] == 10
    r = G.eval([0, 2, 1, 3], BIG)
    assert list(r["profile"]) == [4, 7, 9, 6]
    r = G.eval([0, 1, 0, 2, 3], BIG)
    assert list(r["free"]) == [1, 4, 3, 4, 4] and list(r["profile"]) == [4, 6, 6, 9, 6] and r["dur"] == 11
    r = G.eval([0, 1, 3, 2], BIG)
    assert (r["status"], r["dur"], r["peak"]) == (-1, 10, -1)
    # recomputed sink: only its last copy is the retained result
    G = make_graph(2, [(0, 1)], [1, 1], [7, 2], 3)
    r = G.eval([0, 1, 1], BIG)
    assert list(r["free"]) == [2, 1, 2] and list(r["profile"]) == [7, 9, 9]
    # star: consumers after a recomputation read the newest copy
    G = make_graph(4, [(0, 1), (0, 2), (0, 3)], [1] * 4, [1] * 4, 2)
    r = G.eval([0, 1, 0, 2, 3], BIG)
    assert list(r["free"]) == [1, 4, 4, 4, 4] and list(r["profile"]) == [1, 2, 2, 3, 4]
    # malformed sequences
    G = make_graph(3, [(0, 1)], [1, 2, 3], [1, 1, 1], 2)
    for bad in ([0, 1], [0, 1, 1], [0, 1, 3], [0, 1, -1], [0, 0, 0, 1, 2], [0, 1, 2, 0, 1, 2, 0]):
        r = G.eval(bad, BIG)
        assert (r["status"], r["peak"], r["dur"]) == (-2, -1, -1), bad
    assert G.eval([2, 0, 1], BIG)["status"] == 1
    assert G.eval([1, 0, 2], BIG)["status"] == -1
    # isolated node is a sink; budget test is "<="
    r = G.eval([2, 0, 1], 3)
    assert list(r["profile"]) == [1, 2, 3] and r["status"] == 1 and G.eval([2, 0, 1], 2)["status"] == 0


# ---------------------------------------------------------------- brute force / definitions
def _random_dag(rnd, n, p):
    return [(u, v) for u in range(n) for v in range(u + 1, n) if rnd.random() < p]


def pin_topological_orders(make_graph, n_graphs=12):
    """All topological orders of small DAGs against textbook liveness; any of them is
    dependency-feasible (Section 2.4)."""
    rnd = random.Random(11)
    for k in range(n_graphs):
        n = rnd.randint(3, 6)
        edges = _random_dag(rnd, n, 0.45)
        m = [rnd.randint(1, 30) for _ in range(n)]
        w = [rnd.randint(1, 9) for _ in range(n)]
        G = make_graph(n, edges, w, m, 2)
        for order in defs.topological_orders(n, edges):
            r = G.eval(order, BIG)
            assert r["status"] == 1 and r["dur"] == sum(w)
            assert list(r["profile"]) == defs.no_remat_profile(n, edges, m, order)


def pin_exhaustive(make_graph):
    """Every sequence over n <= 4 nodes up to length 6 (C = 3) against the set definition."""
    rnd = random.Random(3)
    graphs = [(3, [(0, 1), (1, 2)]), (3, [(0, 2), (1, 2)]), (4, [(0, 1), (1, 2), (2, 3), (0, 3)]),
              (4, [(0, 1), (0, 2), (1, 3), (2, 3)]), (4, [(0, 2), (1, 2), (1, 3)]), (3, [])]
    for n, edges in graphs:
        m = [rnd.randint(1, 20) for _ in range(n)]
        w = [rnd.randint(1, 9) for _ in range(n)]
        M = sum(m) * 2 // 3
        G = make_graph(n, edges, w, m, 3)
        for T in range(max(n - 1, 1), 7):
            for seq in itertools.product(range(n), repeat=T):
                seq = list(seq)
                st, peak, dur, prof = defs.set_definition(n, edges, w, m, 3, seq, M)
                r = G.eval(seq, M)
                assert (r["status"], r["peak"], r["dur"]) == (st, peak, dur), (n, edges, seq)
                if st >= 0:
                    assert list(r["profile"]) == prof, (n, edges, seq)


def pin_node_caps(make_graph):
    """Per-node caps C_v (Section 2): hand cases on the paper's 4-node graph, then every sequence up
    to length 6 on two small graphs against the set definition with the same caps."""
    n, edges = 4, [(0, 1), (1, 2), (2, 3), (0, 3)]
    G = make_graph(n, edges, [2, 3, 4, 5], [1, 1, 1, 1], 2)
    seq = [0, 1, 2, 0, 3]
    base = G.eval(seq, BIG)
    assert base["status"] == 1 and base["peak"] == 3
    G.set_caps([1, 2, 2, 2])                      # node 0 may not be recomputed
    r = G.eval(seq, BIG)
    assert (r["status"], r["peak"], r["dur"]) == (-2, -1, -1)
    assert G.eval([0, 1, 2, 3], BIG)["status"] == 1
    G.set_caps([2, 1, 1, 1])                      # only node 0 may be: unchanged result
    r = G.eval(seq, BIG)
    assert (r["status"], r["peak"], r["dur"]) == (1, 3, 16) and list(r["profile"]) == list(base["profile"])
    assert G.eval([0, 1, 1, 2, 3], BIG)["status"] == -2
    G.set_caps(None)                              # uniform cap again
    assert G.eval([0, 1, 1, 2, 3], BIG)["status"] == 1
    rnd = random.Random(5)
    for n, edges, caps in [(4, [(0, 1), (0, 2), (1, 3), (2, 3)], [1, 3, 2, 1]), (3, [(0, 1), (1, 2)], [3, 1, 2])]:
        m = [rnd.randint(1, 20) for _ in range(n)]
        w = [rnd.randint(1, 9) for _ in range(n)]
        M = sum(m) * 2 // 3
        G = make_graph(n, edges, w, m, 3)
        G.set_caps(caps)
        for T in range(n, 7):
            for seq in itertools.product(range(n), repeat=T):
                seq = list(seq)
                st, peak, dur, prof = defs.set_definition(n, edges, w, m, 3, seq, M, caps=caps)
                r = G.eval(seq, M)
                assert (r["status"], r["peak"], r["dur"]) == (st, peak, dur), (n, edges, caps, seq)


def _random_remat_seq(rnd, n, edges, C, p):
    order = rnd.choice(list(itertools.islice(defs.topological_orders(n, edges), 50)))
    seq = list(order)
    for v in range(n):
        for _ in range(C - 1):
            if rnd.random() < p:
                first = seq.index(v)
                seq.insert(rnd.randint(first + 1, len(seq)), v)
    return seq


def pin_random_remat(make_graph, n_cases=150):
    """Random DAGs (n <= 7) with random extra copies: set definition + literal Eqs. 2-5."""
    rnd = random.Random(17)
    for k in range(n_cases):
        n = rnd.randint(3, 7)
        C = rnd.randint(2, 3)
        edges = _random_dag(rnd, n, 0.4)
        m = [rnd.randint(1, 40) for _ in range(n)]
        w = [rnd.randint(0, 9) for _ in range(n)]
        seq = _random_remat_seq(rnd, n, edges, C, 0.4)
        if rnd.random() < 0.25:                       # shuffle a little: may break precedence
            i, j = rnd.randrange(len(seq)), rnd.randrange(len(seq))
            seq[i], seq[j] = seq[j], seq[i]
        M = rnd.randint(max(m), sum(m))
        st, peak, dur, prof = defs.set_definition(n, edges, w, m, C, seq, M)
        G = make_graph(n, edges, w, m, C)
        r = G.eval(seq, M)
        assert (r["status"], r["peak"], r["dur"]) == (st, peak, dur), (n, edges, seq)
        if st >= 0:
            assert list(r["profile"]) == prof
            defs.check_intervals(n, edges, m, seq, list(r["free"]), list(r["profile"]))
            # invariants
            _, pred = defs.succ_lists(n, edges)
            for t, v in enumerate(seq):
                assert r["profile"][t] >= m[v] + sum(m[u] for u in pred[v])
            assert sum(r["profile"]) == sum(m[seq[p]] * (r["free"][p] - p + 1) for p in range(len(seq)))
            # relabelling the nodes changes nothing
            perm = list(range(n))
            rnd.shuffle(perm)
            e2 = [(perm[u], perm[v]) for u, v in edges]
            m2, w2 = [0] * n, [0] * n
            for v in range(n):
                m2[perm[v]], w2[perm[v]] = m[v], w[v]
            r2 = make_graph(n, e2, w2, m2, C).eval([perm[v] for v in seq], M)
            assert (r2["status"], r2["peak"], r2["dur"]) == (st, peak, dur)
            assert list(r2["profile"]) == prof


ALL_PINS = [pin_paper_example, pin_chain, pin_small_cases, pin_topological_orders, pin_exhaustive,
            pin_random_remat, pin_node_caps]


def run_all(make_graph):
    for pin in ALL_PINS:
        pin(make_graph)
