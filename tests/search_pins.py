"""Pins for the search oracle (oracle/moc_search_oracle.c): each takes the bound library so that the
same checks run against altered copies of the source.  Nothing here is shared with the CUDA path."""
from __future__ import annotations

import itertools
import os
import random

import numpy as np

import oracle
from defs import set_definition

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def pin_philox_kat(lib):
    """Published known-answer vectors of the generator."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        out = oracle.philox4x32_10(v[0:4], v[4:6], lib=lib)
        assert [int(x) for x in out] == v[6:10], (r, [hex(int(x)) for x in out])


def list_edit(seq, r0, r1, r2, kinds=7):
    """The three edits restated with Python list operations."""
    s = list(seq)
    T = len(s)
    if T == 0:
        return None
    enabled = [o for o in range(3) if kinds >> o & 1]
    op, q = enabled[r0 % len(enabled)], r1 % T
    if op == 0:
        s.insert(r2 % (T + 1), s[q])
    elif op == 1:
        del s[q]
    else:
        x = s.pop(q)
        s.insert(r2 % T, x)
    return s


def pin_edits(lib):
    # hand-written cases: seq = [5, 6, 7, 8]
    seq = [5, 6, 7, 8]
    cases = [
        ((0, 1, 0), [6, 5, 6, 7, 8]),      # insert a copy of seq[1] in front of index 0
        ((0, 1, 4), [5, 6, 7, 8, 6]),      # ... at the very end (index T)
        ((3, 2, 8), [5, 6, 7, 7, 8]),      # r0 = 3 -> insert; in front of index 8 mod 5 = 3
        ((1, 0, 0), [6, 7, 8]),            # delete element 0
        ((1, 7, 5), [5, 6, 7]),            # delete element 7 mod 4 = 3
        ((2, 0, 3), [6, 7, 8, 5]),         # move element 0 to the end of the shortened sequence
        ((2, 3, 0), [8, 5, 6, 7]),         # move the last element to the front
        ((2, 1, 1), [5, 6, 7, 8]),         # move to its own place: unchanged
        ((5, 2, 6), [5, 6, 7, 8]),         # r0 = 5 -> move element 2 in front of index 6 mod 4 = 2
    ]
    for (r0, r1, r2), want in cases:
        got = oracle.mutate(seq, r0, r1, r2, lib=lib)
        assert list(got) == want, ((r0, r1, r2), list(got), want)
    assert oracle.mutate([], 1, 2, 3, lib=lib) is None
    assert list(oracle.mutate([4], 1, 0, 0, lib=lib)) == []
    # against the list restatement, with draws over the full 32-bit range
    rnd = random.Random(7)
    for _ in range(3000):
        T = rnd.randint(1, 12)
        s = [rnd.randint(0, 5) for _ in range(T)]
        r = [rnd.getrandbits(32) for _ in range(3)]
        if rnd.random() < 0.5:
            r = [x % 16 for x in r]
        got = oracle.mutate(s, *r, lib=lib)
        assert list(got) == list_edit(s, *r), (s, r)
        # the multiset changes by exactly the edit's element
        op = r[0] % 3
        assert len(got) == T + (1, -1, 0)[op]
        # restricted kinds of edit: the (r0 mod k)-th enabled kind
        kinds = rnd.randint(1, 7)
        got = oracle.mutate(s, *r, kinds=kinds, lib=lib)
        assert list(got) == list_edit(s, *r, kinds=kinds), (s, r, kinds)
    # moves only: a permutation of the sequence; hand cases with r0 arbitrary
    assert list(oracle.mutate(seq, 0, 0, 3, kinds=4, lib=lib)) == [6, 7, 8, 5]
    assert list(oracle.mutate(seq, 1, 3, 0, kinds=4, lib=lib)) == [8, 5, 6, 7]
    assert list(oracle.mutate(seq, 1, 0, 0, kinds=5, lib=lib)) == [5, 6, 7, 8]   # insert|move, r0 = 1 -> move element 0 to index 0
    assert list(oracle.mutate(seq, 2, 1, 0, kinds=3, lib=lib)) == [6, 5, 6, 7, 8]   # insert|delete, r0 = 2 -> insert


def key_of(ev, M):
    peak, dur, st = ev
    return (float("inf"), float("inf")) if st < 0 else (max(peak, M), dur)


def pin_accept(lib):
    M = 10
    evs = [(p, d, s) for p in (7, 10, 11, 15) for d in (3, 4) for s in (0, 1)] + [(-1, 9, -1), (-1, -1, -2)]
    for c in evs:
        for p in evs:
            want = c[2] >= 0 and key_of(c, M) <= key_of(p, M)
            assert oracle.accept(c, p, M, lib=lib) == want, (c, p)
    # Phase 1 then Phase 2 of the paper: below the budget only the duration matters
    assert oracle.accept((3, 5, 1), (9, 5, 1), M, lib=lib) and oracle.accept((9, 5, 1), (3, 5, 1), M, lib=lib)
    assert not oracle.accept((9, 6, 1), (3, 5, 1), M, lib=lib)
    assert oracle.accept((11, 99, 0), (12, 1, 0), M, lib=lib)       # over budget: the peak decides first
    assert not oracle.accept((11, 1, 0), (10, 99, 1), M, lib=lib)   # never leave the feasible region


def _tiny_problem():
    # diamond with a heavy source: recomputing node 0 late lowers the peak
    n, edges = 5, [(0, 1), (1, 2), (2, 3), (0, 3), (3, 4)]
    w = [2, 3, 4, 5, 1]
    m = [6, 2, 2, 1, 1]
    return n, edges, w, m


def python_generation_loop(make_graph, lib, n, edges, w, m, C, rows, M, seed, gen0, n_gen, chain0=0, kinds=7, samples=1):
    """The generation loop restated in Python over the separately pinned pieces, with the
    set-definition evaluator of defs.py in place of the oracle's evaluator."""
    def ev(s):
        st, pk, du, _ = set_definition(n, edges, w, m, C, list(s), M)
        return (pk, du, st)
    rows = [list(r) for r in rows]
    evs = [ev(r) for r in rows]
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for gen in range(gen0, gen0 + n_gen):
        for c, r in enumerate(rows):
            best = None                                   # (key, e, child, evaluation): smallest key, then lowest e
            for e_i in range(samples):
                x = oracle.philox4x32_10([gen, chain0 + c, e_i, 0], key, lib=lib)
                child = list_edit(r, int(x[0]), int(x[1]), int(x[2]), kinds)
                if child is None:
                    continue
                e = ev(child)
                if e[2] < 0:
                    continue
                if best is None or (key_of(e, M), e_i) < (best[0], best[1]):
                    best = (key_of(e, M), e_i, child, e)
            if best is not None and best[0] <= key_of(evs[c], M):
                rows[c], evs[c] = best[2], best[3]
    return rows, evs


def pin_search_loop(make_graph, lib):
    n, edges, w, m = _tiny_problem()
    C = 2
    g = make_graph(n, edges, w, m, C)
    P0 = g.eval(np.arange(n), 1 << 60)["peak"]
    rnd = random.Random(3)
    for M in (P0, P0 * 8 // 10, 1):
        for seed in (1, (0xABCDEF01 << 32) | 0x12345678):
            rows = [list(range(n)) for _ in range(6)] + [[0, 1, 2, 0, 3, 4], [4, 3, 2, 1, 0], [0, 1, 2]]
            seqs = np.array([x for r in rows for x in r], np.int32)
            lens = np.array([len(r) for r in rows], np.int32)
            chain0 = 0 if M == P0 else 1000
            kinds = 7 if seed == 1 else (4 if M == 1 else 6)
            samples = 1 if M == P0 else (3 if seed == 1 else 5)
            S = oracle.OracleSearch(g, seqs, lens, M, seed, chain0=chain0, kinds=kinds, samples=samples)
            done = 0
            for n_gen in (1, 7, 40):
                before = [key_of((S.peak[c], S.dur[c], S.status[c]), M) for c in range(S.P)]
                S.run(n_gen)
                want_rows, want_ev = python_generation_loop(make_graph, lib, n, edges, w, m, C, rows, M, seed, done, n_gen, chain0, kinds, samples)
                done += n_gen
                for c in range(S.P):
                    assert list(S.row(c)) == want_rows[c], (M, seed, c)
                    assert (int(S.peak[c]), int(S.dur[c]), int(S.status[c])) == want_ev[c]
                    after = key_of(want_ev[c], M)
                    assert after <= before[c]                     # the key never increases
                rows = want_rows
            assert S.generation == done


def pin_sample_ties(make_graph, lib):
    """Four nodes without edges: every order has the same peak and duration, so all samples of a
    generation tie and the first one (e = 0) must be taken."""
    n, edges, w, m, C = 4, [], [1, 2, 3, 4], [5, 5, 5, 5], 2
    g = make_graph(n, edges, w, m, C)
    rows = [[0, 1, 2, 3], [3, 2, 1, 0], [1, 0, 3, 2]]
    seqs = np.array([x for r in rows for x in r], np.int32)
    lens = np.array([len(r) for r in rows], np.int32)
    S = oracle.OracleSearch(g, seqs, lens, 100, seed=5, kinds=4, samples=4)
    S.run(12)
    want_rows, want_ev = python_generation_loop(make_graph, lib, n, edges, w, m, C, rows, 100, 5, 0, 12, 0, 4, 4)
    for c in range(3):
        assert list(S.row(c)) == want_rows[c], c
    # the same draws with one sample take the e = 0 proposal too
    S1 = oracle.OracleSearch(g, seqs, lens, 100, seed=5, kinds=4, samples=1)
    S1.run(12)
    for c in range(3):
        assert list(S1.row(c)) == list(S.row(c))


def pin_search_reaches_optimum(make_graph, lib):
    """On a graph small enough to enumerate every sequence, enough generations reach the best key."""
    n, edges, w, m = _tiny_problem()
    C = 2
    g = make_graph(n, edges, w, m, C)
    P0 = g.eval(np.arange(n), 1 << 60)["peak"]
    M = P0 * 8 // 10
    best = None
    for T in range(n, 8):
        for s in itertools.product(range(n), repeat=T):
            st, pk, du, _ = set_definition(n, edges, w, m, C, list(s), M)
            if st >= 0:
                k = (max(pk, M), du)
                best = k if best is None or k < best else best
    P = 32
    seqs = np.tile(np.arange(n, dtype=np.int32), P)
    lens = np.full(P, n, np.int32)
    S = oracle.OracleSearch(g, seqs, lens, M, seed=11)
    S.run(300)
    b = S.best()
    assert b >= 0
    got = (max(int(S.peak[b]), M), int(S.dur[b]))
    # sequences of up to 7 steps are enumerated; the search may also use longer ones
    assert got <= best, (got, best)
    st, pk, du, _ = set_definition(n, edges, w, m, C, list(S.row(b)), M)
    assert (pk, du) == (int(S.peak[b]), int(S.dur[b])) and st == int(S.status[b])
    # best = lowest index among the chains with the smallest key
    keys = [key_of((S.peak[c], S.dur[c], S.status[c]), M) for c in range(P)]
    assert b == keys.index(min(keys))
    # chains are independent: chain c's history does not depend on the other rows
    seqs2 = seqs.copy()
    seqs2[n:2 * n] = seqs2[n:2 * n][::-1]          # chain 1 starts from an invalid order
    S2 = oracle.OracleSearch(g, seqs2, lens, M, seed=11)
    S2.run(300)
    for c in (0, 2, 31):
        assert list(S2.row(c)) == list(S.row(c))
    # a population split in two (second half numbered from chain0 = 16) gives the same chains
    half = P // 2
    Sa = oracle.OracleSearch(g, seqs[:half * n], lens[:half], M, seed=11)
    Sb = oracle.OracleSearch(g, seqs[half * n:], lens[half:], M, seed=11, chain0=half)
    Sa.run(300)
    Sb.run(300)
    for c in range(P):
        part, k = (Sa, c) if c < half else (Sb, c - half)
        assert list(part.row(k)) == list(S.row(c))


def run_all(make_graph, lib):
    pin_philox_kat(lib)
    pin_edits(lib)
    pin_accept(lib)
    pin_search_loop(make_graph, lib)
    pin_sample_ties(make_graph, lib)
    pin_search_reaches_optimum(make_graph, lib)
