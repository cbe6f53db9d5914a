"""Pins for the interval-form oracle (oracle/moc_interval_oracle.c); every pin takes a graph factory
so that the same checks run against altered copies of the source.  Nothing is shared with the CUDA
path."""
from __future__ import annotations

import random

import numpy as np

import defs
from pins import read_golden, ints

BIG = 1 << 60
EQ2, EQ3, EQ4, EQ5, EQ6, EQ7, EQ8, STAGE = 1, 2, 4, 8, 16, 32, 64, 128


def paper_solution():
    g = read_golden("paper_fig2_worked_example.txt")
    n = int(g["n"])
    e = ints(g["edges"])
    edges = list(zip(e[0::2], e[1::2]))
    rows = np.array([ints(g[f"interval_node_{v}"]) for v in range(n)], np.int32)
    s, en, a = rows[:, 0::3].copy(), rows[:, 1::3].copy(), rows[:, 2::3].copy()
    return g, n, edges, s, en, a


def pin_paper_intervals(make_graph):
    """Section 2, Figs. 2-3: the worked example in the paper's own variables, staged events."""
    g, n, edges, s, e, a = paper_solution()
    w = [2, 3, 4, 5]
    G = make_graph(n, edges, w, ints(g["m"]), 2)
    topo = np.arange(1, n + 1, dtype=np.int32)
    r = G.check_intervals(s, e, a, 3, topo_index=topo)
    assert r["mask"] == 0 and r["peak"] == int(g["peak"]) and r["dur"] == 2 * 2 + 3 + 4 + 5
    assert list(r["usage"]) == ints(g["usage_by_event"])
    assert r["usage"][0] == 1 and r["usage"][6] == 2          # text: event 1 uses m_1, event 7 m_1 + m_3
    assert int(np.argmax(r["usage"])) + 1 == 10               # text: peak realised at event 10
    assert list(G.intervals_to_sequence(s, e, a, staged=True)) == ints(g["seq"])
    assert sorted(s[a == 1].tolist()) == ints(g["filled_events"])
    # budget one below the peak: only Eq. 4 fails (and <= is not <)
    assert G.check_intervals(s, e, a, 2, topo_index=topo)["mask"] == EQ4
    return G, s, e, a, topo


def pin_each_constraint(make_graph):
    """One violation at a time, planted in the paper's solution."""
    G, s, e, a, topo = pin_paper_intervals(make_graph)

    def chk(s2, e2, a2, staged=True, M=3, D=None):
        return G.check_intervals(s2, e2, a2, M, D=D, topo_index=topo if staged else None)

    def edit(arr, v, i, val):
        out = arr.copy()
        out[v, i] = val
        return out
    assert chk(edit(s, 1, 1, 7), e, a)["mask"] == EQ2                         # inactive slot with s > e
    assert chk(edit(s, 1, 1, 5), edit(e, 1, 1, 5), a)["mask"] == EQ3          # second slot starts before the first ends
    r = chk(s, edit(e, 0, 0, 2), a)                                          # node 0 dropped before node 1 runs at event 3
    assert r["mask"] == EQ5 and list(r["usage"][:3]) == [1, 1, 1]
    assert chk(s, edit(e, 0, 1, 9), a)["mask"] == EQ5                         # ... or before node 3 runs at event 10
    assert chk(s, e, edit(a, 0, 1, 0))["mask"] == EQ5                         # deactivating the recomputation
    assert chk(s, e, edit(a, 2, 0, 0))["mask"] == EQ5 | EQ7
    for args in ((edit(s, 3, 0, 0), e, a), (edit(s, 3, 0, 11), e, a), (s, edit(e, 0, 0, 11), a),
                 (s, e, edit(a, 1, 1, 2)), (s, e, edit(a, 1, 1, -1))):
        r = chk(*args)
        assert (r["mask"], r["peak"], r["dur"]) == (EQ8, -1, -1)
    # staged rule: node 0 may be recomputed at event 1 of a stage only (events 1, 2, 4, 7)
    assert chk(edit(s, 0, 1, 8), e, a)["mask"] == STAGE
    assert chk(edit(s, 0, 1, 4), e, a)["mask"] == 0                           # stage 3, event 1: allowed, costs nothing here
    # first interval away from the last event of its stage (node 1 at event 2 = stage 2 event 1 is node 0's column)
    assert chk(edit(s, 1, 0, 2), e, a)["mask"] & STAGE
    # node 0 first computed at event 2 (its own column, stage 2) instead of the last event of stage 1
    assert chk(edit(s, 0, 0, 2), e, a)["mask"] == STAGE
    # Eq. 7 names the FIRST slot: node 1 with an inactive first and an active second slot
    s7, e7, a7 = edit(s, 1, 1, 3), edit(edit(e, 1, 0, 3), 1, 1, 6), edit(edit(a, 1, 0, 0), 1, 1, 1)
    assert chk(s7, e7, a7)["mask"] == EQ7
    # plain model (D = C*n = 8): the same sequence [0,1,2,0,3] with one event per step, inactive slots
    # parked on the unused events 6, 7, 8
    ps = np.array([[1, 4], [2, 6], [3, 7], [5, 8]], np.int32)
    pe = np.array([[2, 5], [3, 6], [5, 7], [5, 8]], np.int32)
    r = chk(ps, pe, a, staged=False)
    assert (r["mask"], r["peak"], r["dur"]) == (0, 3, 16) and list(r["usage"]) == [1, 2, 2, 2, 3, 0, 0, 0]
    assert list(G.intervals_to_sequence(ps, pe, a)) == [0, 1, 2, 0, 3]
    assert chk(edit(ps, 1, 1, 7), edit(pe, 1, 1, 7), a, staged=False)["mask"] == EQ6      # nodes 1 and 2 both start at 7
    assert chk(edit(ps, 3, 1, 5), edit(pe, 3, 1, 5), a, staged=False)["mask"] == 0        # two slots of ONE node may share
    assert chk(edit(ps, 2, 1, 5), edit(pe, 2, 1, 5), a, staged=False)["mask"] == EQ6      # inactive slots count too
    assert G.intervals_to_sequence(edit(ps, 1, 0, 1), pe, a) is None                      # two computations in event 1
    # Eq. 5 is strict on the producer's side: a consumer in the producer's own event is not served
    r = chk(edit(ps, 1, 0, 1), edit(pe, 1, 0, 3), a, staged=False)
    assert r["mask"] == EQ5 | EQ6


def intervals_from_sequence(G, n, C, seq, staged_topo=None):
    """Interval form of a valid sequence, from the separately pinned sequence evaluator: step p
    becomes event p+1 (plain model) or the event of its stage and column (staged model, identity
    order), its end the event of its free step; unused slots are parked so that Eqs. 2, 3, 6 hold."""
    r = G.eval(seq, BIG)
    assert r["status"] >= 0
    T = len(seq)
    if staged_topo is None:
        ev = np.arange(1, T + 1)
    else:
        ev, stage = np.zeros(T, np.int64), 0
        seen = set()
        for p, v in enumerate(seq):
            if v not in seen:                     # first copy: last event of stage v+1
                stage = v + 1
                seen.add(v)
                ev[p] = stage * (stage + 1) // 2
            else:                                 # a recomputation inside the coming stage
                ev[p] = -1
        # recomputations belong to the stage of the next first copy
        nxt = None
        for p in range(T - 1, -1, -1):
            if ev[p] > 0:
                nxt = seq[p] + 1
            else:
                assert nxt is not None
                ev[p] = nxt * (nxt - 1) // 2 + seq[p] + 1
    s = np.zeros((n, C), np.int32)
    e = np.zeros((n, C), np.int32)
    a = np.zeros((n, C), np.int32)
    cnt = [0] * n
    for p, v in enumerate(seq):
        s[v, cnt[v]], e[v, cnt[v]], a[v, cnt[v]] = ev[p], ev[r["free"][p]], 1
        cnt[v] += 1
    spare = T + 1
    for v in range(n):
        for i in range(cnt[v], C):
            if staged_topo is None:
                s[v, i] = e[v, i] = spare
                spare += 1
            else:
                s[v, i] = e[v, i] = e[v, i - 1]
    return s, e, a, r


def pin_against_sequence_evaluator(make_graph, n_cases=60):
    """Random valid sequences: their interval form passes every constraint with the evaluator's peak
    and duration and converts back to the sequence; stretching an end never lowers the peak; cutting
    an end that is needed breaks Eq. 5."""
    rnd = random.Random(11)
    for case in range(n_cases):
        n = rnd.randint(3, 8)
        edges = [(u, v) for u in range(n) for v in range(u + 1, n) if rnd.random() < 0.4]
        C = rnd.randint(2, 3)
        m = [rnd.randint(1, 30) for _ in range(n)]
        w = [rnd.randint(1, 9) for _ in range(n)]
        G = make_graph(n, edges, w, m, C)
        staged = case % 2 == 1
        if staged:
            # stage j: some already computed nodes again in index order, then node j
            seq, cnt = [], [0] * n
            for j in range(n):
                for k in range(j):
                    if cnt[k] < C and rnd.random() < 0.25:
                        seq.append(k)
                        cnt[k] += 1
                seq.append(j)
                cnt[j] += 1
            topo = np.arange(1, n + 1, dtype=np.int32)
        else:
            order = rnd.choice(list(defs.topological_orders(n, edges))[:40])
            seq, cnt = list(order), [1] * n
            for v in range(n):
                if cnt[v] < C and rnd.random() < 0.4:
                    seq.insert(rnd.randint(seq.index(v) + 1, len(seq)), v)
                    cnt[v] += 1
            topo = None
        s, e, a, r = intervals_from_sequence(G, n, C, seq, staged_topo=topo)
        got = G.check_intervals(s, e, a, r["peak"], topo_index=topo)
        assert got["mask"] == 0 and got["peak"] == r["peak"] and got["dur"] == r["dur"], (n, edges, seq, got)
        assert list(G.intervals_to_sequence(s, e, a, staged=staged)) == seq
        ev = sorted(s[a == 1].tolist())
        assert [int(got["usage"][t - 1]) for t in ev] == [int(x) for x in r["profile"]]
        assert G.check_intervals(s, e, a, r["peak"] - 1, topo_index=topo)["mask"] == EQ4
        # an interval that ends one event later (where Eq. 3 still holds) never lowers the usage
        v, i = rnd.randrange(n), 0
        limit = s[v, 1] if C > 1 else len(got["usage"])
        if e[v, i] + 1 <= min(limit, len(got["usage"])):
            e2 = e.copy()
            e2[v, i] += 1
            g2 = G.check_intervals(s, e2, a, BIG, topo_index=topo)
            assert g2["mask"] & ~EQ6 == 0 and (g2["usage"] >= got["usage"]).all() and g2["usage"].sum() == got["usage"].sum() + m[v]
        # cutting an interval below its last consumer breaks Eq. 5 (the evaluator's ends are minimal)
        cand = [(v, i) for v in range(n) for i in range(C) if a[v, i] and e[v, i] > s[v, i]
                and any(seq[p] == v for p in range(len(seq)))]
        cand = [(v, i) for v, i in cand if any(u == v for u, _ in edges)]
        if cand:
            v, i = rnd.choice(cand)
            e2 = e.copy()
            e2[v, i] -= 1
            assert G.check_intervals(s, e2, a, BIG, topo_index=topo)["mask"] & EQ5, (n, edges, seq, v, i)


def run_all(make_graph):
    pin_each_constraint(make_graph)
    pin_against_sequence_evaluator(make_graph)
