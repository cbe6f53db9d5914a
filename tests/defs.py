"""Independent, definition-level checkers used to pin the CPU oracle (pure Python, tiny inputs).

Nothing here is shared with oracle/ or with the CUDA path.  Two routes are provided:

* ``set_definition``: for every step t, the set of copies resident at t, written from the point of
  view of the *consumers* (successor lists and a forward search), not by the sequential
  last-copy simulation the oracle uses.
* ``check_intervals``: takes retention intervals [s, e] and verifies the paper's Eqs. 2-5 on them
  literally, plus minimality of every interval end.
"""
from __future__ import annotations

import itertools


def succ_lists(n, edges):
    succ = [set() for _ in range(n)]
    pred = [set() for _ in range(n)]
    for u, v in edges:
        succ[u].add(v)
        pred[v].add(u)
    return succ, pred


def set_definition(n, edges, w, m, C, seq, M, caps=None):
    """(status, peak, dur, profile) straight from the definitions; O(T^2).  caps: per-node C_v."""
    T = len(seq)
    succ, pred = succ_lists(n, edges)
    if T < n or T > C * n or any(v < 0 or v >= n for v in seq):
        return -2, -1, -1, None
    for v in range(n):
        k = sum(1 for x in seq if x == v)
        if k < 1 or k > (C if caps is None else caps[v]):
            return -2, -1, -1, None
    dur = sum(w[v] for v in seq)
    # Eq. 5: each consumer needs an earlier copy of every predecessor
    for t, v in enumerate(seq):
        for u in pred[v]:
            if not any(seq[p] == u for p in range(t)):
                return -1, -1, dur, None
    last = {v: max(p for p in range(T) if seq[p] == v) for v in range(n)}
    profile = []
    for t in range(T):
        resident = 0
        for p in range(t + 1):
            u = seq[p]
            live = (p == t)
            if not live and not succ[u] and p == last[u]:
                live = True                      # result of the computation, kept to the end
            if not live:
                # is there a consumer at t' >= t that reads THIS copy (no newer copy of u in between)?
                for t2 in range(p + 1, T):
                    if seq[t2] == u:
                        break                    # a newer copy takes over from here on
                    if t2 >= t and seq[t2] in succ[u]:
                        live = True
                        break
            if live:
                resident += m[u]
        profile.append(resident)
    peak = max(profile)
    return (1 if peak <= M else 0), peak, dur, profile


def check_intervals(n, edges, m, seq, free, profile):
    """Literal check of Eqs. 2-5 for the intervals [s=p, e=free[p]] and of their minimality."""
    T = len(seq)
    succ, pred = succ_lists(n, edges)
    copies = {v: [p for p in range(T) if seq[p] == v] for v in range(n)}
    for p in range(T):
        assert p <= free[p] <= T - 1, "Eq. 2 / domain"
    for v in range(n):
        for a, b in zip(copies[v], copies[v][1:]):
            assert free[a] <= b, "Eq. 3: intervals of one node overlap"
    for t in range(T):
        for u in pred[seq[t]]:
            assert any(p + 1 <= t <= free[p] for p in copies[u]), "Eq. 5 violated"
    for t in range(T):
        assert profile[t] == sum(m[seq[p]] for p in range(T) if p <= t <= free[p]), "Eq. 4 sum"
    # minimality: an interval longer than its compute step ends at a consumer that needs it,
    # or belongs to the final copy of a sink (kept as the result)
    for p in range(T):
        u = seq[p]
        if free[p] == p:
            continue
        if not succ[u] and p == copies[u][-1]:
            assert free[p] == T - 1
            continue
        e = free[p]
        assert seq[e] in succ[u], "interval ends at a non-consumer"
        others = [q for q in copies[u] if q != p and q + 1 <= e <= free[q]]
        assert not others, "two intervals of one node cover the same consumer"


def topological_orders(n, edges):
    _, pred = succ_lists(n, edges)
    for perm in itertools.permutations(range(n)):
        pos = {v: i for i, v in enumerate(perm)}
        if all(pos[u] < pos[v] for u, v in edges):
            yield list(perm)


def no_remat_profile(n, edges, m, order):
    """Textbook liveness for an order without recomputation: at step t the output of order[t] plus
    every earlier output that still has a consumer at a position >= t, plus finished sinks."""
    succ, _ = succ_lists(n, edges)
    pos = {v: i for i, v in enumerate(order)}
    prof = []
    for t in range(len(order)):
        tot = 0
        for u in order[:t + 1]:
            if pos[u] == t or not succ[u] or any(pos[v] >= t for v in succ[u]):
                tot += m[u]
        prof.append(tot)
    return prof
