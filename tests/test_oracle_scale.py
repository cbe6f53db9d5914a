"""Invariants of the oracle on the five synthetic configurations (reduced batch sizes, no GPU)."""
import numpy as np
import pytest

from oracle import OracleGraph
from paper_2304_14463_b200 import workloads as W

BIG = 1 << 60
SMALL_B = [256, 256, 128, 48, 8]


def _pred_sum(n, edges, m):
    s = m.copy()
    np.add.at(s, edges[:, 1], m[edges[:, 0]])
    return s


@pytest.mark.parametrize("idx", range(W.N_CONFIGS))
def test_invariants(idx):
    wl = W.make(idx, seed=2, B=SMALL_B[idx])
    G = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    ident = G.eval(np.arange(wl.n), BIG)
    assert ident["status"] == 1 and ident["dur"] == wl.w.sum()
    P0 = ident["peak"]
    lower = _pred_sum(wl.n, wl.edges, wl.m)
    sinks = np.ones(wl.n, bool)
    sinks[wl.edges[:, 0]] = False
    peak, dur, status, _ = G.eval_batch(wl.seqs, wl.lens, P0 * 80 // 100, n_threads=2)
    rows = W.unpack(wl.seqs, wl.lens)
    assert (status >= 0).all()                      # generated schedules respect precedence
    for b, seq in enumerate(rows):
        assert dur[b] == wl.w[seq].sum() >= wl.w.sum()
        assert peak[b] >= lower.max()
        assert peak[b] <= wl.m[seq].sum()
        assert status[b] == (1 if peak[b] <= P0 * 80 // 100 else 0)
    for b in range(0, len(rows), max(1, len(rows) // 6)):
        seq = rows[b]
        r = G.eval(seq, BIG)
        assert (r["peak"], r["dur"]) == (peak[b], dur[b])
        assert (r["profile"] >= lower[seq]).all()
        assert r["profile"][-1] >= wl.m[sinks].sum()
        assert r["profile"].sum() == (wl.m[seq] * (r["free"] - np.arange(len(seq)) + 1)).sum()
        assert r["profile"].max() == r["peak"]
        # feasibility shortcut: precedence holds iff first[u] < first[v] on every edge
        first = np.full(wl.n, len(seq))
        np.minimum.at(first, seq, np.arange(len(seq)))
        assert (first[wl.edges[:, 0]] < first[wl.edges[:, 1]]).all()


def test_mutated_batches_cover_all_statuses():
    wl = W.make(1, seed=3, B=512)
    G = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    seqs, lens = W.mutate(wl.seqs, wl.lens, wl.n, wl.C, seed=5, frac=0.25)
    peak, dur, status, _ = G.eval_batch(seqs, lens, np.median(G.eval_batch(wl.seqs, wl.lens, BIG)[0]))
    assert set(np.unique(status)) == {-2, -1, 0, 1}
    assert ((status == -2) == (dur == -1)).all() and ((status < 0) == (peak == -1)).all()
    # thread count does not change results
    p2, d2, s2, used = G.eval_batch(seqs, lens, int(np.median(peak[peak > 0])), n_threads=4)
    p1, d1, s1, _ = G.eval_batch(seqs, lens, int(np.median(peak[peak > 0])), n_threads=1)
    assert used == 4 and (p1 == p2).all() and (d1 == d2).all() and (s1 == s2).all()
