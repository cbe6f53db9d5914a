"""Shape and determinism of the synthetic input generators (no GPU)."""
import numpy as np
import pytest

from paper_2304_14463_b200 import workloads as W

EXPECT = [(20, 40), (100, 236), (442, 1247), (1000, 2994), (5000, 15000)]


@pytest.mark.parametrize("idx", range(W.N_CONFIGS))
def test_graph_shape(idx):
    edges, w, m = W.make_graph(idx, seed=1)
    n, n_edges = EXPECT[idx]
    assert edges.shape == (n_edges, 2) and len(w) == n and len(m) == n
    assert (edges[:, 0] < edges[:, 1]).all() and edges.min() >= 0 and edges.max() < n   # ids topological
    assert len({(int(u), int(v)) for u, v in edges}) == n_edges                          # distinct
    assert w.min() >= 1 and m.min() >= 1
    e2, w2, m2 = W.make_graph(idx, seed=1)
    assert (edges == e2).all() and (w == w2).all() and (m == m2).all()
    if idx != 3:
        assert not (W.make_graph(idx, seed=2)[0] == edges).all()


def test_training_graph_structure():
    edges, _, _ = W.make_graph(2)
    E = {(int(u), int(v)) for u, v in edges}
    F = 221
    b = lambda i: 2 * F - 1 - i
    assert all((i, i + 1) in E for i in range(F - 1)) and all((i, b(i)) in E for i in range(F))
    assert all((b(i + 1), b(i)) in E for i in range(F - 1))
    skips = [(u, v) for u, v in E if v < F and v - u >= 2]
    assert len(skips) == 293 and all(2 <= v - u <= 8 for u, v in skips)
    assert all((b(v), b(u)) in E for u, v in skips)
    out = np.zeros(2 * F, int)
    np.add.at(out, edges[:, 0], 1)
    assert (out == 0).sum() == 1 and out[b(0)] == 0      # single sink b_0


@pytest.mark.parametrize("idx", range(W.N_CONFIGS))
def test_schedules(idx):
    s = W.spec(idx)
    wl = W.make(idx, seed=1, B=64, n_threads=1)
    wl2 = W.make(idx, seed=1, B=64, n_threads=3)
    assert (wl.seqs == wl2.seqs).all() and (wl.lens == wl2.lens).all()    # thread-count independent
    assert wl.lens.min() >= wl.n and wl.lens.max() <= wl.meta["t_cap"]
    for seq in W.unpack(wl.seqs, wl.lens):
        cnt = np.bincount(seq, minlength=wl.n)
        assert cnt.min() >= 1 and cnt.max() <= wl.C
        first = np.full(wl.n, len(seq))
        np.minimum.at(first, seq, np.arange(len(seq)))
        assert (first[wl.edges[:, 0]] < first[wl.edges[:, 1]]).all()
    expect_T = wl.n * (1 + (s["C"] - 1) * s["p"])
    assert abs(wl.lens.mean() - expect_T) < 0.05 * expect_T


def test_pack_unpack_mutate():
    wl = W.make(0, seed=1, B=200)
    rows = W.unpack(wl.seqs, wl.lens)
    s2, l2 = W.pack(rows)
    assert (s2 == wl.seqs).all() and (l2 == wl.lens).all()
    s3, l3 = W.mutate(wl.seqs, wl.lens, wl.n, wl.C, seed=1, frac=0.5)
    assert len(l3) == len(wl.lens) and l3.sum() == len(s3)
    assert (l3 != wl.lens).any() and (s3.max() == wl.n or s3.min() == -1)
