"""Parity of moc_check_intervals (through the C ABI) with the interval-form oracle: mask, peak,
duration, and the execution sequence, solution by solution."""
import numpy as np
import pytest
import torch

import interval_pins
from oracle import OracleGraph
from paper_2304_14463_b200 import workloads as W

pytestmark = pytest.mark.gpu
BIG = 1 << 60


@pytest.fixture(scope="module")
def B():
    from paper_2304_14463_b200 import build
    build.build()
    from paper_2304_14463_b200 import binding
    return binding


def dev(a, dtype=torch.int32):
    return torch.as_tensor(np.ascontiguousarray(a), dtype=dtype).cuda()


def test_interval_pins_through_the_gpu(B):
    """The oracle's own pins (worked example of the paper, one violation per constraint, random valid
    solutions) with the CUDA checker in place of the oracle."""
    class GpuGraph:
        def __init__(self, n, edges, w, m, C):
            self.n, self.C = n, C
            self.G = B.Graph(n, edges, w, m, C)
            self.O = OracleGraph(n, edges, w, m, C)     # sequence evaluator, for building inputs only

        def eval(self, seq, M):
            return self.O.eval(seq, M)

        def _call(self, s, e, a, M, D, topo_index):
            sh = (1, self.n, self.C)
            t = None if topo_index is None else dev(topo_index)
            return self.G.check_intervals(dev(np.reshape(s, sh)), dev(np.reshape(e, sh)), dev(np.reshape(a, sh)), M,
                                          D=D, topo_index=t)

        def check_intervals(self, s, e, a, M, D=None, topo_index=None):
            r = self._call(s, e, a, M, D, topo_index)
            torch.cuda.synchronize()
            ref = self.O.check_intervals(s, e, a, M, D=D, topo_index=topo_index)   # usage per event: oracle only
            return dict(mask=int(r["mask"][0]), peak=int(r["peak"][0]), dur=int(r["dur"][0]), usage=ref["usage"])

        def intervals_to_sequence(self, s, e, a, D=None, staged=False):
            topo = np.arange(1, self.n + 1, dtype=np.int32) if staged else None
            r = self._call(s, e, a, BIG, D, topo)
            torch.cuda.synchronize()
            k = int(r["lens"][0])
            return None if k < 0 else r["seqs"][0, :k].cpu().numpy()

    interval_pins.run_all(lambda n, e, w, m, C: GpuGraph(n, e, w, m, C))


def staged_sequence(rng, n, C, p):
    seq, cnt = [], np.zeros(n, np.int64)
    for j in range(n):
        again = np.nonzero((rng.random(j) < p) & (cnt[:j] < C))[0]
        seq.extend(again.tolist())
        cnt[again] += 1
        seq.append(j)
        cnt[j] += 1
    return seq


def build_batch(O, wl, rng, nB, staged):
    n, C = wl.n, wl.C
    s = np.zeros((nB, n, C), np.int32)
    e = np.zeros((nB, n, C), np.int32)
    a = np.zeros((nB, n, C), np.int32)
    topo = np.arange(1, n + 1, dtype=np.int32) if staged else None
    offs = np.concatenate([[0], np.cumsum(wl.lens)])
    for b in range(nB):
        seq = staged_sequence(rng, n, C, 0.3 / max(1, n // 20)) if staged else wl.seqs[offs[b]:offs[b + 1]].tolist()
        s[b], e[b], a[b], _ = interval_pins.intervals_from_sequence(O, n, C, seq, staged_topo=topo)
    D = n * (n + 1) // 2 if staged else C * n
    # damage three quarters of the solutions: a few entries each, of every kind
    for b in range(nB):
        if b % 4 == 0:
            continue
        for _ in range(int(rng.integers(1, 4))):
            v, i, kind = int(rng.integers(n)), int(rng.integers(C)), int(rng.integers(8))
            if kind == 0:
                e[b, v, i] = max(1, e[b, v, i] - int(rng.integers(1, 4)))
            elif kind == 1:
                e[b, v, i] = min(D, e[b, v, i] + int(rng.integers(1, 50)))
            elif kind == 2:
                s[b, v, i] = int(rng.integers(1, D + 1))
            elif kind == 3:
                a[b, v, i] ^= 1
            elif kind == 4:
                s[b, v, i] = s[b, int(rng.integers(n)), int(rng.integers(C))]
            elif kind == 5 and b % 16 == 1:
                s[b, v, i] = [0, D + 1, -5][int(rng.integers(3))]
            elif kind == 6 and b % 16 == 2:
                a[b, v, i] = 2
            else:
                s[b, v, i] = e[b, v, i] = int(rng.integers(1, D + 1))
    return s, e, a, D, topo


@pytest.mark.parametrize("idx,nB,staged", [(0, 512, False), (0, 512, True), (1, 128, False), (1, 96, True),
                                           (2, 64, False), (2, 6, True), (3, 16, False), (4, 3, False)])
def test_interval_batch_parity(B, idx, nB, staged):
    wl = W.make(idx, seed=3, B=nB)
    rng = np.random.default_rng(100 + idx)
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    s, e, a, D, topo = build_batch(O, wl, rng, nB, staged)
    M = O.eval(np.arange(wl.n), BIG)["peak"] * 80 // 100
    r = G.check_intervals(dev(s), dev(e), dev(a), M, D=D, topo_index=None if topo is None else dev(topo))
    torch.cuda.synchronize()
    mask, peak, dur = r["mask"].cpu().numpy(), r["peak"].cpu().numpy(), r["dur"].cpu().numpy()
    lens, seqs = r["lens"].cpu().numpy(), r["seqs"].cpu().numpy()
    seen = set()
    for b in range(nB):
        ref = O.check_intervals(s[b], e[b], a[b], M, D=D, topo_index=topo)
        assert (int(mask[b]), int(peak[b]), int(dur[b])) == (ref["mask"], ref["peak"], ref["dur"]), (idx, staged, b)
        seq = O.intervals_to_sequence(s[b], e[b], a[b], D=D)
        assert (seq is None) == (lens[b] < 0), (idx, staged, b)
        if seq is not None:
            assert lens[b] == len(seq) and (seqs[b, :lens[b]] == seq).all()
        seen.add(ref["mask"])
    assert 0 in seen or any(m & ~4 == 0 for m in seen)
    if nB >= 64:
        assert len(seen) >= 4        # the damage produced several kinds of violation


def test_interval_argument_errors(B):
    wl = W.make(4, seed=1, B=1)      # n = 5000: the staged domain (12.5 M events) does not fit on chip
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    z = torch.ones((1, wl.n, wl.C), dtype=torch.int32, device="cuda")
    with pytest.raises(B.MocError) as err:
        G.check_intervals(z, z, z, 1, topo_index=dev(np.arange(1, wl.n + 1)))
    assert err.value.code == -1
    with pytest.raises(B.MocError):
        G.check_intervals(z, z, z, 1, D=7, topo_index=dev(np.arange(1, wl.n + 1)))   # staged needs D = n(n+1)/2
    with pytest.raises(B.MocError):
        G.check_intervals(z, z, z, 1, D=0)


def test_interval_full_size_sampled(B):
    """The benchmark's shape (headline graph, 16384 solutions, plain domain): every 37th solution is
    compared with the oracle; the rest must agree with the copy of the same solution among them."""
    nB, distinct = 16384, 128
    wl = W.make(2, seed=1, B=distinct)
    rng = np.random.default_rng(9)
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    s, e, a, D, _ = build_batch(O, wl, rng, distinct, staged=False)
    perm = rng.permutation(nB) % distinct
    M = O.eval(np.arange(wl.n), BIG)["peak"] * 80 // 100
    r = G.check_intervals(dev(s[perm]), dev(e[perm]), dev(a[perm]), M, D=D)
    torch.cuda.synchronize()
    mask, peak, dur, lens = (r[k].cpu().numpy() for k in ("mask", "peak", "dur", "lens"))
    ref = {}
    for b in range(0, nB, 37):
        k = int(perm[b])
        if k not in ref:
            x = O.check_intervals(s[k], e[k], a[k], M, D=D)
            ref[k] = (x["mask"], x["peak"], x["dur"])
        assert (int(mask[b]), int(peak[b]), int(dur[b])) == ref[k], b
    first = {}
    for b in range(nB):
        k = int(perm[b])
        got = (int(mask[b]), int(peak[b]), int(dur[b]), int(lens[b]))
        assert first.setdefault(k, got) == got, b
