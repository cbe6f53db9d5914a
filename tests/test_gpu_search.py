"""Parity of the search entry points (through the C ABI) with the search oracle: after any number of
generations every chain's sequence, length, evaluation and acceptance count are identical."""
import os

import numpy as np
import pytest
import torch

from oracle import OracleGraph, OracleSearch
from paper_2304_14463_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2304_14463_b200 import build
    build.build()
    from paper_2304_14463_b200 import binding
    return binding


def dev(a, dtype=torch.int32):
    return torch.as_tensor(np.ascontiguousarray(a), dtype=dtype).cuda()


def assert_state_equal(S, OS, what=""):
    st = S.state()
    torch.cuda.synchronize()
    lens = st["lens"].cpu().numpy()
    assert (lens == OS.lens).all(), f"{what}: lengths differ at {np.nonzero(lens != OS.lens)[0][:5]}"
    for k, want in (("peak", OS.peak), ("dur", OS.dur), ("status", OS.status)):
        got = st[k].cpu().numpy()
        assert (got == want).all(), f"{what}: {k} differs at {np.nonzero(got != want)[0][:5]}"
    rows = st["rows"].cpu().numpy()
    for c in range(OS.P):
        assert (rows[c, :lens[c]] == OS.pop[c, :lens[c]]).all(), f"{what}: sequence of chain {c} differs"
    assert int(st["accepted"].sum()) == OS.accepted
    b = S.best()
    ob = OS.best()
    assert b["index"] == ob and b["accepted"] == OS.accepted
    if ob >= 0:
        assert (b["peak"], b["dur"], b["status"]) == (int(OS.peak[ob]), int(OS.dur[ob]), int(OS.status[ob]))
        assert (b["seq"] == OS.row(ob)).all()


def make_pair(B, wl, seqs, lens, M, seed):
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    S = B.Search(G, dev(seqs), dev(lens), M, seed)
    OS = OracleSearch(O, seqs, lens, M, seed, stride=S.info()["stride"])
    return G, O, S, OS


@pytest.mark.parametrize("idx,P,gens", [(0, 1024, (1, 2, 40)), (1, 512, (1, 9, 20)), (2, 384, (1, 6, 25)),
                                        (3, 96, (1, 5)), (4, 24, (1, 4))])
def test_search_parity(B, idx, P, gens):
    """Every configuration (C = 2 warp kernel and C = 3 group kernel), 1/16 of the start population
    damaged, budget 80 % of the no-rematerialization peak; state compared after each call."""
    wl = W.make(idx, seed=1, B=P)
    seqs, lens = W.mutate(wl.seqs, wl.lens, wl.n, wl.C, seed=5, frac=1 / 16)
    assert (lens <= wl.C * wl.n).all()
    O0 = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    M = O0.eval(np.arange(wl.n), 1 << 60)["peak"] * 80 // 100
    G, O, S, OS = make_pair(B, wl, seqs, lens, M, seed=(idx + 1) * 0x9E3779B97F4A7C15 % (1 << 64))
    assert_state_equal(S, OS, "start")
    for g in gens:
        S.run(g)
        OS.run(g)
        assert_state_equal(S, OS, f"config {idx} after {OS.generation} generations")
    assert S.info()["generation"] == OS.generation
    assert OS.accepted > 0


def test_search_from_identity_reaches_budget(B):
    """Chains that all start from the identity order: over budget at first (Phase 1), then feasible
    chains only trade duration (Phase 2); the key of every chain never increases."""
    wl = W.make(0, seed=2, B=256)
    n = wl.n
    seqs = np.tile(np.arange(n, dtype=np.int32), 256)
    lens = np.full(256, n, np.int32)
    O0 = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    P0 = O0.eval(np.arange(n), 1 << 60)["peak"]
    M = P0 * 90 // 100
    G, O, S, OS = make_pair(B, wl, seqs, lens, M, seed=77)
    prev = None
    for g in (10, 50, 200):
        S.run(g)
        OS.run(g)
        assert_state_equal(S, OS, f"after {OS.generation}")
        key = np.stack([np.maximum(OS.peak, M), OS.dur], 1)
        if prev is not None:
            assert ((key[:, 0] < prev[:, 0]) | ((key[:, 0] == prev[:, 0]) & (key[:, 1] <= prev[:, 1]))).all()
        prev = key


def test_search_split_invariance_and_errors(B):
    wl = W.make(2, seed=3, B=64)
    O0 = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    M = O0.eval(np.arange(wl.n), 1 << 60)["peak"] * 80 // 100
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    a = B.Search(G, dev(wl.seqs), dev(wl.lens), M, 5)
    b = B.Search(G, dev(wl.seqs), dev(wl.lens), M, 5)
    a.run(12)
    for k in (0, 5, 1, 6):
        b.run(k)
    sa, sb = a.state(), b.state()
    torch.cuda.synchronize()
    for k in ("rows", "lens", "peak", "dur", "status", "accepted"):
        assert torch.equal(sa[k], sb[k])
    assert B.moc_last_launch_count() >= 0
    # a population split over two handles evolves like the unsplit one
    half = 32
    offs = np.concatenate([[0], np.cumsum(wl.lens)])
    lo = B.Search(G, dev(wl.seqs[:offs[half]]), dev(wl.lens[:half]), M, 5)
    hi = B.Search(G, dev(wl.seqs[offs[half]:]), dev(wl.lens[half:]), M, 5, first_chain=half)
    lo.run(12)
    hi.run(12)
    sl, sh = lo.state(), hi.state()
    torch.cuda.synchronize()
    for k in ("rows", "lens", "peak", "dur", "status", "accepted"):
        assert torch.equal(torch.cat([sl[k], sh[k]]), sa[k])
    # a length beyond C*n is refused
    lens = wl.lens.copy()
    seqs = np.concatenate([wl.seqs, np.zeros(2 * wl.C * wl.n, np.int32)])
    lens[-1] = wl.C * wl.n + 1
    with pytest.raises(B.MocError) as e:
        B.Search(G, dev(seqs), dev(lens), M, 5)
    assert e.value.code == -1
    # an all-invalid population has no best chain
    bad = np.zeros(4 * wl.n, np.int32)
    s = B.Search(G, dev(bad), dev(np.full(4, wl.n, np.int32)), M, 1)
    assert s.best()["index"] == -1


@pytest.mark.parametrize("kinds", [4, 3, 5, 6, 1, 2])
def test_search_restricted_kinds(B, kinds):
    """Masks of enabled edits; moves only keeps every length and searches over orders."""
    wl = W.make(1, seed=2, B=256)
    O0 = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    M = O0.eval(np.arange(wl.n), 1 << 60)["peak"] * 80 // 100
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    S = B.Search(G, dev(wl.seqs), dev(wl.lens), M, 21)
    S.set_kinds(kinds)
    OS = OracleSearch(O, wl.seqs, wl.lens, M, 21, stride=S.info()["stride"], kinds=kinds)
    for g in (3, 30):
        S.run(g)
        OS.run(g)
        assert_state_equal(S, OS, f"kinds {kinds} after {OS.generation}")
    if kinds == 4:
        assert (OS.lens == wl.lens).all()
    with pytest.raises(B.MocError):
        S.set_kinds(0)
    with pytest.raises(B.MocError):
        S.set_kinds(8)


def test_search_full_size(B):
    """The benchmark's shape: the headline graph with 16384 chains, every chain compared."""
    wl = W.make(2, seed=1)
    O0 = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    M = O0.eval(np.arange(wl.n), 1 << 60)["peak"] * 80 // 100
    G, O, S, OS = make_pair(B, wl, wl.seqs, wl.lens, M, seed=1)
    assert OS.P == 16384
    for g in (1, 3):
        S.run(g)
        OS.run(g)
        assert_state_equal(S, OS, f"full size after {OS.generation}")


@pytest.mark.parametrize("idx,P,samples", [(0, 512, 1), (0, 512, 5), (1, 256, 4), (2, 256, 1), (2, 192, 16), (2, 64, 40)])
def test_search_incremental_parity(B, idx, P, samples):
    """Proposals scored from the cached evaluation (moc_search_set_samples): one or several per chain
    and generation; every chain identical to the search oracle after each call."""
    wl = W.make(idx, seed=3, B=P)
    O0 = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    M = O0.eval(np.arange(wl.n), 1 << 60)["peak"] * 80 // 100
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    S = B.Search(G, dev(wl.seqs), dev(wl.lens), M, 17)
    S.set_samples(samples, incremental=True)
    OS = OracleSearch(O, wl.seqs, wl.lens, M, 17, stride=S.info()["stride"], samples=samples)
    for g in (1, 2, 25):
        S.run(g)
        OS.run(g)
        assert_state_equal(S, OS, f"config {idx}, {samples} samples, after {OS.generation}")
    assert OS.accepted > 0
    if samples == 1:
        # back to proposals evaluated from scratch, and forth again: same chains as the oracle throughout
        S.set_samples(1, incremental=False)
        S.run(7)
        OS.run(7)
        assert_state_equal(S, OS, "after switching to full evaluation")
        S.set_samples(1, incremental=True)
        S.run(7)
        OS.run(7)
        assert_state_equal(S, OS, "after switching back")


def _run_scored(B, n, edges, w, m, C, seqs, lens, M, samples, mode, gens, caps=None, kinds=7, what=""):
    G = B.Graph(n, edges, w, m, C)
    O = OracleGraph(n, edges, w, m, C)
    if caps is not None:
        G.set_caps(caps)
        O.set_caps(caps)
    S = B.Search(G, dev(seqs), dev(lens), M, 23)
    if kinds != 7:
        S.set_kinds(kinds)
    S.set_samples(samples, incremental=mode)
    OS = OracleSearch(O, seqs, lens, M, 23, stride=S.info()["stride"], kinds=kinds, samples=samples)
    for g in gens:
        S.run(g)
        OS.run(g)
        assert_state_equal(S, OS, f"{what}: mode {mode}, {samples} samples, after {OS.generation}")
    return S, OS


@pytest.mark.parametrize("mode", [2, 3])
@pytest.mark.parametrize("idx,P,samples", [(0, 256, 5), (1, 128, 33), (2, 96, 16), (2, 48, 70)])
def test_search_scoring_kernels_agree_with_oracle(B, idx, P, samples, mode):
    """The two scoring kernels of the search on the cached evaluation, each forced: a warp per proposal (2) and
    a warp per chain (3; fewer proposals than lanes, a pass and a bit, more than two passes)."""
    wl = W.make(idx, seed=4, B=P)
    O0 = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    M = O0.eval(np.arange(wl.n), 1 << 60)["peak"] * 80 // 100
    S, OS = _run_scored(B, wl.n, wl.edges, wl.w, wl.m, wl.C, wl.seqs, wl.lens, M, samples, mode, (1, 3, 20), what=f"config {idx}")
    assert OS.accepted > 0
    # the other kernel takes over the same chains in mid-search
    S.set_samples(samples, incremental=5 - mode)
    S.run(5)
    OS.run(5)
    assert_state_equal(S, OS, "after switching the scoring kernel")


@pytest.mark.parametrize("mode", [2, 3])
def test_search_scoring_caps_kinds_and_wide(B, mode):
    """Per-node caps, restricted kinds of edit and 64-bit memory sums through both scoring kernels."""
    wl = W.make(1, seed=6, B=96)
    rng = np.random.default_rng(11)
    caps = np.where(rng.random(wl.n) < 0.5, 1, 2).astype(np.int32)
    rows = [np.arange(wl.n, dtype=np.int32) for _ in range(96)]           # the identity order respects every cap
    seqs, lens = W.pack(rows)
    O0 = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    M = O0.eval(np.arange(wl.n), 1 << 60)["peak"] * 80 // 100
    _, OS = _run_scored(B, wl.n, wl.edges, wl.w, wl.m, wl.C, seqs, lens, M, 12, mode, (2, 30), caps=caps, what="caps")
    assert OS.accepted > 0
    for kinds in (1, 3, 6):
        _run_scored(B, wl.n, wl.edges, wl.w, wl.m, wl.C, wl.seqs, wl.lens, M, 9, mode, (1, 12), kinds=kinds, what=f"kinds {kinds}")
    big = wl.m * (1 << 33)
    _, OS = _run_scored(B, wl.n, wl.edges, wl.w, big, wl.C, wl.seqs, wl.lens, M * (1 << 33), 40, mode, (1, 15), what="wide")
    assert OS.accepted > 0 and int(OS.peak.max()) > (1 << 40)


def _layered_dense(width, layers, seed):
    """Every node of a layer feeds every node of the next: in-degree = out-degree = width."""
    rng = np.random.default_rng(seed)
    n = width * layers
    edges = np.array([(a * width + i, (a + 1) * width + k) for a in range(layers - 1) for i in range(width)
                      for k in range(width)], np.int32)
    return n, edges, rng.integers(1, 50, n).astype(np.int64), rng.integers(1, 1000, n).astype(np.int64)


def test_search_chain_kernel_in_rounds(B):
    """In-degree 30: one proposal may need 64 entries of the 128-entry correction list of a warp, so a pass with
    more than two admissible proposals is scored in several rounds.  A copy inserted behind the node's first one
    is always admissible, so with inserts only about half of the 32 proposals of a pass are."""
    n, edges, w, m = _layered_dense(30, 3, 2)
    rng = np.random.default_rng(3)
    rows = []
    for _ in range(48):
        r = np.concatenate([rng.permutation(30) + 30 * a for a in range(3)]).astype(np.int32)
        rows.append(r)
    seqs, lens = W.pack(rows)
    O0 = OracleGraph(n, edges, w, m, 2)
    M = O0.eval(np.arange(n), 1 << 60)["peak"] * 90 // 100
    for mode in (3, 2):
        _run_scored(B, n, edges, w, m, 2, seqs, lens, M, 32, mode, (1, 2, 10), kinds=1, what="dense, inserts")
        _, OS = _run_scored(B, n, edges, w, m, 2, seqs, lens, M, 48, mode, (1, 8), what="dense, all kinds")
        assert OS.accepted > 0


def test_search_chain_kernel_refuses_what_it_cannot_hold(B):
    """A graph whose rows and correction lists do not fit four warps of an SM: the warp-per-chain kernel is
    refused when asked for by name, and the automatic choice scores with a warp per proposal instead."""
    n = 1700
    edges = np.array([(i, n - 1) for i in range(n - 1)], np.int32)          # in-degree 1699
    rng = np.random.default_rng(1)
    w, m = rng.integers(1, 9, n).astype(np.int64), rng.integers(1, 99, n).astype(np.int64)
    rows = [np.concatenate([rng.permutation(n - 1), [n - 1]]).astype(np.int32) for _ in range(6)]
    seqs, lens = W.pack(rows)
    G = B.Graph(n, edges, w, m, 2)
    S = B.Search(G, dev(seqs), dev(lens), 1 << 60, 5)
    with pytest.raises(B.MocError) as e:
        S.set_samples(8, incremental=3)
    assert e.value.code == -1 and "in-degree" in str(e.value)
    O = OracleGraph(n, edges, w, m, 2)
    S.set_samples(8, incremental=1)
    OS = OracleSearch(O, seqs, lens, 1 << 60, 5, stride=S.info()["stride"], samples=8)
    S.run(3)
    OS.run(3)
    assert_state_equal(S, OS, "star graph, automatic choice")


def test_search_incremental_errors(B):
    wl = W.make(1, seed=3, B=32)
    O0 = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    M = O0.eval(np.arange(wl.n), 1 << 60)["peak"] * 80 // 100
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    seqs = wl.seqs.copy()
    seqs[:wl.lens[0]] = seqs[:wl.lens[0]][::-1]            # chain 0 starts from an invalid order
    S = B.Search(G, dev(seqs), dev(wl.lens), M, 1)
    with pytest.raises(B.MocError) as e:
        S.set_samples(4, incremental=True)
    assert e.value.code == -1
    with pytest.raises(B.MocError):
        S.set_samples(4, incremental=False)                 # several samples need the incremental evaluation
    with pytest.raises(B.MocError):
        S.set_samples(0, incremental=True)
    with pytest.raises(B.MocError):
        S.set_samples(4, incremental=4)                     # modes are 0..3
    S.run(3)                                                # still usable in the old way
    wl3 = W.make(3, seed=1, B=8)                            # C = 3: outside the incremental evaluation
    G3 = B.Graph(wl3.n, wl3.edges, wl3.w, wl3.m, wl3.C)
    S3 = B.Search(G3, dev(wl3.seqs), dev(wl3.lens), 1 << 60, 1)
    with pytest.raises(B.MocError):
        S3.set_samples(2, incremental=True)


# ------------------------------------------------------------------ a population split over two ranks
def _rank_worker(rank, world, port, q):
    import os
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    sys.path.insert(0, root)
    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2304_14463_b200 import binding, sharding, workloads
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    torch.cuda.set_device(0)                        # both ranks share the one GPU; nothing waits on a peer's kernel
    wl = workloads.make(1, seed=6, B=192, n_threads=1)
    G = binding.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    M = workloads.budget_from_peak(G.no_remat_peak(), 85)
    my_seqs, my_lens = sharding.shard_batch(wl.seqs, wl.lens, rank, world)
    b0, b1 = sharding.shard_range(len(wl.lens), rank, world)
    S = binding.Search(G, torch.from_numpy(np.ascontiguousarray(my_seqs)).cuda(), torch.from_numpy(np.ascontiguousarray(my_lens)).cuda(),
                       M, seed=11, first_chain=b0)
    S.run(25)
    st = S.state()
    torch.cuda.synchronize()
    mine = S.best()
    got = sharding.best_over_ranks(mine, M, b0, wl.C * wl.n)
    lens_all = [torch.zeros(len(wl.lens), dtype=torch.int64) for _ in range(world)]
    part = torch.zeros(len(wl.lens), dtype=torch.int64)
    part[b0:b1] = st["lens"].cpu().to(torch.int64)
    dist.all_gather(lens_all, part)
    if rank == 0:
        full = binding.Search(G, torch.from_numpy(wl.seqs).cuda(), torch.from_numpy(wl.lens).cuda(), M, seed=11)
        full.run(25)
        fs = full.state()
        fb = full.best()
        torch.cuda.synchronize()
        same_lens = bool((sum(lens_all) == fs["lens"].cpu().to(torch.int64)).all())
        q.put((same_lens, got["index"] == fb["index"], bool((got["seq"] == fb["seq"]).all()),
               (got["peak"], got["dur"], got["status"]) == (fb["peak"], fb["dur"], fb["status"])))
    dist.barrier()
    dist.destroy_process_group()


def test_population_split_over_two_ranks_on_the_gpu():
    """Two processes (gloo for the host-side exchange), each driving a CUDA search handle on its half of
    the chains with their global chain numbers: the chains evolve exactly as in the unsplit CUDA run and
    the best chain over the ranks is the unsplit best."""
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 33500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    out = q.get(timeout=300)
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    assert out == (True, True, True, True)
