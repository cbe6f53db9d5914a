"""Parity of the CUDA path (through the C ABI) with the CPU oracle: bit-exact on peak, duration,
status, and -- for moc_mem_profile -- on every profile entry and free step."""
import numpy as np
import pytest
import torch

import pins
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


def gpu_eval(G, seqs, lens, M):
    peak, dur, st = G.eval_batch(dev(seqs), dev(lens), M)
    torch.cuda.synchronize()
    return peak.cpu().numpy(), dur.cpu().numpy(), st.cpu().numpy()


def assert_batch_equal(G, O, seqs, lens, M, what=""):
    gp, gd, gs = gpu_eval(G, seqs, lens, M)
    op, od, os_, _ = O.eval_batch(seqs, lens, M, n_threads=4)
    bad = np.nonzero((gp != op) | (gd != od) | (gs != os_))[0]
    assert len(bad) == 0, f"{what}: {len(bad)} of {len(lens)} differ, first {bad[:5]}: gpu " \
                          f"{gp[bad[:3]], gd[bad[:3]], gs[bad[:3]]} oracle {op[bad[:3]], od[bad[:3]], os_[bad[:3]]}"
    return op, od, os_


# ------------------------------------------------------------------ the oracle's pins, on the GPU
def test_pins_through_the_gpu(B):
    class GpuGraph:
        def __init__(self, n, edges, w, m, C):
            self.G = B.Graph(n, edges, w, m, C)

        def set_caps(self, caps):
            self.G.set_caps(caps)

        def eval(self, seq, M):
            seq = np.asarray(seq, np.int32)
            p, d, s = gpu_eval(self.G, seq, np.array([len(seq)], np.int32), M)
            prof, free, st = self.G.mem_profile(dev(seq))
            torch.cuda.synchronize()
            assert (int(st[0]) < 0) == (int(s[0]) < 0) and (int(s[0]) >= 0 or int(st[0]) == int(s[0]))
            return dict(peak=int(p[0]), dur=int(d[0]), status=int(s[0]),
                        profile=prof.cpu().numpy(), free=free.cpu().numpy())

    for pin in (pins.pin_paper_example, pins.pin_small_cases, pins.pin_random_remat, pins.pin_node_caps):
        pin(lambda n, e, w, m, C: GpuGraph(n, e, w, m, C))


# ------------------------------------------------------------------ the five configurations
SMALL_B = [1024, 4096, 2048, 512, 64]


@pytest.mark.parametrize("idx", range(W.N_CONFIGS))
@pytest.mark.parametrize("seed", [1, 2, 3])
def test_config_parity_mutated(B, idx, seed):
    """Reduced batches, 1/16 of the sequences damaged, budgets that make both 0 and 1 occur."""
    wl = W.make(idx, seed=seed, B=SMALL_B[idx])
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    P0 = O.eval(np.arange(wl.n), BIG)["peak"]
    assert G.no_remat_peak() == P0
    seqs, lens = W.mutate(wl.seqs, wl.lens, wl.n, wl.C, seed=seed, frac=1 / 16)
    peaks = O.eval_batch(seqs, lens, BIG)[0]
    median = int(np.median(peaks[peaks >= 0]))
    seen = set()
    for M in [W.budget_from_peak(P0, p) for p in wl.budget_pcts] + [P0, median]:
        _, _, st = assert_batch_equal(G, O, seqs, lens, M, f"{wl.name} seed {seed} M {M}")
        seen |= set(np.unique(st).tolist())
    assert {-2, 0, 1} <= seen and (idx == 4 or -1 in seen)


@pytest.mark.parametrize("idx", range(W.N_CONFIGS))
def test_config_parity_full_size(B, idx):
    """The full batch of every configuration in the launch shape the benchmark times."""
    wl = W.make(idx, seed=1)
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    P0 = G.no_remat_peak()
    for pct in wl.budget_pcts:
        assert_batch_equal(G, O, wl.seqs, wl.lens, W.budget_from_peak(P0, pct), f"{wl.name} {pct}%")


@pytest.mark.parametrize("idx", [0, 1, 2, 3, 4])
def test_wide_arithmetic(B, idx):
    """Output sizes scaled so that sums need 64 bits."""
    wl = W.make(idx, seed=4, B=min(SMALL_B[idx], 256))
    m = wl.m * (1 << 24) + 12345
    O = OracleGraph(wl.n, wl.edges, wl.w * (1 << 30), m, wl.C)
    G = B.Graph(wl.n, wl.edges, wl.w * (1 << 30), m, wl.C)
    assert G.info()["wide"]
    seqs, lens = W.mutate(wl.seqs, wl.lens, wl.n, wl.C, seed=9, frac=1 / 8)
    peaks = O.eval_batch(seqs, lens, BIG)[0]
    assert peaks.max() > (1 << 32)
    assert_batch_equal(G, O, seqs, lens, int(np.median(peaks[peaks >= 0])), wl.name)


@pytest.mark.parametrize("idx", [0, 2, 3])
def test_mem_profile_parity(B, idx):
    wl = W.make(idx, seed=5, B=24)
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    seqs, lens = W.mutate(wl.seqs, wl.lens, wl.n, wl.C, seed=2, frac=0.3)
    for seq in W.unpack(seqs, lens):
        r = O.eval(seq, BIG)
        prof, free, st = G.mem_profile(dev(seq))
        torch.cuda.synchronize()
        assert int(st[0]) == r["status"]
        assert (prof.cpu().numpy() == r["profile"]).all() and (free.cpu().numpy() == r["free"]).all()
    prof, free, st = G.mem_profile(dev(seq), want_free=False)
    torch.cuda.synchronize()
    assert free is None and (prof.cpu().numpy() == r["profile"]).all()


# ------------------------------------------------------------------ every kernel family
LANE_SHAPES = [(0, 0), (32, 32), (16, 32), (16, 16), (8, 32), (8, 24), (8, 16), (8, 8)]


@pytest.mark.parametrize("idx", [0, 1, 2])
@pytest.mark.parametrize("a,b", LANE_SHAPES)
def test_lane_kernel_shapes(B, idx, a, b):
    """The sequence-per-lane kernel in every group size and with few and many warps: damaged batches of
    the three configurations it serves, a batch size that leaves the last group ragged."""
    wl = W.make(idx, seed=7, B=[333, 1500, 777][idx])
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G.set_kernel(B.MOC_KERNEL_LANE, a, b)
    seqs, lens = W.mutate(wl.seqs, wl.lens, wl.n, wl.C, seed=5, frac=1 / 8)
    peaks = O.eval_batch(seqs, lens, BIG)[0]
    assert_batch_equal(G, O, seqs, lens, int(np.median(peaks[peaks >= 0])), f"lane {a}x{b} {wl.name}")


@pytest.mark.parametrize("kind", ["group", "warp", "lane", "block"])
@pytest.mark.parametrize("idx", [0, 1, 2])
def test_kernel_families_agree_with_oracle(B, idx, kind):
    """Each family forced in turn on the full batch of the configurations all of them can serve."""
    wl = W.make(idx, seed=2)
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G.set_kernel({"group": B.MOC_KERNEL_GROUP, "warp": B.MOC_KERNEL_WARP, "lane": B.MOC_KERNEL_LANE,
                  "block": B.MOC_KERNEL_BLOCK}[kind])
    assert_batch_equal(G, O, wl.seqs, wl.lens, W.budget_from_peak(G.no_remat_peak(), 80), f"{kind} {wl.name}")
    assert B.moc_last_launch_count() >= 1


@pytest.mark.parametrize("idx", range(W.N_CONFIGS))
@pytest.mark.parametrize("threads", [0, 64, 160, 1024])
def test_block_kernel_shapes(B, idx, threads):
    """The block-per-sequence kernel with packed words on damaged batches of every configuration (C = 2 and 3),
    with few and many threads per sequence."""
    wl = W.make(idx, seed=8, B=[300, 400, 200, 96, 24][idx])
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G.set_kernel(B.MOC_KERNEL_BLOCK, threads, 0)
    seqs, lens = W.mutate(wl.seqs, wl.lens, wl.n, wl.C, seed=6, frac=1 / 8)
    peaks = O.eval_batch(seqs, lens, BIG)[0]
    _, _, st = assert_batch_equal(G, O, seqs, lens, int(np.median(peaks[peaks >= 0])), f"block {threads} {wl.name}")
    assert {0, 1} <= set(st.tolist()) and (idx == 4 or -2 in st)


@pytest.mark.parametrize("C", [1, 2, 3, 4])
def test_block_kernel_every_cap_and_wide(B, C):
    """Caps 1..4, per-node caps, and sums that need 64 bits, on sequences with up to four copies per node."""
    wl = W.make(1, seed=3, B=64)
    rng = np.random.default_rng(C)
    rows = []
    for _ in range(200):
        r = list(rng.permutation(wl.n)) if rng.random() < 0.1 else list(range(wl.n))
        for v in range(wl.n):
            for _ in range(int(rng.integers(0, 5)) if rng.random() < 0.15 else 0):
                r.insert(int(rng.integers(r.index(v) + 1, len(r) + 1)), v)
        rows.append(r)
    seqs, lens = W.pack(rows)
    for scale, caps in ((1, None), (1 << 26, None), (1, np.asarray(rng.integers(1, C + 1, wl.n), np.int32))):
        m = wl.m * scale
        O = OracleGraph(wl.n, wl.edges, wl.w, m, C)
        G = B.Graph(wl.n, wl.edges, wl.w, m, C)
        if caps is not None:
            O.set_caps(caps)
            G.set_caps(caps)
        G.set_kernel(B.MOC_KERNEL_BLOCK)
        peaks = O.eval_batch(seqs, lens, BIG)[0]
        M = int(np.median(peaks[peaks >= 0])) if (peaks >= 0).any() else 1
        _, _, st = assert_batch_equal(G, O, seqs, lens, M, f"block C={C} scale={scale} caps={caps is not None}")
    assert G.info()["wide"] is False or scale > 1


def test_lane_kernel_refuses_what_it_cannot_serve(B):
    wl = W.make(3, seed=1, B=8)                          # C = 3
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G.set_kernel(B.MOC_KERNEL_LANE)
    with pytest.raises(B.MocError):
        G.eval_batch(dev(wl.seqs), dev(wl.lens), BIG)
    G.set_kernel(B.MOC_KERNEL_AUTO)
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    assert_batch_equal(G, O, wl.seqs, wl.lens, BIG, "auto after a refused kind")


# ------------------------------------------------------------------ launch shapes, alignment, edges
@pytest.mark.parametrize("tps,spb", [(0, 0), (0, 4), (0, 8), (0, 12), (0, 16), (32, 1), (32, 8), (32, 16), (64, 4), (128, 2), (256, 1), (256, 3),
                                     (512, 1), (512, 2), (1024, 1)])
def test_every_launch_shape(B, tps, spb):
    wl = W.make(2, seed=6, B=700)
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G.set_launch(tps, spb)
    seqs, lens = W.mutate(wl.seqs, wl.lens, wl.n, wl.C, seed=3, frac=1 / 8)
    peaks = O.eval_batch(seqs, lens, BIG)[0]
    assert_batch_equal(G, O, seqs, lens, int(np.median(peaks[peaks >= 0])), f"shape {tps}x{spb}")


@pytest.mark.parametrize("C", [1, 2, 3, 4, 5, 8])
def test_every_copy_cap(B, C):
    n = 150
    edges = W.layered_dag(n, 400, 10, seed=C)
    w = W.weights_uniform(n, 1, 9, 1, 1)
    m = W.weights_lognormal(n, 5.0, 1.0, 1, 2)
    seqs, lens = W.schedules(n, edges, C, 0.35, 300, seed=C)
    seqs, lens = W.mutate(seqs, lens, n, C, seed=C, frac=1 / 8)
    O = OracleGraph(n, edges, w, m, C)
    G = B.Graph(n, edges, w, m, C)
    peaks = O.eval_batch(seqs, lens, BIG)[0]
    assert_batch_equal(G, O, seqs, lens, int(np.median(peaks[peaks >= 0])), f"C={C}")
    # the cap is what makes a sequence malformed: the same sequences under a smaller cap
    if C > 1:
        O2 = OracleGraph(n, edges, w, m, C - 1)
        B.moc_graph_set_max_copies(G.h, C - 1)
        assert_batch_equal(G, O2, seqs, lens, BIG, f"C={C} evaluated with cap {C - 1}")


def test_unaligned_rows_and_views(B):
    """Rows start at every 4-byte phase; the packed array itself starts off a 16-byte boundary."""
    wl = W.make(1, seed=7, B=500)
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    op, od, os_, _ = O.eval_batch(wl.seqs, wl.lens, BIG)
    for shift in (1, 2, 3):
        buf = torch.zeros(len(wl.seqs) + 8, dtype=torch.int32, device="cuda")
        view = buf[shift:shift + len(wl.seqs)]
        view.copy_(dev(wl.seqs))
        assert view.data_ptr() % 16 == 4 * shift
        peak, dur, st = G.eval_batch(view, dev(wl.lens), BIG)
        torch.cuda.synchronize()
        assert (peak.cpu().numpy() == op).all() and (dur.cpu().numpy() == od).all() and (st.cpu().numpy() == os_).all()


def test_rows_found_in_kernel(B):
    """Batches small enough for the warp-per-sequence kernel to locate its rows itself: ranges that
    do not divide evenly, fewer sequences than warps, a length array off a 16-byte boundary, very
    long and negative lengths in front of valid rows."""
    wl = W.make(2, seed=10, B=1500)
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    rows = W.unpack(wl.seqs, wl.lens)
    for nb in (1, 2, 11, 13, 445, 1499):
        seqs, lens = W.pack(rows[:nb])
        assert_batch_equal(G, O, seqs, lens, BIG, f"{nb} sequences")
        assert B.moc_last_launch_count() == 1
    seqs, lens = W.mutate(wl.seqs, wl.lens, wl.n, wl.C, seed=6, frac=0.2)
    lens = lens.copy()
    junk = np.full(3000, 7, np.int32)
    lens2 = np.concatenate([[-5, 3000], lens, [0, -1]]).astype(np.int32)     # a 3000-step malformed row first
    seqs2 = np.concatenate([junk, seqs]).astype(np.int32)
    op, od, os_, _ = O.eval_batch(seqs2, lens2, 10 ** 6)
    buf = torch.zeros(len(lens2) + 3, dtype=torch.int32, device="cuda")
    view = buf[1:1 + len(lens2)]
    view.copy_(dev(lens2))
    assert view.data_ptr() % 16 == 4
    peak, dur, st = G.eval_batch(dev(seqs2), view, 10 ** 6)
    torch.cuda.synchronize()
    assert (peak.cpu().numpy() == op).all() and (dur.cpu().numpy() == od).all() and (st.cpu().numpy() == os_).all()
    assert os_[0] == -2 and os_[1] == -2 and os_[-1] == -2


def test_degenerate_batches(B):
    n = 5
    edges = [(0, 1), (1, 2), (0, 3)]
    w = np.arange(1, 6)
    m = np.array([5, 1, 2, 3, 4])
    O = OracleGraph(n, edges, w, m, 2)
    G = B.Graph(n, edges, w, m, 2)
    # B = 0: nothing happens
    e = torch.empty(0, dtype=torch.int32, device="cuda")
    p, d, s = G.eval_batch(e, e, 10)
    assert p.numel() == 0 and B.moc_last_launch_count() == 0
    # zero, negative, too short, exactly n, exactly C*n, too long
    rows = [[], [0, 1, 2], [0, 1, 2, 3, 4], [0, 0, 1, 1, 2, 2, 3, 3, 4, 4], [0, 1, 2, 3, 4] * 2 + [0], [4, 3, 2, 1, 0]]
    seqs, lens = W.pack(rows)
    lens = np.concatenate([lens, [-3]]).astype(np.int32)
    assert_batch_equal(G, O, seqs, lens, 9, "degenerate")
    # single isolated node
    O1, G1 = OracleGraph(1, [], [7], [3], 2), B.Graph(1, [], [7], [3], 2)
    seqs, lens = W.pack([[0], [0, 0], [0, 0, 0], [1]])
    assert_batch_equal(G1, O1, seqs, lens, 3, "single node")
    # duplicate edges are merged
    G2 = B.Graph(n, edges + edges, w, m, 2)
    assert G2.info()["n_edges"] == 3
    # mem_profile of an empty and of a malformed sequence
    prof, free, st = G.mem_profile(torch.empty(0, dtype=torch.int32, device="cuda"))
    torch.cuda.synchronize()
    assert int(st[0]) == -2
    prof, free, st = G.mem_profile(dev([0, 1, 2, 3, 9]))
    torch.cuda.synchronize()
    assert int(st[0]) == -2 and (prof.cpu().numpy() == -1).all() and (free.cpu().numpy() == -1).all()


def test_determinism_and_reuse(B):
    wl = W.make(2, seed=8, B=3000)
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    s, l = dev(wl.seqs), dev(wl.lens)
    a = [t.clone() for t in G.eval_batch(s, l, 12345678)]
    for _ in range(3):
        b = G.eval_batch(s, l, 12345678)
        torch.cuda.synchronize()
        assert all(torch.equal(x, y) for x, y in zip(a, b))
    # a smaller batch after a larger one on the same handle
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    assert_batch_equal(G, O, wl.seqs[:int(wl.lens[:10].sum())], wl.lens[:10], BIG, "reuse")
    assert B.moc_last_launch_count() == 1          # the warp-per-sequence kernel finds its rows itself
    G.set_launch(64, 4)                            # the group kernel runs behind the offsets kernel
    assert_batch_equal(G, O, wl.seqs[:int(wl.lens[:10].sum())], wl.lens[:10], BIG, "reuse, group kernel")
    assert B.moc_last_launch_count() == 2


def test_handles_of_different_size_interleaved(B):
    """Two graphs that use the same kernels with very different shared-memory footprints."""
    big = W.make(2, seed=11, B=600)
    small = W.make(0, seed=11, B=600)
    Gb, Gs = B.Graph(big.n, big.edges, big.w, big.m, big.C), B.Graph(small.n, small.edges, small.w, small.m, small.C)
    Ob, Os = OracleGraph(big.n, big.edges, big.w, big.m, big.C), OracleGraph(small.n, small.edges, small.w, small.m, small.C)
    for shape in ((0, 0), (128, 2)):
        Gb.set_launch(*shape)
        Gs.set_launch(*shape)
        for _ in range(2):
            assert_batch_equal(Gb, Ob, big.seqs, big.lens, BIG, "large graph")
            assert_batch_equal(Gs, Os, small.seqs, small.lens, BIG, "small graph")


def test_timing_hook(B):
    wl = W.make(2, seed=8, B=2000)
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    s, l = dev(wl.seqs), dev(wl.lens)
    ref = [t.clone() for t in G.eval_batch(s, l, BIG)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    G.set_timing_events(e0, e1)
    out = G.eval_batch(s, l, BIG)
    G.set_timing_events(None, None)
    torch.cuda.synchronize()
    assert 0.0 < e0.elapsed_time(e1) < 50.0 and all(torch.equal(a, b) for a, b in zip(ref, out))
    with pytest.raises(B.MocError):
        B._check(B.lib.moc_graph_set_timing_events(G.h, None, 1), "half a pair")


def test_host_entry_point(B):
    wl = W.make(1, seed=9, B=2000)
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    seqs = torch.from_numpy(wl.seqs).pin_memory()
    lens = torch.from_numpy(wl.lens).pin_memory()
    peak = torch.empty(wl.B, dtype=torch.int64).pin_memory()
    dur = torch.empty(wl.B, dtype=torch.int64).pin_memory()
    st = torch.empty(wl.B, dtype=torch.int32).pin_memory()
    M = 30000
    G.eval_batch_host(seqs, lens, M, peak, dur, st)
    op, od, os_, _ = O.eval_batch(wl.seqs, wl.lens, M)
    assert (peak.numpy() == op).all() and (dur.numpy() == od).all() and (st.numpy() == os_).all()
    # pageable numpy arrays work too
    p2, d2, s2 = np.empty(wl.B, np.int64), np.empty(wl.B, np.int64), np.empty(wl.B, np.int32)
    G.eval_batch_host(wl.seqs, wl.lens, M, p2, d2, s2)
    assert (p2 == op).all() and (d2 == od).all() and (s2 == os_).all()


def test_host_entry_point_u16(B):
    """16-bit node ids from the host: same results, ids >= n stay out of range, odd lengths and tails."""
    wl = W.make(2, seed=4, B=777)
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    seqs, lens = W.mutate(wl.seqs, wl.lens, wl.n, wl.C, seed=2, frac=1 / 8)
    seqs = np.where(seqs < 0, 65535, seqs).astype(np.int32)          # what 16 bits can carry of a damaged id
    M = O.eval(np.arange(wl.n), BIG)["peak"] * 80 // 100
    op, od, os_, _ = O.eval_batch(seqs, lens, M)
    s16 = torch.from_numpy(seqs.astype(np.uint16)).pin_memory()
    l = torch.from_numpy(lens).pin_memory()
    peak = torch.empty(len(lens), dtype=torch.int64).pin_memory()
    dur = torch.empty(len(lens), dtype=torch.int64).pin_memory()
    st = torch.empty(len(lens), dtype=torch.int32).pin_memory()
    for _ in range(2):
        G.eval_batch_host16(s16, l, M, peak, dur, st)
        assert (peak.numpy() == op).all() and (dur.numpy() == od).all() and (st.numpy() == os_).all()
    assert (os_ == -2).any() and (os_ >= 0).any()
    # pageable, unaligned source
    buf = np.zeros(len(seqs) + 1, np.uint16)
    buf[1:] = seqs
    p2, d2, s2 = np.empty(len(lens), np.int64), np.empty(len(lens), np.int64), np.empty(len(lens), np.int32)
    G.eval_batch_host16(buf[1:], lens, M, p2, d2, s2)
    assert (p2 == op).all() and (d2 == od).all() and (s2 == os_).all()


def test_host_entry_points_in_chunks(B):
    """A batch large enough to travel in several chunks (copy of one chunk under the evaluation of the
    one before), cut at sequence boundaries that do not divide the batch evenly; damaged sequences and
    a zero-length one sit at chunk edges like anywhere else."""
    wl = W.make(2, seed=11, B=5003)
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    seqs, lens = W.mutate(wl.seqs, wl.lens, wl.n, wl.C, seed=3, frac=1 / 8)
    seqs = np.where(seqs < 0, 65535, seqs).astype(np.int32)
    M = O.eval(np.arange(wl.n), BIG)["peak"] * 80 // 100
    op, od, os_, _ = O.eval_batch(seqs, lens, M)
    l = torch.from_numpy(lens).pin_memory()
    outs = [torch.empty(len(lens), dtype=dt).pin_memory() for dt in (torch.int64, torch.int64, torch.int32)]
    for rep in range(2):
        G.eval_batch_host(torch.from_numpy(seqs).pin_memory(), l, M, *outs)
        assert B.moc_last_launch_count() >= 3
        assert (outs[0].numpy() == op).all() and (outs[1].numpy() == od).all() and (outs[2].numpy() == os_).all()
        for o in outs:
            o.zero_()
        G.eval_batch_host16(torch.from_numpy(seqs.astype(np.uint16)).pin_memory(), l, M, *outs)
        assert B.moc_last_launch_count() >= 6
        assert (outs[0].numpy() == op).all() and (outs[1].numpy() == od).all() and (outs[2].numpy() == os_).all()
    # the device entry point on the same handle in between is not disturbed
    assert_batch_equal(G, O, seqs[:int(np.clip(lens[:100], 0, None).sum())], lens[:100], M, "after host calls")


def test_state_in_global_memory(B):
    """A graph whose per-sequence state exceeds shared memory (and > 65534 steps per sequence)."""
    n, C = 40000, 2
    edges = W.layered_dag(n, 3 * n, 40, seed=3)
    w = W.weights_uniform(n, 1, 100, 3, 1)
    m = W.weights_lognormal(n, 8.0, 2.0, 3, 2)
    seqs, lens = W.schedules(n, edges, C, 0.7, 6, seed=11)
    assert lens.max() > 65534
    seqs, lens = W.mutate(seqs, lens, n, C, seed=1, frac=0.34)
    O = OracleGraph(n, edges, w, m, C)
    G = B.Graph(n, edges, w, m, C)
    peaks = O.eval_batch(seqs, lens, BIG)[0]
    assert_batch_equal(G, O, seqs, lens, int(np.median(peaks[peaks >= 0])), "global state")
    seq = W.unpack(seqs, lens)[int(np.argmax(peaks >= 0))]
    r = O.eval(seq, BIG)
    prof, free, st = G.mem_profile(dev(seq))
    torch.cuda.synchronize()
    assert int(st[0]) == 1 and (prof.cpu().numpy() == r["profile"]).all() and (free.cpu().numpy() == r["free"]).all()


def test_sampled_invariants_at_full_size(B):
    """Properties that hold at any size, on the benchmark workload (no oracle involved)."""
    wl = W.make(2, seed=1)
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    peak, dur, st = gpu_eval(G, wl.seqs, wl.lens, BIG)
    lower = wl.m.copy()
    np.add.at(lower, wl.edges[:, 1], wl.m[wl.edges[:, 0]])
    assert (st == 1).all() and (peak >= lower.max()).all()
    offs = np.concatenate([[0], np.cumsum(wl.lens)])
    wsum = np.add.reduceat(wl.w[wl.seqs], offs[:-1])
    msum = np.add.reduceat(wl.m[wl.seqs], offs[:-1])
    assert (dur == wsum).all() and (peak <= msum).all()


@pytest.mark.parametrize("idx", [1, 2, 3])
def test_node_caps_parity(B, idx):
    """Random per-node caps C_v on the warp-per-sequence kernel (C = 2) and the group kernel (C = 3)."""
    wl = W.make(idx, seed=2, B=[0, 2048, 1024, 256][idx])
    rng = np.random.default_rng(idx)
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    seqs, lens = W.mutate(wl.seqs, wl.lens, wl.n, wl.C, seed=4, frac=1 / 16)
    M = O.eval(np.arange(wl.n), BIG)["peak"] * 80 // 100
    for frac_one in (0.02, 0.5, 1.0):
        caps = np.where(rng.random(wl.n) < frac_one, 1, rng.integers(1, wl.C + 1, wl.n)).astype(np.int32)
        O.set_caps(caps)
        G.set_caps(caps)
        _, _, st = assert_batch_equal(G, O, seqs, lens, M, f"caps {frac_one}")
        assert (st == -2).any()
    O.set_caps(None)
    G.set_caps(None)
    _, _, st = assert_batch_equal(G, O, seqs, lens, M, "caps cleared")
    assert (st >= 0).any()
    with pytest.raises(B.MocError):
        G.set_caps(np.full(wl.n, wl.C + 1, np.int32))
