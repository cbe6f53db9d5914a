"""moc_eval_batch_noalloc: the entry point for callers that cannot allocate device memory (their
framework owns all of it, or they cannot afford the allocator's locks and synchronisation).  It
keeps its scratch in a fixed array inside the library, shared by all calls, so the test runs two
calls in a row -- a large batch, then a smaller, different one that leaves stale entries behind --
and wants each to equal moc_eval_batch bit for bit.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from oracle import OracleGraph
from paper_2304_14463_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2304_14463_b200 import build
    build.build()
    from paper_2304_14463_b200 import binding
    return binding


def _outputs(n):
    return (torch.empty(n, dtype=torch.int64, device="cuda"), torch.empty(n, dtype=torch.int64, device="cuda"),
            torch.empty(n, dtype=torch.int32, device="cuda"))


def test_two_calls_match_the_allocating_entry_point(B):
    wl = W.make(2, seed=12, B=3000)
    seqs, lens = W.mutate(wl.seqs, wl.lens, wl.n, wl.C, seed=4, frac=1 / 8)
    G = B.Graph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    M = W.budget_from_peak(G.no_remat_peak(), 85)
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    batches = [(seqs, lens), (np.ascontiguousarray(seqs[int(lens[:5].sum()):int(lens[:905].sum())]), lens[5:905])]
    for s, l in batches:
        ds, dl = torch.from_numpy(s).cuda(), torch.from_numpy(np.ascontiguousarray(l)).cuda()
        ref = G.eval_batch(ds, dl, M)
        outs = _outputs(len(l))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        got = B.moc_eval_batch_noalloc(G.h, ds, dl, M, *outs)
        assert B.moc_last_launch_count() == 2
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before          # nothing was allocated on the device
        for r, g in zip(ref, got):
            assert torch.equal(r, g)
        op, od, os_, _ = O.eval_batch(s, np.ascontiguousarray(l), M)
        assert (got[0].cpu().numpy() == op).all() and (got[1].cpu().numpy() == od).all() and (got[2].cpu().numpy() == os_).all()
        assert set(ref[2].unique().tolist()) >= {-2, 0, 1}


def test_other_kernels_and_two_handles_share_the_scratch(B):
    """The thread-group kernel (C = 3, 64-bit sums) through the same entry point, and two handles of
    different size taking turns on one stream: every call rewrites the shared offsets before use."""
    cases = []
    for idx, nB in ((3, 96), (1, 700), (3, 64), (0, 300)):
        wl = W.make(idx, seed=21 + idx, B=nB)
        seqs, lens = W.mutate(wl.seqs, wl.lens, wl.n, wl.C, seed=2, frac=1 / 8)
        m = wl.m * (1 << 24) if not cases else wl.m          # the first handle sums in 64 bits
        G = B.Graph(wl.n, wl.edges, wl.w, m, wl.C)
        O = OracleGraph(wl.n, wl.edges, wl.w, m, wl.C)
        cases.append((G, O, seqs, lens, W.budget_from_peak(G.no_remat_peak(), 90)))
    assert cases[0][0].info()["wide"]
    dev = [(torch.from_numpy(s).cuda(), torch.from_numpy(l).cuda(), _outputs(len(l))) for _, _, s, l, _ in cases]
    for rep in range(2):                                   # all calls queued back to back, then checked
        for (G, _, _, _, M), (ds, dl, outs) in zip(cases, dev):
            B.moc_eval_batch_noalloc(G.h, ds, dl, M, *outs)
    torch.cuda.synchronize()
    for (G, O, s, l, M), (_, _, outs) in zip(cases, dev):
        op, od, os_, _ = O.eval_batch(s, l, M)
        assert (outs[0].cpu().numpy() == op).all() and (outs[1].cpu().numpy() == od).all() and (outs[2].cpu().numpy() == os_).all()


def test_limits_are_reported_not_exceeded(B):
    G = B.Graph(3, [(0, 1)], [1, 1, 1], [1, 2, 3], 2)
    n = B.MOC_NOALLOC_MAX_B + 1
    lens = torch.full((n,), 3, dtype=torch.int32, device="cuda")
    seqs = torch.arange(3, dtype=torch.int32, device="cuda").repeat(n)
    with pytest.raises(B.MocError) as e:
        B.moc_eval_batch_noalloc(G.h, seqs, lens, 10, *_outputs(n))
    assert e.value.code == -1 and "exceeds" in str(e.value)
    # exactly the maximum is accepted and correct
    got = B.moc_eval_batch_noalloc(G.h, seqs[:-3], lens[:-1], 10, *_outputs(n - 1))
    torch.cuda.synchronize()
    assert (got[0] == 5).all() and (got[1] == 3).all() and (got[2] == 1).all()
    # a graph whose state needs a global workspace is refused with a clear message
    big = 40000
    Gb = B.Graph(big, [], np.ones(big, np.int64), np.ones(big, np.int64), 2)
    with pytest.raises(B.MocError) as e:
        B.moc_eval_batch_noalloc(Gb.h, torch.arange(big, dtype=torch.int32, device="cuda"),
                                 torch.tensor([big], dtype=torch.int32, device="cuda"), 10, *_outputs(1))
    assert e.value.code == -1 and "workspace" in str(e.value)
