"""moc_eval_batch_noalloc: the entry point for callers that cannot allocate device memory (their
framework owns all of it, or they cannot afford the allocator's locks and synchronisation).  It
keeps its scratch in a fixed array inside the library, shared by all calls, so the test runs two
calls in a row -- a large batch, then a smaller, different one that leaves stale entries behind --
and wants each to equal moc_eval_batch bit for bit.  Collected last on purpose."""
import numpy as np
import pytest
import torch

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
    M = B.budget_from_peak(G.no_remat_peak(), 85)
    batches = [(seqs, lens), (np.ascontiguousarray(seqs[int(lens[:5].sum()):int(lens[:905].sum())]), lens[5:905])]
    for s, l in batches:
        ds, dl = torch.from_numpy(s).cuda(), torch.from_numpy(np.ascontiguousarray(l)).cuda()
        ref = G.eval_batch(ds, dl, M)
        got = B.moc_eval_batch_noalloc(G.h, ds, dl, M, *_outputs(len(l)))
        assert B.moc_last_launch_count() == 2
        torch.cuda.synchronize()
        for r, g in zip(ref, got):
            assert torch.equal(r, g)
        assert set(ref[2].unique().tolist()) >= {-2, 0, 1}


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
