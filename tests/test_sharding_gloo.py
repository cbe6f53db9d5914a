"""The multi-GPU host logic on CPU: two gloo ranks each take their block of one batch, evaluate it
(with the CPU oracle standing in for the device), and the gathered results equal the unsharded ones."""
import os
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import torch
    import torch.distributed as dist
    from oracle import OracleGraph
    from paper_2304_14463_b200 import sharding, workloads
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = workloads.make(1, seed=5, B=301, n_threads=1)
    seqs, lens = workloads.mutate(wl.seqs, wl.lens, wl.n, wl.C, seed=2, frac=0.1)
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    my_seqs, my_lens = sharding.shard_batch(seqs, lens, rank, world)
    peak, dur, st, _ = O.eval_batch(my_seqs, my_lens, 30000)
    b0, b1 = sharding.shard_range(len(lens), rank, world)
    full = torch.zeros(3, len(lens), dtype=torch.int64)
    full[0, b0:b1] = torch.from_numpy(peak)
    full[1, b0:b1] = torch.from_numpy(dur)
    full[2, b0:b1] = torch.from_numpy(st.astype(np.int64))
    dist.all_reduce(full)                                   # blocks are disjoint: sum = gather
    t = torch.tensor([0.5 + rank], dtype=torch.float64)     # stand-in per-rank times
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    units = torch.tensor([float(np.clip(my_lens, 0, None).sum())], dtype=torch.float64)
    dist.all_reduce(units)
    if rank == 0:
        rp, rd, rs, _ = O.eval_batch(seqs, lens, 30000)
        ok = bool((full[0].numpy() == rp).all() and (full[1].numpy() == rd).all() and (full[2].numpy() == rs).all())
        q.put((ok, float(t[0]), float(units[0]), float(np.clip(lens, 0, None).sum())))
    dist.destroy_process_group()


def test_two_ranks_cover_the_batch():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    ok, tmax, units, total = q.get(timeout=120)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    assert ok and tmax == 1.5 and units == total


def test_shard_ranges():
    from paper_2304_14463_b200 import sharding
    for B in (0, 1, 7, 16384):
        for world in (1, 2, 3, 8):
            r = [sharding.shard_range(B, k, world) for k in range(world)]
            assert r[0][0] == 0 and r[-1][1] == B and all(a[1] == b[0] for a, b in zip(r, r[1:]))
            assert max(b - a for a, b in r) - min(b - a for a, b in r) <= 1
    assert sharding.aggregate_throughput([10, 30], [1.0, 2.0]) == 20.0


def _search_worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from oracle import OracleGraph, OracleSearch
    from paper_2304_14463_b200 import sharding, workloads
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = workloads.make(0, seed=4, B=97, n_threads=1)
    O = OracleGraph(wl.n, wl.edges, wl.w, wl.m, wl.C)
    M = O.eval(np.arange(wl.n), 1 << 60)["peak"] * 85 // 100
    out = []
    for case in ("normal", "rank0_all_invalid"):
        seqs, lens = wl.seqs.copy(), wl.lens.copy()
        if case == "rank0_all_invalid":
            b0, b1 = sharding.shard_range(len(lens), 0, world)
            offs = np.concatenate([[0], np.cumsum(lens)])
            seqs[:offs[b1]] = 0                             # rank 0 starts with invalid chains only
        my_seqs, my_lens = sharding.shard_batch(seqs, lens, rank, world)
        b0, _ = sharding.shard_range(len(lens), rank, world)
        S = OracleSearch(O, my_seqs, my_lens, M, seed=9, chain0=b0)   # the oracle stands in for the device
        S.run(0 if case == "rank0_all_invalid" else 60)
        b = S.best()
        mine = dict(index=b, peak=int(S.peak[b]) if b >= 0 else -1, dur=int(S.dur[b]) if b >= 0 else -1,
                    status=int(S.status[b]) if b >= 0 else -2, seq=S.row(b) if b >= 0 else np.zeros(0, np.int32))
        got = sharding.best_over_ranks(mine, M, b0, wl.C * wl.n)
        if rank == 0:
            full = OracleSearch(O, seqs, lens, M, seed=9)
            full.run(0 if case == "rank0_all_invalid" else 60)
            fb = full.best()
            out.append(got["index"] == fb and (got["seq"] == full.row(fb)).all()
                       and (got["peak"], got["dur"], got["status"]) == (int(full.peak[fb]), int(full.dur[fb]), int(full.status[fb]))
                       and (case == "normal" or got["rank"] == 1))
    if rank == 0:
        q.put(out)
    dist.destroy_process_group()


def test_two_ranks_search_best():
    """A population split over two ranks (global chain numbers) evolves like the unsplit one, and the
    best chain over the ranks is the unsplit best, also when one rank has no valid chain."""
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_search_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    out = q.get(timeout=180)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    assert out == [True, True]
