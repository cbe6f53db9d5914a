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
