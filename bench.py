#!/usr/bin/env python
"""Throughput of batched schedule evaluation: schedule-steps evaluated per second.

One "step" of the benchmark is one pass of the whole evaluation (offsets, occurrence table, free
steps, memory profile, reductions) over one batch of B candidate sequences, through the C ABI.
Workload: the training-graph-shaped configuration n=442, m=1247, B=16384, C=2, budget = 80 % of the
no-rematerialization peak.  Inputs are synthetic and seeded; a ring of distinct batches larger than
the L2 cache is cycled so that every timed pass reads its sequences from HBM.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

With N > 1 (under torchrun) every rank evaluates its own ring of batches on its own GPU: sequences
are independent, no collective is on the data path; the reported value is the total over ranks
divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

WORKLOAD_IDX = 2   # the configuration the headline metric is quoted on; --workload times another one
METRIC = "schedule_steps_per_s_n442_B16384"
UNIT = "steps/s"
PCT = 80
L2_BYTES = 126 * 1024 * 1024
# One ncu capture of a full-size launch of the evaluation kernel (flushed caches): DRAM traffic
# (dram__bytes_read.sum + dram__bytes_write.sum) and executed warp instructions (smsp__inst_executed.sum),
# valid for the kernel source whose hash is recorded with them; printed as null once the source differs.
NCU_CAPTURE = {
    "traffic_bytes": 34868992,
    "warp_instructions": 29312076,
    "source": "ncu --set full, one launch of eval_pair_kernel<int, 5>: dram read 34.87 MB, write 0 "
              "(the 0.33 MB of results were still in L2)",
    "kernel_sha256": "f4611319144c97b5c27d312d28a869f55b24c70d391af1598de5709fc93334a1",
}
KERNEL_SOURCES = ["paper_2304_14463_b200/csrc/moc_pair_kernel.cuh"]


def kernel_sha256():
    import hashlib
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        with open(os.path.join(ROOT, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def workload_config(base, M, ring_len, ring_bytes):
    """The `config` object of the JSON line; both arms print exactly this for the same workload."""
    return {"workload": f"{base.name}: n={base.n} m={len(base.edges)} B={base.B} C={base.C} "
                        f"M={PCT}% of no-remat peak ({M})",
            "sum_T_per_step": int(base.total_steps), "per_gpu_batch": int(base.B),
            "cold_l2": f"ring of {ring_len} distinct batches, {ring_bytes / 1e6:.0f} MB of inputs > {L2_BYTES / 1e6:.0f} MB L2"}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4)}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.002)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def make_ring(workloads, n_batches, rank, idx=WORKLOAD_IDX):
    """Distinct batches of one configuration (same graph, different schedule seeds)."""
    base = workloads.make(idx, seed=1)
    s = workloads.spec(idx)
    ring = [(base.seqs, base.lens)]
    for k in range(1, n_batches):
        seqs, lens = workloads.schedules(base.n, base.edges, base.C, s["p"], s["B"],
                                         seed=100003 * (rank + 1) + k, t_cap=base.meta["t_cap"])
        ring.append((seqs, lens))
    return base, ring


def run_reference(args):
    """The CPU oracle, as it stands, on the host cores: a bounded sample of the same workload (the same
    ring of batches as the GPU arm; every step evaluates one whole batch)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2304_14463_b200 import workloads
    from oracle import OracleGraph
    base, ring = make_ring(workloads, args.ring, 0, args.workload)
    ring_bytes = sum(4 * int(l.sum()) + 4 * len(l) for _, l in ring)
    O = OracleGraph(base.n, base.edges, base.w, base.m, base.C)
    cores = len(os.sched_getaffinity(0))
    P0 = O.eval(np.arange(base.n), 1 << 62)["peak"]
    M = workloads.budget_from_peak(P0, PCT)
    for i in range(args.warmup):
        O.eval_batch(ring[i % len(ring)][0], ring[i % len(ring)][1], M, n_threads=cores)
    t0 = time.perf_counter()
    used, steps = cores, 0
    for i in range(args.steps):
        seqs, lens = ring[i % len(ring)]
        _, _, _, used = O.eval_batch(seqs, lens, M, n_threads=cores)
        steps += int(lens.sum())
    dt = time.perf_counter() - t0
    value = steps / dt
    line = {"impl": "reference", "metric": METRIC if args.workload == WORKLOAD_IDX else f"schedule_steps_per_s_{base.name}",
            "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64",
            "data": "synthetic",
            "config": workload_config(base, M, len(ring), ring_bytes),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": used, "kind": "oracle",
                             "sample": f"one whole batch ({base.B} sequences, about {base.total_steps} steps) per step, "
                                       f"{args.steps} steps"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_search(args):
    """Throughput of the search entry points: generations of P chains on the headline graph.  Prints a
    JSON line of its own (the default run's line is the evaluation metric)."""
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py --mode search needs a CUDA device")
    torch.cuda.set_device(0)
    import __graft_entry__
    __graft_entry__.build()
    from paper_2304_14463_b200 import binding, workloads
    P = args.chains
    base = workloads.make(WORKLOAD_IDX, seed=1, B=P)
    G = binding.Graph(base.n, base.edges, base.w, base.m, base.C)
    P0 = G.no_remat_peak()
    M = workloads.budget_from_peak(P0, PCT)
    d_seqs, d_lens = torch.from_numpy(base.seqs).cuda(), torch.from_numpy(base.lens).cuda()
    S = binding.Search(G, d_seqs, d_lens, M, seed=1)
    if args.incremental or args.samples > 1:
        S.set_samples(args.samples, incremental=True)
    stride = S.info()["stride"]
    steps, warm = (200 if args.steps is None else args.steps), max(3, 20 if args.warmup is None else args.warmup)
    S.run(warm)
    per_call = binding.moc_last_launch_count()
    torch.cuda.synchronize()
    lens0 = S.state(want_rows=False)["lens"].double().sum().item()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    stream = torch.cuda.current_stream()
    with ClockSampler(0) as clocks:
        e0.record(stream)
        S.run(steps)
        e1.record(stream)
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    launches = binding.moc_last_launch_count()
    lens1 = S.state(want_rows=False)["lens"].double().sum().item()
    mean_T = 0.5 * (lens0 + lens1) / P
    best = S.best()
    # bytes one generation has to move: proposal kernel reads the row and writes the proposal,
    # the evaluation reads the proposal; per chain about 60 bytes of state and results
    alg_bytes = P * (3 * 4 * mean_T + 100)
    peak_gbs, peak_kind = load_peaks()
    sum_w = int(base.w.sum())
    E = args.samples
    inc = args.incremental or E > 1
    line = {"metric": "search_proposals_per_s_n442", "value": P * E * steps / (ms * 1e-3), "unit": "proposals/s",
            "n_gpus": 1, "steps": steps, "warmup": warm, "ms_per_step": ms / steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
            "config": {"workload": f"search on {base.name}: n={base.n} m={len(base.edges)} C={base.C} chains={P} "
                                   f"M={PCT}% of no-remat peak ({M}), {E} proposal(s) per chain and generation, "
                                   + ("scored from the cached evaluation" if inc else "written out and evaluated from scratch"),
                       "mean_T": mean_T,
                       "cold_l2": f"rows of the chains: {2 * P * stride * 4 / 1e6:.0f} MB > {L2_BYTES / 1e6:.0f} MB L2"},
            "schedule_steps_per_s": P * E * mean_T * steps / (ms * 1e-3),
            "gpu_launches": launches, "launches_per_generation": (per_call - (0 if inc else 1)) / warm,
            "roofline": {"bound": "hbm", "achieved": alg_bytes / (ms / steps * 1e-3) / 1e9, "peak": peak_gbs, "unit": "GB/s",
                         "frac": alg_bytes / (ms / steps * 1e-3) / 1e9 / peak_gbs, "peak_kind": f"of {peak_kind}",
                         "traffic": None, "algorithmic_bytes_per_generation": alg_bytes,
                         "note": "whole generation (proposal kernel + evaluation kernel), not one kernel; bytes as if "
                                 "every proposal were written out and read back"} if not inc else None,
            "result": {"generations": S.info()["generation"], "best_status": best["status"], "best_peak": best["peak"],
                       "best_dur": best["dur"], "tdi_percent": 100.0 * (best["dur"] - sum_w) / sum_w if best["index"] >= 0 else None,
                       "accepted": best["accepted"], "no_remat_peak": P0, "budget": M},
            "clocks": clocks.summary()}
    if not args.no_cpu_baseline:
        from oracle import OracleGraph, OracleSearch
        Pc = min(P, 1024)
        O = OracleGraph(base.n, base.edges, base.w, base.m, base.C)
        offs = np.concatenate([[0], np.cumsum(base.lens)])
        OS = OracleSearch(O, base.seqs[:offs[Pc]], base.lens[:Pc], M, seed=1, stride=stride, samples=E)
        OS.run(1)
        t0, gens = time.perf_counter(), 0
        while time.perf_counter() - t0 < 8.0:
            OS.run(1 if E > 4 else 4)
            gens += 1 if E > 4 else 4
        dt = time.perf_counter() - t0
        # parity of the sample: the same chains, the same number of generations, on the GPU
        S2 = binding.Search(G, torch.from_numpy(base.seqs[:offs[Pc]]).cuda(), d_lens[:Pc].contiguous(), M, seed=1)
        if inc:
            S2.set_samples(E, incremental=True)
        S2.run(OS.generation)
        st = S2.state()
        torch.cuda.synchronize()
        same = bool((st["lens"].cpu().numpy() == OS.lens).all() and (st["peak"].cpu().numpy() == OS.peak).all()
                    and (st["dur"].cpu().numpy() == OS.dur).all() and (st["status"].cpu().numpy() == OS.status).all())
        line["cpu_baseline"] = {"value": Pc * E * gens / dt, "unit": "proposals/s", "cores": 1, "kind": "oracle",
                                "sample": f"{Pc} chains, {gens} generations, one core (the search oracle is sequential)"}
        line["parity_sample"] = same
    print(json.dumps(line))


def run_intervals(args):
    """Throughput of moc_check_intervals: solutions in interval form on the headline graph (plain event
    domain D = C*n).  Prints a JSON line of its own."""
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py --mode intervals needs a CUDA device")
    torch.cuda.set_device(0)
    import __graft_entry__
    __graft_entry__.build()
    from paper_2304_14463_b200 import binding, workloads
    nB, distinct = 16384, 1024
    base = workloads.make(WORKLOAD_IDX, seed=1, B=distinct)
    n, C = base.n, base.C
    G = binding.Graph(n, base.edges, base.w, base.m, C)
    M = workloads.budget_from_peak(G.no_remat_peak(), PCT)
    # interval form of `distinct` valid sequences: starts = steps, ends = the free steps the library's
    # own profile entry point reports; unused slots parked on the events after the last step
    offs = np.concatenate([[0], np.cumsum(base.lens)])
    s = np.zeros((distinct, n, C), np.int32)
    e = np.zeros((distinct, n, C), np.int32)
    a = np.zeros((distinct, n, C), np.int32)
    d_all = torch.from_numpy(base.seqs).cuda()
    for b in range(distinct):
        seq = base.seqs[offs[b]:offs[b + 1]]
        _, free, _ = G.mem_profile(d_all[offs[b]:offs[b + 1]])
        free = free.cpu().numpy()
        order = np.argsort(seq, kind="stable")
        slot = np.zeros(len(seq), np.int64)
        sv = seq[order]
        slot[order] = np.arange(len(seq)) - np.searchsorted(sv, sv, side="left")
        s[b, seq, slot] = np.arange(1, len(seq) + 1)
        e[b, seq, slot] = free + 1
        a[b, seq, slot] = 1
        spare = np.nonzero(a[b].reshape(-1) == 0)[0]
        s[b].reshape(-1)[spare] = e[b].reshape(-1)[spare] = np.arange(len(seq) + 1, len(seq) + 1 + len(spare))
    rep = nB // distinct
    ring = []
    for k in range(4):
        perm = np.random.default_rng(k).permutation(nB) % distinct
        ring.append([torch.from_numpy(x[perm]).cuda() for x in (s, e, a)])
    D = C * n
    outs = dict(peak=torch.empty(nB, dtype=torch.int64, device="cuda"), dur=torch.empty(nB, dtype=torch.int64, device="cuda"),
                mask=torch.empty(nB, dtype=torch.int32, device="cuda"))
    import ctypes
    stream = torch.cuda.current_stream()

    def step(i):
        ss, ee, aa = ring[i % len(ring)]
        rc = binding.lib.moc_check_intervals(G.h, ss.data_ptr(), ee.data_ptr(), aa.data_ptr(), nB, D, None, M,
                                             outs["peak"].data_ptr(), outs["dur"].data_ptr(), outs["mask"].data_ptr(),
                                             None, None, ctypes.c_void_p(stream.cuda_stream))
        assert rc == 0, binding.lib.moc_last_error()
    steps, warm = (200 if args.steps is None else args.steps), max(3, 10 if args.warmup is None else args.warmup)
    for i in range(warm):
        step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(0) as clocks:
        e0.record(stream)
        for i in range(steps):
            step(i)
        e1.record(stream)
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    alg_bytes = nB * (12 * n * C + 20)
    peak_gbs, peak_kind = load_peaks()
    ok = int((outs["mask"] == 0).sum())
    line = {"metric": "interval_solutions_checked_per_s_n442", "value": nB / (ms * 1e-3), "unit": "solutions/s", "n_gpus": 1,
            "steps": steps, "warmup": warm, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int64", "data": "synthetic",
            "config": {"workload": f"moc_check_intervals on {base.name}: n={n} C={C} D={D} B={nB} ({distinct} distinct valid "
                                   f"solutions, shuffled copies), M={PCT}% of no-remat peak",
                       "cold_l2": f"ring of 4 batches, {4 * alg_bytes / 1e6:.0f} MB > {L2_BYTES / 1e6:.0f} MB L2"},
            "gpu_launches": steps, "solutions_without_violation_but_budget": int(((outs["mask"] & ~4) == 0).sum()), "solutions_ok": ok,
            "roofline": {"bound": "hbm", "achieved": alg_bytes / (ms * 1e-3) / 1e9, "peak": peak_gbs, "unit": "GB/s",
                         "frac": alg_bytes / (ms * 1e-3) / 1e9 / peak_gbs, "peak_kind": f"of {peak_kind}",
                         "traffic": 173843712 + 4957440,
                         "traffic_source": "ncu, one launch of this workload: dram read 173.84 MB, write 4.96 MB",
                         "algorithmic_bytes_per_launch": alg_bytes},
            "clocks": clocks.summary()}
    if not args.no_cpu_baseline:
        from oracle import OracleGraph
        O = OracleGraph(n, base.edges, base.w, base.m, C)
        t0, k = time.perf_counter(), 0
        same = True
        pk, msk = outs["peak"].cpu().numpy(), outs["mask"].cpu().numpy()
        perm = np.random.default_rng((steps - 1) % 4).permutation(nB) % distinct
        while time.perf_counter() - t0 < 8.0 and k < nB:
            r = O.check_intervals(s[perm[k]], e[perm[k]], a[perm[k]], M, D=D)
            same = same and r["peak"] == pk[k] and r["mask"] == msk[k]
            k += 1
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": k / dt, "unit": "solutions/s", "cores": 1, "kind": "oracle",
                                "sample": f"the first {k} solutions of the last batch, one core"}
        line["parity_sample"] = bool(same)
    print(json.dumps(line))


def run_edits(args):
    """Throughput of the incremental evaluation: random single edits of the headline batch's sequences,
    scored from the cached parents.  Prints a JSON line of its own."""
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py --mode edits needs a CUDA device")
    torch.cuda.set_device(0)
    import __graft_entry__
    __graft_entry__.build()
    from paper_2304_14463_b200 import binding, workloads
    base = workloads.make(WORKLOAD_IDX, seed=1)
    P, per_parent = base.B, 16
    G = binding.Graph(base.n, base.edges, base.w, base.m, base.C)
    M = workloads.budget_from_peak(G.no_remat_peak(), PCT)
    cache = binding.EditCache(G, P)
    d_seqs, d_lens = torch.from_numpy(base.seqs).cuda(), torch.from_numpy(base.lens).cuda()
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    cache.build(d_seqs, d_lens, M)
    torch.cuda.synchronize()
    e0.record(stream)
    cache.build(d_seqs, d_lens, M)
    e1.record(stream)
    torch.cuda.synchronize()
    build_ms = e0.elapsed_time(e1)
    nE = P * per_parent
    ring = []
    for k in range(4):
        rng = np.random.default_rng(k)
        parent = rng.permutation(nE).astype(np.int32) % P
        T = base.lens[parent]
        op = rng.integers(0, 3, nE).astype(np.int32)
        q = (rng.integers(0, 1 << 30, nE) % T).astype(np.int32)
        j = (rng.integers(0, 1 << 30, nE) % np.where(op == 0, T + 1, T)).astype(np.int32)
        ring.append([torch.from_numpy(x).cuda() for x in (parent, op, q, j)] + [parent, op, q, j])
    out = (torch.empty(nE, dtype=torch.int64, device="cuda"), torch.empty(nE, dtype=torch.int64, device="cuda"),
           torch.empty(nE, dtype=torch.int32, device="cuda"))
    window = torch.zeros(nE, dtype=torch.int32, device="cuda")
    steps, warm = (100 if args.steps is None else args.steps), max(3, 5 if args.warmup is None else args.warmup)
    for i in range(warm):
        r = ring[i % 4]
        cache.eval_edits(r[0], r[1], r[2], r[3], M, out=out, window=window)
    torch.cuda.synchronize()
    mean_window = float(window.double().mean())
    with ClockSampler(0) as clocks:
        e0.record(stream)
        for i in range(steps):
            r = ring[i % 4]
            cache.eval_edits(r[0], r[1], r[2], r[3], M, out=out)
        e1.record(stream)
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    last = ring[(steps - 1) % 4]
    st = out[2].cpu().numpy()
    # ---- second figure: admissible edits only (random edits are mostly refused early: precedence, copy count).
    # The admissible edits of the four batches, repeated to the same batch size, timed the same way.
    adm = []
    for r in ring:
        cache.eval_edits(r[0], r[1], r[2], r[3], M, out=out)
        torch.cuda.synchronize()
        keep = np.nonzero(out[2].cpu().numpy() >= 0)[0]
        adm.append([a[keep] for a in r[4:8]])
    pool = [np.concatenate([a[k] for a in adm]) for k in range(4)]
    adm_ms, adm_frac = None, float(np.mean([len(a[0]) for a in adm])) / nE
    if len(pool[0]) > 0:
        idx = np.resize(np.arange(len(pool[0])), nE)
        d_adm = [torch.from_numpy(np.ascontiguousarray(x[idx])).cuda() for x in pool]
        for _ in range(warm):
            cache.eval_edits(d_adm[0], d_adm[1], d_adm[2], d_adm[3], M, out=out)
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(steps):
            cache.eval_edits(d_adm[0], d_adm[1], d_adm[2], d_adm[3], M, out=out)
        e1.record(stream)
        torch.cuda.synchronize()
        adm_ms = e0.elapsed_time(e1) / steps
        assert bool((out[2] >= 0).all())
    mean_T = float(base.lens.mean())
    msz = 8 if G.info()["wide"] else 4
    # per edit: the record (16 B), the result (20 B), the cached usage over the recomputed window, two
    # extrema, and about a dozen position / free-step words of the edited node and its neighbours
    alg_bytes = nE * (36 + msz * mean_window + 2 * msz + 64)
    peak_gbs, peak_kind = load_peaks()
    line = {"metric": "edits_scored_per_s_n442", "value": nE / (ms * 1e-3), "unit": "edits/s", "n_gpus": 1, "steps": steps,
            "warmup": warm, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int64" if msz == 8 else "int32", "data": "synthetic",
            "config": {"workload": f"moc_eval_edits on {base.name}: n={base.n} C={base.C}, {P} cached parents, {per_parent} random "
                                   f"edits each (insert / delete / move), M={PCT}% of no-remat peak",
                       "cold_l2": f"cache of the parents: {P * (4 + 3 * msz) * (2 * base.n) / 1e6:.0f} MB > {L2_BYTES / 1e6:.0f} MB L2",
                       "mean_T": mean_T, "mean_recomputed_steps": mean_window},
            "equivalent_schedule_steps_per_s": nE * mean_T / (ms * 1e-3), "cache_build_ms": build_ms, "gpu_launches": steps,
            "admissible_only": None if adm_ms is None else {
                "value": nE / (adm_ms * 1e-3), "unit": "edits/s", "ms_per_step": adm_ms,
                "share_of_random_edits_that_are_admissible": adm_frac,
                "note": "a batch of the same size made of edits whose status is 0 or 1 (none refused for precedence or copy count)"},
            "status_counts": {str(k): int((st == k).sum()) for k in (1, 0, -1, -2, -3)},
            "roofline": {"bound": "hbm", "achieved": alg_bytes / (ms * 1e-3) / 1e9, "peak": peak_gbs, "unit": "GB/s",
                         "frac": alg_bytes / (ms * 1e-3) / 1e9 / peak_gbs, "peak_kind": f"of {peak_kind}",
                         "traffic": 101489664 + 3884544,
                         "traffic_source": "ncu, one launch of this workload (edit_eval_lanes_kernel): dram read 101.49 MB, write 3.88 MB",
                         "algorithmic_bytes_per_launch": alg_bytes},
            "clocks": clocks.summary()}
    if not args.no_cpu_baseline:
        import oracle
        from oracle import OracleGraph
        O = OracleGraph(base.n, base.edges, base.w, base.m, base.C)
        offs = np.concatenate([[0], np.cumsum(base.lens)])
        pk, du = out[0].cpu().numpy(), out[1].cpu().numpy()
        t0, k, same = time.perf_counter(), 0, True
        while time.perf_counter() - t0 < 8.0 and k < nE:
            c = last[4][k]
            child = oracle.mutate(base.seqs[offs[c]:offs[c + 1]], int(last[5][k]), int(last[6][k]), int(last[7][k]))
            r = O.eval(child, M)
            same = same and (r["peak"], r["dur"], r["status"]) == (int(pk[k]), int(du[k]), int(st[k]))
            k += 1
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": k / dt, "unit": "edits/s", "cores": 1, "kind": "oracle",
                                "sample": f"the first {k} edits of the last batch: edit + full evaluation, one core"}
        line["parity_sample"] = bool(same)
    print(json.dumps(line))


def time_oracle(base, M, budget_s=6.0):
    from oracle import OracleGraph
    O = OracleGraph(base.n, base.edges, base.w, base.m, base.C)
    cores = len(os.sched_getaffinity(0))
    O.eval_batch(base.seqs, base.lens, M, n_threads=cores)
    out = {}
    for label, threads, share in (("all", cores, 0.6), ("one", 1, 0.4)):
        reps, t0 = 0, time.perf_counter()
        used = threads
        while True:
            res = O.eval_batch(base.seqs, base.lens, M, n_threads=threads)
            used = res[3]
            reps += 1
            dt = time.perf_counter() - t0
            if dt > budget_s * share and reps >= 2:
                break
        out[label] = (base.total_steps * reps / dt, used, reps, res)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--ring", type=int, default=16, help="distinct input batches cycled through")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", type=int, default=WORKLOAD_IDX,
                    help="index 0..4 of the configuration to time (default: the headline one)")
    ap.add_argument("--kernel", default="auto", choices=["auto", "group", "warp", "lane", "block"],
                    help="evaluation kernel family to time (default: the library's own choice)")
    ap.add_argument("--mode", default="eval", choices=["eval", "search", "intervals", "edits"],
                    help="eval: the headline evaluation metric; search: generations of the search entry points; "
                         "intervals: the interval-form checker; edits: the incremental evaluation of single edits")
    ap.add_argument("--chains", type=int, default=32768, help="--mode search: number of chains")
    ap.add_argument("--samples", type=int, default=1, help="--mode search: proposals per chain and generation")
    ap.add_argument("--incremental", action="store_true",
                    help="--mode search: score proposals from the cached evaluation (implied by --samples > 1)")
    args = ap.parse_args()
    if args.mode == "search" and args.impl != "reference":
        return run_search(args)
    if args.mode == "intervals" and args.impl != "reference":
        return run_intervals(args)
    if args.mode == "edits" and args.impl != "reference":
        return run_edits(args)
    if args.impl == "reference":
        args.steps = 5 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        return run_reference(args)
    args.steps = 4000 if args.steps is None else args.steps
    args.warmup = max(3, 200 if args.warmup is None else args.warmup)

    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path (use --impl reference for the oracle)")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    import __graft_entry__
    if rank == 0:
        __graft_entry__.build()
    if world > 1:
        dist.barrier()
    from paper_2304_14463_b200 import binding, workloads

    base, ring_host = make_ring(workloads, args.ring, rank, args.workload)
    G = binding.Graph(base.n, base.edges, base.w, base.m, base.C)
    G.set_kernel({"auto": binding.MOC_KERNEL_AUTO, "group": binding.MOC_KERNEL_GROUP, "warp": binding.MOC_KERNEL_WARP,
                  "lane": binding.MOC_KERNEL_LANE, "block": binding.MOC_KERNEL_BLOCK}[args.kernel])
    M = workloads.budget_from_peak(G.no_remat_peak(), PCT)
    ring = []
    for seqs, lens in ring_host:
        B = len(lens)
        ring.append(dict(seqs=torch.from_numpy(seqs).cuda(), lens=torch.from_numpy(lens).cuda(),
                         peak=torch.empty(B, dtype=torch.int64, device="cuda"),
                         dur=torch.empty(B, dtype=torch.int64, device="cuda"),
                         st=torch.empty(B, dtype=torch.int32, device="cuda"),
                         steps=int(lens.sum()), B=B))
    ring_bytes = sum(4 * r["steps"] + 4 * r["B"] for r in ring)
    stream = torch.cuda.current_stream()

    def step(i):
        r = ring[i % len(ring)]
        G.eval_batch(r["seqs"], r["lens"], M, out_peak=r["peak"], out_dur=r["dur"], out_feasible=r["st"])

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident throughput: K steps back to back on one stream.  A short region (the
    # driver's --steps 20 is about a millisecond) is repeated and the median region reported, so
    # that one slow launch does not decide the figure and the clock sampler sees the GPU under load.
    for i in range(args.warmup):
        step(i)
    launches_per_step = binding.moc_last_launch_count()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(min(args.steps, 20)):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    est_ms = e0.elapsed_time(e1) / min(args.steps, 20) * args.steps
    repeats = 1 if est_ms >= 100.0 else int(min(200, max(25, 100.0 / max(est_ms, 1e-3))))
    barrier()
    region_ms = []
    with ClockSampler(local_rank) as clocks:
        for r in range(repeats):
            e0.record(stream)
            for i in range(args.steps):
                step(r * args.steps + i)
            e1.record(stream)
            barrier()
            region_ms.append(e0.elapsed_time(e1))
    ms = float(np.median(region_ms))
    # every region runs the same number of steps over the ring; count the steps of the median-length one
    steps_done = sum(ring[i % len(ring)]["steps"] for i in range(args.steps))

    # ---- the same region again with the library's measurement hook: an event pair around every
    # launch of the evaluation kernel alone (the dominant kernel), on the launching stream
    n_k = min(args.steps, 512)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_k)]
    for i in range(n_k):
        G.set_timing_events(evs[i][0], evs[i][1])
        step(i)
    G.set_timing_events(None, None)
    torch.cuda.synchronize()
    kern_ms = np.array([a.elapsed_time(b) for a, b in evs])
    gap_ms = np.array([evs[i][1].elapsed_time(evs[i + 1][0]) for i in range(n_k - 1)]) if n_k > 1 else np.zeros(1)

    # ---- the same steps replayed from one CUDA graph: what is left when the host's launch path is taken out
    graph_ms = None
    try:
        n_g = min(len(ring) * 4, 64)
        cg = torch.cuda.CUDAGraph()
        with torch.cuda.graph(cg):
            for i in range(n_g):
                step(i)
        cg.replay()
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = max(1, args.steps // n_g)
        g0.record()
        for _ in range(reps):
            cg.replay()
        g1.record()
        torch.cuda.synchronize()
        graph_ms = g0.elapsed_time(g1) / (reps * n_g)
    except Exception as ex:                       # capture is a measurement aid, never a requirement
        graph_ms = None
        print(f"# CUDA graph capture skipped: {ex}", file=sys.stderr)

    # ---- end to end: host buffers in, host buffers out, through the host entry point
    hr = []
    for seqs, lens in ring_host[:4]:
        B = len(lens)
        hr.append(dict(seqs=torch.from_numpy(seqs).pin_memory(), lens=torch.from_numpy(lens).pin_memory(),
                       peak=torch.empty(B, dtype=torch.int64).pin_memory(),
                       dur=torch.empty(B, dtype=torch.int64).pin_memory(),
                       st=torch.empty(B, dtype=torch.int32).pin_memory(), steps=int(lens.sum()), B=B))
    n_e2e = max(3, min(args.steps, 64))
    # pinned host -> device bandwidth of this machine for the same bytes: what the end-to-end figures are bound by
    d_tmp = torch.empty_like(hr[0]["seqs"], device="cuda")
    for _ in range(3):
        d_tmp.copy_(hr[0]["seqs"], non_blocking=True)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(10):
        d_tmp.copy_(hr[0]["seqs"], non_blocking=True)
    torch.cuda.synchronize()
    link_gbs = 10 * hr[0]["seqs"].numel() * 4 / (time.perf_counter() - t0) / 1e9
    del d_tmp
    for i in range(2 * len(hr)):                      # every pinned buffer has travelled before the clock starts
        r = hr[i % len(hr)]
        G.eval_batch_host(r["seqs"], r["lens"], M, r["peak"], r["dur"], r["st"])
    barrier()
    t0 = time.perf_counter()
    e2e_steps = 0
    for i in range(n_e2e):
        r = hr[i % len(hr)]
        G.eval_batch_host(r["seqs"], r["lens"], M, r["peak"], r["dur"], r["st"])
        e2e_steps += r["steps"]
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0

    # ---- the same with 16-bit node ids on the host side (half the bytes over the host link)
    e2e16_s, e2e16_steps = None, 0
    if base.n <= 65535:
        hr16 = [dict(r, seqs=torch.from_numpy(r["seqs"].numpy().astype(np.uint16)).pin_memory()) for r in hr]
        for i in range(2 * len(hr16)):
            r = hr16[i % len(hr16)]
            G.eval_batch_host16(r["seqs"], r["lens"], M, r["peak"], r["dur"], r["st"])
        barrier()
        t0 = time.perf_counter()
        for i in range(n_e2e):
            r = hr16[i % len(hr16)]
            G.eval_batch_host16(r["seqs"], r["lens"], M, r["peak"], r["dur"], r["st"])
            e2e16_steps += r["steps"]
        torch.cuda.synchronize()
        e2e16_s = time.perf_counter() - t0

    # ---- max over ranks
    if world > 1:
        t = torch.tensor([ms, e2e_s, e2e16_s or 0.0], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms, e2e_s = float(t[0]), float(t[1])
        e2e16_s = float(t[2]) if e2e16_s is not None else None
        tot = torch.tensor([steps_done, e2e_steps, e2e16_steps], dtype=torch.float64, device="cuda")
        dist.all_reduce(tot, op=dist.ReduceOp.SUM)
        steps_done, e2e_steps, e2e16_steps = float(tot[0]), float(tot[1]), float(tot[2])

    if rank == 0:
        peak_gbs, peak_kind = load_peaks()
        r0 = ring[0]
        alg_bytes = 4 * r0["steps"] + 4 * r0["B"] + 20 * r0["B"]
        kernel_ms = float(np.mean(kern_ms))
        sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count
        capture_ok = args.workload == WORKLOAD_IDX and args.kernel == "auto" and NCU_CAPTURE["kernel_sha256"] == kernel_sha256()
        if launches_per_step == 1:
            # one kernel per step: the timed region itself (K back-to-back launches between two CUDA
            # events) is the cleaner per-launch figure; the per-launch event pairs add record overhead
            kernel_ms = min(kernel_ms, ms / args.steps)
        info = G.info()
        line = {
            "metric": METRIC if args.workload == WORKLOAD_IDX else f"schedule_steps_per_s_{base.name}", "value": steps_done / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int64" if info["wide"] else "int32", "data": "synthetic",
            "config": workload_config(base, M, len(ring), ring_bytes), "kernel_family": args.kernel,
            "timed_regions": repeats, "region_ms_median_min_max": [ms, float(np.min(region_ms)), float(np.max(region_ms))],
            "gpu_launches": launches_per_step * args.steps,
            "e2e": {"value": e2e_steps / e2e_s, "unit": UNIT,
                    "h2d_bytes_per_step": 4 * hr[0]["steps"] + 4 * hr[0]["B"], "d2h_bytes_per_step": 20 * hr[0]["B"],
                    "steps": n_e2e, "api": "moc_eval_batch_host (pinned host buffers)", "link_gbs": link_gbs,
                    "link_frac": (4 * hr[0]["steps"] + 4 * hr[0]["B"]) / (e2e_s / n_e2e) / 1e9 / link_gbs},
            "e2e_u16": None if e2e16_s is None else {
                "value": e2e16_steps / e2e16_s, "unit": UNIT, "h2d_bytes_per_step": 2 * hr[0]["steps"] + 4 * hr[0]["B"],
                "d2h_bytes_per_step": 20 * hr[0]["B"], "steps": n_e2e,
                "api": "moc_eval_batch_host16 (node ids as uint16 in pinned host buffers)", "link_gbs": link_gbs,
                "link_frac": (2 * hr[0]["steps"] + 4 * hr[0]["B"]) / (e2e16_s / n_e2e) / 1e9 / link_gbs},
            "roofline": {"bound": "hbm", "achieved": alg_bytes / (kernel_ms * 1e-3) / 1e9, "peak": peak_gbs,
                         "unit": "GB/s", "frac": alg_bytes / (kernel_ms * 1e-3) / 1e9 / peak_gbs,
                         "peak_kind": f"of {peak_kind}",
                         "traffic": NCU_CAPTURE["traffic_bytes"] if capture_ok else None,
                         "traffic_source": NCU_CAPTURE["source"] if capture_ok else
                                           "no capture of this kernel source and workload (the recorded one is stale)",
                         "algorithmic_bytes_per_launch": alg_bytes, "kernel_ms": kernel_ms,
                         "kernel": "evaluation kernel (CUDA events around each launch, mean of %d)" % n_k,
                         "between_kernels_ms": float(np.mean(gap_ms)),
                         "graph_replay_ms_per_step": graph_ms,
                         "note": "the kernel is bound on chip (shared-memory data pipe, instruction issue), not by HBM: see profiles/"},
            "clocks": clocks.summary(),
        }
        if capture_ok:
            # Second view of the same launch: the limits ncu shows are instruction issue and the shared-memory
            # pipe.  Issue peak = SMs x 4 schedulers x 1 warp instruction per clock.
            sm_mhz = line["clocks"]["sm_mhz"] or 1965.0
            issue_peak = sm_count * 4 * sm_mhz * 1e6
            line["issue_roofline"] = {"bound": "alu", "achieved": NCU_CAPTURE["warp_instructions"] / (kernel_ms * 1e-3) / 1e9,
                                      "peak": issue_peak / 1e9, "unit": "G warp instructions/s",
                                      "frac": NCU_CAPTURE["warp_instructions"] / (kernel_ms * 1e-3) / issue_peak,
                                      "note": "executed (not algorithmic) instructions of one launch from the ncu capture; "
                                              "context for the HBM fraction above, not a replacement"}
        if not args.no_cpu_baseline:
            o = time_oracle(base, M)
            res = o["all"][3]
            torch.cuda.synchronize()
            same = bool((ring[0]["peak"].cpu().numpy() == res[0]).all() and (ring[0]["dur"].cpu().numpy() == res[1]).all()
                        and (ring[0]["st"].cpu().numpy() == res[2]).all())
            line["cpu_baseline"] = {"value": o["all"][0], "unit": UNIT, "cores": o["all"][1], "kind": "oracle",
                                    "sample": f"the full first batch ({base.B} sequences, {base.total_steps} steps), "
                                              f"{o['all'][2]} passes on all cores",
                                    "one_core_value": o["one"][0]}
            line["parity_first_batch"] = same
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
