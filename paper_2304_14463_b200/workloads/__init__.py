"""Seeded synthetic workloads: compute DAGs, node weights and packed batches of candidate sequences.

Data generation only -- no part of the schedule evaluation lives here.  The generators stand in for
the paper's evaluation graphs (Section 4.1: random layered graphs, training graphs, real-world
graphs), which are not distributed with it; node/edge counts follow the paper's figures and tables
(G1 = (100, 236), the real-world graph of Fig. 1 = (442, 1247), G4-scale n = 1000) and C follows
Section 4.3 (C_v = 2) or is raised to 3 for the two largest cases.

The five named configurations:

  0  layered   n=20   m=40    L=4   w~U[1,10]   m~U[1,100]        B=1024   C=2 p=0.5
  1  layered   n=100  m=236   L=10  w~U[1,20]   m~LN(4,1)         B=65536  C=2 p=0.2
  2  training  n=442  m=1247  221 forward ops, 293 skips span 2-8
                                     w~U[1,50]   m~LN(6,1.5)       B=16384  C=2 p=0.2
  3  resnet    n=1000 m=2994  500 forward ops   w~LN(3,1) m~LN(7,1.5)  B=4096 C=3 p=0.3
  4  layered   n=5000 m=15000 L=50  w~U[1,100]  m~LN(8,2)         B=1024   C=3 p=0.3, T <= 2n

The memory budget M is a percentage of the peak of the identity order 0..n-1 (the "input
topological order" of Section 2.3); computing that peak is evaluation, so callers do it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "workloads.c")
_LIB = os.path.join(_HERE, "libmoc_workloads.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.run(["gcc", "-O2", "-std=gnu11", "-shared", "-fPIC", "-pthread", "-o", tmp, _SRC, "-lm"],
                       check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        P, i32, i64, u64, f64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64, ctypes.c_double
        lib.wl_weights_uniform.restype = None
        lib.wl_weights_uniform.argtypes = [i32, i64, i64, u64, u64, P]
        lib.wl_weights_lognormal.restype = None
        lib.wl_weights_lognormal.argtypes = [i32, f64, f64, u64, u64, P]
        lib.wl_layered_dag.restype = i64
        lib.wl_layered_dag.argtypes = [i32, i64, i32, u64, P]
        lib.wl_training_dag.restype = i64
        lib.wl_training_dag.argtypes = [i32, i32, i32, i32, u64, P]
        lib.wl_resnet_dag.restype = i64
        lib.wl_resnet_dag.argtypes = [i32, i64, P]
        lib.wl_schedules.restype = i32
        lib.wl_schedules.argtypes = [i32, i64, P, i32, f64, i32, i64, u64, i32, i64, P, P]
        lib.wl_pack.restype = i64
        lib.wl_pack.argtypes = [i64, i64, P, P, P]
        _lib = lib
    return _lib


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def weights_uniform(n, lo, hi, seed, stream):
    out = np.empty(n, np.int64)
    _load().wl_weights_uniform(n, lo, hi, seed, stream, _ptr(out))
    return out


def weights_lognormal(n, mu, sigma, seed, stream):
    """max(1, round(exp(mu + sigma*z))), z standard normal (Box-Muller in double)."""
    out = np.empty(n, np.int64)
    _load().wl_weights_lognormal(n, mu, sigma, seed, stream, _ptr(out))
    return out


def layered_dag(n, m, L, seed):
    edges = np.empty((m, 2), np.int32)
    got = _load().wl_layered_dag(n, m, L, seed, _ptr(edges))
    if got != m:
        raise ValueError(f"layered_dag({n},{m},{L}) not constructible")
    return edges


def training_dag(F, n_skips, smin, smax, seed):
    m = 3 * F - 2 + 2 * n_skips
    edges = np.empty((m, 2), np.int32)
    got = _load().wl_training_dag(F, n_skips, smin, smax, seed, _ptr(edges))
    if got != m:
        raise ValueError("training_dag not constructible")
    return edges


def resnet_dag(F):
    cap = 8 * F
    edges = np.empty((cap, 2), np.int32)
    got = _load().wl_resnet_dag(F, cap, _ptr(edges))
    if got < 0:
        raise ValueError("resnet_dag failed")
    return np.ascontiguousarray(edges[:got])


def schedules(n, edges, C, p, B, seed, t_cap=None, n_threads=None):
    """B schedules (random Kahn order + random extra copies) -> packed (seqs[int32], lens[int32])."""
    t_cap = C * n if t_cap is None else min(int(t_cap), C * n)
    n_threads = n_threads or min(16, os.cpu_count() or 1)
    edges = np.ascontiguousarray(edges, np.int32)
    strided = np.empty((B, t_cap), np.int32)
    lens = np.empty(B, np.int32)
    rc = _load().wl_schedules(n, len(edges), _ptr(edges), C, p, t_cap, B, seed, n_threads, t_cap,
                              _ptr(strided), _ptr(lens))
    if rc != 0:
        raise ValueError("schedules: bad arguments")
    packed = np.empty(int(lens.sum()), np.int32)
    _load().wl_pack(B, t_cap, _ptr(strided), _ptr(lens), _ptr(packed))
    return packed, lens


def pack(rows):
    """List of 1-D int arrays -> packed (seqs, lens)."""
    lens = np.array([len(r) for r in rows], np.int32)
    seqs = np.concatenate([np.asarray(r, np.int32) for r in rows]) if rows else np.empty(0, np.int32)
    return np.ascontiguousarray(seqs, np.int32), lens


def unpack(seqs, lens):
    offs = np.concatenate([[0], np.cumsum(np.clip(lens, 0, None))])
    return [seqs[offs[b]:offs[b + 1]] for b in range(len(lens))]


def mutate(seqs, lens, n, C, seed, frac=1.0 / 16):
    """Damages about ``frac`` of the schedules so that dependency violations and malformed
    sequences occur: swap two positions / delete the first copy of a node / overwrite one id with
    n or -1 / append copies of one node until it has C+1.  Returns new packed (seqs, lens)."""
    rs = np.random.RandomState(seed)
    rows = [r.copy() for r in unpack(seqs, lens)]
    for b in range(len(rows)):
        if rs.rand() >= frac:
            continue
        r = rows[b]
        kind = rs.randint(4)
        if kind == 0 and len(r) >= 2:
            i, j = rs.randint(len(r), size=2)
            r[i], r[j] = r[j], r[i]
        elif kind == 1 and len(r) >= 1:
            v = r[rs.randint(len(r))]
            first = int(np.argmax(r == v))
            rows[b] = np.delete(r, first)
        elif kind == 2 and len(r) >= 1:
            r[rs.randint(len(r))] = n if rs.rand() < 0.5 else -1
        else:
            v = rs.randint(n)
            have = int((r == v).sum())
            rows[b] = np.concatenate([r, np.full(max(C + 1 - have, 1), v, np.int32)])
    return pack(rows)


@dataclass
class Workload:
    name: str
    n: int
    edges: np.ndarray          # (m, 2) int32, (u, v): v consumes u
    w: np.ndarray              # (n,) int64 durations
    m: np.ndarray              # (n,) int64 output sizes
    C: int
    seqs: np.ndarray           # packed int32
    lens: np.ndarray           # (B,) int32
    budget_pcts: tuple = (80,)
    meta: dict = field(default_factory=dict)

    @property
    def B(self):
        return len(self.lens)

    @property
    def total_steps(self):
        return int(self.lens.sum())


_SPECS = [
    dict(name="layered_n20", kind="layered", n=20, m=40, L=4, w=("u", 1, 10), mem=("u", 1, 100),
         B=1024, C=2, p=0.5, pcts=(80,)),
    dict(name="layered_n100", kind="layered", n=100, m=236, L=10, w=("u", 1, 20), mem=("ln", 4.0, 1.0),
         B=65536, C=2, p=0.2, pcts=(80,)),
    dict(name="training_n442", kind="training", n=442, F=221, skips=293, w=("u", 1, 50),
         mem=("ln", 6.0, 1.5), B=16384, C=2, p=0.2, pcts=(80,)),
    dict(name="resnet_n1000", kind="resnet", n=1000, F=500, w=("ln", 3.0, 1.0), mem=("ln", 7.0, 1.5),
         B=4096, C=3, p=0.3, pcts=(70, 80, 90)),
    dict(name="layered_n5000", kind="layered", n=5000, m=15000, L=50, w=("u", 1, 100),
         mem=("ln", 8.0, 2.0), B=1024, C=3, p=0.3, pcts=(80,), t_cap_mult=2),
]
N_CONFIGS = len(_SPECS)


def budget_from_peak(peak: int, pct: int) -> int:
    """M = floor(peak * pct / 100): a budget given as a percentage of a no-rematerialization peak
    (Section 4.3; the budgets printed there equal this rounding of a common integer peak)."""
    return int(peak) * int(pct) // 100


def spec(idx):
    return dict(_SPECS[idx])


def _weights(desc, n, seed, stream):
    if desc[0] == "u":
        return weights_uniform(n, desc[1], desc[2], seed, stream)
    return weights_lognormal(n, desc[1], desc[2], seed, stream)


def make_graph(idx, seed=1):
    s = _SPECS[idx]
    if s["kind"] == "layered":
        edges = layered_dag(s["n"], s["m"], s["L"], seed * 1000 + idx)
    elif s["kind"] == "training":
        edges = training_dag(s["F"], s["skips"], 2, 8, seed * 1000 + idx)
    else:
        edges = resnet_dag(s["F"])
    w = _weights(s["w"], s["n"], seed * 1000 + idx, 1)
    m = _weights(s["mem"], s["n"], seed * 1000 + idx, 2)
    return edges, w, m


def make(idx, seed=1, B=None, n_threads=None):
    """Configuration ``idx`` (0..4) with ``B`` schedules (default: the configuration's batch)."""
    s = _SPECS[idx]
    edges, w, m = make_graph(idx, seed)
    B = s["B"] if B is None else int(B)
    t_cap = s["n"] * s.get("t_cap_mult", s["C"])
    seqs, lens = schedules(s["n"], edges, s["C"], s["p"], B, seed * 7919 + idx, t_cap=t_cap,
                           n_threads=n_threads)
    return Workload(s["name"], s["n"], edges, w, m, s["C"], seqs, lens, tuple(s["pcts"]),
                    dict(seed=seed, p=s["p"], t_cap=t_cap, kind=s["kind"]))
