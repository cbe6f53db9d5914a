"""CPU oracle (test infrastructure only) for the evaluation of rematerialization sequences.

This package wraps ``moc_oracle.c`` -- the plain sequential statement of the paper's Eqs. 1-8 for
one given sequence -- with ctypes.  Only the tests, the smoke check and the timed CPU baseline of
the benchmark may import it.  It imports nothing from the CUDA package and the CUDA package
imports nothing from here.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moc_oracle.c")
_SRC_SEARCH = os.path.join(_HERE, "moc_search_oracle.c")
_SRC_INTERVAL = os.path.join(_HERE, "moc_interval_oracle.c")
_HDR = os.path.join(_HERE, "moc_oracle_graph.h")
_LIB = os.path.join(_HERE, "libmoc_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compiles moc_oracle.c and moc_search_oracle.c and moc_interval_oracle.c into libmoc_oracle.so next to them (gcc -O2);
    returns the path."""
    newest = max(os.path.getmtime(f) for f in (_SRC, _SRC_SEARCH, _SRC_INTERVAL, _HDR))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest:
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.run(["gcc", "-O2", "-std=c11", "-shared", "-fPIC", "-pthread", "-o", tmp, _SRC,
                        _SRC_SEARCH, _SRC_INTERVAL], check=True)
        os.replace(tmp, _LIB)
    return _LIB


def load_library(path):
    """Binds the entry points of an oracle shared library (the tests also load altered builds)."""
    lib = ctypes.CDLL(path)
    P = ctypes.c_void_p
    lib.moc_oracle_graph_create.restype = P
    lib.moc_oracle_graph_create.argtypes = [ctypes.c_int32, ctypes.c_int64, P, P, P, ctypes.c_int32]
    lib.moc_oracle_graph_destroy.restype = None
    lib.moc_oracle_graph_destroy.argtypes = [P]
    lib.moc_oracle_graph_set_caps.restype = ctypes.c_int32
    lib.moc_oracle_graph_set_caps.argtypes = [P, P]
    lib.moc_oracle_eval.restype = None
    lib.moc_oracle_eval.argtypes = [P, P, ctypes.c_int32, ctypes.c_int64, P, P, P, P, P]
    lib.moc_oracle_eval_batch.restype = ctypes.c_int32
    lib.moc_oracle_eval_batch.argtypes = [P, P, P, ctypes.c_int64, ctypes.c_int64, P, P, P,
                                          ctypes.c_int32]
    if hasattr(lib, "moc_oracle_check_intervals"):
        lib.moc_oracle_check_intervals.restype = None
        lib.moc_oracle_check_intervals.argtypes = [P, P, P, P, ctypes.c_int64, P, ctypes.c_int64, P, P, P, P]
        lib.moc_oracle_intervals_to_sequence.restype = ctypes.c_int32
        lib.moc_oracle_intervals_to_sequence.argtypes = [P, P, P, P, ctypes.c_int64, P]
    if hasattr(lib, "moc_oracle_search_run"):
        u32, u64, i32, i64 = ctypes.c_uint32, ctypes.c_uint64, ctypes.c_int32, ctypes.c_int64
        lib.moc_oracle_philox4x32_10.restype = None
        lib.moc_oracle_philox4x32_10.argtypes = [P, P, P]
        lib.moc_oracle_mutate.restype = i32
        lib.moc_oracle_mutate.argtypes = [P, i32, u32, u32, u32, u32, P]
        lib.moc_oracle_accept.restype = i32
        lib.moc_oracle_accept.argtypes = [i64, i64, i32, i64, i64, i32, i64]
        lib.moc_oracle_search_run.restype = None
        lib.moc_oracle_search_run.argtypes = [P, P, P, P, P, P, i32, i32, i64, u64, u32, u32, u32, u32, u32, P]
        lib.moc_oracle_search_best.restype = i32
        lib.moc_oracle_search_best.argtypes = [P, P, P, i32, i64]
    return lib


def _load():
    global _lib
    if _lib is None:
        _lib = load_library(build())
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


class OracleGraph:
    """DAG G=(V,E) with durations w and output sizes m; (u, v) in ``edges`` means v consumes u."""

    def __init__(self, n, edges, w, m, C=2, lib=None):
        self._lib = lib if lib is not None else _load()
        self.n = int(n)
        self.C = int(C)
        self.edges = np.ascontiguousarray(np.asarray(edges, dtype=np.int32).reshape(-1, 2))
        self.w = np.ascontiguousarray(w, dtype=np.int64)
        self.m = np.ascontiguousarray(m, dtype=np.int64)
        assert self.w.shape == (self.n,) and self.m.shape == (self.n,)
        self._h = self._lib.moc_oracle_graph_create(self.n, len(self.edges), _ptr(self.edges),
                                                  _ptr(self.w), _ptr(self.m), self.C)
        if not self._h:
            raise ValueError("oracle: bad graph (id out of range, self-loop, n<=0 or C<1)")

    def __del__(self):
        if getattr(self, "_h", None):
            self._lib.moc_oracle_graph_destroy(self._h)
            self._h = None

    def set_caps(self, caps):
        """Per-node caps C_v in [1, C] (None: uniform C again)."""
        if caps is None:
            self._lib.moc_oracle_graph_set_caps(self._h, None)
            return
        caps = np.ascontiguousarray(caps, dtype=np.int32)
        assert caps.shape == (self.n,)
        if self._lib.moc_oracle_graph_set_caps(self._h, _ptr(caps)) != 0:
            raise ValueError("oracle: cap outside [1, C]")

    def eval(self, seq, M):
        """One sequence -> dict(peak, dur, status, profile[T], free[T])."""
        seq = np.ascontiguousarray(seq, dtype=np.int32)
        T = len(seq)
        peak = np.zeros(1, np.int64)
        dur = np.zeros(1, np.int64)
        status = np.zeros(1, np.int32)
        profile = np.zeros(max(T, 1), np.int64)
        free = np.zeros(max(T, 1), np.int32)
        self._lib.moc_oracle_eval(self._h, _ptr(seq), T, int(M), _ptr(peak), _ptr(dur), _ptr(status),
                                _ptr(profile), _ptr(free))
        return dict(peak=int(peak[0]), dur=int(dur[0]), status=int(status[0]),
                    profile=profile[:T].copy(), free=free[:T].copy())

    def check_intervals(self, s, e, a, M, D=None, topo_index=None):
        """One solution in interval form ([n, C] int32 arrays s, e, a) -> dict(mask, peak, dur).
        topo_index (1-based index of every node in the input topological order) selects the staged
        model; D defaults to C*n (plain) or n(n+1)/2 (staged)."""
        s = np.ascontiguousarray(s, dtype=np.int32).reshape(self.n, self.C)
        e = np.ascontiguousarray(e, dtype=np.int32).reshape(self.n, self.C)
        a = np.ascontiguousarray(a, dtype=np.int32).reshape(self.n, self.C)
        ti = None if topo_index is None else np.ascontiguousarray(topo_index, dtype=np.int32)
        if D is None:
            D = self.C * self.n if ti is None else self.n * (self.n + 1) // 2
        peak, dur, mask = np.zeros(1, np.int64), np.zeros(1, np.int64), np.zeros(1, np.int32)
        usage = np.full(int(D), -1, np.int64)
        self._lib.moc_oracle_check_intervals(self._h, _ptr(s), _ptr(e), _ptr(a), int(D),
                                             None if ti is None else _ptr(ti), int(M), _ptr(peak), _ptr(dur), _ptr(mask),
                                             _ptr(usage))
        return dict(mask=int(mask[0]), peak=int(peak[0]), dur=int(dur[0]), usage=usage)

    def intervals_to_sequence(self, s, e, a, D=None, staged=False):
        """Execution sequence of a solution in interval form, or None when it has none."""
        s = np.ascontiguousarray(s, dtype=np.int32).reshape(self.n, self.C)
        e = np.ascontiguousarray(e, dtype=np.int32).reshape(self.n, self.C)
        a = np.ascontiguousarray(a, dtype=np.int32).reshape(self.n, self.C)
        if D is None:
            D = self.n * (self.n + 1) // 2 if staged else self.C * self.n
        out = np.zeros(self.n * self.C, np.int32)
        k = self._lib.moc_oracle_intervals_to_sequence(self._h, _ptr(s), _ptr(e), _ptr(a), int(D), _ptr(out))
        return None if k < 0 else out[:k].copy()

    def eval_batch(self, seqs, lens, M, n_threads=1):
        """Packed batch -> (peak[B], dur[B], status[B], threads_used)."""
        seqs = np.ascontiguousarray(seqs, dtype=np.int32)
        lens = np.ascontiguousarray(lens, dtype=np.int32)
        B = len(lens)
        assert int(np.clip(lens, 0, None).sum()) <= len(seqs)
        peak = np.zeros(B, np.int64)
        dur = np.zeros(B, np.int64)
        status = np.zeros(B, np.int32)
        used = self._lib.moc_oracle_eval_batch(self._h, _ptr(seqs), _ptr(lens), B, int(M), _ptr(peak),
                                             _ptr(dur), _ptr(status), int(n_threads))
        return peak, dur, status, int(used)


# ---- local search over sequences (moc_search_oracle.c) ----------------------------------------------

def philox4x32_10(ctr, key, lib=None):
    """One block of Philox4x32-10: ctr = 4 uint32, key = 2 uint32 -> 4 uint32."""
    lib = lib if lib is not None else _load()
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, np.uint32)
    lib.moc_oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def mutate(seq, r0, r1, r2, kinds=7, lib=None):
    """The proposal the draws (r0, r1, r2) make from ``seq`` with the enabled kinds of edit (bit 0
    insert, bit 1 delete, bit 2 move); None for an empty sequence."""
    lib = lib if lib is not None else _load()
    seq = np.ascontiguousarray(seq, dtype=np.int32)
    child = np.zeros(len(seq) + 2, np.int32)
    Tc = lib.moc_oracle_mutate(_ptr(seq), len(seq), int(r0), int(r1), int(r2), int(kinds), _ptr(child))
    return None if Tc < 0 else child[:Tc].copy()


def accept(child, parent, M, lib=None):
    """child, parent = (peak, dur, status) -> bool: the proposal replaces the chain's sequence."""
    lib = lib if lib is not None else _load()
    return bool(lib.moc_oracle_accept(int(child[0]), int(child[1]), int(child[2]), int(parent[0]),
                                      int(parent[1]), int(parent[2]), int(M)))


class OracleSearch:
    """P chains of the search: rows of ``stride`` ints with lengths and evaluations."""

    def __init__(self, graph: OracleGraph, seqs, lens, M, seed, stride=None, chain0=0, kinds=7, samples=1):
        self.g = graph
        self._lib = graph._lib
        self.M = int(M)
        self.seed = int(seed)
        self.chain0 = int(chain0)
        self.kinds = int(kinds)
        self.samples = int(samples)
        lens = np.ascontiguousarray(lens, dtype=np.int32)
        self.P = len(lens)
        self.stride = int(stride) if stride is not None else graph.C * graph.n
        self.pop = np.zeros((self.P, self.stride), np.int32)
        offs = np.concatenate([[0], np.cumsum(np.clip(lens, 0, None))])
        for c in range(self.P):
            assert lens[c] <= self.stride
            self.pop[c, :max(lens[c], 0)] = seqs[offs[c]:offs[c + 1]]
        self.lens = np.clip(lens, 0, None).astype(np.int32)
        self.peak, self.dur, self.status, _ = graph.eval_batch(seqs, lens, self.M)
        self.generation = 0
        self.accepted = 0

    def run(self, n_gen):
        acc = np.zeros(1, np.int64)
        self._lib.moc_oracle_search_run(self.g._h, _ptr(self.pop), _ptr(self.lens), _ptr(self.peak),
                                        _ptr(self.dur), _ptr(self.status), self.P, self.stride, self.M,
                                        self.seed, self.generation, int(n_gen), self.chain0, self.kinds, self.samples, _ptr(acc))
        self.generation += int(n_gen)
        self.accepted += int(acc[0])
        return int(acc[0])

    def best(self):
        return int(self._lib.moc_oracle_search_best(_ptr(self.peak), _ptr(self.dur), _ptr(self.status),
                                                    self.P, self.M))

    def row(self, c):
        return self.pop[c, :self.lens[c]].copy()
