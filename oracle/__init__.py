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
_LIB = os.path.join(_HERE, "libmoc_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compiles moc_oracle.c into libmoc_oracle.so next to it (gcc -O2); returns the path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.run(["gcc", "-O2", "-std=c11", "-shared", "-fPIC", "-pthread", "-o", tmp, _SRC],
                       check=True)
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
    lib.moc_oracle_eval.restype = None
    lib.moc_oracle_eval.argtypes = [P, P, ctypes.c_int32, ctypes.c_int64, P, P, P, P, P]
    lib.moc_oracle_eval_batch.restype = ctypes.c_int32
    lib.moc_oracle_eval_batch.argtypes = [P, P, P, ctypes.c_int64, ctypes.c_int64, P, P, P,
                                          ctypes.c_int32]
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
