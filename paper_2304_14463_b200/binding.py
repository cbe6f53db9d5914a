"""Thin ctypes binding of libmoc_b200.so (argument marshalling only; see include/moc.h).

Function names mirror the C ABI.  PyTorch supplies device memory and streams: tensors are passed as
``data_ptr()`` and the stream as ``torch.cuda.current_stream().cuda_stream``.  If the CUDA library
has not been built, importing this module raises -- there is no CPU path.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
# MOC_B200_LIB selects another build of the same library (e.g. one compiled with other flags)
LIB_PATH = os.environ.get("MOC_B200_LIB") or os.path.join(_HERE, "libmoc_b200.so")

MOC_OK = 0
ERROR_NAMES = {-1: "MOC_ERR_ARG", -2: "MOC_ERR_RANGE", -3: "MOC_ERR_CYCLE", -4: "MOC_ERR_OVERFLOW",
               -5: "MOC_ERR_CUDA", -6: "MOC_ERR_NOMEM"}
EXPORTS = ["moc_graph_create", "moc_graph_set_max_copies", "moc_graph_destroy", "moc_graph_info",
           "moc_eval_batch", "moc_eval_batch_host", "moc_mem_profile", "moc_graph_set_launch",
           "moc_last_launch_count", "moc_last_error", "moc_eval_batch_noalloc", "moc_graph_set_timing_events",
           "moc_search_create", "moc_search_run", "moc_search_state", "moc_search_best", "moc_search_info",
           "moc_search_destroy", "moc_search_set_kinds", "moc_graph_set_node_caps", "moc_check_intervals",
           "moc_cache_create", "moc_cache_build", "moc_eval_edits", "moc_cache_destroy", "moc_eval_batch_host16", "moc_search_set_samples",
           "moc_graph_set_kernel"]

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2304_14463_b200.build` "
                      "(nvcc, sm_100a). There is no CPU fallback.")

lib = ctypes.CDLL(LIB_PATH)
_P, _i32, _i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
lib.moc_graph_create.restype = ctypes.c_int
lib.moc_graph_create.argtypes = [_i32, _i64, _P, _P, _P, ctypes.POINTER(_P)]
lib.moc_graph_set_max_copies.restype = ctypes.c_int
lib.moc_graph_set_max_copies.argtypes = [_P, _i32]
lib.moc_graph_set_node_caps.restype = ctypes.c_int
lib.moc_graph_set_node_caps.argtypes = [_P, _P]
lib.moc_graph_destroy.restype = None
lib.moc_graph_destroy.argtypes = [_P]
lib.moc_graph_info.restype = ctypes.c_int
lib.moc_graph_info.argtypes = [_P, _P, _P, _P, _P]
lib.moc_eval_batch.restype = ctypes.c_int
lib.moc_eval_batch.argtypes = [_P, _P, _P, _i32, _i64, _P, _P, _P, _P]
lib.moc_eval_batch_host.restype = ctypes.c_int
lib.moc_eval_batch_host.argtypes = [_P, _P, _i64, _P, _i32, _i64, _P, _P, _P, _P]
lib.moc_eval_batch_host16.restype = ctypes.c_int
lib.moc_eval_batch_host16.argtypes = [_P, _P, _i64, _P, _i32, _i64, _P, _P, _P, _P]
lib.moc_eval_batch_noalloc.restype = ctypes.c_int
lib.moc_eval_batch_noalloc.argtypes = [_P, _P, _P, _i32, _i64, _P, _P, _P, _P]
lib.moc_mem_profile.restype = ctypes.c_int
lib.moc_mem_profile.argtypes = [_P, _P, _i32, _P, _P, _P, _P]
lib.moc_graph_set_launch.restype = ctypes.c_int
lib.moc_graph_set_launch.argtypes = [_P, _i32, _i32]
lib.moc_graph_set_kernel.restype = ctypes.c_int
lib.moc_graph_set_kernel.argtypes = [_P, _i32, _i32, _i32]
lib.moc_graph_set_timing_events.restype = ctypes.c_int
lib.moc_graph_set_timing_events.argtypes = [_P, _P, _P]
lib.moc_check_intervals.restype = ctypes.c_int
lib.moc_check_intervals.argtypes = [_P, _P, _P, _P, _i32, _i64, _P, _i64, _P, _P, _P, _P, _P, _P]
lib.moc_cache_create.restype = ctypes.c_int
lib.moc_cache_create.argtypes = [_P, _i32, ctypes.POINTER(_P)]
lib.moc_cache_build.restype = ctypes.c_int
lib.moc_cache_build.argtypes = [_P, _P, _P, _i32, _i64, _P, _P, _P, _P]
lib.moc_eval_edits.restype = ctypes.c_int
lib.moc_eval_edits.argtypes = [_P, _P, _P, _P, _P, _i32, _i64, _P, _P, _P, _P, _P]
lib.moc_cache_destroy.restype = None
lib.moc_cache_destroy.argtypes = [_P]
lib.moc_search_create.restype = ctypes.c_int
lib.moc_search_create.argtypes = [_P, _P, _P, _i32, _i64, ctypes.c_uint64, ctypes.c_uint32, _P, ctypes.POINTER(_P)]
lib.moc_search_run.restype = ctypes.c_int
lib.moc_search_run.argtypes = [_P, _i32, _P]
lib.moc_search_set_kinds.restype = ctypes.c_int
lib.moc_search_set_kinds.argtypes = [_P, ctypes.c_uint32]
lib.moc_search_set_samples.restype = ctypes.c_int
lib.moc_search_set_samples.argtypes = [_P, _i32, _i32]
lib.moc_search_state.restype = ctypes.c_int
lib.moc_search_state.argtypes = [_P, _P, _P, _P, _P, _P, _P, _P]
lib.moc_search_best.restype = ctypes.c_int
lib.moc_search_best.argtypes = [_P, _P, _P, _P]
lib.moc_search_info.restype = ctypes.c_int
lib.moc_search_info.argtypes = [_P, _P, _P, _P]
lib.moc_search_destroy.restype = None
lib.moc_search_destroy.argtypes = [_P]
lib.moc_last_launch_count.restype = ctypes.c_int
lib.moc_last_launch_count.argtypes = []
lib.moc_last_error.restype = ctypes.c_char_p
lib.moc_last_error.argtypes = []


class MocError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        text = lib.moc_last_error().decode(errors="replace")
        super().__init__(f"{where}: {ERROR_NAMES.get(code, code)}: {text}")


def _check(rc, where):
    if rc != MOC_OK:
        raise MocError(rc, where)


def _stream():
    import torch
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev(t, dtype, name):
    import torch
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of {dtype}")
    return ctypes.c_void_p(t.data_ptr())


def _host(a, dtype, name):
    """numpy array or CPU torch tensor -> pointer (the object must stay alive during the call)."""
    import numpy as np
    try:
        import torch
        if isinstance(a, torch.Tensor):
            if a.is_cuda or not a.is_contiguous():
                raise TypeError(f"{name}: expected a contiguous CPU tensor")
            if a.numpy().dtype != np.dtype(dtype):
                raise TypeError(f"{name}: expected dtype {dtype}")
            return ctypes.c_void_p(a.data_ptr())
    except ImportError:
        pass
    if not (isinstance(a, np.ndarray) and a.dtype == np.dtype(dtype) and a.flags.c_contiguous):
        raise TypeError(f"{name}: expected a C-contiguous numpy array of {dtype}")
    return ctypes.c_void_p(a.ctypes.data)


def moc_graph_create(n, edges, w, m):
    """edges: (k, 2) int32 host array of (u, v) = v consumes u; w, m: int64 host arrays of n."""
    import numpy as np
    edges = np.ascontiguousarray(np.asarray(edges, np.int32).reshape(-1, 2))
    w = np.ascontiguousarray(w, np.int64)
    m = np.ascontiguousarray(m, np.int64)
    if w.shape != (n,) or m.shape != (n,):
        raise ValueError("w and m must have n entries")
    h = _P()
    rc = lib.moc_graph_create(int(n), len(edges), edges.ctypes.data if len(edges) else None,
                              w.ctypes.data, m.ctypes.data, ctypes.byref(h))
    _check(rc, "moc_graph_create")
    return h


def moc_graph_set_max_copies(g, C):
    _check(lib.moc_graph_set_max_copies(g, int(C)), "moc_graph_set_max_copies")


def moc_graph_set_node_caps(g, caps):
    """caps: n ints (host), each in [1, C]; None restores the uniform cap."""
    import numpy as np
    if caps is None:
        _check(lib.moc_graph_set_node_caps(g, None), "moc_graph_set_node_caps")
        return
    caps = np.ascontiguousarray(caps, np.int32)
    _check(lib.moc_graph_set_node_caps(g, caps.ctypes.data), "moc_graph_set_node_caps")


def moc_graph_set_launch(g, threads_per_sequence=0, sequences_per_block=0):
    _check(lib.moc_graph_set_launch(g, int(threads_per_sequence), int(sequences_per_block)),
           "moc_graph_set_launch")


MOC_KERNEL_AUTO, MOC_KERNEL_GROUP, MOC_KERNEL_WARP, MOC_KERNEL_LANE, MOC_KERNEL_BLOCK = 0, 1, 2, 3, 4


def moc_graph_set_kernel(g, kind=MOC_KERNEL_AUTO, a=0, b=0):
    _check(lib.moc_graph_set_kernel(g, int(kind), int(a), int(b)), "moc_graph_set_kernel")


def moc_graph_set_timing_events(g, before=None, after=None):
    """before/after: torch.cuda.Event(enable_timing=True) recorded around the evaluation kernel of
    every following moc_eval_batch on this handle; None, None switches the hook off."""
    def raw(ev):
        if ev is None:
            return None
        if not ev.cuda_event:          # torch creates the CUDA event lazily, on the first record
            ev.record()
        return ctypes.c_void_p(ev.cuda_event)
    _check(lib.moc_graph_set_timing_events(g, raw(before), raw(after)), "moc_graph_set_timing_events")


def moc_graph_destroy(g):
    lib.moc_graph_destroy(g)


def moc_graph_info(g):
    n, ne, C, wide = _i32(), _i64(), _i32(), _i32()
    _check(lib.moc_graph_info(g, ctypes.byref(n), ctypes.byref(ne), ctypes.byref(C), ctypes.byref(wide)),
           "moc_graph_info")
    return dict(n=n.value, n_edges=ne.value, C=C.value, wide=bool(wide.value))


def _check_outputs(lens, outs):
    """The C ABI cannot see device buffer sizes: a short output would be overrun by the kernel."""
    B = lens.numel()
    for name, t in outs:
        if t.numel() < B:
            raise ValueError(f"{name} has {t.numel()} entries, the batch has {B} sequences")
        if t.device != lens.device:
            raise ValueError(f"{name} is on {t.device}, lens on {lens.device}")


def moc_eval_batch(g, seqs, lens, M, out_peak=None, out_dur=None, out_feasible=None):
    """Device tensors in, device tensors out (allocated with torch if not given). Asynchronous."""
    import torch
    B = lens.numel()
    if out_peak is None:
        out_peak = torch.empty(B, dtype=torch.int64, device=lens.device)
    if out_dur is None:
        out_dur = torch.empty(B, dtype=torch.int64, device=lens.device)
    if out_feasible is None:
        out_feasible = torch.empty(B, dtype=torch.int32, device=lens.device)
    _check_outputs(lens, (("out_peak", out_peak), ("out_dur", out_dur), ("out_feasible", out_feasible)))
    rc = lib.moc_eval_batch(g, _dev(seqs, torch.int32, "seqs"), _dev(lens, torch.int32, "lens"), B, int(M),
                            _dev(out_peak, torch.int64, "out_peak"), _dev(out_dur, torch.int64, "out_dur"),
                            _dev(out_feasible, torch.int32, "out_feasible"), _stream())
    _check(rc, "moc_eval_batch")
    return out_peak, out_dur, out_feasible


MOC_NOALLOC_MAX_B = 65536


def moc_eval_batch_noalloc(g, seqs, lens, M, out_peak, out_dur, out_feasible):
    """moc_eval_batch for callers that must not allocate: every tensor, outputs included, is passed
    in, and the library keeps its packing offsets in a fixed array of its own device image (at most
    MOC_NOALLOC_MAX_B sequences per call; calls on one device must not overlap on the GPU)."""
    import torch
    _check_outputs(lens, (("out_peak", out_peak), ("out_dur", out_dur), ("out_feasible", out_feasible)))
    rc = lib.moc_eval_batch_noalloc(g, _dev(seqs, torch.int32, "seqs"), _dev(lens, torch.int32, "lens"),
                                    lens.numel(), int(M), _dev(out_peak, torch.int64, "out_peak"),
                                    _dev(out_dur, torch.int64, "out_dur"),
                                    _dev(out_feasible, torch.int32, "out_feasible"), _stream())
    _check(rc, "moc_eval_batch_noalloc")
    return out_peak, out_dur, out_feasible


def moc_eval_batch_host(g, seqs, lens, M, out_peak, out_dur, out_feasible):
    """Host arrays (numpy or CPU tensors, ideally pinned) in and out; returns after the results landed."""
    import numpy as np
    B = int(lens.shape[0])
    rc = lib.moc_eval_batch_host(g, _host(seqs, np.int32, "seqs"), int(seqs.shape[0]), _host(lens, np.int32, "lens"),
                                 B, int(M), _host(out_peak, np.int64, "out_peak"), _host(out_dur, np.int64, "out_dur"),
                                 _host(out_feasible, np.int32, "out_feasible"), _stream())
    _check(rc, "moc_eval_batch_host")
    return out_peak, out_dur, out_feasible


def moc_eval_batch_host16(g, seqs, lens, M, out_peak, out_dur, out_feasible):
    """moc_eval_batch_host with uint16 node ids (n <= 65535): half the bytes over the host link."""
    import numpy as np
    B = int(lens.shape[0])
    rc = lib.moc_eval_batch_host16(g, _host(seqs, np.uint16, "seqs"), int(seqs.shape[0]), _host(lens, np.int32, "lens"),
                                   B, int(M), _host(out_peak, np.int64, "out_peak"), _host(out_dur, np.int64, "out_dur"),
                                   _host(out_feasible, np.int32, "out_feasible"), _stream())
    _check(rc, "moc_eval_batch_host16")
    return out_peak, out_dur, out_feasible


def moc_mem_profile(g, seq, want_free=True):
    """One device sequence -> (profile[int64], free[int32] or None, status[int32 tensor of 1])."""
    import torch
    T = seq.numel()
    profile = torch.empty(T, dtype=torch.int64, device=seq.device)
    free = torch.empty(T, dtype=torch.int32, device=seq.device) if want_free else None
    status = torch.empty(1, dtype=torch.int32, device=seq.device)
    rc = lib.moc_mem_profile(g, _dev(seq, torch.int32, "seq"), T, _dev(profile, torch.int64, "profile"),
                             _dev(free, torch.int32, "free") if want_free else None,
                             _dev(status, torch.int32, "status"), _stream())
    _check(rc, "moc_mem_profile")
    return profile, free, status


def moc_last_launch_count():
    return lib.moc_last_launch_count()


def moc_check_intervals(g, s, e, a, M, D, topo_index=None, want_seqs=True):
    """Device tensors s, e, a of shape [B, n, C] (int32) -> dict of device tensors mask, peak, dur and,
    with want_seqs, seqs [B, n*C] and lens."""
    import torch
    B, K = s.shape[0], s.shape[1] * s.shape[2]
    peak = torch.empty(B, dtype=torch.int64, device=s.device)
    dur = torch.empty(B, dtype=torch.int64, device=s.device)
    mask = torch.empty(B, dtype=torch.int32, device=s.device)
    seqs = torch.full((B, K), -1, dtype=torch.int32, device=s.device) if want_seqs else None
    lens = torch.empty(B, dtype=torch.int32, device=s.device) if want_seqs else None
    rc = lib.moc_check_intervals(g, _dev(s, torch.int32, "s"), _dev(e, torch.int32, "e"), _dev(a, torch.int32, "a"),
                                 B, int(D), _dev(topo_index, torch.int32, "topo_index") if topo_index is not None else None,
                                 int(M), _dev(peak, torch.int64, "peak"), _dev(dur, torch.int64, "dur"),
                                 _dev(mask, torch.int32, "mask"),
                                 _dev(seqs, torch.int32, "seqs") if want_seqs else None,
                                 _dev(lens, torch.int32, "lens") if want_seqs else None, _stream())
    _check(rc, "moc_check_intervals")
    return dict(mask=mask, peak=peak, dur=dur, seqs=seqs, lens=lens)


def moc_search_create(g, seqs, lens, M, seed, first_chain=0):
    """Device tensors (packed sequences, lengths) -> search handle; synchronous."""
    import torch
    h = _P()
    rc = lib.moc_search_create(g, _dev(seqs, torch.int32, "seqs"), _dev(lens, torch.int32, "lens"), lens.numel(),
                               int(M), ctypes.c_uint64(int(seed)), ctypes.c_uint32(int(first_chain)), _stream(),
                               ctypes.byref(h))
    _check(rc, "moc_search_create")
    return h


def moc_search_run(s, n_generations):
    _check(lib.moc_search_run(s, int(n_generations), _stream()), "moc_search_run")


MOC_EDIT_INSERT, MOC_EDIT_DELETE, MOC_EDIT_MOVE = 1, 2, 4


def moc_search_set_kinds(s, kinds):
    _check(lib.moc_search_set_kinds(s, int(kinds)), "moc_search_set_kinds")


def moc_search_info(s):
    P, stride, gen = _i32(), _i32(), ctypes.c_uint32()
    _check(lib.moc_search_info(s, ctypes.byref(P), ctypes.byref(stride), ctypes.byref(gen)), "moc_search_info")
    return dict(P=P.value, stride=stride.value, generation=gen.value)


def moc_search_state(s, want_rows=True):
    """-> dict of device tensors: rows [P, stride] (or None), lens, peak, dur, status, accepted."""
    import torch
    info = moc_search_info(s)
    P = info["P"]
    rows = torch.zeros((P, info["stride"]), dtype=torch.int32, device="cuda") if want_rows else None
    lens = torch.empty(P, dtype=torch.int32, device="cuda")
    peak = torch.empty(P, dtype=torch.int64, device="cuda")
    dur = torch.empty(P, dtype=torch.int64, device="cuda")
    status = torch.empty(P, dtype=torch.int32, device="cuda")
    acc = torch.empty(P, dtype=torch.int32, device="cuda")
    rc = lib.moc_search_state(s, ctypes.c_void_p(rows.data_ptr()) if want_rows else None,
                              ctypes.c_void_p(lens.data_ptr()), ctypes.c_void_p(peak.data_ptr()),
                              ctypes.c_void_p(dur.data_ptr()), ctypes.c_void_p(status.data_ptr()),
                              ctypes.c_void_p(acc.data_ptr()), _stream())
    _check(rc, "moc_search_state")
    return dict(rows=rows, lens=lens, peak=peak, dur=dur, status=status, accepted=acc)


def moc_search_best(s, max_len):
    """-> (seq tensor of max_len ints on the device, out_best tensor of 6 int64 on the device)."""
    import torch
    seq = torch.zeros(max_len, dtype=torch.int32, device="cuda")
    best = torch.empty(6, dtype=torch.int64, device="cuda")
    _check(lib.moc_search_best(s, ctypes.c_void_p(seq.data_ptr()), ctypes.c_void_p(best.data_ptr()), _stream()),
           "moc_search_best")
    return seq, best


def moc_search_destroy(s):
    lib.moc_search_destroy(s)


class Graph:
    """Owns a moc_graph handle (created on the current CUDA device)."""

    def __init__(self, n, edges, w, m, C=2):
        self.n = int(n)
        self.h = moc_graph_create(n, edges, w, m)
        try:
            moc_graph_set_max_copies(self.h, C)
        except Exception:
            moc_graph_destroy(self.h)
            self.h = None
            raise
        self.C = int(C)

    def close(self, _destroy=lib.moc_graph_destroy):
        if getattr(self, "h", None):
            _destroy(self.h)
            self.h = None

    __del__ = close

    def info(self):
        return moc_graph_info(self.h)

    def set_max_copies(self, C):
        moc_graph_set_max_copies(self.h, C)
        self.C = int(C)

    def set_caps(self, caps):
        if caps is not None and len(caps) != self.n:
            raise ValueError("caps must have n entries")
        moc_graph_set_node_caps(self.h, caps)

    def set_timing_events(self, before=None, after=None):
        moc_graph_set_timing_events(self.h, before, after)

    def set_launch(self, threads_per_sequence=0, sequences_per_block=0):
        moc_graph_set_launch(self.h, threads_per_sequence, sequences_per_block)

    def set_kernel(self, kind=MOC_KERNEL_AUTO, a=0, b=0):
        moc_graph_set_kernel(self.h, kind, a, b)

    def eval_batch(self, seqs, lens, M, **out):
        return moc_eval_batch(self.h, seqs, lens, M, **out)

    def eval_batch_host(self, seqs, lens, M, out_peak, out_dur, out_feasible):
        return moc_eval_batch_host(self.h, seqs, lens, M, out_peak, out_dur, out_feasible)

    def eval_batch_host16(self, seqs, lens, M, out_peak, out_dur, out_feasible):
        return moc_eval_batch_host16(self.h, seqs, lens, M, out_peak, out_dur, out_feasible)

    def mem_profile(self, seq, want_free=True):
        return moc_mem_profile(self.h, seq, want_free)

    def check_intervals(self, s, e, a, M, D=None, topo_index=None, want_seqs=True):
        if D is None:
            D = self.n * (self.n + 1) // 2 if topo_index is not None else self.C * self.n
        return moc_check_intervals(self.h, s, e, a, M, D, topo_index, want_seqs)

    def no_remat_peak(self):
        """Peak of the identity order 0..n-1 (the input topological order when ids are topological),
        the reference point for budgets given in percent (Section 4.3)."""
        import torch
        seq = torch.arange(self.n, dtype=torch.int32, device="cuda")
        lens = torch.tensor([self.n], dtype=torch.int32, device="cuda")
        peak, _, st = self.eval_batch(seq, lens, (1 << 62))
        torch.cuda.synchronize()
        if int(st[0]) != 1:
            raise ValueError("identity order is not a topological order of this graph")
        return int(peak[0])


class Search:
    """Owns a moc_search handle; keeps its Graph alive."""

    def __init__(self, graph: Graph, seqs, lens, M, seed, first_chain=0):
        self.graph = graph
        self.M = int(M)
        self.h = moc_search_create(graph.h, seqs, lens, M, seed, first_chain)

    def close(self, _destroy=lib.moc_search_destroy):
        if getattr(self, "h", None):
            _destroy(self.h)
            self.h = None

    __del__ = close

    def run(self, n_generations):
        moc_search_run(self.h, n_generations)

    def set_kinds(self, kinds):
        moc_search_set_kinds(self.h, kinds)

    def set_samples(self, samples, incremental=True):
        """samples proposals per chain and generation; incremental: False / 0 written out and evaluated from
        scratch, True / 1 scored from the cached evaluation (the library picks the kernel), 2 with a warp per
        proposal, 3 with a warp per chain (MOC_SEARCH_*)."""
        _check(lib.moc_search_set_samples(self.h, int(samples), int(incremental)), "moc_search_set_samples")

    def info(self):
        return moc_search_info(self.h)

    def state(self, want_rows=True):
        return moc_search_state(self.h, want_rows)

    def best(self):
        """-> dict(index, seq (numpy), peak, dur, status, accepted); synchronises."""
        import torch
        seq, b = moc_search_best(self.h, self.graph.C * self.graph.n)
        torch.cuda.synchronize()
        b = b.cpu().numpy()
        return dict(index=int(b[0]), seq=seq[:int(b[1])].cpu().numpy(), peak=int(b[2]), dur=int(b[3]),
                    status=int(b[4]), accepted=int(b[5]))


MOC_STATUS_PARENT_INVALID = -3
MOC_SEARCH_WRITTEN_OUT, MOC_SEARCH_SCORE_AUTO, MOC_SEARCH_SCORE_EDIT, MOC_SEARCH_SCORE_CHAIN = 0, 1, 2, 3


class EditCache:
    """Owns a moc_cache handle: evaluated parents on the device, from which single edits are scored."""

    def __init__(self, graph: Graph, max_parents):
        self.graph = graph
        h = _P()
        _check(lib.moc_cache_create(graph.h, int(max_parents), ctypes.byref(h)), "moc_cache_create")
        self.h = h

    def close(self, _destroy=lib.moc_cache_destroy):
        if getattr(self, "h", None):
            _destroy(self.h)
            self.h = None

    __del__ = close

    def build(self, seqs, lens, M):
        """Device tensors (packed parents) -> (peak, dur, status) device tensors of the parents."""
        import torch
        P = lens.numel()
        peak = torch.empty(P, dtype=torch.int64, device=lens.device)
        dur = torch.empty(P, dtype=torch.int64, device=lens.device)
        st = torch.empty(P, dtype=torch.int32, device=lens.device)
        rc = lib.moc_cache_build(self.h, _dev(seqs, torch.int32, "seqs"), _dev(lens, torch.int32, "lens"), P, int(M),
                                 _dev(peak, torch.int64, "peak"), _dev(dur, torch.int64, "dur"),
                                 _dev(st, torch.int32, "status"), _stream())
        _check(rc, "moc_cache_build")
        return peak, dur, st

    def eval_edits(self, parent, op, q, j, M, out=None, window=None):
        """int32 device tensors of B edits -> (peak, dur, status) device tensors; window: optional int32
        device tensor that receives the number of recomputed steps per edit."""
        import torch
        B = parent.numel()
        if out is None:
            out = (torch.empty(B, dtype=torch.int64, device=parent.device), torch.empty(B, dtype=torch.int64, device=parent.device),
                   torch.empty(B, dtype=torch.int32, device=parent.device))
        rc = lib.moc_eval_edits(self.h, _dev(parent, torch.int32, "parent"), _dev(op, torch.int32, "op"),
                                _dev(q, torch.int32, "q"), _dev(j, torch.int32, "j"), B, int(M),
                                _dev(out[0], torch.int64, "peak"), _dev(out[1], torch.int64, "dur"),
                                _dev(out[2], torch.int32, "status"),
                                _dev(window, torch.int32, "window") if window is not None else None, _stream())
        _check(rc, "moc_eval_edits")
        return out
