"""The C-ABI library: it loads, exports every symbol the header declares, and its host-side
validation returns the documented error codes.  No kernel is launched (runs without a GPU)."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2304_14463_b200 import workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2304_14463_b200 import build
    build.build()
    from paper_2304_14463_b200 import binding
    return binding


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "moc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(moc_[a-z0-9_]+)\s*\(", text)))


def test_exports_match_header(binding):
    names = declared_symbols()
    assert "moc_graph_create" in names and "moc_eval_batch" in names and "moc_mem_profile" in names
    for name in names:
        assert hasattr(binding.lib, name), f"{name} declared in moc.h but not exported"
    assert sorted(binding.EXPORTS) == names


def _create(binding, n, edges, w, m):
    edges = np.asarray(edges, np.int32).reshape(-1, 2)
    w = np.asarray(w, np.int64)
    m = np.asarray(m, np.int64)
    h = ctypes.c_void_p()
    rc = binding.lib.moc_graph_create(n, len(edges), edges.ctypes.data if len(edges) else None,
                                      w.ctypes.data, m.ctypes.data, ctypes.byref(h))
    return rc, h


def test_create_validation(binding):
    one = [1, 1, 1]
    assert _create(binding, 3, [(0, 3)], one, one)[0] == -2            # endpoint out of range
    assert _create(binding, 3, [(-1, 1)], one, one)[0] == -2
    assert _create(binding, 3, [(1, 1)], one, one)[0] == -3            # self-loop
    assert _create(binding, 3, [(0, 1), (1, 2), (2, 0)], one, one)[0] == -3   # cycle
    assert _create(binding, 3, [], [1, -1, 1], one)[0] == -4           # negative weight
    assert _create(binding, 3, [], one, [1 << 59, 1 << 59, 1 << 59])[0] == -4  # 8*sum >= 2^62
    assert _create(binding, 0, [], [], [])[0] == -1
    rc, h = _create(binding, 3, [(0, 1), (1, 2), (2, 0)], one, one)
    assert rc == -3 and not h.value and b"cycle" in binding.lib.moc_last_error()
    assert binding.lib.moc_graph_create(3, 0, None, None, None, ctypes.byref(h)) == -1
    assert binding.lib.moc_graph_create(3, 0, None, None, None, None) == -1


def test_null_handles(binding):
    lib = binding.lib
    lib.moc_graph_destroy(None)
    assert lib.moc_graph_set_max_copies(None, 2) == -1
    assert lib.moc_graph_info(None, None, None, None, None) == -1
    assert lib.moc_eval_batch(None, None, None, 0, 0, None, None, None, None) == -1
    assert lib.moc_mem_profile(None, None, 0, None, None, None, None) == -1
    assert lib.moc_graph_set_launch(None, 0, 0) == -1
    assert lib.moc_graph_set_kernel(None, 0, 0, 0) == -1
    assert lib.moc_last_error() != b""
    # the later entry points: search, interval form, incremental evaluation
    h = ctypes.c_void_p()
    assert lib.moc_graph_set_node_caps(None, None) == -1
    assert lib.moc_search_create(None, None, None, 1, 0, 0, 0, None, ctypes.byref(h)) == -1 and not h.value
    assert lib.moc_search_run(None, 1, None) == -1
    assert lib.moc_search_set_kinds(None, 7) == -1
    assert lib.moc_search_state(None, None, None, None, None, None, None, None) == -1
    assert lib.moc_search_best(None, None, None, None) == -1
    assert lib.moc_search_info(None, None, None, None) == -1
    lib.moc_search_destroy(None)
    assert lib.moc_check_intervals(None, None, None, None, 1, 8, None, 0, None, None, None, None, None, None) == -1
    assert lib.moc_cache_create(None, 1, ctypes.byref(h)) == -1 and not h.value
    assert lib.moc_cache_build(None, None, None, 1, 0, None, None, None, None) == -1
    assert lib.moc_eval_edits(None, None, None, None, None, 1, 0, None, None, None, None, None) == -1
    lib.moc_cache_destroy(None)
    assert b"moc_eval_edits" in lib.moc_last_error() or lib.moc_last_error() != b""


def test_no_device_is_an_error_not_a_fallback(binding):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    rc, h = _create(binding, 3, [(0, 1)], [1, 1, 1], [1, 1, 1])
    assert rc in (-5, -6) and not h.value           # MOC_ERR_CUDA: no CPU path behind the ABI


def test_budget_rounding_matches_printed_budgets():
    """M = floor(P0*pct/100) reproduces the budgets printed under the plots of Section 4.3."""
    path = os.path.join(ROOT, "tests", "golden", "budget_rounding.txt")
    rows = [l for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for line in rows:
        p0 = int(line.split(":")[1].split("|")[0])
        budgets = [int(x) for x in line.split("|")[1].split()]
        assert [workloads.budget_from_peak(p0, pct) for pct in (90, 85, 80, 75)] == budgets
