"""The C-ABI library loads and exports every symbol the header declares; host-side argument
checks answer without a GPU."""
import ctypes as C
import os
import re

import pytest

from paper_2407_14057_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "lazyllm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b((?:lazy_|aux_cache_)\w+)\s*\(", text)
    return sorted(set(names))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = _declared_functions()
    assert "lazy_prefill_init" in names and "lazy_prefill_run" in names
    assert "lazy_decode_step" in names and "aux_cache_revive" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in lazyllm.h but not exported"
    assert sorted(binding.exported_names()) == names


def test_strerror_and_workspace_validation(lib):
    assert lib.lazy_strerror(0) == b"ok"
    assert b"schedule" in lib.lazy_strerror(-2)
    cfg = binding.lazy_model_cfg(2, 256, 4, 64, 688, 1024, 1e-6, 1e4, binding.LAZY_F32, 1, 256, 4)
    sched, keep = binding._make_schedule(((1, 5000),))
    assert lib.lazy_prefill_workspace_bytes(C.byref(cfg), C.byref(sched)) > 0
    bad, keep2 = binding._make_schedule(((0, 5000),))           # layer 0 cannot be a pruning point
    assert lib.lazy_prefill_workspace_bytes(C.byref(cfg), C.byref(bad)) == 0
    bad, keep3 = binding._make_schedule(((1, 5000), (1, 4000)))  # not strictly increasing
    assert lib.lazy_prefill_workspace_bytes(C.byref(cfg), C.byref(bad)) == 0
    bad, keep4 = binding._make_schedule(((1, 12000),))
    assert lib.lazy_prefill_workspace_bytes(C.byref(cfg), C.byref(bad)) == 0
    cfg.n_heads = 3                                               # heads * head_dim != d_model
    assert lib.lazy_prefill_workspace_bytes(C.byref(cfg), C.byref(sched)) == 0


def test_null_arguments_are_rejected_without_touching_the_device(lib):
    assert lib.lazy_prefill_run(None, None, None, None, 1, None) == -1
    assert lib.lazy_decode_step(None, None, None, None, None) == -1
    assert lib.aux_cache_revive(None, None, 0, 0, None, 0, None) == -1
    assert lib.lazy_k_gemm(None, 0, 0, None, None, None, None, 1, 8, 8) == -1
    assert lib.lazy_prune_op_workspace_bytes(0, 256, 4, 64, 1, 16) == 0


def test_keep_count_of_the_library_matches_the_worked_values(lib):
    """Host arithmetic only: the count the library sizes every buffer with, against the hand-worked
    fixture (Section 3.2, top-percentile selection as a count)."""
    with open(os.path.join(ROOT, "tests", "golden", "keep_counts.txt")) as f:
        rows = [l for l in f if l.strip() and not l.startswith("#")]
    for line in rows:
        N, bp, want = [int(t) for t in line.split("|")]
        assert lib.lazy_keep_count(N, bp, N) == want
    assert lib.lazy_keep_count(100, 7000, 50) == 50          # clamped to the rows present
    assert lib.lazy_keep_count(100, 1, 100) == 1             # never below one row
    assert lib.lazy_keep_count(0, 5000, 1) == 0 and lib.lazy_keep_count(10, 0, 10) == 0   # bad arguments
    assert lib.lazy_keep_count(10, 10001, 10) == 0


def test_wait_selftest_rejects_bad_arguments_without_a_device(lib):
    assert lib.lazy_k_wait_selftest(None, 2, 1000) == -1
    assert lib.lazy_k_wait_selftest(None, 0, 0) == -1
    assert lib.lazy_k_wait_selftest(None, 0, 200000) == -1     # limits above 0.1 s are refused
