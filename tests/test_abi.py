"""CPU-side checks of the boundary: the library builds for sm_100a, loads, exports every
symbol the header declares, and rejects bad arguments on the host without a GPU."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2608_08097_b200 import build, binding
    build.build()
    return binding


def header_symbols():
    text = open(os.path.join(ROOT, "include", "oasis.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(oasis_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    syms = header_symbols()
    assert set(syms) == set(L.SYMBOLS)
    lib = L.lib()
    for s in syms:
        assert getattr(lib, s) is not None
    assert L.lib().oasis_version().decode() == "0.1"


def test_oracle_and_library_share_nothing():
    """The checker and the product do not import, include or link each other."""
    pkg = os.path.join(ROOT, "paper_2608_08097_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text, f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2608_08097_b200" not in text and "oasis.h" not in text, f


def test_dims_validation(L):
    lib = L.lib()
    good = L.Dims(2, 32, 8, 64)
    null = ctypes.c_void_p(0)
    one = ctypes.c_void_p(4096)      # non-null, 16-byte aligned, never dereferenced on the host

    def summ(d):
        dc = d.c()
        return lib.oasis_build_summaries(ctypes.byref(dc), one, one, one, one, 1, one, null)

    assert summ(L.Dims(2, 32, 8, 64, head_dim=64)) == 2 and "head_dim" in L.last_error()
    assert summ(L.Dims(2, 32, 8, 64, block_size=32)) == 2 and "block_size" in L.last_error()
    assert summ(L.Dims(2, 30, 8, 64)) == 1 and "multiple" in L.last_error()
    assert summ(L.Dims(2, 32, 8, 0)) == 1
    dc = good.c()
    assert lib.oasis_build_summaries(ctypes.byref(dc), null, one, one, one, 1, one, null) == 1
    assert lib.oasis_build_summaries(ctypes.byref(dc), ctypes.c_void_p(4104), one, one, one, 1, one, null) == 1
    assert "aligned" in L.last_error()
    assert lib.oasis_build_summaries(ctypes.byref(dc), one, one, one, one, 65, one, null) == 1
    assert lib.oasis_build_summaries(None, one, one, one, one, 1, one, null) == 1


def test_argument_validation_of_each_call(L):
    lib = L.lib()
    dc = L.Dims(2, 32, 8, 64).c()
    d = ctypes.byref(dc)
    null, one = ctypes.c_void_p(0), ctypes.c_void_p(4096)
    dense = 4 * 32 * 128
    assert lib.oasis_score_blocks(d, one, dense, 4, one, one, 0, null, null) == 1          # scores NULL
    assert lib.oasis_score_blocks(d, one, dense, 0, one, one, 0, one, null) == 1           # n_draft
    assert lib.oasis_score_blocks(d, one, dense, 4, one, one, 7, one, null) == 1           # reduce mode
    assert lib.oasis_score_blocks(d, one, dense - 8, 4, one, one, 0, one, null) == 1       # stride too small
    assert lib.oasis_score_blocks(d, one, dense, 40, one, one, 0, one, null) == 2          # 160 rows
    assert "rows" in L.last_error()
    assert lib.oasis_select_topk(d, one, one, one, 5, 0, one, one, null, null, null) == 1  # k = 0
    assert lib.oasis_select_topk(d, one, one, one, 5, 4096, one, one, null, null, null) == 1
    assert lib.oasis_select_topk(d, one, one, one, 5, 8, one, one, one, null, null) == 1   # only one list
    big = L.Dims(2, 32, 8, 60000).c()
    assert lib.oasis_select_topk(ctypes.byref(big), one, one, one, 5, 8, one, one, null, null, null) == 2
    assert lib.oasis_stage_blocks(one, one, one, -1, one, null) == 1
    assert lib.oasis_stage_blocks(one, one, one, 0, one, null) == 0                        # nothing to do
    assert lib.oasis_stage_blocks(null, one, one, 3, one, null) == 1
    assert lib.oasis_sparse_attn(d, one, 5, one, one, one, 0, one, 1.0, one, null, null, 0, null) == 1
    assert lib.oasis_sparse_attn(d, one, 40, one, one, one, 130, one, 1.0, one, null, null, 0, null) == 2
    need = lib.oasis_attn_workspace_bytes(d, 5, 130)
    assert need > 0                                                                          # 16 rows on 148 SMs: split
    assert lib.oasis_sparse_attn(d, one, 5, one, one, one, 130, one, 1.0, one, null, null, 0, null) == 4
    assert "workspace" in L.last_error()
    assert lib.oasis_sparse_attn(d, one, 5, one, one, one, 130, one, 1.0, one, null, one, need - 1, null) == 4
    assert lib.oasis_plan_delta(d, one, 130, 128, one, one, one, 128, 130, 2, 130, 200, 1, one, one, null, null) == 1
    assert lib.oasis_plan_delta(d, one, 130, 128, one, one, one, 128, 130, 2, 100, 6, 1, one, one, null, null) == 1
    assert lib.oasis_plan_delta(d, one, 130, 128, one, one, one, 128, 129, 2, 130, 6, 1, one, one, null, null) == 1
    assert lib.oasis_plan_delta(d, one, 129, 128, one, one, one, 128, 130, 2, 130, 6, 1, one, one, null, null) == 1
    empty = L.Dims(0, 32, 8, 64).c()
    assert lib.oasis_score_blocks(ctypes.byref(empty), one, dense, 4, one, one, 0, one, null) == 0


def test_workspace_query_matches_plan(L):
    lib = L.lib()
    # one row per SM pair or more: no split, no workspace
    dc = L.Dims(64, 32, 8, 64).c()
    assert lib.oasis_attn_workspace_bytes(ctypes.byref(dc), 5, 130) == 0
    assert lib.oasis_attn_workspace_bytes(ctypes.byref(dc), 0, 130) == 0


def test_missing_library_fails_loudly(monkeypatch):
    from paper_2608_08097_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/liboasis.so")
    with pytest.raises(binding.OasisError, match="no CPU fallback"):
        binding.lib()
