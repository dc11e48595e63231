"""C-ABI checks that need no GPU: the library loads, exports every declared symbol, and
rejects bad arguments before launching anything."""

import ctypes
import os
import re

import pytest

from paper_2606_13392_b200 import binding as B
from paper_2606_13392_b200.build import build_library
from paper_2606_13392_b200.inputs import CONFIGS

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_library()
    return B.lib()


def declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if f.endswith(".h"):
            text = open(os.path.join(inc, f)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names.update(re.findall(r"\b(msa_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert "msa_index_scores" in names and "msa_topk_select" in names
    assert "msa_sparse_attn_prefill" in names and "msa_sparse_attn_decode" in names
    for n in names:
        assert hasattr(lib, n), "library does not export %s" % n
    assert set(B.EXPORTS) <= set(names)


def test_status_strings(lib):
    assert B.status_string(0) == "ok"
    assert "workspace" in B.status_string(3)
    assert B.status_string(99) == "unknown status"


def test_argument_validation_without_launch(lib):
    shape = B.shape_of(CONFIGS["c1"])
    null = ctypes.c_void_p(0)
    i64 = ctypes.c_int64
    # range outside the sequence
    assert lib.msa_index_scores(ctypes.byref(shape), null, null, i64(10), i64(10), i64(15), null,
                                i64(4), null) == 1
    # null pointers with a non-empty range
    assert lib.msa_index_scores(ctypes.byref(shape), null, null, i64(0), i64(1), i64(1), null,
                                i64(4), null) == 1
    # an empty range is a valid no-op
    assert lib.msa_index_scores(ctypes.byref(shape), null, null, i64(0), i64(0), i64(0), null,
                                i64(4), null) == 0
    assert lib.msa_topk_select(ctypes.byref(shape), null, i64(4), i64(0), i64(0), i64(0), null, null) == 0
    # bad shapes
    bad = B.shape_of(CONFIGS["c1"].scaled(n_q_heads=7, n_kv_heads=2))
    assert lib.msa_topk_select(ctypes.byref(bad), null, i64(4), i64(0), i64(0), i64(0), null, null) == 1
    bad = B.shape_of(CONFIGS["c1"].scaled(top_k=100000))
    assert lib.msa_topk_select(ctypes.byref(bad), null, i64(4), i64(0), i64(0), i64(0), null, null) == 2
    bad = B.shape_of(CONFIGS["c1"].scaled(head_dim=100))
    assert lib.msa_topk_select(ctypes.byref(bad), null, i64(4), i64(0), i64(0), i64(0), null, null) == 2
    assert lib.msa_index_scores(None, null, null, i64(0), i64(0), i64(0), null, i64(4), null) == 1
    # order of the blocks inside a score row: 0 or 1; run order exists for B_k 64 and 128 only,
    # and the decode calls take block order only
    bad = B.shape_of(CONFIGS["c1"], score_runs=2)
    assert lib.msa_topk_select(ctypes.byref(bad), null, i64(8), i64(0), i64(0), i64(0), null, null) == 1
    bad = B.shape_of(CONFIGS["c1"].scaled(block_size=16), score_runs=1)
    assert lib.msa_topk_select(ctypes.byref(bad), null, i64(8), i64(0), i64(0), i64(0), null, null) == 2
    runs = B.shape_of(CONFIGS["c1"], score_runs=1)
    assert lib.msa_topk_select(ctypes.byref(runs), null, i64(8), i64(0), i64(0), i64(0), null, null) == 0
    assert lib.msa_topk_select_decode(ctypes.byref(runs), null, i64(8), null, ctypes.c_int32(0), i64(0), null,
                                      null) == 2


def test_run_order_columns_are_a_permutation_inside_every_run():
    # msa_shape_t.score_runs = 1: the columns of a run of eight hold its blocks 0 2 4 6 1 3 5 7
    # (B_k = 128: one block per epilogue thread and key tile) or 0 1 4 5 2 3 6 7 (B_k = 64: two).
    from paper_2606_13392_b200 import api
    for bk, holds in ((128, [0, 2, 4, 6, 1, 3, 5, 7]), (64, [0, 1, 4, 5, 2, 3, 6, 7])):
        cols = api.run_order_columns(24, bk).tolist()
        assert sorted(cols) == list(range(24))
        for run in range(3):
            assert [cols.index(8 * run + c) - 8 * run for c in range(8)] == holds
        assert api.run_order_columns(13, bk).tolist() == cols[:13]


def test_workspace_queries(lib):
    for name in ("c1", "c2", "c3", "c4"):
        cfg = CONFIGS[name]
        shape = B.shape_of(cfg)
        mn, pf = B.msa_prefill_forward_workspace_bytes(shape, cfg.T)
        assert 0 < mn <= pf
        hmn, hpf = B.msa_prefill_forward_host_workspace_bytes(shape, cfg.T)
        assert hmn > mn and hpf >= hmn
        amn, apf = B.msa_sparse_attn_prefill_workspace_bytes(shape, cfg.T, cfg.T)
        assert 0 < amn <= apf <= pf
    assert B.msa_sparse_attn_decode_workspace_bytes(B.shape_of(CONFIGS["c5"]), 32) > 0
    # fp8 K/V caches: room for the bf16 copies of the visible K and V rows in front of the rest,
    # and half the K/V staging in the host-buffer call
    for name, q_count, kv_len in (("c3", 1000, 131072), ("p1m", 1048576, 1048576), ("c1", 7, 100)):
        cfg = CONFIGS[name]
        s16, s8 = B.shape_of(cfg), B.shape_of(cfg.scaled(kv_fp8=True))
        copies = 2 * ((kv_len * cfg.n_kv_heads * cfg.head_dim * 2 + 255) // 256 * 256)
        a16 = B.msa_sparse_attn_prefill_workspace_bytes(s16, q_count, kv_len)
        a8 = B.msa_sparse_attn_prefill_workspace_bytes(s8, q_count, kv_len)
        assert a8 == (a16[0] + copies, a16[1] + copies)
    s16, s8 = B.shape_of(CONFIGS["c3"]), B.shape_of(CONFIGS["c3"].scaled(kv_fp8=True))
    T = CONFIGS["c3"].T
    kv_bytes = T * 8 * 128
    h16, h8 = B.msa_prefill_forward_host_workspace_bytes(s16, T), B.msa_prefill_forward_host_workspace_bytes(s8, T)
    f16, f8 = B.msa_prefill_forward_workspace_bytes(s16, T), B.msa_prefill_forward_workspace_bytes(s8, T)
    assert h8[0] - f8[0] == h16[0] - f16[0] - 2 * kv_bytes
    # a workspace below the minimum is refused before any launch
    shape = B.shape_of(CONFIGS["c2"])
    one = ctypes.c_void_p(256)  # non-null, never dereferenced on this path
    code = lib.msa_prefill_forward(ctypes.byref(shape), one, one, one, one, one, ctypes.c_int64(32768),
                                   one, None, one, one, ctypes.c_size_t(16), None)
    assert code == 3


def test_varlen_validation_and_workspace(lib):
    shape = B.shape_of(CONFIGS["c3"])
    one = ctypes.c_void_p(256)  # non-null, never dereferenced on these paths
    i64x3 = (ctypes.c_int64 * 3)
    args = lambda cu, n: (ctypes.byref(shape), one, one, one, one, one, cu, ctypes.c_int32(n), one, None, one,
                          one, ctypes.c_size_t(16), None)
    assert lib.msa_prefill_forward_varlen(*args(None, 2)) == 1                  # no offsets
    assert lib.msa_prefill_forward_varlen(*args(i64x3(0, 500, 400), 2)) == 1    # decreasing
    assert lib.msa_prefill_forward_varlen(*args(i64x3(0, 0, 0), 2)) == 0        # nothing to do
    assert lib.msa_prefill_forward_varlen(*args(i64x3(0, 500, 900), -1)) == 1
    assert lib.msa_prefill_forward_varlen(*args(i64x3(0, 500, 900), 2)) == 3    # workspace too small
    # a batch of several sequences runs as one packed problem: its workspace holds the batch's maps (row
    # and block offsets, per-row and per-block arrays) in front of the stage buffers, and a larger
    # workspace buys longer query ranges as in the single-sequence call
    cu = [0, 300, 5000, 5100]
    mn, pf = B.msa_prefill_forward_varlen_workspace_bytes(shape, cu)
    m1, p1 = B.msa_prefill_forward_workspace_bytes(shape, 4700)
    rows, blocks = 5100, 3 + 37 + 1
    maps = 2 * rows * 4 + blocks * 4
    assert m1 <= mn <= m1 + maps + 64 * 1024 and mn <= pf
    # one sequence: exactly the single-sequence call
    mn, pf = B.msa_prefill_forward_varlen_workspace_bytes(shape, [0, 4700])
    assert (mn, pf) == (m1, p1)
    mn, pf = B.msa_prefill_forward_varlen_workspace_bytes(shape, [100, 4800])
    assert (mn, pf) == (m1, p1)


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError, match="missing"):
        B.lib()
