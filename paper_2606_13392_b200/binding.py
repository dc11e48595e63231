"""Thin ctypes binding over ``libmsa_b200.so`` (the C ABI of ``include/msa.h``).

Argument marshalling only: tensors become device pointers, the current torch stream
becomes the stream argument, status codes become exceptions.  Every step of the path runs
in the CUDA kernels of the library.  If the library is missing this module raises; there
is no CPU fallback.
"""

from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

from .inputs import MSAConfig

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmsa_b200.so")
_lib: Optional[ctypes.CDLL] = None

c_i64, c_i32, c_vp, c_sz = ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p, ctypes.c_size_t

EXPORTS = [
    "msa_status_string", "msa_check_async_status", "msa_index_scores", "msa_index_scores_decode",
    "msa_topk_select", "msa_topk_select_decode", "msa_sparse_attn_prefill",
    "msa_sparse_attn_prefill_workspace_bytes", "msa_sparse_attn_prefill_static",
    "msa_sparse_attn_decode",
    "msa_sparse_attn_decode_workspace_bytes", "msa_index_topk_fused", "msa_index_lse_prefill",
    "msa_index_lse_prefill_workspace_bytes", "msa_prefill_forward",
    "msa_prefill_forward_workspace_bytes", "msa_prefill_forward_varlen",
    "msa_prefill_forward_varlen_workspace_bytes", "msa_prefill_forward_host",
    "msa_prefill_forward_host_workspace_bytes", "msa_decode_forward", "msa_decode_forward_host",
    "msa_launch_count", "msa_profile_begin", "msa_profile_end", "msa_index_scores_plan", "msa_debug_set_wait",
]


class MsaShape(ctypes.Structure):
    _fields_ = [("n_q_heads", c_i32), ("n_kv_heads", c_i32), ("head_dim", c_i32),
                ("idx_dim", c_i32), ("block_size", c_i32), ("top_k", c_i32),
                ("softmax_scale", ctypes.c_float), ("index_scale", ctypes.c_float),
                ("idx_fp8", c_i32), ("kv_fp8", c_i32), ("q_fp8", c_i32), ("score_runs", c_i32)]


class MsaError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s (status %d)" % (where, status_string(code), code))


def lib() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "CUDA library %s is missing: build it with "
                "`python -m paper_2606_13392_b200.build` (needs nvcc, sm_100a)" % LIB_PATH)
        _lib = ctypes.CDLL(LIB_PATH)
        _lib.msa_status_string.restype = ctypes.c_char_p
        _lib.msa_status_string.argtypes = [c_i32]
        _lib.msa_launch_count.restype = c_i64
        for name in EXPORTS:
            if name not in ("msa_status_string", "msa_launch_count"):
                getattr(_lib, name).restype = c_i32
    return _lib


def status_string(code: int) -> str:
    return lib().msa_status_string(code).decode()


def shape_of(cfg: MSAConfig, softmax_scale: float = 0.0, index_scale: float = 0.0, score_runs: int = 0) -> MsaShape:
    return MsaShape(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.idx_dim, cfg.block_size,
                    cfg.top_k, softmax_scale, index_scale, 1 if cfg.idx_fp8 else 0, 1 if cfg.kv_fp8 else 0,
                    1 if getattr(cfg, "q_fp8", False) else 0, score_runs)


def _ptr(t) -> c_vp:
    if t is None:
        return c_vp(0)
    assert t.is_contiguous(), "tensors passed to the C ABI must be contiguous"
    return c_vp(t.data_ptr())


def _dev(t: Optional[torch.Tensor]):
    if t is not None:
        assert t.is_cuda, "device pointer expected"
    return _ptr(t)


def _idx(shape, t: Optional[torch.Tensor], host: bool = False):
    """An index-branch operand: its element size must match the shape's idx_fp8 flag."""
    if t is not None:
        want = 1 if shape.idx_fp8 else 2
        assert t.element_size() == want, "index operand element size %d, shape expects %d" % (
            t.element_size(), want)
    return _host(t) if host else _dev(t)


def _kv(shape, t: Optional[torch.Tensor]):
    """A K or V tensor (device): its element size must match the shape's kv_fp8 flag."""
    if t is not None:
        want = 1 if shape.kv_fp8 else 2
        assert t.element_size() == want, "K/V cache element size %d, shape expects %d" % (t.element_size(), want)
    return _dev(t)


def _q(shape, t: Optional[torch.Tensor], host: bool = False):
    """The Q tensor: its element size must match the shape's q_fp8 flag."""
    if t is not None:
        want = 1 if shape.q_fp8 else 2
        assert t.element_size() == want, "Q element size %d, shape expects %d" % (t.element_size(), want)
    return _host(t) if host else _dev(t)


def _host(t: Optional[torch.Tensor]):
    if t is not None:
        assert not t.is_cuda, "host pointer expected"
    return _ptr(t)


def _stream(stream=None) -> c_vp:
    s = torch.cuda.current_stream() if stream is None else stream
    return c_vp(s.cuda_stream)


def _check(code: int, where: str) -> None:
    if code != 0:
        raise MsaError(code, where)


def launch_count() -> int:
    return int(lib().msa_launch_count())


STAGES = ["index_scores", "topk_select", "schedule", "attn_prefill", "combine",
          "index_scores_decode", "attn_decode", "combine_decode", "index_lse"]


def profile_begin() -> None:
    _check(lib().msa_profile_begin(), "msa_profile_begin")


def profile_end():
    """-> {stage: (ms, launches)} summed since profile_begin(); synchronises the device."""
    ms = (ctypes.c_float * len(STAGES))()
    n = (c_i64 * len(STAGES))()
    _check(lib().msa_profile_end(ms, n), "msa_profile_end")
    return {STAGES[i]: (float(ms[i]), int(n[i])) for i in range(len(STAGES))}


def check_async_status() -> Tuple[int, int]:
    """(status, detail) of the device-side status word; clears it.  Synchronises."""
    detail = c_i32(0)
    code = lib().msa_check_async_status(ctypes.byref(detail))
    return int(code), int(detail.value)


# ------------------------------------------------------------------ the four stages
def msa_index_scores(shape, q_idx, k_idx, q_begin, q_count, kv_len, scores, ld_scores, stream=None):
    _check(lib().msa_index_scores(ctypes.byref(shape), _idx(shape, q_idx), _idx(shape, k_idx), c_i64(q_begin),
                                  c_i64(q_count), c_i64(kv_len), _dev(scores), c_i64(ld_scores),
                                  _stream(stream)), "msa_index_scores")


def msa_index_scores_decode(shape, q_idx, k_idx_cache, seq_offsets, seq_lens, batch, max_seq_len,
                            scores, ld_scores, stream=None):
    _check(lib().msa_index_scores_decode(ctypes.byref(shape), _idx(shape, q_idx), _idx(shape, k_idx_cache),
                                         _dev(seq_offsets), _dev(seq_lens), c_i32(batch),
                                         c_i64(max_seq_len), _dev(scores), c_i64(ld_scores),
                                         _stream(stream)), "msa_index_scores_decode")


def msa_topk_select(shape, scores, ld_scores, q_begin, q_count, kv_len, block_idx, stream=None):
    _check(lib().msa_topk_select(ctypes.byref(shape), _dev(scores), c_i64(ld_scores), c_i64(q_begin),
                                 c_i64(q_count), c_i64(kv_len), _dev(block_idx), _stream(stream)),
           "msa_topk_select")


def msa_topk_select_decode(shape, scores, ld_scores, seq_lens, batch, max_seq_len, block_idx, stream=None):
    _check(lib().msa_topk_select_decode(ctypes.byref(shape), _dev(scores), c_i64(ld_scores),
                                        _dev(seq_lens), c_i32(batch), c_i64(max_seq_len), _dev(block_idx),
                                        _stream(stream)), "msa_topk_select_decode")


def msa_index_scores_plan(shape, q_count, kv_len) -> Tuple[bool, int]:
    """(runs on the tensor cores?, index heads per CTA) for msa_index_scores on the current device."""
    tc, nh = c_i32(0), c_i32(0)
    _check(lib().msa_index_scores_plan(ctypes.byref(shape), c_i64(q_count), c_i64(kv_len), ctypes.byref(tc),
                                       ctypes.byref(nh)), "msa_index_scores_plan")
    return bool(tc.value), int(nh.value)


def msa_debug_set_wait(wait_limit_cycles: int = 0, producer_delay_cycles: int = 0) -> None:
    """Test hook: shortens the device-side bounded waits (0 = the production limit) and makes the
    copy-issuing role of the tensor-core kernels start late by the given number of SM cycles."""
    _check(lib().msa_debug_set_wait(c_i64(wait_limit_cycles), c_i64(producer_delay_cycles)), "msa_debug_set_wait")


def msa_sparse_attn_prefill_workspace_bytes(shape, q_count, kv_len) -> Tuple[int, int]:
    mn, pf = c_sz(0), c_sz(0)
    _check(lib().msa_sparse_attn_prefill_workspace_bytes(ctypes.byref(shape), c_i64(q_count),
                                                         c_i64(kv_len), ctypes.byref(mn),
                                                         ctypes.byref(pf)),
           "msa_sparse_attn_prefill_workspace_bytes")
    return int(mn.value), int(pf.value)


def msa_sparse_attn_prefill(shape, q, k, v, block_idx, q_begin, q_count, kv_len, out, lse,
                            workspace, stream=None):
    _check(lib().msa_sparse_attn_prefill(ctypes.byref(shape), _q(shape, q), _kv(shape, k), _kv(shape, v),
                                         _dev(block_idx), c_i64(q_begin), c_i64(q_count),
                                         c_i64(kv_len), _dev(out), _dev(lse), _dev(workspace),
                                         c_sz(workspace.numel() * workspace.element_size()),
                                         _stream(stream)), "msa_sparse_attn_prefill")


STATIC_SCRATCH_BYTES = 64 << 20


def msa_sparse_attn_prefill_static(shape, q, k, v, block_idx, q_begin, q_count, kv_len, out, lse,
                                   stream=None):
    """Stage 3 (prefill) for callers that may not allocate device memory.

    Same inputs and outputs as :func:`msa_sparse_attn_prefill`, but no workspace argument:
    the scratch is a fixed array of ``STATIC_SCRATCH_BYTES`` inside the library's device
    image.  Meant for hosts that cannot call ``cudaMalloc`` or ask torch for a buffer at
    that point (a plug-in inside an engine that owns all device memory, code running after
    the memory pool was frozen).  Raises ``MsaError`` (workspace) when fewer than
    ``min(q_count, 16)`` queries fit the array.  Calls that overlap on the GPU race on the
    shared array; make the first call on a device outside any stream capture.
    """
    _check(lib().msa_sparse_attn_prefill_static(ctypes.byref(shape), _dev(q), _dev(k), _dev(v),
                                                _dev(block_idx), c_i64(q_begin), c_i64(q_count),
                                                c_i64(kv_len), _dev(out), _dev(lse),
                                                _stream(stream)), "msa_sparse_attn_prefill_static")


def msa_sparse_attn_decode_workspace_bytes(shape, batch) -> int:
    mn = c_sz(0)
    _check(lib().msa_sparse_attn_decode_workspace_bytes(ctypes.byref(shape), c_i32(batch),
                                                        ctypes.byref(mn)),
           "msa_sparse_attn_decode_workspace_bytes")
    return int(mn.value)


def msa_sparse_attn_decode(shape, q, k_cache, v_cache, cache_tokens, seq_offsets, seq_lens, batch,
                           block_idx, out, lse, workspace, stream=None):
    _check(lib().msa_sparse_attn_decode(ctypes.byref(shape), _dev(q), _kv(shape, k_cache), _kv(shape, v_cache),
                                        c_i64(cache_tokens), _dev(seq_offsets), _dev(seq_lens),
                                        c_i32(batch), _dev(block_idx), _dev(out), _dev(lse),
                                        _dev(workspace),
                                        c_sz(workspace.numel() * workspace.element_size()),
                                        _stream(stream)), "msa_sparse_attn_decode")


# ------------------------------------------------------------------ whole path
def msa_prefill_forward_workspace_bytes(shape, T) -> Tuple[int, int]:
    mn, pf = c_sz(0), c_sz(0)
    _check(lib().msa_prefill_forward_workspace_bytes(ctypes.byref(shape), c_i64(T), ctypes.byref(mn),
                                                     ctypes.byref(pf)),
           "msa_prefill_forward_workspace_bytes")
    return int(mn.value), int(pf.value)


def msa_prefill_forward(shape, q, k, v, q_idx, k_idx, T, out, lse, block_idx, workspace, stream=None):
    _check(lib().msa_prefill_forward(ctypes.byref(shape), _q(shape, q), _kv(shape, k), _kv(shape, v), _idx(shape, q_idx),
                                     _idx(shape, k_idx), c_i64(T), _dev(out), _dev(lse), _dev(block_idx),
                                     _dev(workspace),
                                     c_sz(workspace.numel() * workspace.element_size()),
                                     _stream(stream)), "msa_prefill_forward")


def msa_index_topk_fused(shape, q_idx, k_idx, q_begin, q_count, kv_len, block_idx, stream=None):
    _check(lib().msa_index_topk_fused(ctypes.byref(shape), _idx(shape, q_idx), _idx(shape, k_idx), c_i64(q_begin),
                                      c_i64(q_count), c_i64(kv_len), _dev(block_idx), _stream(stream)),
           "msa_index_topk_fused")


def msa_index_lse_prefill_workspace_bytes(shape, q_count, kv_len) -> Tuple[int, int]:
    mn, pf = c_sz(0), c_sz(0)
    _check(lib().msa_index_lse_prefill_workspace_bytes(ctypes.byref(shape), c_i64(q_count), c_i64(kv_len),
                                                       ctypes.byref(mn), ctypes.byref(pf)),
           "msa_index_lse_prefill_workspace_bytes")
    return int(mn.value), int(pf.value)


def msa_index_lse_prefill(shape, q_idx, k_idx, block_idx, q_begin, q_count, kv_len, lse_idx, workspace,
                          stream=None):
    _check(lib().msa_index_lse_prefill(ctypes.byref(shape), _idx(shape, q_idx), _idx(shape, k_idx), _dev(block_idx),
                                       c_i64(q_begin), c_i64(q_count), c_i64(kv_len), _dev(lse_idx),
                                       _dev(workspace), c_sz(workspace.numel() * workspace.element_size()),
                                       _stream(stream)), "msa_index_lse_prefill")


def _cu_array(cu_seqlens):
    cu = [int(c) for c in cu_seqlens]
    return (c_i64 * len(cu))(*cu), len(cu) - 1


def msa_prefill_forward_varlen_workspace_bytes(shape, cu_seqlens) -> Tuple[int, int]:
    arr, n = _cu_array(cu_seqlens)
    mn, pf = c_sz(0), c_sz(0)
    _check(lib().msa_prefill_forward_varlen_workspace_bytes(ctypes.byref(shape), arr, c_i32(n),
                                                            ctypes.byref(mn), ctypes.byref(pf)),
           "msa_prefill_forward_varlen_workspace_bytes")
    return int(mn.value), int(pf.value)


def msa_prefill_forward_varlen(shape, q, k, v, q_idx, k_idx, cu_seqlens, out, lse, block_idx, workspace,
                               stream=None):
    arr, n = _cu_array(cu_seqlens)
    _check(lib().msa_prefill_forward_varlen(ctypes.byref(shape), _q(shape, q), _kv(shape, k), _kv(shape, v), _idx(shape, q_idx),
                                            _idx(shape, k_idx), arr, c_i32(n), _dev(out), _dev(lse),
                                            _dev(block_idx), _dev(workspace),
                                            c_sz(workspace.numel() * workspace.element_size()),
                                            _stream(stream)), "msa_prefill_forward_varlen")


def msa_prefill_forward_host_workspace_bytes(shape, T) -> Tuple[int, int]:
    mn, pf = c_sz(0), c_sz(0)
    _check(lib().msa_prefill_forward_host_workspace_bytes(ctypes.byref(shape), c_i64(T),
                                                          ctypes.byref(mn), ctypes.byref(pf)),
           "msa_prefill_forward_host_workspace_bytes")
    return int(mn.value), int(pf.value)


def msa_prefill_forward_host(shape, q, k, v, q_idx, k_idx, T, out, lse, block_idx, workspace,
                             stream=None):
    """q..k_idx, out, lse, block_idx are HOST tensors (pinned for full copy rate)."""
    _check(lib().msa_prefill_forward_host(ctypes.byref(shape), _q(shape, q, True), _host(k), _host(v),
                                          _idx(shape, q_idx, True), _idx(shape, k_idx, True), c_i64(T), _host(out),
                                          _host(lse), _host(block_idx), _dev(workspace),
                                          c_sz(workspace.numel() * workspace.element_size()),
                                          _stream(stream)), "msa_prefill_forward_host")


def msa_decode_forward(shape, q, q_idx, k_cache, v_cache, k_idx_cache, cache_tokens, seq_offsets,
                       seq_lens, batch, max_seq_len, scores, ld_scores, block_idx, out, lse,
                       workspace, stream=None):
    _check(lib().msa_decode_forward(ctypes.byref(shape), _dev(q), _idx(shape, q_idx), _kv(shape, k_cache),
                                    _kv(shape, v_cache), _idx(shape, k_idx_cache), c_i64(cache_tokens),
                                    _dev(seq_offsets), _dev(seq_lens), c_i32(batch),
                                    c_i64(max_seq_len), _dev(scores), c_i64(ld_scores),
                                    _dev(block_idx), _dev(out), _dev(lse), _dev(workspace),
                                    c_sz(workspace.numel() * workspace.element_size()),
                                    _stream(stream)), "msa_decode_forward")


def msa_decode_forward_host(shape, q_host, q_idx_host, q_dev, q_idx_dev, k_cache, v_cache,
                            k_idx_cache, cache_tokens, seq_offsets, seq_lens, batch, max_seq_len,
                            scores, ld_scores, block_idx, out_dev, out_host, workspace, stream=None):
    _check(lib().msa_decode_forward_host(ctypes.byref(shape), _host(q_host), _idx(shape, q_idx_host, True),
                                         _dev(q_dev), _idx(shape, q_idx_dev), _kv(shape, k_cache), _kv(shape, v_cache),
                                         _idx(shape, k_idx_cache), c_i64(cache_tokens), _dev(seq_offsets),
                                         _dev(seq_lens), c_i32(batch), c_i64(max_seq_len),
                                         _dev(scores), c_i64(ld_scores), _dev(block_idx),
                                         _dev(out_dev), _host(out_host), _dev(workspace),
                                         c_sz(workspace.numel() * workspace.element_size()),
                                         _stream(stream)), "msa_decode_forward_host")


# ------------------------------------------------------------------ allocation helpers
def score_ld(kv_len: int, block_size: int) -> int:
    """Row pitch (in floats) for a scores buffer: B rounded up to a multiple of 4."""
    return (-(-kv_len // block_size) + 3) // 4 * 4


def alloc_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)
