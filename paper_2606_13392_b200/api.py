"""Convenience layer over the binding: allocates outputs/workspaces with torch and calls the
C ABI.  No arithmetic happens here."""

from __future__ import annotations

from typing import Dict, Optional

import torch

from . import binding as B
from .inputs import MSAConfig


def prefill_forward(cfg: MSAConfig, x: Dict[str, torch.Tensor], workspace: Optional[torch.Tensor] = None,
                    want_lse: bool = True, workspace_bytes: Optional[int] = None):
    """Algorithm 1 lines 3-5 on device tensors q,k,v,q_idx,k_idx -> (out, lse, block_idx)."""
    shape = B.shape_of(cfg)
    T = x["q"].shape[0]
    dev = x["q"].device
    out = torch.empty(x["q"].shape, dtype=torch.bfloat16, device=dev)  # (Q itself may be fp8)
    lse = torch.empty((T, cfg.n_q_heads), dtype=torch.float32, device=dev) if want_lse else None
    block_idx = torch.empty((T, cfg.n_kv_heads, cfg.top_k), dtype=torch.int32, device=dev)
    if workspace is None:
        mn, pf = B.msa_prefill_forward_workspace_bytes(shape, T)
        workspace = B.alloc_workspace(pf if workspace_bytes is None else max(mn, workspace_bytes), dev)
    B.msa_prefill_forward(shape, x["q"], x["k"], x["v"], x["q_idx"], x["k_idx"], T, out, lse,
                          block_idx, workspace)
    return out, lse, block_idx


def prefill_forward_varlen(cfg: MSAConfig, x: Dict[str, torch.Tensor], cu_seqlens,
                           workspace: Optional[torch.Tensor] = None, want_lse: bool = True):
    """The same for sequences packed token-major; cu_seqlens: n_seqs+1 row offsets (host ints).
    block_idx holds block numbers relative to each row's own sequence."""
    shape = B.shape_of(cfg)
    T = x["q"].shape[0]
    dev = x["q"].device
    out = torch.empty(x["q"].shape, dtype=torch.bfloat16, device=dev)
    lse = torch.empty((T, cfg.n_q_heads), dtype=torch.float32, device=dev) if want_lse else None
    block_idx = torch.empty((T, cfg.n_kv_heads, cfg.top_k), dtype=torch.int32, device=dev)
    if workspace is None:
        _, pf = B.msa_prefill_forward_varlen_workspace_bytes(shape, cu_seqlens)
        workspace = B.alloc_workspace(pf, dev)
    B.msa_prefill_forward_varlen(shape, x["q"], x["k"], x["v"], x["q_idx"], x["k_idx"], cu_seqlens, out, lse,
                                 block_idx, workspace)
    return out, lse, block_idx


def index_lse(cfg: MSAConfig, q_idx: torch.Tensor, k_idx: torch.Tensor, block_idx: torch.Tensor,
              q_begin: int = 0, q_count: Optional[int] = None, kv_len: Optional[int] = None,
              workspace_bytes: Optional[int] = None) -> torch.Tensor:
    """Section 4.3: log-sum-exp of the index scores over the selected blocks, rows
    [q_begin, q_begin+q_count); q_idx and block_idx hold the whole sequence's rows."""
    shape = B.shape_of(cfg)
    kv_len = k_idx.shape[0] if kv_len is None else kv_len
    q_count = q_idx.shape[0] - q_begin if q_count is None else q_count
    out = torch.empty((q_count, cfg.n_kv_heads), dtype=torch.float32, device=q_idx.device)
    mn, pf = B.msa_index_lse_prefill_workspace_bytes(shape, q_count, kv_len)
    ws = B.alloc_workspace(pf if workspace_bytes is None else max(mn, workspace_bytes), q_idx.device)
    B.msa_index_lse_prefill(shape, q_idx[q_begin:q_begin + q_count], k_idx, block_idx[q_begin:q_begin + q_count],
                            q_begin, q_count, kv_len, out, ws)
    return out


def index_scores(cfg: MSAConfig, q_idx: torch.Tensor, k_idx: torch.Tensor, q_begin: int, q_count: int,
                 kv_len: Optional[int] = None, score_runs: int = 0) -> torch.Tensor:
    """Eq. 6 for rows [q_begin, q_begin+q_count); q_idx holds the whole sequence's rows.
    score_runs = 1: the columns of a row come in run order (run_order_columns gives the map)."""
    shape = B.shape_of(cfg, score_runs=score_runs)
    kv_len = k_idx.shape[0] if kv_len is None else kv_len
    ld = B.score_ld(kv_len, cfg.block_size)
    if score_runs:
        ld = (ld + 7) // 8 * 8
    scores = torch.full((q_count, cfg.n_kv_heads, ld), float("nan"), dtype=torch.float32,
                        device=q_idx.device)
    B.msa_index_scores(shape, q_idx[q_begin:q_begin + q_count], k_idx, q_begin, q_count, kv_len,
                       scores, ld)
    return scores


def run_order_columns(n_blocks: int, block_size: int) -> torch.Tensor:
    """Column of block b in a score row in run order (msa_shape_t.score_runs = 1), for b < n_blocks."""
    n = 128 // block_size
    b = torch.arange(n_blocks, dtype=torch.int64)
    w = b % 8
    return (b - w) + 4 * ((w // n) % 2) + n * (w // (2 * n)) + (w % n)


def topk_select(cfg: MSAConfig, scores: torch.Tensor, q_begin: int, kv_len: int, score_runs: int = 0) -> torch.Tensor:
    shape = B.shape_of(cfg, score_runs=score_runs)
    q_count, _, ld = scores.shape
    block_idx = torch.empty((q_count, cfg.n_kv_heads, cfg.top_k), dtype=torch.int32,
                            device=scores.device)
    B.msa_topk_select(shape, scores, ld, q_begin, q_count, kv_len, block_idx)
    return block_idx


def sparse_attn_prefill(cfg: MSAConfig, q, k, v, block_idx, q_begin: int = 0,
                        workspace_bytes: Optional[int] = None):
    shape = B.shape_of(cfg)
    q_count, kv_len = q.shape[0], k.shape[0]
    out = torch.empty(q.shape, dtype=torch.bfloat16, device=q.device)
    lse = torch.empty((q_count, cfg.n_q_heads), dtype=torch.float32, device=q.device)
    mn, pf = B.msa_sparse_attn_prefill_workspace_bytes(shape, q_count, kv_len)
    ws = B.alloc_workspace(pf if workspace_bytes is None else max(mn, workspace_bytes), q.device)
    B.msa_sparse_attn_prefill(shape, q, k, v, block_idx, q_begin, q_count, kv_len, out, lse, ws)
    return out, lse


def decode_forward(cfg: MSAConfig, x: Dict[str, torch.Tensor]):
    """One decode step for a batch of cached sequences -> (out, lse, block_idx, scores)."""
    shape = B.shape_of(cfg)
    batch = x["q"].shape[0]
    dev = x["q"].device
    max_len = int(max(cfg.seq_lens))
    ld = B.score_ld(max_len, cfg.block_size)
    scores = torch.empty((batch, cfg.n_kv_heads, ld), dtype=torch.float32, device=dev)
    block_idx = torch.empty((batch, cfg.n_kv_heads, cfg.top_k), dtype=torch.int32, device=dev)
    out = torch.empty_like(x["q"])
    lse = torch.empty((batch, cfg.n_q_heads), dtype=torch.float32, device=dev)
    ws = B.alloc_workspace(B.msa_sparse_attn_decode_workspace_bytes(shape, batch), dev)
    B.msa_decode_forward(shape, x["q"], x["q_idx"], x["k_cache"], x["v_cache"], x["k_idx_cache"],
                         x["k_cache"].shape[0], x["seq_offsets"], x["seq_lens"], batch, max_len,
                         scores, ld, block_idx, out, lse, ws)
    return out, lse, block_idx, scores
