"""CPU oracle for the MSA forward path: TEST INFRASTRUCTURE ONLY.

Thin ctypes loader around ``msa_oracle.c`` (plain C, double precision, OpenMP over query
rows).  Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the product path never does.  Nothing here imports the CUDA package.

Function-to-passage map:
  index_scores   Eq. 6 (token scores, causal block max, -inf for invisible blocks)
  topk_select    Eq. 7 + Local Block rule (Section 3.2), exp-free ranking (Section 4.1)
  sparse_attn    Eq. 8 (softmax attention over visible tokens of the selected blocks)
  dense_attn     Eq. 1 (dense causal GQA attention)
  combine        Section 4.2, "Two-phase forward" (LSE-weighted merge of partials)
  flops_gqa / flops_msa   Section 3.3 (complexity formulas)
"""

from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "msa_oracle.c")
_LIB = os.path.join(_HERE, "libmsa_oracle.so")
_lib: Optional[ctypes.CDLL] = None


def build(force: bool = False) -> str:
    """Compiles msa_oracle.c with gcc (IEEE arithmetic: no -ffast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.msa_oracle_combine.restype = ctypes.c_double
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, "oracle inputs are bf16 bit patterns (uint16)"
    return a


def _pos(pos) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(pos, dtype=np.int64))


def n_threads() -> int:
    return len(os.sched_getaffinity(0))


def _idx(a) -> np.ndarray:
    """Index-branch operand: bf16 bit patterns (uint16) or fp8 E4M3 bit patterns (uint8)."""
    a = np.asarray(a)
    assert a.dtype in (np.uint16, np.uint8), "index operands are uint16 (bf16) or uint8 (E4M3) bit patterns"
    return np.ascontiguousarray(a)


def index_scores(q_idx, k_idx, pos, block_size: int, scale: Optional[float] = None) -> np.ndarray:
    """Eq. 6.  q_idx [n,H_kv,d_idx], k_idx [L,d_idx] (both u16 = bf16 or both u8 = E4M3), pos [n]
    -> M [n,H_kv,B] f64."""
    q_idx, k_idx, pos = _idx(q_idx), _idx(k_idx), _pos(pos)
    assert q_idx.dtype == k_idx.dtype
    n, H_kv, d_idx = q_idx.shape
    L = k_idx.shape[0]
    assert k_idx.shape[1] == d_idx and len(pos) == n
    assert n == 0 or (pos.min() >= 0 and pos.max() < L)
    if scale is None:
        scale = 1.0 / np.sqrt(d_idx)
    B = -(-L // block_size)
    M = np.empty((n, H_kv, B), dtype=np.float64)
    _load().msa_oracle_index_scores(_p(q_idx), _p(k_idx), _p(pos), ctypes.c_int64(n),
                                    ctypes.c_int64(L), H_kv, d_idx, block_size,
                                    ctypes.c_double(scale), _p(M), int(q_idx.dtype == np.uint8))
    return M


def topk_select(M, pos, L: int, block_size: int, top_k: int) -> np.ndarray:
    """Eq. 7 + forced local block.  M [n,H_kv,B] f64 -> I [n,H_kv,k] int32 (ascending, -1 pad)."""
    M = np.ascontiguousarray(M, dtype=np.float64)
    pos = _pos(pos)
    n, H_kv, B = M.shape
    assert B == -(-L // block_size)
    I = np.empty((n, H_kv, top_k), dtype=np.int32)
    _load().msa_oracle_topk_select(_p(M), _p(pos), ctypes.c_int64(n), ctypes.c_int64(L),
                                   H_kv, block_size, top_k, _p(I))
    return I


def index_lse(q_idx, k_idx, I, pos, block_size: int, scale: Optional[float] = None) -> np.ndarray:
    """Section 4.3 (LSE fusion): log-sum-exp of the index scores over the visible tokens of the
    selected blocks.  q_idx [n,H_kv,d_idx] u16, k_idx [L,d_idx] u16, I [n,H_kv,k] int32 -> [n,H_kv] f64."""
    q_idx, k_idx, pos = _idx(q_idx), _idx(k_idx), _pos(pos)
    assert q_idx.dtype == k_idx.dtype
    I = np.ascontiguousarray(I, dtype=np.int32)
    n, H_kv, d_idx = q_idx.shape
    L = k_idx.shape[0]
    assert k_idx.shape[1] == d_idx and len(pos) == n and I.shape[:2] == (n, H_kv)
    if scale is None:
        scale = 1.0 / np.sqrt(d_idx)
    out = np.empty((n, H_kv), dtype=np.float64)
    _load().msa_oracle_index_lse(_p(q_idx), _p(k_idx), _p(I), _p(pos), ctypes.c_int64(n),
                                 ctypes.c_int64(L), H_kv, d_idx, block_size, I.shape[2],
                                 ctypes.c_double(scale), _p(out), int(q_idx.dtype == np.uint8))
    return out


def sparse_attn(q, K, V, I, pos, block_size: int, scale: Optional[float] = None):
    """Eq. 8.  q [n,H_q,d] (u16 = bf16 or u8 = fp8 E4M3), K,V [L,H_kv,d] (both u16 or both u8),
    I [n,H_kv,k] -> (O [n,H_q,d], LSE [n,H_q]) f64."""
    q, K, V, pos = _idx(q), _idx(K), _idx(V), _pos(pos)
    assert K.dtype == V.dtype
    I = np.ascontiguousarray(I, dtype=np.int32)
    n, H_q, d = q.shape
    L, H_kv, _ = K.shape
    k = I.shape[2]
    assert V.shape == K.shape and I.shape[:2] == (n, H_kv) and H_q % H_kv == 0
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    O = np.empty((n, H_q, d), dtype=np.float64)
    LSE = np.empty((n, H_q), dtype=np.float64)
    _load().msa_oracle_sparse_attn(_p(q), _p(K), _p(V), _p(I), _p(pos), ctypes.c_int64(n),
                                   ctypes.c_int64(L), H_q, H_kv, d, block_size, k,
                                   ctypes.c_double(scale), _p(O), _p(LSE), int(K.dtype == np.uint8),
                                   int(q.dtype == np.uint8))
    return O, LSE


def dense_attn(q, K, V, pos, scale: Optional[float] = None):
    """Eq. 1.  Same layouts as sparse_attn, no block selection."""
    q, K, V, pos = _u16(q), _u16(K), _u16(V), _pos(pos)
    n, H_q, d = q.shape
    L, H_kv, _ = K.shape
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    O = np.empty((n, H_q, d), dtype=np.float64)
    LSE = np.empty((n, H_q), dtype=np.float64)
    _load().msa_oracle_dense_attn(_p(q), _p(K), _p(V), _p(pos), ctypes.c_int64(n),
                                  ctypes.c_int64(L), H_q, H_kv, d, ctypes.c_double(scale),
                                  _p(O), _p(LSE))
    return O, LSE


def combine(O_parts, LSE_parts):
    """Section 4.2 combine.  O_parts [S,d], LSE_parts [S] -> (O [d], LSE)."""
    O_parts = np.ascontiguousarray(O_parts, dtype=np.float64)
    LSE_parts = np.ascontiguousarray(LSE_parts, dtype=np.float64)
    S, d = O_parts.shape
    out = np.empty(d, dtype=np.float64)
    lse = _load().msa_oracle_combine(_p(O_parts), _p(LSE_parts), S, d, _p(out))
    return out, float(lse)


def msa_forward(q, k, v, q_idx, k_idx, pos, block_size: int, top_k: int):
    """Algorithm 1, lines 3-5, for the listed query positions (rows of q, q_idx)."""
    M = index_scores(q_idx, k_idx, pos, block_size)
    I = topk_select(M, pos, k_idx.shape[0], block_size, top_k)
    O, LSE = sparse_attn(q, k, v, I, pos, block_size)
    return M, I, O, LSE


def flops_gqa(N: int, H_q: int, d_h: int) -> float:
    """Section 3.3: F_GQA(N) = 2 H_q d_h N^2."""
    return 2.0 * H_q * d_h * float(N) ** 2


def flops_msa(N: int, H_q: int, H_kv: int, d_h: int, d_idx: int, k: int, B_k: int) -> float:
    """Section 3.3: F_MSA(N) = H_kv d_idx N^2 + 4 H_q d_h N k B_k."""
    return H_kv * d_idx * float(N) ** 2 + 4.0 * H_q * d_h * float(N) * k * B_k
