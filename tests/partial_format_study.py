"""Tolerance study for narrower operand and partial formats in prefill attention (CPU only).

Calls nothing but the oracle, the seeded input generators and numpy/torch dtype conversions.

Section 4.2 says the kernels "also support fp8", which "rescales the absolute IO volume" of the
KV-outer scheme: Q, K, V and the partial buffer.  This script measures, with the oracle's own
arithmetic, what each narrowing costs in accuracy on the synthetic workloads, so that the formats
the CUDA path uses can be chosen on numbers:

  operands    Q, K, V rounded to E4M3 before Eq. 8 (error of the inputs themselves, against the
              oracle on the bf16 inputs; the CUDA path's fp8 mode is compared with the oracle ON
              the decoded fp8 values, so this column is context, not a tolerance)
  P           softmax weights of a block rounded to bf16 / E4M3 before they multiply V
  partials    per-block normalised partial outputs (Section 4.2, two-phase forward) rounded to
              bf16 / fp16 / E4M3 with one fp32 scale per row, then merged with the LSE-weighted combine

    python tests/partial_format_study.py             # prints one table per input scale
"""

from __future__ import annotations

import sys

import numpy as np
import torch

import os
import sys as _sys

_sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

import oracle  # noqa: E402
from paper_2606_13392_b200.inputs import MSAConfig, bits_to_f32, make_prefill_inputs, to_bits  # noqa: E402


def _round(x: np.ndarray, fmt: str) -> np.ndarray:
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float64)).float()
    if fmt == "f64":
        return x
    if fmt == "bf16":
        return t.to(torch.bfloat16).double().numpy()
    if fmt == "f16":
        return t.to(torch.float16).double().numpy()
    if fmt == "e4m3":
        return t.to(torch.float8_e4m3fn).double().numpy()
    if fmt == "e4m3+rowscale":  # one scale per row so that the row's largest magnitude sits at E4M3's 448
        m = t.abs().amax(dim=-1, keepdim=True).clamp_min(1e-30)
        s = 448.0 / m
        return ((t * s).to(torch.float8_e4m3fn).float() / s).double().numpy()
    raise ValueError(fmt)


def block_partials(xb, I_row, pos_i, r, cfg):
    """Per selected block of (query, group r): exact P rows, V rows, partial O and LSE (Eq. 8 restricted
    to one block), computed in double from the bit patterns."""
    G, d, Bk = cfg.group, cfg.head_dim, cfg.block_size
    q = bits_to_f32(xb["q_row"]).astype(np.float64)[r * G:(r + 1) * G]      # [G, d]
    out = []
    for b in I_row:
        if b < 0:
            continue
        j0, j1 = b * Bk, min((b + 1) * Bk, pos_i + 1)
        K = bits_to_f32(xb["k"][j0:j1, r]).astype(np.float64)
        V = bits_to_f32(xb["v"][j0:j1, r]).astype(np.float64)
        z = q @ K.T / np.sqrt(d)
        m = z.max(axis=1, keepdims=True)
        e = np.exp(z - m)
        ell = e.sum(axis=1, keepdims=True)
        out.append((e / ell, V, (m + np.log(ell))[:, 0]))
    return out


def study(cfg: MSAConfig, sharp: bool, n_pos: int = 24):
    x = make_prefill_inputs(cfg, "cpu", sharp=sharp)
    xb = {n: to_bits(t) for n, t in x.items()}
    lo = min(cfg.top_k * cfg.block_size, cfg.T - 1)       # rows that use their whole budget
    pos = np.sort(np.random.default_rng(3).choice(np.arange(lo, cfg.T), size=min(n_pos, cfg.T - lo), replace=False))
    M = oracle.index_scores(xb["q_idx"][pos], xb["k_idx"], pos, cfg.block_size)
    I = oracle.topk_select(M, pos, cfg.T, cfg.block_size, cfg.top_k)
    O_ref, _ = oracle.sparse_attn(xb["q"][pos], xb["k"], xb["v"], I, pos, cfg.block_size)
    # operands rounded to E4M3 (the oracle decodes them itself)
    f8 = lambda t: to_bits(t.to(torch.float8_e4m3fn))
    O_f8, _ = oracle.sparse_attn(f8(x["q"][pos]), f8(x["k"]), f8(x["v"]), I, pos, cfg.block_size)
    rows = {"operands E4M3 (vs bf16 inputs)": O_f8}
    variants = [("P f64, partials f64", "f64", "f64"), ("P bf16, partials bf16 (the CUDA path)", "bf16", "bf16"),
                ("P bf16, partials f16", "bf16", "f16"), ("P bf16, partials E4M3 + row scale", "bf16", "e4m3+rowscale"),
                ("P E4M3, partials bf16", "e4m3", "bf16"), ("P E4M3, partials E4M3 + row scale", "e4m3", "e4m3+rowscale")]
    G, d = cfg.group, cfg.head_dim
    for name, pf, of in variants:
        O = np.zeros_like(O_ref)
        for a, i in enumerate(pos):
            xrow = dict(xb)
            xrow["q_row"] = xb["q"][i]
            for r in range(cfg.n_kv_heads):
                parts = block_partials(xrow, I[a, r], int(i), r, cfg)
                Os = np.stack([_round(_round(P, pf) @ V, of) for P, V, _ in parts])     # [S, G, d]
                Ls = np.stack([L for _, _, L in parts])                                # [S, G]
                for g in range(G):
                    O[a, r * G + g], _ = oracle.combine(Os[:, g, :], Ls[:, g])
        rows[name] = O
    print("%s, %s inputs, %d queries x %d heads (|O| rms %.3g)" % (
        cfg.name, "unscaled N(0,1) ('sharp')" if sharp else "N(0,1)/sqrt(d)", len(pos), cfg.n_q_heads,
        float(np.sqrt(np.mean(O_ref ** 2)))))
    print("  %-42s %10s %10s %10s" % ("variant", "max-abs", "mean-abs", "rel-L2"))
    for name, O in rows.items():
        dlt = O - O_ref
        print("  %-42s %10.3g %10.3g %10.3g" % (name, np.abs(dlt).max(), np.abs(dlt).mean(),
                                                np.linalg.norm(dlt) / np.linalg.norm(O_ref)))


if __name__ == "__main__":
    T = int(sys.argv[1]) if len(sys.argv) > 1 else 12288
    for sharp in (False, True):
        study(MSAConfig("c3-12k", "prefill", T, 64, 8, 128, 64, seed=2), sharp)
        study(MSAConfig("paper-shape-12k", "prefill", T, 64, 4, 128, 16, idx_dim=128, seed=6), sharp)
