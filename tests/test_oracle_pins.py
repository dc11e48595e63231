"""Pins the CPU oracle to things other than itself (no GPU needed).

Each test checks an oracle function against what the paper or the mathematics fixes:
invariants, special cases that reduce to a library routine, or brute force written here
independently in NumPy on tiny inputs.
"""

import itertools
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2606_13392_b200.inputs import (MSAConfig, bits_to_f32, make_decode_inputs, make_prefill_inputs,
                                          to_bits)


def tiny(T=40, Hq=4, Hkv=2, Bk=4, k=3, d=8, di=4, seed=0, sharp=True):
    cfg = MSAConfig("tiny", "prefill", T, Hq, Hkv, Bk, k, head_dim=d, idx_dim=di, seed=seed)
    t = make_prefill_inputs(cfg, "cpu", sharp=sharp)
    return cfg, {n: to_bits(x) for n, x in t.items()}


def f64(bits):
    return bits_to_f32(bits).astype(np.float64)


# ---------------------------------------------------------------- brute force (P4)
def brute_scores(q_idx, k_idx, i, r, Bk):
    """Eq. 6 by enumeration: returns dict block -> max score over visible tokens."""
    qi, ki = f64(q_idx), f64(k_idx)
    out = {}
    for j in range(i + 1):
        s = float(np.dot(qi[i, r], ki[j])) / np.sqrt(qi.shape[-1])
        b = j // Bk
        out[b] = max(out.get(b, -np.inf), s)
    return out


def brute_select(block_scores, i, Bk, k):
    """Eq. 7 + local block by full sort of (score desc, index asc)."""
    loc = i // Bk
    earlier = sorted((b for b in block_scores if b < loc),
                     key=lambda b: (-block_scores[b], b))
    return sorted(earlier[:max(0, k - 1)] + [loc])


def brute_attn(q, K, V, i, h, r, blocks, Bk):
    """Eq. 8 by explicit token-set enumeration."""
    qf, Kf, Vf = f64(q), f64(K), f64(V)
    toks = [j for j in range(i + 1) if j // Bk in blocks]
    z = np.array([np.dot(qf[i, h], Kf[j, r]) for j in toks]) / np.sqrt(qf.shape[-1])
    w = np.exp(z - z.max())
    w /= w.sum()
    o = sum(wj * Vf[j, r] for wj, j in zip(w, toks))
    lse = z.max() + np.log(np.exp(z - z.max()).sum())
    return o, lse, toks


@pytest.mark.parametrize("T,Hq,Hkv,Bk,k", [
    (37, 2, 1, 4, 1), (37, 2, 2, 4, 2), (64, 4, 2, 8, 3), (23, 2, 1, 2, 3), (50, 4, 2, 4, 3),
])
def test_brute_force_tiny(T, Hq, Hkv, Bk, k):
    cfg, x = tiny(T=T, Hq=Hq, Hkv=Hkv, Bk=Bk, k=k, seed=T + k)
    pos = np.arange(T)
    M, I, O, LSE = oracle.msa_forward(x["q"], x["k"], x["v"], x["q_idx"], x["k_idx"],
                                      pos, Bk, k)
    G = Hq // Hkv
    for i in range(T):
        for r in range(Hkv):
            bs = brute_scores(x["q_idx"], x["k_idx"], i, r, Bk)
            for b in range(cfg.n_blocks):
                want = bs.get(b, -np.inf)
                assert M[i, r, b] == pytest.approx(want, rel=1e-12, abs=1e-14)
            sel = brute_select(bs, i, Bk, k)
            got = [b for b in I[i, r] if b >= 0]
            assert got == sel
            assert list(I[i, r, len(sel):]) == [-1] * (k - len(sel))
            for h in range(r * G, (r + 1) * G):
                o, lse, _ = brute_attn(x["q"], x["k"], x["v"], i, h, r, set(sel), Bk)
                np.testing.assert_allclose(O[i, h], o, rtol=1e-11, atol=1e-13)
                assert LSE[i, h] == pytest.approx(lse, rel=1e-12)


# ---------------------------------------------------------------- P1, P9: selection rules
def test_local_block_forced_and_inf_formulation():
    cfg, x = tiny(T=200, Hq=4, Hkv=2, Bk=8, k=5, seed=3)
    pos = np.arange(cfg.T)
    M = oracle.index_scores(x["q_idx"], x["k_idx"], pos, cfg.block_size)
    I = oracle.topk_select(M, pos, cfg.T, cfg.block_size, cfg.top_k)
    for i in pos:
        loc = i // cfg.block_size
        for r in range(cfg.n_kv_heads):
            got = [b for b in I[i, r] if b >= 0]
            assert loc in got and got == sorted(got) and len(set(got)) == len(got)
            assert len(got) == min(cfg.top_k, loc + 1)
            assert max(got) == loc  # nothing beyond the local block
            # Equivalent statement: give the local block +inf and take a plain top-k
            # (stable sort by descending score keeps the lower index first among ties).
            row = M[i, r].copy()
            row[loc] = np.inf
            order = np.argsort(-row, kind="stable")[:min(cfg.top_k, loc + 1)]
            assert sorted(order.tolist()) == got
            if loc < cfg.top_k:
                assert got == list(range(loc + 1))


def test_selection_invariances():
    cfg, x = tiny(T=160, Hq=2, Hkv=2, Bk=4, k=6, seed=5)
    pos = np.arange(cfg.T)
    M = oracle.index_scores(x["q_idx"], x["k_idx"], pos, cfg.block_size)
    I = oracle.topk_select(M, pos, cfg.T, cfg.block_size, cfg.top_k)
    # exact (power-of-two) positive scaling and a per-row shift do not change the set
    I2 = oracle.topk_select(M * 4.0, pos, cfg.T, cfg.block_size, cfg.top_k)
    assert np.array_equal(I, I2)
    shift = np.random.default_rng(0).integers(-8, 8, size=M.shape[:2] + (1,)).astype(np.float64)
    with np.errstate(invalid="ignore"):
        Ms = np.where(np.isfinite(M), np.round(M * 2 ** 20) / 2 ** 20 + shift, M)
        I_a = oracle.topk_select(np.where(np.isfinite(M), np.round(M * 2 ** 20) / 2 ** 20, M),
                                 pos, cfg.T, cfg.block_size, cfg.top_k)
    I_b = oracle.topk_select(Ms, pos, cfg.T, cfg.block_size, cfg.top_k)
    assert np.array_equal(I_a, I_b)


def test_tie_break_lower_index_wins():
    # 6 earlier blocks with equal scores: the lowest indices are taken.
    B, k, Bk = 8, 4, 2
    M = np.full((1, 1, B), -np.inf)
    M[0, 0, :7] = 1.0
    M[0, 0, 6] = 0.5  # local block's own score is irrelevant
    pos = np.array([6 * Bk + 1])
    I = oracle.topk_select(M, pos, B * Bk, Bk, k)
    assert I[0, 0].tolist() == [0, 1, 2, 6]
    M[0, 0, 4] = 2.0
    I = oracle.topk_select(M, pos, B * Bk, Bk, k)
    assert I[0, 0].tolist() == [0, 1, 4, 6]


# ---------------------------------------------------------------- P2: exp-free == top-k of softmax
def test_exp_free_equals_topk_of_softmax():
    cfg, x = tiny(T=256, Hq=2, Hkv=2, Bk=4, k=9, seed=7)
    pos = np.arange(cfg.T)
    M = oracle.index_scores(x["q_idx"], x["k_idx"], pos, cfg.block_size)
    I = oracle.topk_select(M, pos, cfg.T, cfg.block_size, cfg.top_k)
    for i in pos[::3]:
        loc = i // cfg.block_size
        if loc == 0:
            continue
        for r in range(cfg.n_kv_heads):
            row = M[i, r, :loc]
            p = np.exp(row - row.max())
            p /= p.sum()  # softmax over the rankable blocks, in double
            sel = np.array([b for b in I[i, r] if 0 <= b < loc], dtype=int)
            unsel = np.setdiff1d(np.arange(loc), sel)
            assert len(sel) == min(cfg.top_k - 1, loc)
            if len(unsel) and len(sel):
                assert p[sel].min() >= p[unsel].max()


# ---------------------------------------------------------------- P11: torch.topk agrees
def test_matches_torch_topk_away_from_ties():
    cfg, x = tiny(T=512, Hq=2, Hkv=1, Bk=4, k=8, seed=11)
    pos = np.arange(cfg.T)
    M = oracle.index_scores(x["q_idx"], x["k_idx"], pos, cfg.block_size)
    I = oracle.topk_select(M, pos, cfg.T, cfg.block_size, cfg.top_k)
    checked = 0
    for i in pos:
        loc = i // cfg.block_size
        if loc < cfg.top_k:
            continue
        row = torch.from_numpy(M[i, 0, :loc])
        vals, idx = torch.topk(row, cfg.top_k - 1)
        srt = torch.sort(row, descending=True).values
        if srt[cfg.top_k - 2] == srt[cfg.top_k - 1]:
            continue  # boundary tie: torch's choice is unspecified
        assert sorted(idx.tolist() + [loc]) == I[i, 0].tolist()
        checked += 1
    assert checked > 300


# ---------------------------------------------------------------- P8: stage 1 vs library matmul
def test_index_scores_match_matmul_reshape_max():
    cfg, x = tiny(T=96, Hq=4, Hkv=2, Bk=8, k=3, di=16, seed=13)
    pos = np.arange(cfg.T)
    M = oracle.index_scores(x["q_idx"], x["k_idx"], pos, cfg.block_size)
    qi, ki = f64(x["q_idx"]), f64(x["k_idx"])
    S = np.einsum("irc,jc->irj", qi, ki) / np.sqrt(cfg.idx_dim)  # [T,Hkv,T]
    causal = np.arange(cfg.T)[None, :] <= np.arange(cfg.T)[:, None]
    S = np.where(causal[:, None, :], S, -np.inf)
    want = S.reshape(cfg.T, cfg.n_kv_heads, cfg.n_blocks, cfg.block_size).max(-1)
    np.testing.assert_allclose(M, want, rtol=1e-12, atol=1e-14)
    # invisible blocks are exactly -inf, visible ones finite
    for i in range(cfg.T):
        loc = i // cfg.block_size
        assert np.all(np.isfinite(M[i, :, :loc + 1]))
        assert np.all(np.isneginf(M[i, :, loc + 1:]))


def test_index_scores_ragged_last_block():
    cfg, x = tiny(T=45, Hq=2, Hkv=1, Bk=8, k=2, di=8, seed=17)
    pos = np.array([44, 40, 39, 7, 0])
    M = oracle.index_scores(x["q_idx"][pos], x["k_idx"], pos, cfg.block_size)
    assert M.shape == (5, 1, 6)
    qi, ki = f64(x["q_idx"]), f64(x["k_idx"])
    for a, i in enumerate(pos):
        s = (ki[: i + 1] @ qi[i, 0]) / np.sqrt(cfg.idx_dim)
        for b in range(6):
            seg = s[b * 8: (b + 1) * 8]
            want = seg.max() if len(seg) else -np.inf
            assert M[a, 0, b] == pytest.approx(want, rel=1e-12, abs=1e-14)


# ---------------------------------------------------------------- P3: k >= B  ==> dense causal GQA
def test_all_blocks_selected_equals_dense_and_sdpa():
    cfg, x = tiny(T=70, Hq=6, Hkv=2, Bk=8, k=9, d=16, di=8, seed=19, sharp=True)
    assert cfg.top_k >= cfg.n_blocks
    pos = np.arange(cfg.T)
    _, I, O, LSE = oracle.msa_forward(x["q"], x["k"], x["v"], x["q_idx"], x["k_idx"],
                                      pos, cfg.block_size, cfg.top_k)
    Od, LSEd = oracle.dense_attn(x["q"], x["k"], x["v"], pos)
    np.testing.assert_allclose(O, Od, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(LSE, LSEd, rtol=1e-12)
    # library routine: torch SDPA, causal, KV heads repeated per group (adjacent heads)
    G = cfg.group
    q = torch.from_numpy(f64(x["q"])).permute(1, 0, 2)[None]  # [1,Hq,T,d]
    k = torch.from_numpy(f64(x["k"])).permute(1, 0, 2).repeat_interleave(G, 0)[None]
    v = torch.from_numpy(f64(x["v"])).permute(1, 0, 2).repeat_interleave(G, 0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True)
    ref = ref[0].permute(1, 0, 2).numpy()
    np.testing.assert_allclose(O, ref, rtol=1e-9, atol=1e-12)


def test_dense_attn_matches_numpy_definition():
    cfg, x = tiny(T=33, Hq=4, Hkv=2, Bk=4, k=2, d=8, seed=23)
    pos = np.array([0, 1, 17, 32])
    Od, LSEd = oracle.dense_attn(x["q"][pos], x["k"], x["v"], pos)
    qf, Kf, Vf = f64(x["q"]), f64(x["k"]), f64(x["v"])
    for a, t in enumerate(pos):
        for h in range(4):
            r = h // 2
            z = Kf[: t + 1, r] @ qf[t, h] / np.sqrt(8)
            al = np.exp(z) / np.exp(z).sum()
            np.testing.assert_allclose(Od[a, h], al @ Vf[: t + 1, r], rtol=1e-12, atol=1e-14)
            assert LSEd[a, h] == pytest.approx(np.log(np.exp(z).sum()), rel=1e-12)


# ---------------------------------------------------------------- P6: token budget
def test_token_budget():
    cfg, x = tiny(T=130, Hq=2, Hkv=1, Bk=8, k=4, seed=29)
    pos = np.arange(cfg.T)
    M = oracle.index_scores(x["q_idx"], x["k_idx"], pos, cfg.block_size)
    I = oracle.topk_select(M, pos, cfg.T, cfg.block_size, cfg.top_k)
    for i in pos:
        sel = [b for b in I[i, 0] if b >= 0]
        n_tok = sum(min((b + 1) * 8, i + 1) - b * 8 for b in sel)
        assert n_tok <= cfg.top_k * cfg.block_size
        full = (i // 8 >= cfg.top_k - 1) and (i % 8 == 7)
        assert (n_tok == cfg.top_k * cfg.block_size) == full


# ---------------------------------------------------------------- P7: combine identity
def test_combine_identity_any_partition():
    cfg, x = tiny(T=90, Hq=4, Hkv=2, Bk=8, k=5, d=8, seed=31)
    i = 85
    pos = np.array([i])
    qrow = x["q"][pos]
    M = oracle.index_scores(x["q_idx"][pos], x["k_idx"], pos, cfg.block_size)
    I = oracle.topk_select(M, pos, cfg.T, cfg.block_size, cfg.top_k)
    O, LSE = oracle.sparse_attn(qrow, x["k"], x["v"], I, pos, cfg.block_size)
    sel = [int(b) for b in I[0, 0] if b >= 0]
    assert len(sel) == 5
    for parts in ([[0], [1], [2], [3], [4]], [[0, 1, 2, 3, 4]], [[0, 3], [1], [2, 4]],
                  [[4], [0, 1, 2, 3]]):
        for h in range(cfg.n_q_heads):
            r = h // cfg.group
            blocks = [int(b) for b in I[0, r] if b >= 0]
            Op, Lp = [], []
            for part in parts:
                Ipart = np.full((1, cfg.n_kv_heads, cfg.top_k), -1, dtype=np.int32)
                Ipart[0, r, :len(part)] = sorted(blocks[t] for t in part)
                o, l = oracle.sparse_attn(qrow, x["k"], x["v"], Ipart, pos, cfg.block_size)
                Op.append(o[0, h])
                Lp.append(l[0, h])
            o_c, lse_c = oracle.combine(np.stack(Op), np.array(Lp))
            np.testing.assert_allclose(o_c, O[0, h], rtol=1e-12, atol=1e-14)
            assert lse_c == pytest.approx(LSE[0, h], rel=1e-12)


def test_combine_closed_form_two_parts():
    # two parts with LSE ln(1) and ln(3): weights 1/4 and 3/4
    o, lse = oracle.combine(np.array([[4.0, 0.0], [0.0, 8.0]]), np.log(np.array([1.0, 3.0])))
    np.testing.assert_allclose(o, [1.0, 6.0], rtol=1e-14)
    assert lse == pytest.approx(np.log(4.0), rel=1e-14)
    # an empty part (LSE = -inf) is ignored
    o, lse = oracle.combine(np.array([[4.0, 0.0], [7.0, 7.0]]), np.array([0.0, -np.inf]))
    np.testing.assert_allclose(o, [4.0, 0.0])
    assert lse == 0.0


# ---------------------------------------------------------------- P10: decode == last prefill row; causality
def test_decode_is_last_row_and_future_tokens_do_not_matter():
    cfg, x = tiny(T=77, Hq=4, Hkv=2, Bk=8, k=4, seed=37)
    pos = np.arange(cfg.T)
    M, I, O, LSE = oracle.msa_forward(x["q"], x["k"], x["v"], x["q_idx"], x["k_idx"],
                                      pos, cfg.block_size, cfg.top_k)
    for L in (1, 8, 9, 40, 77):
        p = np.array([L - 1])
        Md, Id, Od, Ld = oracle.msa_forward(x["q"][p], x["k"][:L], x["v"][:L],
                                            x["q_idx"][p], x["k_idx"][:L], p,
                                            cfg.block_size, cfg.top_k)
        nb = -(-L // cfg.block_size)
        np.testing.assert_array_equal(Md[0], M[L - 1][:, :nb])
        np.testing.assert_array_equal(Id[0], I[L - 1])
        np.testing.assert_array_equal(Od[0], O[L - 1])
        np.testing.assert_array_equal(Ld[0], LSE[L - 1])


# ---------------------------------------------------------------- P12: softmax sanity
def test_output_in_convex_hull_and_lse_finite():
    cfg, x = tiny(T=120, Hq=4, Hkv=2, Bk=8, k=3, d=8, seed=41)
    pos = np.arange(cfg.T)
    _, I, O, LSE = oracle.msa_forward(x["q"], x["k"], x["v"], x["q_idx"], x["k_idx"],
                                      pos, cfg.block_size, cfg.top_k)
    Vf = f64(x["v"])
    assert np.all(np.isfinite(LSE)) and np.all(np.isfinite(O))
    for i in pos[::7]:
        for h in range(cfg.n_q_heads):
            r = h // cfg.group
            toks = [j for j in range(i + 1) if j // 8 in set(I[i, r].tolist())]
            lo, hi = Vf[toks, r].min(0), Vf[toks, r].max(0)
            assert np.all(O[i, h] >= lo - 1e-12) and np.all(O[i, h] <= hi + 1e-12)
    # a query at position 0 sees one token: output is exactly that value row, LSE = z
    np.testing.assert_allclose(O[0, 0], Vf[0, 0], rtol=1e-15)


def test_group_sharing_uses_adjacent_heads():
    # Make KV head 1's values distinct constants: heads 2,3 (group 1) must output them.
    cfg, x = tiny(T=24, Hq=4, Hkv=2, Bk=4, k=2, d=8, seed=43)
    v = torch.zeros(24, 2, 8, dtype=torch.bfloat16)
    v[:, 0] = 1.0
    v[:, 1] = -2.0
    pos = np.arange(24)
    _, _, O, _ = oracle.msa_forward(x["q"], x["k"], to_bits(v), x["q_idx"], x["k_idx"], pos, 4, 2)
    np.testing.assert_allclose(O[:, 0:2], 1.0, rtol=1e-14)
    np.testing.assert_allclose(O[:, 2:4], -2.0, rtol=1e-14)


# ---------------------------------------------------------------- P5: printed FLOPs ratio
def test_index_lse_brute_force_dense_limit_and_bounds():
    # Section 4.3 (LSE fusion).  (a) token-by-token enumeration; (b) with every visible block
    # selected it is the log-sum-exp of the whole causal score row, which scipy computes from an
    # einsum; (c) it is the log-sum-exp of per-block log-sum-exps (the reduction the paper
    # describes), for any split of the list; (d) it lies between the largest selected block score
    # and that plus the log of the number of tokens summed.
    from scipy.special import logsumexp
    cfg, x = tiny(T=61, Hq=4, Hkv=2, Bk=4, k=4, di=8, seed=21)
    pos = np.arange(cfg.T)
    M = oracle.index_scores(x["q_idx"], x["k_idx"], pos, cfg.block_size)
    I = oracle.topk_select(M, pos, cfg.T, cfg.block_size, cfg.top_k)
    got = oracle.index_lse(x["q_idx"], x["k_idx"], I, pos, cfg.block_size)
    qi, ki = f64(x["q_idx"]), f64(x["k_idx"])
    for i in range(cfg.T):
        for r in range(cfg.n_kv_heads):
            blocks = [b for b in I[i, r] if b >= 0]
            z = np.array([np.dot(qi[i, r], ki[j]) / np.sqrt(cfg.idx_dim)
                          for j in range(i + 1) if j // cfg.block_size in blocks])
            want = np.log(np.exp(z - z.max()).sum()) + z.max()
            assert abs(got[i, r] - want) < 1e-12
            # (d)
            top = max(M[i, r, b] for b in blocks)
            assert top - 1e-12 <= got[i, r] <= top + np.log(len(z)) + 1e-12
            # (c): two sub-lists, each padded with -1
            if len(blocks) >= 2:
                a, b2 = blocks[:1], blocks[1:]
                Ia = np.full((1, 1, cfg.top_k), -1, np.int32); Ia[0, 0, :len(a)] = a
                Ib = np.full((1, 1, cfg.top_k), -1, np.int32); Ib[0, 0, :len(b2)] = b2
                la = oracle.index_lse(x["q_idx"][i:i + 1, r:r + 1], x["k_idx"], Ia, [i], cfg.block_size)[0, 0]
                lb = oracle.index_lse(x["q_idx"][i:i + 1, r:r + 1], x["k_idx"], Ib, [i], cfg.block_size)[0, 0]
                assert abs(np.logaddexp(la, lb) - got[i, r]) < 1e-12
    # (b)
    k_all = cfg.n_blocks
    I_all = oracle.topk_select(M, pos, cfg.T, cfg.block_size, k_all)
    dense = oracle.index_lse(x["q_idx"], x["k_idx"], I_all, pos, cfg.block_size)
    S = np.einsum("irc,jc->irj", qi, ki) / np.sqrt(cfg.idx_dim)
    causal = np.arange(cfg.T)[None, :] <= np.arange(cfg.T)[:, None]
    S = np.where(causal[:, None, :], S, -np.inf)
    np.testing.assert_allclose(dense, logsumexp(S, axis=-1), rtol=0, atol=1e-12)
    # an all-padding list has nothing to sum
    I_none = np.full((1, 1, 3), -1, np.int32)
    assert np.isneginf(oracle.index_lse(x["q_idx"][:1, :1], x["k_idx"], I_none, [0], cfg.block_size)[0, 0])


def test_fp8_index_operands_decode_and_scores():
    # The oracle's E4M3 decoding against torch's own conversion for all 256 codes (through a
    # one-element score: q = code, k = 1.0), and Eq. 6 on fp8 operands against an einsum on the
    # torch-decoded values.
    codes = np.arange(256, dtype=np.uint8)
    want = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    one = torch.tensor([1.0]).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    q = codes.reshape(256, 1, 1)                    # [n, H_kv=1, d_idx=1]
    k = np.repeat(one.reshape(1, 1), 256, axis=0)   # [L, 1]: every key is 1.0
    M = oracle.index_scores(q, k, np.arange(256), block_size=1, scale=1.0)
    got = np.array([M[i, 0, i] for i in range(256)])
    finite = np.isfinite(want)
    assert np.array_equal(got[finite], want[finite])
    assert list(np.nonzero(~finite)[0]) == [0x7F, 0xFF]  # the two NaN codes; a NaN is never a maximum
    cfg = MSAConfig("tiny8", "prefill", 50, 4, 2, 4, 3, head_dim=8, idx_dim=16, seed=5, idx_fp8=True)
    t = make_prefill_inputs(cfg, "cpu", sharp=True)
    assert t["q_idx"].dtype == torch.float8_e4m3fn
    qi, ki = t["q_idx"].to(torch.float64).numpy(), t["k_idx"].to(torch.float64).numpy()
    pos = np.arange(cfg.T)
    M = oracle.index_scores(to_bits(t["q_idx"]), to_bits(t["k_idx"]), pos, cfg.block_size)
    S = np.einsum("irc,jc->irj", qi, ki) / np.sqrt(cfg.idx_dim)
    causal = np.arange(cfg.T)[None, :] <= np.arange(cfg.T)[:, None]
    S = np.where(causal[:, None, :], S, -np.inf)
    pad = cfg.n_blocks * cfg.block_size - cfg.T
    S = np.pad(S, ((0, 0), (0, 0), (0, pad)), constant_values=-np.inf)
    np.testing.assert_allclose(M, S.reshape(cfg.T, cfg.n_kv_heads, cfg.n_blocks, cfg.block_size).max(-1),
                               rtol=1e-12, atol=1e-14)
    # and the log-sum-exp of the same operands, dense limit
    from scipy.special import logsumexp
    I_all = oracle.topk_select(M, pos, cfg.T, cfg.block_size, cfg.n_blocks)
    dense = oracle.index_lse(to_bits(t["q_idx"]), to_bits(t["k_idx"]), I_all, pos, cfg.block_size)
    np.testing.assert_allclose(dense, logsumexp(S, axis=-1), rtol=0, atol=1e-12)


def test_flops_model_printed_ratio():
    path = os.path.join(os.path.dirname(__file__), "golden", "flops_reduction_1m.txt")
    vals = {}
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        key, val = line.split()
        vals[key] = float(val)
    N = int(vals["N"])
    ratio = oracle.flops_gqa(N, int(vals["H_q"]), int(vals["d_h"])) / oracle.flops_msa(
        N, int(vals["H_q"]), int(vals["H_kv"]), int(vals["d_h"]), int(vals["d_idx"]),
        int(vals["k"]), int(vals["B_k"]))
    assert round(ratio, 1) == vals["ratio"]
    # closed forms of the two terms
    assert oracle.flops_gqa(10, 3, 5) == 2 * 3 * 5 * 100
    assert oracle.flops_msa(10, 4, 2, 5, 7, 3, 2) == 2 * 7 * 100 + 4 * 4 * 5 * 10 * 3 * 2


def test_fp8_kv_sparse_attention_equals_bf16_of_the_same_values():
    # Section 4.2 (the kernels also support fp8): K and V stored as fp8 E4M3.  Every E4M3 value is
    # exactly a bf16 value, so the oracle on fp8 K/V must give, bit for bit, what it gives on the bf16
    # tensors torch converts those fp8 tensors to (an independent decoding), and a visibly different
    # result from the unrounded bf16 caches.
    cfg = MSAConfig("kv8", "decode", 0, 8, 2, 16, 3, head_dim=32, idx_dim=16, seed=5, seq_lens=(70, 33), kv_fp8=True)
    x = make_decode_inputs(cfg, "cpu", sharp=True)
    assert x["k_cache"].dtype == torch.float8_e4m3fn and x["q"].dtype == torch.bfloat16
    L = cfg.seq_lens[0]
    K8, V8 = x["k_cache"][:L], x["v_cache"][:L]
    pos = np.array([L - 1])
    I = np.array([[[0, 2, 4], [1, 3, 4]]], dtype=np.int32)
    q = to_bits(x["q"][:1])
    O8, L8 = oracle.sparse_attn(q, to_bits(K8), to_bits(V8), I, pos, cfg.block_size)
    Ob, Lb = oracle.sparse_attn(q, to_bits(K8.to(torch.bfloat16)), to_bits(V8.to(torch.bfloat16)), I, pos, cfg.block_size)
    assert np.array_equal(O8, Ob) and np.array_equal(L8, Lb)
    xb = make_decode_inputs(cfg.scaled(kv_fp8=False), "cpu", sharp=True)
    Of, _ = oracle.sparse_attn(q, to_bits(xb["k_cache"][:L]), to_bits(xb["v_cache"][:L]), I, pos, cfg.block_size)
    assert 1e-4 < np.abs(Of - O8).max() < 0.2  # the rounding of K and V is there, and is small


def test_fp8_q_sparse_attention_equals_bf16_of_the_same_values():
    # Q stored as fp8 E4M3 as well (Section 4.2): the oracle on fp8 Q, K, V must give, bit for bit, what
    # it gives on the bf16 tensors torch converts them to (torch's decoding is independent of the
    # oracle's), a visibly different result from the unrounded Q, and the dense result when every block
    # is selected (the same SDPA pin as the bf16 path, on the decoded values).
    cfg = MSAConfig("q8", "prefill", 90, 8, 2, 16, 6, head_dim=32, idx_dim=16, seed=9, kv_fp8=True, q_fp8=True)
    x = make_prefill_inputs(cfg, "cpu", sharp=True)
    assert x["q"].dtype == torch.float8_e4m3fn and x["k"].dtype == torch.float8_e4m3fn
    pos = np.array([5, 31, 32, 89])
    I = np.tile(np.arange(6, dtype=np.int32), (len(pos), cfg.n_kv_heads, 1))
    for a, i in enumerate(pos):
        I[a][:, (i // cfg.block_size) + 1:] = -1
    q8, k8, v8 = x["q"][pos], x["k"], x["v"]
    O8, L8 = oracle.sparse_attn(to_bits(q8), to_bits(k8), to_bits(v8), I, pos, cfg.block_size)
    bf = torch.bfloat16
    Ob, Lb = oracle.sparse_attn(to_bits(q8.to(bf)), to_bits(k8.to(bf)), to_bits(v8.to(bf)), I, pos, cfg.block_size)
    assert np.array_equal(O8, Ob) and np.array_equal(L8, Lb)
    xq = make_prefill_inputs(cfg.scaled(q_fp8=False), "cpu", sharp=True)
    Of, _ = oracle.sparse_attn(to_bits(xq["q"][pos]), to_bits(k8), to_bits(v8), I, pos, cfg.block_size)
    assert 1e-4 < np.abs(Of - O8).max() < 0.3  # the rounding of Q is there, and is small
    # every visible block selected: torch SDPA on the decoded values (heads repeated per group)
    G = cfg.group
    qf, kf, vf = q8.float(), k8.float(), v8.float()
    for a, i in enumerate(pos):
        kk = kf[: i + 1].repeat_interleave(G, dim=1).permute(1, 0, 2)   # [H_q, i+1, d]
        vv = vf[: i + 1].repeat_interleave(G, dim=1).permute(1, 0, 2)
        ref = torch.nn.functional.scaled_dot_product_attention(qf[a][:, None, :], kk, vv)[:, 0, :]
        assert np.abs(ref.double().numpy() - O8[a]).max() < 2e-5
