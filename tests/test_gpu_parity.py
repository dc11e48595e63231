"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element,
on the same seeded inputs.  Sizes here are ones the oracle finishes in seconds; full-size
configurations are covered on sampled query positions in test_gpu_full_configs.py."""

import numpy as np
import pytest
import torch

import oracle
from paper_2606_13392_b200 import api
from paper_2606_13392_b200 import binding as B
from paper_2606_13392_b200.inputs import (CONFIGS, MSAConfig, make_decode_inputs,
                                          make_prefill_inputs, sample_positions, to_bits)
from parity_utils import check_attn, check_scores, check_selection

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _bits(x):
    return {n: to_bits(t) for n, t in x.items() if t.dtype == torch.bfloat16}


def _assert_clean():
    code, detail = B.check_async_status()
    assert code == 0, "device status %d detail %d" % (code, detail)


def run_prefill_case(cfg: MSAConfig, sharp: bool, n_sample: int, ws_bytes=None):
    x = make_prefill_inputs(cfg, DEV, sharp=sharp)
    T = cfg.T
    pos = np.arange(T) if n_sample >= T else sample_positions(T, cfg.block_size, cfg.top_k, n_sample, 7)
    pos_t = torch.from_numpy(pos).to(DEV)
    # the oracle needs every key/value row but only the sampled query rows
    kb, vb, kib = to_bits(x["k"]), to_bits(x["v"]), to_bits(x["k_idx"])
    qb, qib = to_bits(x["q"][pos_t]), to_bits(x["q_idx"])[pos]

    # --- whole path on the GPU
    out, lse, I = api.prefill_forward(cfg, x, workspace_bytes=ws_bytes)
    torch.cuda.synchronize()
    _assert_clean()

    # --- stage 1 at the sampled rows (one call per run of consecutive positions)
    M_gpu = np.empty((len(pos), cfg.n_kv_heads, cfg.n_blocks), dtype=np.float32)
    runs = np.split(np.arange(len(pos)), np.where(np.diff(pos) != 1)[0] + 1)
    for run in runs:
        q0, qc = int(pos[run[0]]), len(run)
        s = api.index_scores(cfg, x["q_idx"], x["k_idx"], q0, qc)
        M_gpu[run] = s[:, :, :cfg.n_blocks].cpu().numpy()
    M_ref = oracle.index_scores(qib, kib, pos, cfg.block_size)
    score_err = check_scores(M_gpu, M_ref, pos, cfg.block_size)

    # --- stage 2: the GPU's own pipeline against the oracle's selection
    I_ref = oracle.topk_select(M_ref, pos, T, cfg.block_size, cfg.top_k)
    I_gpu = I[pos_t].cpu().numpy()
    exact, n_rows = check_selection(I_gpu, I_ref, M_ref, pos, cfg.block_size, cfg.top_k)

    # --- stage 3: oracle attention on the GPU's index lists
    O_ref, LSE_ref = oracle.sparse_attn(qb, kb, vb, I_gpu, pos, cfg.block_size)
    o = out[pos_t].float().cpu().numpy()
    stats = check_attn(o, lse[pos_t].cpu().numpy(), O_ref, LSE_ref, cfg.name)
    stats.update(score_err=score_err, exact_sets=exact, rows=n_rows)
    return stats


@pytest.mark.parametrize("sharp", [False, True])
def test_c1_full(sharp):
    stats = run_prefill_case(CONFIGS["c1"], sharp, n_sample=10 ** 9)
    assert stats["exact_sets"] >= 0.999
    print("c1", sharp, stats)


@pytest.mark.parametrize("sharp", [False, True])
def test_c2_shape_reduced_length(sharp):
    cfg = CONFIGS["c2"].scaled(name="c2-4k", T=4096 + 37)  # ragged last block
    stats = run_prefill_case(cfg, sharp, n_sample=384)
    assert stats["exact_sets"] >= 0.999
    print("c2-4k", sharp, stats)


@pytest.mark.parametrize("sharp", [False, True])
def test_c3_shape_reduced_length(sharp):
    cfg = CONFIGS["c3"].scaled(name="c3-12k", T=12288 + 5)
    stats = run_prefill_case(cfg, sharp, n_sample=256)
    assert stats["exact_sets"] >= 0.999
    print("c3-12k", sharp, stats)


def test_c3_shape_small_workspace_many_passes():
    # Same numbers must come out when the workspace forces many query ranges / score chunks.
    cfg = CONFIGS["c3"].scaled(name="c3-6k", T=6144 + 77)
    x = make_prefill_inputs(cfg, DEV, sharp=True)
    shape = B.shape_of(cfg)
    mn, pf = B.msa_prefill_forward_workspace_bytes(shape, cfg.T)
    o1, l1, i1 = api.prefill_forward(cfg, x, workspace_bytes=pf)
    o2, l2, i2 = api.prefill_forward(cfg, x, workspace_bytes=mn)
    torch.cuda.synchronize()
    _assert_clean()
    assert torch.equal(i1, i2)
    assert torch.equal(o1, o2) and torch.equal(l1, l2)


def test_varlen_batch_equals_sequence_by_sequence():
    # Packed sequences of different lengths (one shorter than a block, one empty): every sequence
    # must come out exactly as from its own single-sequence call, and one of them is checked
    # against the oracle through the packed call's outputs.
    cfg = CONFIGS["c3"].scaled(name="c3-varlen", T=0, top_k=8)
    lens = [1000, 37, 0, 4096 + 5, 129, 2500]
    cu = np.concatenate([[0], np.cumsum(lens)]).tolist()
    total = cu[-1]
    x = make_prefill_inputs(cfg.scaled(T=total), DEV, sharp=False)
    out, lse, I = api.prefill_forward_varlen(cfg.scaled(T=total), x, cu)
    torch.cuda.synchronize()
    _assert_clean()
    for s, L in enumerate(lens):
        if L == 0:
            continue
        a, b = cu[s], cu[s + 1]
        xs = {n: t[a:b].contiguous() for n, t in x.items()}
        o1, l1, i1 = api.prefill_forward(cfg.scaled(T=L), xs)
        torch.cuda.synchronize()
        assert torch.equal(I[a:b], i1), "sequence %d index lists" % s
        assert torch.equal(out[a:b], o1) and torch.equal(lse[a:b], l1), "sequence %d outputs" % s
    # oracle on the fourth sequence, positions relative to that sequence
    s = 3
    a, b, L = cu[s], cu[s + 1], lens[s]
    pos = sample_positions(L, cfg.block_size, cfg.top_k, 64, 11)
    pos_t = torch.from_numpy(pos).to(DEV)
    kb, vb, kib = to_bits(x["k"][a:b]), to_bits(x["v"][a:b]), to_bits(x["k_idx"][a:b])
    qb, qib = to_bits(x["q"][a:b][pos_t]), to_bits(x["q_idx"][a:b][pos_t])
    M_ref = oracle.index_scores(qib, kib, pos, cfg.block_size)
    I_ref = oracle.topk_select(M_ref, pos, L, cfg.block_size, cfg.top_k)
    I_gpu = I[a:b][pos_t].cpu().numpy()
    exact, n_rows = check_selection(I_gpu, I_ref, M_ref, pos, cfg.block_size, cfg.top_k)
    assert exact >= 0.999
    O_ref, LSE_ref = oracle.sparse_attn(qb, kb, vb, I_gpu, pos, cfg.block_size)
    check_attn(out[a:b][pos_t].float().cpu().numpy(), lse[a:b][pos_t].cpu().numpy(), O_ref, LSE_ref, "varlen")


@pytest.mark.parametrize("ws", ["preferred", "minimum"])
def test_varlen_short_and_long_sequences_in_one_batch(ws):
    # Short and long sequences mixed, an empty one, one of exactly 64 blocks: the batch runs as one
    # problem per stage (one fused index + Top-k launch, one reverse index / attention / merge per
    # query range, which spans sequence boundaries; many ranges with the minimum workspace).
    # Every sequence must come out exactly as from its own call.
    cfg = CONFIGS["c3"].scaled(name="c3-varlen-mix", T=0, top_k=8)
    lens = [3000, 700, 9000, 0, 500, 64, 100, 2000, 1500, 12000, 300, 8192]
    cu = np.concatenate([[0], np.cumsum(lens)]).tolist()
    total = cu[-1]
    x = make_prefill_inputs(cfg.scaled(T=total), DEV, sharp=False)
    shape = B.shape_of(cfg.scaled(T=total))
    mn, pf = B.msa_prefill_forward_varlen_workspace_bytes(shape, cu)
    workspace = B.alloc_workspace(pf if ws == "preferred" else mn, DEV)
    for rep in range(2):  # (the second call starts behind the first one's joins)
        out, lse, I = api.prefill_forward_varlen(cfg.scaled(T=total), x, cu, workspace=workspace)
    torch.cuda.synchronize()
    _assert_clean()
    for s, L in enumerate(lens):
        if L == 0:
            continue
        a, b = cu[s], cu[s + 1]
        xs = {n: t[a:b].contiguous() for n, t in x.items()}
        o1, l1, i1 = api.prefill_forward(cfg.scaled(T=L), xs)
        torch.cuda.synchronize()
        assert torch.equal(I[a:b], i1), "sequence %d index lists" % s
        assert torch.equal(out[a:b], o1) and torch.equal(lse[a:b], l1), "sequence %d outputs" % s


@pytest.mark.parametrize("name,T,Hq,Hkv,Bk,k,di,sharp", [
    ("c3 shape", 6144 + 77, 64, 8, 128, 64, 64, False),
    ("c3 shape, sharp", 5000, 64, 8, 128, 16, 64, True),
    ("paper regime", 4096 + 3, 64, 4, 128, 16, 128, True),
    ("B_k 64", 3000, 16, 2, 64, 8, 64, True),
    ("generic shape", 700, 6, 3, 16, 5, 32, True),
])
def test_index_lse_matches_oracle(name, T, Hq, Hkv, Bk, k, di, sharp):
    # Section 4.3: log-sum-exp of the index scores over the visible tokens of the selected blocks,
    # on the GPU's own selection; full sequence on the GPU, sampled rows in the oracle; the
    # smallest workspace as well (many query ranges).
    cfg = MSAConfig("lse", "prefill", T, Hq, Hkv, Bk, k, head_dim=128, idx_dim=di, seed=T)
    x = make_prefill_inputs(cfg, DEV, sharp=sharp)
    _, _, I = api.prefill_forward(cfg, x)
    got = api.index_lse(cfg, x["q_idx"], x["k_idx"], I)
    got_small = api.index_lse(cfg, x["q_idx"], x["k_idx"], I, workspace_bytes=0)
    torch.cuda.synchronize()
    _assert_clean()
    assert torch.equal(got, got_small)
    pos = sample_positions(T, Bk, k, 160, 5)
    pos_t = torch.from_numpy(pos).to(DEV)
    want = oracle.index_lse(to_bits(x["q_idx"][pos_t]), to_bits(x["k_idx"]), I[pos_t].cpu().numpy(), pos, Bk)
    err = np.abs(got[pos_t].cpu().numpy().astype(np.float64) - want)
    assert np.isfinite(want).all() and err.max() <= 2e-3, (name, float(err.max()))
    # a sub-range call gives the same rows
    q0, qc = T // 3, min(500, T - T // 3)
    sub = api.index_lse(cfg, x["q_idx"], x["k_idx"], I, q_begin=q0, q_count=qc)
    torch.cuda.synchronize()
    assert torch.equal(sub, got[q0:q0 + qc])


@pytest.mark.parametrize("T,Hq,Hkv,Bk,k,di,ties", [
    (4096 + 77, 64, 4, 128, 16, 128, False),   # the paper's regime
    (3000, 16, 2, 64, 8, 64, False),           # B_k 64: two blocks per thread and key tile
    (2500, 24, 3, 128, 16, 64, False),         # an odd number of index heads: one head per CTA
    (2048 + 5, 8, 1, 128, 1, 64, False),       # k = 1: the local block only
    (5000, 32, 4, 128, 12, 128, True),         # many exactly equal scores
])
def test_fused_index_topk_equals_separate_calls(T, Hq, Hkv, Bk, k, di, ties):
    # Eq. 6 + Eq. 7 in one kernel must write the very list the two calls write (ties included).
    cfg = MSAConfig("fused", "prefill", T, Hq, Hkv, Bk, k, head_dim=128, idx_dim=di, seed=T)
    x = make_prefill_inputs(cfg, DEV, sharp=True)
    if ties:  # keys repeat with period 7 blocks: block maxima of different blocks coincide exactly
        period = 7 * Bk
        x["k_idx"] = x["k_idx"][:period].repeat((T + period - 1) // period, 1)[:T].contiguous()
    shape = B.shape_of(cfg)
    I_f = torch.full((T, Hkv, k), -7, dtype=torch.int32, device=DEV)
    B.msa_index_topk_fused(shape, x["q_idx"], x["k_idx"], 0, T, T, I_f)
    M = api.index_scores(cfg, x["q_idx"], x["k_idx"], 0, T)
    I_s = api.topk_select(cfg, M, 0, T)
    torch.cuda.synchronize()
    _assert_clean()
    assert torch.equal(I_f, I_s), int((I_f != I_s).any(dim=2).sum())
    # a range that starts inside the sequence
    q0, qc = T // 2 + 3, T - (T // 2 + 3)
    I_r = torch.full((qc, Hkv, k), -7, dtype=torch.int32, device=DEV)
    B.msa_index_topk_fused(shape, x["q_idx"][q0:], x["k_idx"], q0, qc, T, I_r)
    torch.cuda.synchronize()
    assert torch.equal(I_r, I_s[q0:])


def test_single_item_tiles_many_ranges():
    # Few selections per query and the smallest workspace: nearly every (block, head) tile of a
    # query range holds a single item, so the K/V tile buffers change owner with every item.
    cfg = CONFIGS["c3"].scaled(name="c3-lone", T=4096 + 19, top_k=4)
    mn, _ = B.msa_prefill_forward_workspace_bytes(B.shape_of(cfg), cfg.T)
    run_prefill_case(cfg, sharp=False, n_sample=96, ws_bytes=mn)


@pytest.mark.parametrize("T,Hq,Hkv,Bk,k,d,di", [
    (1, 8, 1, 64, 8, 128, 64),        # a single token
    (63, 8, 1, 64, 8, 128, 64),       # less than one block
    (65, 16, 2, 64, 4, 128, 64),      # one token into the second block
    (300, 4, 2, 8, 3, 32, 16),        # tiny blocks, generic shapes
    (257, 6, 3, 16, 5, 64, 32),       # G = 2, H_kv = 3
    (1000, 16, 1, 32, 40, 128, 64),   # k larger than the number of blocks: dense causal
    (777, 32, 2, 128, 2, 128, 64),    # G = 16, k = 2 (local + one)
    (500, 8, 1, 64, 1, 128, 64),      # k = 1: local block only
])
def test_odd_shapes_full(T, Hq, Hkv, Bk, k, d, di):
    cfg = MSAConfig("odd", "prefill", T, Hq, Hkv, Bk, k, head_dim=d, idx_dim=di, seed=T)
    stats = run_prefill_case(cfg, True, n_sample=10 ** 9)
    assert stats["exact_sets"] >= 0.995
    if k >= cfg.n_blocks:  # every visible block selected: equals dense causal GQA (Eq. 1)
        x = make_prefill_inputs(cfg, DEV, sharp=True)
        xb = _bits(x)
        out, lse, _ = api.prefill_forward(cfg, x)
        Od, Ld = oracle.dense_attn(xb["q"], xb["k"], xb["v"], np.arange(T))
        check_attn(out.float().cpu().numpy(), lse.cpu().numpy(), Od, Ld, "dense")


def test_topk_bit_exact_on_arbitrary_scores():
    # Stage 2 alone on fp32 scores with many exact ties: sets must equal the oracle's bit for
    # bit (same values, same total order).
    g = torch.Generator(device="cpu").manual_seed(5)
    for (T, Bk, k, Hkv) in [(4096, 4, 64, 2), (3000, 2, 33, 1), (2048, 1, 128, 1), (5000, 8, 17, 3),
                            (9000, 1, 64, 1)]:
        cfg = MSAConfig("tk", "prefill", T, Hkv, Hkv, Bk, k)
        nb = cfg.n_blocks
        ld = B.score_ld(T, Bk)
        # coarse values => plenty of ties; a few +/-0 and -inf-free rows
        M = torch.randint(-50, 50, (T, Hkv, ld), generator=g).float() * 0.25
        M[::7] = torch.randn((len(range(0, T, 7)), Hkv, ld), generator=g)
        M[3::11] = -0.0
        Md = M.to(DEV)
        I = api.topk_select(cfg, Md, 0, T).cpu().numpy()
        pos = np.arange(T)
        I_ref = oracle.topk_select(M[:, :, :nb].double().numpy(), pos, T, Bk, k)
        assert np.array_equal(I, I_ref), (T, Bk, k)


def test_topk_row_offsets_and_ranges():
    cfg = MSAConfig("tk2", "prefill", 6000, 2, 2, 4, 32)
    ld = B.score_ld(cfg.T, cfg.block_size)
    g = torch.Generator(device="cpu").manual_seed(9)
    M = torch.randn((cfg.T, 2, ld), generator=g)
    I_ref = oracle.topk_select(M[:, :, :cfg.n_blocks].double().numpy(), np.arange(cfg.T), cfg.T, 4, 32)
    for q0, qc in [(0, 1), (5, 100), (4097, 1903), (5999, 1)]:
        I = api.topk_select(cfg, M[q0:q0 + qc].contiguous().to(DEV), q0, cfg.T).cpu().numpy()
        assert np.array_equal(I, I_ref[q0:q0 + qc])


def run_decode_case(cfg: MSAConfig, sharp: bool):
    x = make_decode_inputs(cfg, DEV, sharp=sharp)
    out, lse, I, scores = api.decode_forward(cfg, x)
    torch.cuda.synchronize()
    _assert_clean()
    offs = x["seq_offsets"].cpu().numpy()
    res = []
    for s, L in enumerate(cfg.seq_lens):
        sl = slice(int(offs[s]), int(offs[s]) + L)
        kb, vb = to_bits(x["k_cache"][sl]), to_bits(x["v_cache"][sl])
        kib = to_bits(x["k_idx_cache"][sl])
        pos = np.array([L - 1])
        nb = -(-L // cfg.block_size)
        M_ref = oracle.index_scores(to_bits(x["q_idx"][s:s + 1]), kib, pos, cfg.block_size)
        M_gpu = scores[s:s + 1, :, :nb].cpu().numpy()
        check_scores(M_gpu, M_ref, pos, cfg.block_size)
        nb_max = -(-max(cfg.seq_lens) // cfg.block_size)
        assert torch.isneginf(scores[s, :, nb:nb_max]).all()
        I_ref = oracle.topk_select(M_ref, pos, L, cfg.block_size, cfg.top_k)
        I_gpu = I[s:s + 1].cpu().numpy()
        exact, _ = check_selection(I_gpu, I_ref, M_ref, pos, cfg.block_size, cfg.top_k)
        O_ref, LSE_ref = oracle.sparse_attn(to_bits(x["q"][s:s + 1]), kb, vb, I_gpu, pos, cfg.block_size)
        st = check_attn(out[s:s + 1].float().cpu().numpy(), lse[s:s + 1].cpu().numpy(), O_ref, LSE_ref,
                        "decode seq %d" % s)
        st["exact"] = exact
        res.append(st)
    return res


@pytest.mark.parametrize("sharp", [False, True])
def test_decode_small_batch_mixed_lengths(sharp):
    cfg = CONFIGS["c5"].scaled(name="c5-small", seq_lens=(1, 127, 128, 129, 8192, 8200, 20000, 16384 + 64))
    res = run_decode_case(cfg, sharp)
    assert np.mean([r["exact"] for r in res]) >= 0.95


@pytest.mark.parametrize("kv8,idx8,G", [(False, False, 8), (True, False, 8), (False, False, 16), (True, True, 16)])
def test_decode_cache_slack_may_hold_anything(kv8, idx8, G):
    # A growing cache: every sequence owns `capacity` rows of which the first seq_lens[s] are
    # written.  The rows behind them (up to the end of the local block and beyond) hold NaN bit
    # patterns here; the step must give exactly what it gives on a packed cache.
    lens = (1, 100, 129, 5000, 8191, 8193, 12345)
    cfg = CONFIGS["c5"].scaled(name="c5-slack", n_kv_heads=64 // G, seq_lens=lens, kv_fp8=kv8, idx_fp8=idx8,
                               idx_dim=128 if idx8 else 64)
    x = make_decode_inputs(cfg, DEV, sharp=True)
    out, lse, I, scores = api.decode_forward(cfg, x)
    cap = 12345 + 300
    offs = x["seq_offsets"].cpu().numpy()

    def strided(t, nan_bits):
        wide = torch.empty((cap * len(lens),) + tuple(t.shape[1:]), dtype=t.dtype, device=DEV)
        wide.view(torch.uint8 if t.element_size() == 1 else torch.int16).fill_(nan_bits)
        for s_, L in enumerate(lens):
            wide[s_ * cap: s_ * cap + L] = t[int(offs[s_]): int(offs[s_]) + L]
        return wide

    y = dict(x)
    y["k_cache"] = strided(x["k_cache"], 0x7F if kv8 else 0x7FC0)
    y["v_cache"] = strided(x["v_cache"], 0x7F if kv8 else 0x7FC0)
    y["k_idx_cache"] = strided(x["k_idx_cache"], 0x7F if idx8 else 0x7FC0)
    y["seq_offsets"] = torch.arange(len(lens), dtype=torch.int64, device=DEV) * cap
    out2, lse2, I2, scores2 = api.decode_forward(cfg, y)
    torch.cuda.synchronize()
    _assert_clean()
    assert torch.equal(I, I2)
    assert torch.isfinite(out2.float()).all() and torch.isfinite(lse2).all()
    assert torch.equal(out, out2) and torch.equal(lse, lse2)


def test_decode_topk_row_longer_than_the_score_pitch_is_reported():
    # seq_lens is a device array: a length beyond what the score rows hold must not be read past
    # the row.  The row's list comes back as all -1 and the status word names a bad index.
    cfg = CONFIGS["c5"].scaled(name="c5-pitch", seq_lens=(4096, 4096))
    shape = B.shape_of(cfg)
    ld = B.score_ld(4096, cfg.block_size)
    scores = torch.randn((2, cfg.n_kv_heads, ld), device=DEV)
    lens = torch.tensor([4096, 4096 * 9], dtype=torch.int32, device=DEV)   # the second one lies
    idx = torch.full((2, cfg.n_kv_heads, cfg.top_k), -5, dtype=torch.int32, device=DEV)
    with pytest.raises(B.MsaError):   # the pitch cannot hold the stated maximum
        B.msa_topk_select_decode(shape, scores, ld, lens, 2, 4096 * 9, idx)
    B.msa_topk_select_decode(shape, scores, ld, lens, 2, 4096, idx)
    code, _ = B.check_async_status()
    assert code == 6  # MSA_ERR_BAD_INDEX
    loc = 4095 // cfg.block_size   # fewer visible blocks than top_k: all of them, then padding
    assert bool((idx[1] == -1).all()) and bool((idx[0, :, loc] == loc).all()) and bool((idx[0, :, loc + 1] == -1).all())
    assert B.check_async_status()[0] == 0


def test_decode_generic_shape():
    cfg = MSAConfig("dec-odd", "decode", 0, 6, 3, 16, 5, head_dim=64, idx_dim=32, seed=3,
                    seq_lens=(5, 16, 17, 400, 1000))
    run_decode_case(cfg, True)


def test_decode_equals_last_prefill_row():
    # The decode call on a cache of length L gives row L-1 of the prefill call (same kernels'
    # arithmetic may differ in order, so compare within tolerance, and sets exactly).
    cfg = CONFIGS["c3"].scaled(name="c3-9k", T=9000)
    x = make_prefill_inputs(cfg, DEV, sharp=True)
    out, lse, I = api.prefill_forward(cfg, x)
    dcfg = cfg.scaled(mode="decode", seq_lens=(cfg.T,))
    xd = {"q": x["q"][-1:].contiguous(), "q_idx": x["q_idx"][-1:].contiguous(), "k_cache": x["k"],
          "v_cache": x["v"], "k_idx_cache": x["k_idx"],
          "seq_offsets": torch.zeros(1, dtype=torch.int64, device=DEV),
          "seq_lens": torch.tensor([cfg.T], dtype=torch.int32, device=DEV)}
    od, ld_, Id, _ = api.decode_forward(dcfg, xd)
    assert torch.equal(Id[0], I[-1])
    assert torch.allclose(od[0].float(), out[-1].float(), atol=2e-2)
    assert torch.allclose(ld_[0], lse[-1], atol=2e-3)


def test_bad_block_index_is_reported_not_dereferenced():
    cfg = CONFIGS["c1"]
    x = make_prefill_inputs(cfg, DEV)
    out, lse, I = api.prefill_forward(cfg, x)
    bad = I.clone()
    bad[100, 0, 0] = 10 ** 6   # far outside the sequence
    bad[200, 0, 1] = -7        # not the padding value
    o2, _ = api.sparse_attn_prefill(cfg, x["q"], x["k"], x["v"], bad)
    code, _ = B.check_async_status()
    assert code == 6  # MSA_ERR_BAD_INDEX
    assert torch.isfinite(o2.float()).all()
    assert B.check_async_status()[0] == 0  # cleared


@pytest.mark.parametrize("name,T,ws_scale", [("c1", 2048, 1.0), ("c3", 5000, 0.0), ("c3", 9001, 1.0), ("odd", 300, 1.0),
                                             ("c3-kv8", 5000, 0.0), ("c3-kv8", 9001, 1.0)])
def test_host_forward_matches_device_forward(name, T, ws_scale):
    # The host-buffer form (copies overlapped with compute on a second stream, output copied
    # back range by range) must give exactly what the device form gives.
    if name == "odd":
        cfg = MSAConfig("odd", "prefill", T, 4, 2, 8, 3, head_dim=32, idx_dim=16, seed=1)  # generic kernels
    else:
        cfg = CONFIGS[name[:2]].scaled(name=name + "-host", T=T, kv_fp8=name.endswith("kv8"))  # kv8: K, V uploaded as fp8
    shape = B.shape_of(cfg)
    x = make_prefill_inputs(cfg, DEV, sharp=True)
    out, lse, I = api.prefill_forward(cfg, x)
    host = {n: t.cpu().pin_memory() for n, t in x.items()}
    out_h = torch.empty(out.shape, dtype=torch.bfloat16).pin_memory()
    lse_h = torch.empty(lse.shape, dtype=torch.float32).pin_memory()
    I_h = torch.empty(I.shape, dtype=torch.int32).pin_memory()
    mn, pf = B.msa_prefill_forward_host_workspace_bytes(shape, T)
    ws = B.alloc_workspace(int(mn + ws_scale * (pf - mn)), DEV)
    for _ in range(2):  # twice: the second call reuses the staging area while nothing else runs
        out_h.zero_(); lse_h.zero_(); I_h.zero_()
        B.msa_prefill_forward_host(shape, host["q"], host["k"], host["v"], host["q_idx"], host["k_idx"], T,
                                   out_h, lse_h, I_h, ws)
        assert torch.equal(I_h, I.cpu())
        assert torch.equal(out_h, out.cpu())
        assert torch.equal(lse_h, lse.cpu())
    _assert_clean()


def test_sink_block_selected_by_every_query():
    # Real workloads have an attention sink: one early block that nearly every query selects
    # (Section 4.2, "pre-scheduled tile chunking").  Block 0's tile then holds every query of a
    # range, thousands of times the average: the item list must spread it over all CTAs and the
    # results must not change.
    cfg = CONFIGS["c3"].scaled(name="c3-sink", T=16384 + 300)
    x = make_prefill_inputs(cfg, DEV, sharp=True)
    u = torch.zeros(cfg.idx_dim, device=DEV)
    u[0] = 1.0
    x["k_idx"][: cfg.block_size] = (x["k_idx"][: cfg.block_size].float() + 40.0 * u).to(torch.bfloat16)
    x["q_idx"] = (x["q_idx"].float() + 6.0 * u).to(torch.bfloat16)
    T = cfg.T
    pos = sample_positions(T, cfg.block_size, cfg.top_k, 200, 3)
    pos_t = torch.from_numpy(pos).to(DEV)
    out, lse, I = api.prefill_forward(cfg, x)
    torch.cuda.synchronize()
    _assert_clean()
    assert bool((I[cfg.block_size:, :, 0] == 0).all()), "block 0 must be in every list"
    kb, vb, kib = to_bits(x["k"]), to_bits(x["v"]), to_bits(x["k_idx"])
    M_ref = oracle.index_scores(to_bits(x["q_idx"][pos_t]), kib, pos, cfg.block_size)
    I_ref = oracle.topk_select(M_ref, pos, T, cfg.block_size, cfg.top_k)
    I_gpu = I[pos_t].cpu().numpy()
    exact, _ = check_selection(I_gpu, I_ref, M_ref, pos, cfg.block_size, cfg.top_k, eps=1e-4)
    assert exact >= 0.995
    O_ref, LSE_ref = oracle.sparse_attn(to_bits(x["q"][pos_t]), kb, vb, I_gpu, pos, cfg.block_size)
    check_attn(out[pos_t].float().cpu().numpy(), lse[pos_t].cpu().numpy(), O_ref, LSE_ref, "sink")


# The paper's own model regime (Section 5.3): 64 query heads / 4 KV heads (G = 16), d_h = 128,
# B_k = 128, k = 16; d_idx = 128 is the value that reproduces its printed FLOPs ratio.
PAPER_SHAPE = MSAConfig("paper-shape", "prefill", 20000 + 77, 64, 4, 128, 16, head_dim=128, idx_dim=128, seed=6)


@pytest.mark.parametrize("sharp", [False, True])
def test_paper_shape_prefill(sharp):
    stats = run_prefill_case(PAPER_SHAPE, sharp, n_sample=256)
    assert stats["exact_sets"] >= 0.999
    print("paper-shape", sharp, stats)


def test_paper_shape_small_chunks_and_b64():
    # d_idx = 128 with B_k = 64 and a workspace that forces several score chunks and query ranges
    cfg = PAPER_SHAPE.scaled(name="paper-b64", T=9000, block_size=64, top_k=24)
    shape = B.shape_of(cfg)
    mn, pf = B.msa_prefill_forward_workspace_bytes(shape, cfg.T)
    stats = run_prefill_case(cfg, True, n_sample=200, ws_bytes=mn)
    assert stats["exact_sets"] >= 0.999


@pytest.mark.parametrize("sharp", [False, True])
def test_paper_shape_decode(sharp):
    cfg = PAPER_SHAPE.scaled(name="paper-decode", mode="decode", T=0,
                             seq_lens=(1, 130, 4096, 5000, 30000, 16384 + 64))
    res = run_decode_case(cfg, sharp)
    assert np.mean([r["exact"] for r in res]) >= 0.95


def test_decode_g16_b64():
    cfg = MSAConfig("dec-g16", "decode", 0, 32, 2, 64, 12, head_dim=128, idx_dim=64, seed=8,
                    seq_lens=(70, 640, 641, 7000))
    run_decode_case(cfg, True)


# ----------------------------------------------------------------- fp8 E4M3 index operands (Section 4.2)
@pytest.mark.parametrize("name,T,Hq,Hkv,Bk,k,di,sharp", [
    ("paper regime, fused selection", 6144 + 77, 64, 4, 128, 16, 128, True),
    ("paper regime, diffuse", 5000, 64, 4, 128, 16, 128, False),
    ("8 index heads, k 64", 7000, 64, 8, 128, 64, 128, True),
    ("B_k 64", 4096 + 9, 16, 2, 64, 24, 128, True),
    ("short range, generic kernel", 20, 16, 2, 64, 4, 128, True),
    ("generic shape", 700, 6, 3, 16, 5, 32, True),
])
def test_fp8_index_prefill(name, T, Hq, Hkv, Bk, k, di, sharp):
    cfg = MSAConfig("f8", "prefill", T, Hq, Hkv, Bk, k, head_dim=128 if Hq > 6 else 64, idx_dim=di, seed=T,
                    idx_fp8=True)
    stats = run_prefill_case(cfg, sharp, n_sample=200)
    assert stats["exact_sets"] >= 0.999, (name, stats)
    print("fp8", name, stats)


def test_fp8_fused_equals_separate_calls_and_small_workspace():
    cfg = MSAConfig("f8-fused", "prefill", 9000, 64, 4, 128, 16, head_dim=128, idx_dim=128, seed=12, idx_fp8=True)
    x = make_prefill_inputs(cfg, DEV, sharp=True)
    shape = B.shape_of(cfg)
    T = cfg.T
    I_f = torch.full((T, 4, 16), -7, dtype=torch.int32, device=DEV)
    B.msa_index_topk_fused(shape, x["q_idx"], x["k_idx"], 0, T, T, I_f)
    M = api.index_scores(cfg, x["q_idx"], x["k_idx"], 0, T)
    I_s = api.topk_select(cfg, M, 0, T)
    mn, pf = B.msa_prefill_forward_workspace_bytes(shape, T)
    o1, l1, i1 = api.prefill_forward(cfg, x, workspace_bytes=pf)
    o2, l2, i2 = api.prefill_forward(cfg, x, workspace_bytes=mn)  # several ranges: q_idx offsets in bytes
    torch.cuda.synchronize()
    _assert_clean()
    assert torch.equal(I_f, I_s) and torch.equal(i1, I_s) and torch.equal(i2, I_s)
    assert torch.equal(o1, o2) and torch.equal(l1, l2)


def test_fp8_varlen_equals_sequence_by_sequence():
    cfg = MSAConfig("f8-varlen", "prefill", 0, 64, 4, 128, 16, head_dim=128, idx_dim=128, seed=4, idx_fp8=True)
    lens = [1000, 37, 0, 4096 + 5, 2500]
    cu = np.concatenate([[0], np.cumsum(lens)]).tolist()
    x = make_prefill_inputs(cfg.scaled(T=cu[-1]), DEV, sharp=True)
    out, lse, I = api.prefill_forward_varlen(cfg.scaled(T=cu[-1]), x, cu)
    torch.cuda.synchronize()
    _assert_clean()
    for s, L in enumerate(lens):
        if L == 0:
            continue
        a, b = cu[s], cu[s + 1]
        xs = {n: t[a:b].contiguous() for n, t in x.items()}
        o1, l1, i1 = api.prefill_forward(cfg.scaled(T=L), xs)
        torch.cuda.synchronize()
        assert torch.equal(I[a:b], i1) and torch.equal(out[a:b], o1) and torch.equal(lse[a:b], l1), s


@pytest.mark.parametrize("Hkv,di,lens", [
    (4, 128, (1, 130, 4096, 5000, 30000, 16384 + 64)),   # streaming tensor-core kernel
    (3, 32, (5, 16, 17, 400, 1000)),                     # generic kernel
])
def test_fp8_index_decode(Hkv, di, lens):
    big = di == 128
    cfg = MSAConfig("f8-dec", "decode", 0, 64 if big else 6, Hkv, 128 if big else 16, 16 if big else 5,
                    head_dim=128 if big else 64, idx_dim=di, seed=21, seq_lens=lens, idx_fp8=True)
    res = run_decode_case(cfg, True)
    assert np.mean([r["exact"] for r in res]) >= 0.95


def test_fp8_index_lse_matches_oracle():
    cfg = MSAConfig("f8-lse", "prefill", 3000, 64, 4, 128, 16, head_dim=128, idx_dim=128, seed=6, idx_fp8=True)
    x = make_prefill_inputs(cfg, DEV, sharp=True)
    _, _, I = api.prefill_forward(cfg, x)
    got = api.index_lse(cfg, x["q_idx"], x["k_idx"], I)
    torch.cuda.synchronize()
    _assert_clean()
    pos = sample_positions(cfg.T, 128, 16, 160, 5)
    pos_t = torch.from_numpy(pos).to(DEV)
    want = oracle.index_lse(to_bits(x["q_idx"])[pos], to_bits(x["k_idx"]), I[pos_t].cpu().numpy(), pos, 128)
    err = np.abs(got[pos_t].cpu().numpy().astype(np.float64) - want)
    assert np.isfinite(want).all() and err.max() <= 2e-3, float(err.max())


def test_fp8_flag_and_operand_size_must_agree():
    cfg = MSAConfig("f8-bad", "prefill", 256, 16, 2, 64, 4, head_dim=128, idx_dim=128, seed=1)
    x = make_prefill_inputs(cfg, DEV)  # bf16 index operands
    shape = B.shape_of(cfg.scaled(idx_fp8=True))
    with pytest.raises(AssertionError):
        B.msa_index_scores(shape, x["q_idx"], x["k_idx"], 0, 256, 256,
                           torch.empty((256, 2, 4), device=DEV), 4)
    shape.idx_fp8 = 2
    with pytest.raises(B.MsaError):
        B.msa_prefill_forward_workspace_bytes(shape, 256)


# ----------------------------------------------------------------- two-level Top-k on long rows
@pytest.mark.parametrize("T,Hq,Hkv,k,di,ties,sharp", [
    (100000 + 77, 16, 2, 20, 64, False, True),
    (100000 + 77, 16, 2, 20, 64, True, True),     # many exactly equal scores (and equal run maxima)
    (140000, 32, 4, 24, 128, True, False),
    (300000 + 5, 64, 8, 64, 64, False, False),    # the headline shape's head layout and k
])
def test_two_level_topk_long_rows_bit_exact(T, Hq, Hkv, k, di, ties, sharp):
    # Rows of 2 (k-1) runs of 8 blocks and more are selected in two levels (run maxima first, then
    # only the runs that can hold a selected block).  The lists must be the oracle's on the very
    # scores the GPU computed (fp32, exact in fp64), ties included, and the whole-path call must
    # give the same lists as the separate calls.
    cfg = MSAConfig("top2", "prefill", T, Hq, Hkv, 128, k, head_dim=128, idx_dim=di, seed=T + k)
    x = make_prefill_inputs(cfg, DEV, sharp=sharp)
    if ties:  # keys repeat with period 7 blocks: block maxima of different blocks coincide exactly
        period = 7 * 128
        x["k_idx"] = x["k_idx"][:period].repeat((T + period - 1) // period, 1)[:T].contiguous()
    _, _, I = api.prefill_forward(cfg, x)
    torch.cuda.synchronize()
    _assert_clean()
    first_long = 2 * (k - 1) * 8 * 128  # rows from here on take the two-level path
    assert T > first_long + 4096
    nb = cfg.n_blocks
    for q0, qc in [(first_long - 150, 300), ((first_long + T) // 2 + 11, 400), (T - 384, 384)]:
        M = api.index_scores(cfg, x["q_idx"], x["k_idx"], q0, qc)
        I_s = api.topk_select(cfg, M, q0, T)
        torch.cuda.synchronize()
        assert torch.equal(I[q0:q0 + qc], I_s), (q0, int((I[q0:q0 + qc] != I_s).any(dim=2).sum()))
        I_ref = oracle.topk_select(M[:, :, :nb].double().cpu().numpy(), np.arange(q0, q0 + qc), T, 128, k)
        assert np.array_equal(I_s.cpu().numpy(), I_ref), q0


@pytest.mark.parametrize("n_blocks,k,levels", [(3000, 20, 0), (8192, 64, 0), (8192, 64, 5), (5000, 33, 3),
                                               (9000, 17, 0), (8192, 64, -64), (4100, 32, -24), (6000, 128, -16)])
def test_two_level_topk_on_arbitrary_long_score_rows(n_blocks, k, levels):
    # Top-k alone on synthetic score rows: continuous values, values from a handful of levels
    # (whole runs tie, the threshold is shared by hundreds of blocks) and normal values rounded to
    # multiples of 1/|levels| (a few blocks tie with the threshold: the short list of blocks above the
    # run-maxima threshold still decides them by block order); rows at many positions, including
    # ones beyond the candidate list's capacity (n_blocks 9000), which take one level.
    Bk = 16
    T = n_blocks * Bk
    cfg = MSAConfig("top2-raw", "prefill", T, 4, 2, Bk, k, head_dim=64, idx_dim=32, seed=n_blocks)
    g = torch.Generator().manual_seed(n_blocks + k)
    ld = B.score_ld(T, Bk)
    pos = np.unique(np.concatenate([np.arange(T - 40, T), np.linspace(2 * (k - 1) * 8 * Bk - 20, T - 1, 150).astype(np.int64)]))
    runs = np.split(pos, np.where(np.diff(pos) != 1)[0] + 1)
    for run in runs:
        q0, qc = int(run[0]), len(run)
        M = torch.randn((qc, 2, ld), generator=g)
        if levels > 0:
            M = torch.randint(0, levels, (qc, 2, ld), generator=g).float() * 0.5 - 1.0
        elif levels < 0:
            M = torch.round(M * float(-levels)) / float(-levels)
        I = api.topk_select(cfg, M.to(DEV), q0, T).cpu().numpy()
        I_ref = oracle.topk_select(M[:, :, :n_blocks].double().numpy(), np.arange(q0, q0 + qc), T, Bk, k)
        assert np.array_equal(I, I_ref), (q0, qc)


@pytest.mark.parametrize("Bk,n_blocks,k,levels", [(128, 700, 64, 0), (128, 700, 64, 6), (64, 1100, 32, 4),
                                                 (128, 2600, 64, -48), (64, 300, 64, 3), (128, 4200, 16, -16)])
def test_topk_reads_run_ordered_rows_like_block_ordered_ones(Bk, n_blocks, k, levels):
    # Stage 2 alone on synthetic score rows handed over in run order (msa_shape_t.score_runs = 1):
    # the lists must be those of the same rows in block order and the oracle's, with continuous
    # values, with a handful of levels (whole runs tie) and with values rounded to multiples of
    # 1/|levels| (a few ties at the threshold); rows of every length class (one level, two levels with
    # quarters, halves and whole runs as threshold groups).
    T = n_blocks * Bk
    cfg = MSAConfig("top-runs", "prefill", T, 4, 2, Bk, k, head_dim=64, idx_dim=64, seed=n_blocks)
    g = torch.Generator().manual_seed(n_blocks + k)
    ld = (n_blocks + 7) // 8 * 8
    cols = api.run_order_columns(n_blocks, Bk)
    pos = np.unique(np.concatenate([np.arange(T - 24, T), np.linspace(Bk * (k - 1), T - 1, 120).astype(np.int64)]))
    for run in np.split(pos, np.where(np.diff(pos) != 1)[0] + 1):
        q0, qc = int(run[0]), len(run)
        M = torch.randn((qc, 2, ld), generator=g)
        if levels > 0:
            M = torch.randint(0, levels, (qc, 2, ld), generator=g).float() * 0.5 - 1.0
        elif levels < 0:
            M = torch.round(M * float(-levels)) / float(-levels)
        M_runs = torch.full_like(M, float("nan"))   # columns of blocks that do not exist stay NaN
        M_runs[:, :, cols] = M[:, :, :n_blocks]
        I_blk = api.topk_select(cfg, M.to(DEV), q0, T).cpu().numpy()
        I_run = api.topk_select(cfg, M_runs.to(DEV), q0, T, score_runs=1).cpu().numpy()
        I_ref = oracle.topk_select(M[:, :, :n_blocks].double().numpy(), np.arange(q0, q0 + qc), T, Bk, k)
        assert np.array_equal(I_blk, I_ref), (q0, qc)
        assert np.array_equal(I_run, I_ref), (q0, qc)


# ----------------------------------------------------------------- CUDA graphs
def test_decode_and_prefill_calls_replay_from_a_cuda_graph():
    # A decode step is a handful of short kernels: serving loops capture it once and replay it.
    # The calls must be capturable (no allocation, no synchronisation, no host read inside) and a
    # replay on new inputs in the same buffers must give what a plain call gives.
    cfg = CONFIGS["c5"].scaled(name="c5-graph", seq_lens=(129, 4096, 20000, 16384 + 64))
    x = make_decode_inputs(cfg, DEV, sharp=True)
    shape = B.shape_of(cfg)
    batch, max_len = len(cfg.seq_lens), int(max(cfg.seq_lens))
    ld = B.score_ld(max_len, cfg.block_size)
    scores = torch.empty((batch, cfg.n_kv_heads, ld), dtype=torch.float32, device=DEV)
    I = torch.empty((batch, cfg.n_kv_heads, cfg.top_k), dtype=torch.int32, device=DEV)
    out = torch.empty_like(x["q"])
    lse = torch.empty((batch, cfg.n_q_heads), dtype=torch.float32, device=DEV)
    ws = B.alloc_workspace(B.msa_sparse_attn_decode_workspace_bytes(shape, batch), DEV)

    def step():
        B.msa_decode_forward(shape, x["q"], x["q_idx"], x["k_cache"], x["v_cache"], x["k_idx_cache"],
                             x["k_cache"].shape[0], x["seq_offsets"], x["seq_lens"], batch, max_len,
                             scores, ld, I, out, lse, ws)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):  # warm-up outside the capture (attributes are set on first use)
        step()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step()
    # new queries in the captured buffers
    x2 = make_decode_inputs(cfg.scaled(seed=cfg.seed + 1), DEV, sharp=True)
    x["q"].copy_(x2["q"])
    x["q_idx"].copy_(x2["q_idx"])
    g.replay()
    torch.cuda.synchronize()
    _assert_clean()
    got = (out.clone(), lse.clone(), I.clone())
    out.zero_(); lse.zero_(); I.zero_()
    step()
    torch.cuda.synchronize()
    assert torch.equal(got[2], I) and torch.equal(got[0], out) and torch.equal(got[1], lse)

    # the prefill call, same way
    pcfg = CONFIGS["c3"].scaled(name="c3-graph", T=3000)
    px = make_prefill_inputs(pcfg, DEV, sharp=True)
    pshape = B.shape_of(pcfg)
    po = torch.empty_like(px["q"])
    pl = torch.empty((pcfg.T, pcfg.n_q_heads), dtype=torch.float32, device=DEV)
    pi = torch.empty((pcfg.T, pcfg.n_kv_heads, pcfg.top_k), dtype=torch.int32, device=DEV)
    pws = B.alloc_workspace(B.msa_prefill_forward_workspace_bytes(pshape, pcfg.T)[1], DEV)

    def pstep():
        B.msa_prefill_forward(pshape, px["q"], px["k"], px["v"], px["q_idx"], px["k_idx"], pcfg.T, po, pl, pi, pws)
    with torch.cuda.stream(side):
        pstep()
    torch.cuda.synchronize()
    want = (po.clone(), pl.clone(), pi.clone())
    pg = torch.cuda.CUDAGraph()
    with torch.cuda.graph(pg):
        pstep()
    po.zero_(); pl.zero_(); pi.zero_()
    pg.replay()
    torch.cuda.synchronize()
    _assert_clean()
    assert torch.equal(want[2], pi) and torch.equal(want[0], po) and torch.equal(want[1], pl)


# ----------------------------------------------------------------- fp8 E4M3 K/V caches (decode, Section 4.2)
@pytest.mark.parametrize("Hq,Hkv,Bk,k,lens", [
    (64, 8, 128, 64, (1, 127, 128, 129, 8192, 8200, 20000, 16384 + 64)),   # G = 8
    (64, 4, 128, 16, (1, 130, 4096, 5000, 30000)),                          # G = 16, the paper's regime
    (32, 2, 64, 12, (70, 640, 641, 7000)),                                  # G = 16, B_k = 64
    (16, 2, 64, 40, (3000, 64, 65)),                                        # G = 8, B_k = 64, several splits
])
@pytest.mark.parametrize("sharp", [False, True])
def test_fp8_kv_cache_decode(Hq, Hkv, Bk, k, lens, sharp):
    # K and V are dequantised exactly in registers, so against the oracle on the same fp8 values the
    # result must hold the bf16 path's tolerances.
    cfg = MSAConfig("kv8", "decode", 0, Hq, Hkv, Bk, k, head_dim=128, idx_dim=64, seed=len(lens) + k, seq_lens=lens,
                    kv_fp8=True)
    res = run_decode_case(cfg, sharp)
    assert np.mean([r["exact"] for r in res]) >= 0.95


def test_fp8_kv_and_index_decode_together():
    cfg = MSAConfig("kv8-idx8", "decode", 0, 64, 4, 128, 16, head_dim=128, idx_dim=128, seed=3,
                    seq_lens=(129, 4096, 40000), kv_fp8=True, idx_fp8=True)
    run_decode_case(cfg, True)


@pytest.mark.parametrize("Hq,Hkv,Bk,k,T,d", [
    (64, 8, 128, 16, 6144 + 77, 128),   # tensor-core attention path, ragged last block
    (64, 4, 128, 16, 4096 + 1, 128),    # the paper's regime (G = 16)
    (16, 2, 64, 6, 1500, 128),          # B_k = 64
    (6, 3, 16, 5, 333, 64),             # generic kernels
])
@pytest.mark.parametrize("sharp", [False, True])
def test_fp8_kv_cache_prefill(Hq, Hkv, Bk, k, T, d, sharp):
    # Prefill onto fp8 K/V caches: the kernels run on exact bf16 copies of the fp8 values, so the
    # result must (a) hold the bf16 path's tolerances against the oracle on the fp8 values and
    # (b) equal, bit for bit, the bf16 call on the same values widened by torch.
    cfg = MSAConfig("kv8-prefill", "prefill", T, Hq, Hkv, Bk, k, head_dim=d, idx_dim=64, seed=T % 97, kv_fp8=True)
    stats = run_prefill_case(cfg, sharp, n_sample=256)
    assert stats["exact_sets"] >= 0.999
    x = make_prefill_inputs(cfg, DEV, sharp=sharp)
    o8, l8, i8 = api.prefill_forward(cfg, x)
    wide = dict(x, k=x["k"].to(torch.bfloat16), v=x["v"].to(torch.bfloat16))
    o16, l16, i16 = api.prefill_forward(cfg.scaled(kv_fp8=False), wide)
    torch.cuda.synchronize()
    _assert_clean()
    assert torch.equal(i8, i16) and torch.equal(o8, o16) and torch.equal(l8, l16)


def test_fp8_kv_cache_prefill_query_range_and_small_workspace():
    # A chunk of new queries [q_begin, q_begin + q_count) against a longer fp8 cache, with the
    # smallest workspace the library accepts: same numbers as the preferred size, and as the oracle.
    cfg = MSAConfig("kv8-chunk", "prefill", 5000, 64, 8, 128, 8, head_dim=128, idx_dim=64, seed=11, kv_fp8=True)
    x = make_prefill_inputs(cfg, DEV, sharp=True)
    _, _, I = api.prefill_forward(cfg, x)
    q0, qc, L = 3000, 1203, 4500  # the cache holds more rows than the call may see
    o1, l1 = api.sparse_attn_prefill(cfg, x["q"][q0:q0 + qc], x["k"][:L], x["v"][:L], I[q0:q0 + qc].contiguous(), q0)
    o2, l2 = api.sparse_attn_prefill(cfg, x["q"][q0:q0 + qc], x["k"][:L], x["v"][:L], I[q0:q0 + qc].contiguous(), q0,
                                     workspace_bytes=1)
    torch.cuda.synchronize()
    _assert_clean()
    assert torch.equal(o1, o2) and torch.equal(l1, l2)
    pos = np.arange(q0, q0 + qc)[::7]
    O_ref, LSE_ref = oracle.sparse_attn(to_bits(x["q"][q0:q0 + qc][::7]), to_bits(x["k"][:L]), to_bits(x["v"][:L]),
                                        I[q0:q0 + qc][::7].cpu().numpy(), pos, cfg.block_size)
    check_attn(o1[::7].float().cpu().numpy(), l1[::7].cpu().numpy(), O_ref, LSE_ref, "kv8-chunk")


def test_fp8_kv_cache_prefill_varlen_equals_sequence_by_sequence():
    cfg = MSAConfig("kv8-varlen", "prefill", 0, 64, 8, 128, 8, head_dim=128, idx_dim=64, seed=5, kv_fp8=True)
    lens = [700, 0, 2048 + 3, 129]
    cu = np.concatenate([[0], np.cumsum(lens)]).tolist()
    x = make_prefill_inputs(cfg.scaled(T=cu[-1]), DEV, sharp=True)
    out, lse, I = api.prefill_forward_varlen(cfg, x, cu)
    for a, b in zip(cu[:-1], cu[1:]):
        if b == a:
            continue
        o1, l1, i1 = api.prefill_forward(cfg.scaled(T=b - a), {n: t[a:b] for n, t in x.items()})
        assert torch.equal(out[a:b], o1) and torch.equal(lse[a:b], l1) and torch.equal(I[a:b], i1)
    torch.cuda.synchronize()
    _assert_clean()


def test_fp8_kv_cache_is_rejected_where_it_is_not_supported():
    cfg = MSAConfig("kv8-bad", "prefill", 512, 64, 8, 128, 4, head_dim=128, idx_dim=64, seed=1, kv_fp8=True)
    x = make_prefill_inputs(cfg, DEV)
    with pytest.raises(AssertionError):  # bf16 K/V with the flag set
        api.prefill_forward(cfg, make_prefill_inputs(cfg.scaled(kv_fp8=False), DEV))
    I = torch.zeros((cfg.T, cfg.n_kv_heads, cfg.top_k), dtype=torch.int32, device=DEV)
    out, lse = torch.empty_like(x["q"]), torch.empty((cfg.T, cfg.n_q_heads), dtype=torch.float32, device=DEV)
    with pytest.raises(B.MsaError) as e:  # the allocation-free variant takes bf16 K/V only
        B.msa_sparse_attn_prefill_static(B.shape_of(cfg), x["q"], x["k"], x["v"], I, 0, cfg.T, cfg.T, out, lse)
    assert e.value.code == 2  # MSA_ERR_UNSUPPORTED
    dcfg = MSAConfig("kv8-odd", "decode", 0, 6, 3, 16, 5, head_dim=64, idx_dim=32, seed=3, seq_lens=(5, 400), kv_fp8=True)
    xd = make_decode_inputs(dcfg, DEV)
    with pytest.raises(B.MsaError) as e:
        api.decode_forward(dcfg, xd)
    assert e.value.code == 2
    with pytest.raises(AssertionError):  # bf16 caches with the flag set
        api.decode_forward(dcfg, make_decode_inputs(dcfg.scaled(kv_fp8=False), DEV))


def test_fp8_index_decode_d_idx_64():
    # fp8 index keys of 64 elements (C5's shapes): a 64-byte row is one segment of the streaming kernel.
    cfg = MSAConfig("f8-dec64", "decode", 0, 64, 8, 128, 64, head_dim=128, idx_dim=64, seed=21,
                    seq_lens=(1, 130, 4096, 5000, 30000, 16384 + 64), idx_fp8=True, kv_fp8=True)
    res = run_decode_case(cfg, True)
    assert np.mean([r["exact"] for r in res]) >= 0.95


# ---- Q, K and V in fp8 E4M3, read as such by the prefill attention kernel (Section 4.2) ----
@pytest.mark.parametrize("name,T,Hq,Hkv,Bk,k,di,idx8", [
    ("c3 shape", 12288 + 5, 64, 8, 128, 64, 64, False),
    ("c3 shape, few picks", 6144 + 77, 64, 8, 128, 4, 64, False),
    ("paper regime, fp8 index too", 20000 + 77, 64, 4, 128, 16, 128, True),
    ("B_k 64, G 8", 4096 + 37, 16, 2, 64, 8, 64, False),
    ("B_k 64, G 16", 3000, 32, 2, 64, 6, 64, False),
])
@pytest.mark.parametrize("sharp", [False, True])
def test_fp8_qkv_prefill_matches_oracle(name, T, Hq, Hkv, Bk, k, di, idx8, sharp):
    # The oracle is Eq. 8 on the decoded fp8 operands, in double; the kernel's products are exact and
    # everything after S is the bf16 path, so the bf16 path's tolerances apply unchanged.
    cfg = MSAConfig("f8qkv", "prefill", T, Hq, Hkv, Bk, k, head_dim=128, idx_dim=di, seed=T, idx_fp8=idx8,
                    kv_fp8=True, q_fp8=True)
    stats = run_prefill_case(cfg, sharp, n_sample=192)
    assert stats["exact_sets"] >= 0.995
    print(name, sharp, stats)


def test_fp8_qkv_prefill_small_workspace_and_ranges_equal_the_whole_call():
    cfg = CONFIGS["c3"].scaled(name="c3-f8qkv-6k", T=6144 + 77, kv_fp8=True, q_fp8=True)
    shape = B.shape_of(cfg)
    x = make_prefill_inputs(cfg, DEV, sharp=True)
    mn, pf = B.msa_prefill_forward_workspace_bytes(shape, cfg.T)
    # no bf16 copies of K and V: the workspace is that of the bf16 call
    assert (mn, pf) == B.msa_prefill_forward_workspace_bytes(B.shape_of(cfg.scaled(kv_fp8=False, q_fp8=False)), cfg.T)
    o1, l1, i1 = api.prefill_forward(cfg, x, workspace_bytes=pf)
    o2, l2, i2 = api.prefill_forward(cfg, x, workspace_bytes=mn)
    q0 = cfg.T // 2 + 3
    o3, l3 = api.sparse_attn_prefill(cfg, x["q"][q0:], x["k"], x["v"], i1[q0:], q_begin=q0)
    torch.cuda.synchronize()
    _assert_clean()
    assert o1.dtype == torch.bfloat16
    assert torch.equal(i1, i2) and torch.equal(o1, o2) and torch.equal(l1, l2)
    assert torch.equal(o3, o1[q0:]) and torch.equal(l3, l1[q0:])
    # the same values through the widening path (fp8 K/V caches, bf16 Q): S is summed in another order
    # there, nothing else differs
    cfg_w = cfg.scaled(q_fp8=False)
    xw = dict(x)
    xw["q"] = x["q"].to(torch.bfloat16)
    ow, lw, iw = api.prefill_forward(cfg_w, xw)
    assert torch.equal(iw, i1)
    assert (ow.float() - o1.float()).abs().max().item() <= 4e-3 and (lw - l1).abs().max().item() <= 1e-4


def test_fp8_qkv_varlen_and_host_calls():
    cfg = CONFIGS["c3"].scaled(name="c3-f8qkv-var", T=0, top_k=8, kv_fp8=True, q_fp8=True)
    lens = [1000, 37, 0, 4096 + 5, 129]
    cu = np.concatenate([[0], np.cumsum(lens)]).tolist()
    total = cu[-1]
    x = make_prefill_inputs(cfg.scaled(T=total), DEV, sharp=True)
    out, lse, I = api.prefill_forward_varlen(cfg.scaled(T=total), x, cu)
    torch.cuda.synchronize()
    _assert_clean()
    for s, L in enumerate(lens):
        if L == 0:
            continue
        a, b = cu[s], cu[s + 1]
        xs = {n: t[a:b].contiguous() for n, t in x.items()}
        o1, l1, i1 = api.prefill_forward(cfg.scaled(T=L), xs)
        assert torch.equal(I[a:b], i1) and torch.equal(out[a:b], o1) and torch.equal(lse[a:b], l1), "sequence %d" % s
    # host buffers: Q, K, V go up as fp8 bytes
    T = 5000
    cfg = CONFIGS["c3"].scaled(name="c3-f8qkv-host", T=T, kv_fp8=True, q_fp8=True)
    shape = B.shape_of(cfg)
    x = make_prefill_inputs(cfg, DEV, sharp=True)
    out, lse, I = api.prefill_forward(cfg, x)
    host = {n: t.cpu().pin_memory() for n, t in x.items()}
    out_h = torch.empty(out.shape, dtype=torch.bfloat16).pin_memory()
    lse_h = torch.empty(lse.shape, dtype=torch.float32).pin_memory()
    I_h = torch.empty(I.shape, dtype=torch.int32).pin_memory()
    mn, pf = B.msa_prefill_forward_host_workspace_bytes(shape, T)
    ws = B.alloc_workspace(pf, DEV)
    B.msa_prefill_forward_host(shape, host["q"], host["k"], host["v"], host["q_idx"], host["k_idx"], T, out_h, lse_h, I_h, ws)
    assert torch.equal(I_h, I.cpu()) and torch.equal(out_h, out.cpu()) and torch.equal(lse_h, lse.cpu())
    _assert_clean()


def test_fp8_q_is_rejected_where_it_is_not_supported():
    x = make_prefill_inputs(CONFIGS["c1"].scaled(T=300), DEV)
    q8 = x["q"].to(torch.float8_e4m3fn)
    k8, v8 = x["k"].to(torch.float8_e4m3fn), x["v"].to(torch.float8_e4m3fn)
    I = torch.zeros((300, 1, 8), dtype=torch.int32, device=DEV)
    out = torch.empty(x["q"].shape, dtype=torch.bfloat16, device=DEV)
    ws = B.alloc_workspace(1 << 26, DEV)
    # fp8 Q with bf16 K/V
    bad = B.shape_of(CONFIGS["c1"].scaled(q_fp8=True))
    with pytest.raises(B.MsaError) as e:
        B.msa_sparse_attn_prefill(bad, q8, x["k"], x["v"], I, 0, 300, 300, out, None, ws)
    assert e.value.code == 2
    # a shape outside the tensor-core kernel (d_h = 64)
    odd = MSAConfig("odd8", "prefill", 300, 8, 1, 64, 8, head_dim=64, idx_dim=64, kv_fp8=True, q_fp8=True)
    xo = make_prefill_inputs(odd, DEV)
    with pytest.raises(B.MsaError) as e:
        B.msa_sparse_attn_prefill(B.shape_of(odd), xo["q"], xo["k"], xo["v"], I, 0, 300, 300,
                                  torch.empty(xo["q"].shape, dtype=torch.bfloat16, device=DEV), None, ws)
    assert e.value.code == 2
    # decode calls
    dcfg = CONFIGS["c5"].scaled(seq_lens=(300,), kv_fp8=True, q_fp8=True, n_kv_heads=1, n_q_heads=8)
    sh = B.shape_of(dcfg)
    with pytest.raises(B.MsaError) as e:
        B.msa_sparse_attn_decode(sh, x["q"][:1].contiguous(), k8, v8, 300, torch.zeros(1, dtype=torch.int64, device=DEV),
                                 torch.tensor([300], dtype=torch.int32, device=DEV), 1, I[:1].contiguous(),
                                 out[:1].contiguous(), None, ws)
    assert e.value.code == 2


@pytest.mark.parametrize("base,lens,ws", [
    ("c3", [9000, 130, 2500, 1], "minimum"),
    ("c3", [9000, 130, 2500, 1], "preferred"),
    ("c2", [700, 5000, 0, 64, 3000, 8192 + 9, 31, 1500], "preferred"),
    ("c2", [700, 5000, 0, 64, 3000, 8192 + 9, 31, 1500], "minimum"),
])
def test_varlen_batch_with_larger_top_k_and_a_row_offset(base, lens, ws):
    # top_k above the fused kernel's limit: stages 1-2 run on groups of consecutive sequences (one
    # scoring launch and one Top-k launch per group: one group with the preferred workspace, several
    # - and the single-sequence path for a sequence that does not fit - with the minimum), stage 3
    # once over the batch; the batch starts at a row offset inside the tensors (cu_seqlens[0] > 0).
    cfg = CONFIGS[base].scaled(name=base + "-varlen-k", T=0)
    cu = (np.concatenate([[0], np.cumsum(lens)]) + 384).tolist()
    total = cu[-1] + 77   # rows before and after the batch that the call must leave alone
    x = make_prefill_inputs(cfg.scaled(T=total), DEV, sharp=True)
    shape = B.shape_of(cfg)
    out = torch.full((total, cfg.n_q_heads, 128), 7.0, dtype=torch.bfloat16, device=DEV)
    lse = torch.full((total, cfg.n_q_heads), 7.0, dtype=torch.float32, device=DEV)
    I = torch.full((total, cfg.n_kv_heads, cfg.top_k), -7, dtype=torch.int32, device=DEV)
    mn, pf = B.msa_prefill_forward_varlen_workspace_bytes(shape, cu)
    n0 = B.launch_count()
    B.msa_prefill_forward_varlen(shape, x["q"], x["k"], x["v"], x["q_idx"], x["k_idx"], cu, out, lse, I,
                                 B.alloc_workspace(mn if ws == "minimum" else pf, DEV))
    n_batch = B.launch_count() - n0
    if ws == "preferred":  # as many launches as ONE sequence of the batch's size takes, plus the one that builds the maps
        one = cfg.scaled(T=sum(lens))
        n0 = B.launch_count()
        api.prefill_forward(one, {n: t[:sum(lens)].contiguous() for n, t in x.items()})
        assert n_batch <= B.launch_count() - n0 + 1, (n_batch, B.launch_count() - n0)
    torch.cuda.synchronize()
    _assert_clean()
    assert bool((out[:384] == 7.0).all()) and bool((out[cu[-1]:] == 7.0).all()) and bool((I[:384] == -7).all())
    for s_, L in enumerate(lens):
        if L == 0:
            continue
        a, b = cu[s_], cu[s_ + 1]
        xs = {n: t[a:b].contiguous() for n, t in x.items()}
        o1, l1, i1 = api.prefill_forward(cfg.scaled(T=L), xs)
        assert torch.equal(I[a:b], i1) and torch.equal(out[a:b], o1) and torch.equal(lse[a:b], l1), "sequence %d" % s_
    # oracle on the longest sequence through the batch call's outputs
    s_ = int(np.argmax(lens))
    a, b, L = cu[s_], cu[s_ + 1], lens[s_]
    pos = sample_positions(L, cfg.block_size, cfg.top_k, 48, 5)
    pos_t = torch.from_numpy(pos).to(DEV)
    I_gpu = I[a:b][pos_t].cpu().numpy()
    O_ref, LSE_ref = oracle.sparse_attn(to_bits(x["q"][a:b][pos_t]), to_bits(x["k"][a:b]), to_bits(x["v"][a:b]), I_gpu,
                                        pos, cfg.block_size)
    check_attn(out[a:b][pos_t].float().cpu().numpy(), lse[a:b][pos_t].cpu().numpy(), O_ref, LSE_ref, "varlen k64")
