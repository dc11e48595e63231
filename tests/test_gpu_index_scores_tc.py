"""Eq. 6 on the tensor-core index kernel, element by element against the oracle, in the forms the
kernel takes at full size: ranges long enough that eight (or four, two, one) index heads share a
CTA, deep key prefixes (the key-tile ring wraps many times), a range that starts inside the
sequence, the tile that crosses the diagonal at a large position, both block sizes, both index
widths and fp8 operands, in block order and in run order (the order msa_prefill_forward uses in its
workspace; msa_topk_select must pick the same lists from either).  Every case asserts, through msa_index_scores_plan, that the call it
compares ran on the tensor-core kernel with the expected number of heads per CTA, so that the
comparison cannot silently fall on the generic kernel."""

import numpy as np
import pytest
import torch

import oracle
from paper_2606_13392_b200 import api
from paper_2606_13392_b200 import binding as B
from paper_2606_13392_b200.inputs import CONFIGS, MSAConfig, make_prefill_inputs, to_bits
from parity_utils import check_scores

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _runs(q0: int, qc: int, T: int, n_rows: int, seed: int):
    """Runs of consecutive rows of the range [q0, q0+qc): its first rows, its last rows (the end of
    the sequence when q0+qc = T), a run across a 256-key tile edge in mid-range, and a run across a
    128-query tile edge at a random place."""
    rng = np.random.default_rng(seed)
    mid = (q0 + qc // 2) // 256 * 256
    odd = q0 + int(rng.integers(1, max(2, qc // 128 - 1))) * 128
    starts = [q0, q0 + qc - n_rows, mid - n_rows // 2, odd - n_rows // 2]
    runs = []
    for s in starts:
        s = int(min(max(s, q0), q0 + qc - n_rows))
        runs.append(np.arange(s, s + n_rows, dtype=np.int64))
    return runs


def _index_only_inputs(cfg: MSAConfig, sharp: bool):
    """Q_idx and K_idx of the recipe without drawing Q, K, V at their full size."""
    x = make_prefill_inputs(cfg.scaled(n_q_heads=cfg.n_kv_heads, head_dim=8), DEV, sharp=sharp)
    return x["q_idx"], x["k_idx"]


def check_range(cfg: MSAConfig, q_idx, k_idx, q0: int, qc: int, want_nh: int, n_rows: int = 128, seed: int = 0,
                score_runs: int = 0):
    shape = B.shape_of(cfg, score_runs=score_runs)
    tc, nh = B.msa_index_scores_plan(shape, qc, cfg.T)
    assert tc and nh == want_nh, "expected the tensor-core kernel with %d heads per CTA, got tc=%s nh=%d" % (
        want_nh, tc, nh)
    n0 = B.launch_count()
    M = api.index_scores(cfg, q_idx, k_idx, q0, qc, score_runs=score_runs)   # NaN-filled before the call
    torch.cuda.synchronize()
    assert B.launch_count() == n0 + 1
    code, detail = B.check_async_status()
    assert code == 0, (code, detail)
    nb = cfg.n_blocks
    # columns the call must not touch keep their fill
    nb_written = (nb + 7) // 8 * 8 if score_runs else nb
    assert torch.isnan(M[:, :, nb_written:]).all()
    if not score_runs:
        assert not torch.isnan(M[:, :, :nb]).any()
    cols = api.run_order_columns(nb, cfg.block_size).to(DEV) if score_runs else torch.arange(nb, device=DEV)
    kib = to_bits(k_idx)
    worst = 0.0
    for pos in _runs(q0, qc, cfg.T, n_rows, seed):
        pos_t = torch.from_numpy(pos).to(DEV)
        M_ref = oracle.index_scores(to_bits(q_idx[pos_t]), kib, pos, cfg.block_size)
        M_gpu = M[pos_t - q0][:, :, cols].cpu().numpy()
        if score_runs:  # columns of blocks after the local block are unspecified in run order
            hidden = np.arange(nb)[None, :] > (pos // cfg.block_size)[:, None]
            M_gpu[np.broadcast_to(hidden[:, None, :], M_gpu.shape)] = -np.inf
        worst = max(worst, check_scores(M_gpu, M_ref, pos, cfg.block_size))
    if score_runs:
        # Stage 2 on the run-ordered rows picks, bit for bit, the lists it picks from block-ordered ones.
        M0 = api.index_scores(cfg, q_idx, k_idx, q0, qc)
        I1 = api.topk_select(cfg, M, q0, cfg.T, score_runs=1)
        I0 = api.topk_select(cfg, M0, q0, cfg.T)
        torch.cuda.synchronize()
        assert torch.equal(I0, I1)
    return worst


@pytest.mark.parametrize("name,T,Hkv,Bk,di,fp8,q0,qc,nh", [
    # eight heads per CTA needs 2 * 148 CTAs: at least 296 query tiles
    ("NH8 whole sequence", 40960 + 77, 8, 128, 64, False, 0, 40960 + 77, 8),
    ("NH8 deep range, B_k 64", 50000, 8, 64, 64, False, 50000 - 38016, 38016, 8),
    ("NH4", 30000 + 5, 8, 128, 64, False, 30005 - 19000, 19000, 4),
    ("NH4, four heads in all", 40000, 4, 128, 64, False, 40000 - 37900, 37900, 4),
    ("NH2", 24000, 8, 128, 64, False, 24000 - 9600, 9600, 2),
    ("NH1", 9000 + 3, 8, 64, 64, False, 1000, 8003, 1),
    ("d_idx 128, NH2", 40000 + 9, 4, 128, 128, False, 40009 - 19008, 19008, 2),
    ("d_idx 128, NH1, B_k 64", 12000, 4, 64, 128, False, 3000, 9000, 1),
    ("fp8 operands, NH4", 40000, 4, 128, 128, True, 40000 - 37900, 37900, 4),
    ("fp8 operands, NH8", 41000, 8, 64, 128, True, 41000 - 37900, 37900, 8),
])
@pytest.mark.parametrize("sharp", [False, True])
@pytest.mark.parametrize("score_runs", [0, 1])
def test_tensor_core_scores_match_oracle(name, T, Hkv, Bk, di, fp8, q0, qc, nh, sharp, score_runs):
    top_k = 8 if not score_runs else (64 if Hkv == 8 else 24)  # run order: stage 2 on the rows as well
    cfg = MSAConfig("idx-tc", "prefill", T, Hkv, Hkv, Bk, top_k, head_dim=8, idx_dim=di, seed=T + Hkv, idx_fp8=fp8)
    q_idx, k_idx = _index_only_inputs(cfg, sharp)
    worst = check_range(cfg, q_idx, k_idx, q0, qc, nh, n_rows=96, seed=T, score_runs=score_runs)
    print(name, sharp, score_runs, "max score error %.3g" % worst)


@pytest.mark.parametrize("score_runs", [0, 1])
@pytest.mark.parametrize("name,rows", [("c3", 128), ("c4", 64)])
def test_full_size_chunk_scores_match_oracle(name, rows, score_runs):
    # The last query chunk of the full-size configurations as msa_prefill_forward scores it: 32 768
    # rows (40 960 at c3, where the chunk is the whole tail) against the whole key prefix, eight heads
    # per CTA; thousands of key tiles per CTA at c4.
    cfg = CONFIGS[name]
    q_idx, k_idx = _index_only_inputs(cfg, False)
    qc = 40960
    worst = check_range(cfg, q_idx, k_idx, cfg.T - qc, qc, 8, n_rows=rows, seed=1, score_runs=score_runs)
    print(name, score_runs, "max score error %.3g" % worst)
    del q_idx, k_idx
    torch.cuda.empty_cache()
