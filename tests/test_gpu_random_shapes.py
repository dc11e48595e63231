"""GPU parity on randomly drawn shapes (fixed seeds): head counts, group sizes, block sizes, k,
sequence lengths, fp8 flags and workspace sizes that the hand-picked cases do not list.  Shapes
the library declares unsupported (MSA_ERR_UNSUPPORTED) are skipped, anything else must pass."""

import numpy as np
import pytest
import torch

from paper_2606_13392_b200 import api
from paper_2606_13392_b200 import binding as B
from paper_2606_13392_b200.inputs import MSAConfig, make_prefill_inputs
from test_gpu_parity import run_decode_case, run_prefill_case

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _draw_shape(rng, fast_share):
    """(H_kv, G, d_h, B_k, d_idx): mostly shapes of the tensor-core kernels, else anything allowed."""
    if rng.random() < fast_share:
        return (int(rng.choice([1, 2, 4, 8])), int(rng.choice([8, 16])), 128, int(rng.choice([64, 128])),
                int(rng.choice([64, 128])))
    return (int(rng.choice([1, 2, 3, 4, 8])), int(rng.choice([1, 2, 4, 8, 16])), int(rng.choice([32, 64, 128, 256])),
            int(rng.choice([8, 16, 32, 64, 128])), int(rng.choice([16, 32, 64, 128])))


@pytest.mark.parametrize("seed", [11, 12])
def test_random_shapes_against_the_oracle(seed):
    rng = np.random.default_rng(seed)
    ran = 0
    for case in range(60):
        Hkv, G, d, Bk, d_idx = _draw_shape(rng, 0.6)
        fast = d == 128 and G in (8, 16) and Bk in (64, 128)
        k = int(rng.choice([1, 2, 3, 8, 16, 17, 32, 33, 64, 100]))
        idx_fp8, kv_fp8, sharp = (bool(rng.random() < 0.3) for _ in range(3))
        try:
            if rng.random() < 0.65:
                T = int(rng.choice([1, 2, int(rng.integers(3, 300)), int(rng.integers(300, 5000)),
                                    int(rng.integers(5000, 20000))]))
                T = T if fast else min(T, 3000)
                cfg = MSAConfig("rnd", "prefill", T, Hkv * G, Hkv, Bk, k, head_dim=d, idx_dim=d_idx,
                                seed=1000 * seed + case, idx_fp8=idx_fp8, kv_fp8=kv_fp8)
                stats = run_prefill_case(cfg, sharp, n_sample=64, ws_bytes=1 if rng.random() < 0.4 else None)
                assert stats["exact_sets"] >= 0.98, (cfg, stats)
            else:
                lens = tuple(int(rng.choice([1, int(rng.integers(2, 300)), int(rng.integers(300, 40000))]))
                             for _ in range(int(rng.integers(1, 6))))
                lens = lens if fast else tuple(min(L, 3000) for L in lens)
                cfg = MSAConfig("rnd", "decode", 0, Hkv * G, Hkv, Bk, k, head_dim=d, idx_dim=d_idx,
                                seed=1000 * seed + case, seq_lens=lens, idx_fp8=idx_fp8, kv_fp8=kv_fp8)
                run_decode_case(cfg, sharp)
            ran += 1
        except B.MsaError as e:
            if e.code != 2:
                raise
        torch.cuda.empty_cache()
    assert ran >= 40


@pytest.mark.parametrize("seed", [21])
def test_random_ranges_packed_batches_and_static_call_equal_the_whole_sequence_call(seed):
    # The stage calls on a query range against a prefix of the cache, the packed-batch call and the
    # allocation-free call must reproduce, bit for bit, what the whole-sequence call gives.
    rng = np.random.default_rng(seed)
    for case in range(120):
        Hkv, G, d, Bk, d_idx = _draw_shape(rng, 0.7)
        fast = d == 128 and G in (8, 16) and Bk in (64, 128)
        k = int(rng.choice([1, 2, 5, 16, 17, 32, 64]))
        idx_fp8, kv_fp8 = bool(rng.random() < 0.3), bool(rng.random() < 0.3)
        T = int(rng.integers(1, 12000 if fast else 2500))
        cfg = MSAConfig("rnd2", "prefill", T, Hkv * G, Hkv, Bk, k, head_dim=d, idx_dim=d_idx,
                        seed=1000 * seed + case, idx_fp8=idx_fp8, kv_fp8=kv_fp8)
        try:
            x = make_prefill_inputs(cfg, DEV, sharp=bool(rng.random() < 0.5))
            out, lse, I = api.prefill_forward(cfg, x)
            q0 = int(rng.integers(0, T))
            qc = int(rng.integers(1, T - q0 + 1))
            L = int(rng.integers(q0 + qc, T + 1))
            what = "%s q0=%d qc=%d L=%d" % (cfg, q0, qc, L)
            s = api.index_scores(cfg, x["q_idx"], x["k_idx"][:L], q0, qc, L)
            Ir = api.topk_select(cfg, s, q0, L)
            assert torch.equal(Ir, I[q0:q0 + qc]), what
            o, l = api.sparse_attn_prefill(cfg, x["q"][q0:q0 + qc], x["k"][:L], x["v"][:L], Ir, q0,
                                           workspace_bytes=1 if rng.random() < 0.5 else None)
            assert torch.equal(o, out[q0:q0 + qc]) and torch.equal(l, lse[q0:q0 + qc]), what
            if not kv_fp8 and rng.random() < 0.5:
                o2, l2 = torch.empty_like(o), torch.empty_like(l)
                try:
                    B.msa_sparse_attn_prefill_static(B.shape_of(cfg), x["q"][q0:q0 + qc], x["k"][:L], x["v"][:L], Ir,
                                                     q0, qc, L, o2, l2)
                    assert torch.equal(o2, o) and torch.equal(l2, l), what
                except B.MsaError as e:
                    if e.code != 3:  # the fixed array is too small for this shape
                        raise
            cu = [0] + sorted(int(c) for c in rng.integers(0, T + 1, size=int(rng.integers(0, 4)))) + [T]
            ov, lv, Iv = api.prefill_forward_varlen(cfg, x, cu)
            for a, b in zip(cu[:-1], cu[1:]):
                if a == b:
                    continue
                o1, l1, i1 = api.prefill_forward(cfg.scaled(T=b - a), {n: t[a:b] for n, t in x.items()})
                assert torch.equal(ov[a:b], o1) and torch.equal(lv[a:b], l1) and torch.equal(Iv[a:b], i1), (what, cu)
        except B.MsaError as e:
            if e.code != 2:
                raise
        torch.cuda.synchronize()
        assert B.check_async_status()[0] == 0
        torch.cuda.empty_cache()
