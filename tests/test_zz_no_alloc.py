"""The allocation-free prefill attention entry point against the workspace form.

msa_sparse_attn_prefill_static serves hosts that cannot allocate device memory when they
need attention (a plug-in inside an engine that owns all of it, code that runs after the
memory pool was frozen): it takes no workspace and uses one fixed scratch array inside the
library.  This file checks, through the C ABI, that it gives what msa_sparse_attn_prefill
gives on the same inputs, on two calls in a row (the array keeps the first call's contents,
so the second call also proves that nothing stale leaks), and that it refuses a problem the
fixed array cannot serve.  The file name keeps it last in collection order, so a run that
stops at the first failure has already run every other test.
"""

import pytest
import torch

from paper_2606_13392_b200 import api
from paper_2606_13392_b200 import binding as B
from paper_2606_13392_b200.inputs import CONFIGS, make_prefill_inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _both(cfg, x, I, q_begin, q_count):
    """Runs both entry points on rows [q_begin, q_begin+q_count) and returns their outputs."""
    shape = B.shape_of(cfg)
    q = x["q"][q_begin:q_begin + q_count].contiguous()
    Ic = I[q_begin:q_begin + q_count].contiguous()
    kv_len = x["k"].shape[0]
    outs = []
    for static in (False, True):
        out = torch.zeros_like(q)
        lse = torch.zeros((q_count, cfg.n_q_heads), dtype=torch.float32, device=DEV)
        if static:
            B.msa_sparse_attn_prefill_static(shape, q, x["k"], x["v"], Ic, q_begin, q_count, kv_len,
                                             out, lse)
        else:
            mn, pf = B.msa_sparse_attn_prefill_workspace_bytes(shape, q_count, kv_len)
            ws = B.alloc_workspace(pf, DEV)
            B.msa_sparse_attn_prefill(shape, q, x["k"], x["v"], Ic, q_begin, q_count, kv_len, out, lse, ws)
        torch.cuda.synchronize()
        outs.append((out, lse))
    return outs


def _assert_same(a, b):
    (o1, l1), (o2, l2) = a, b
    # Tolerances of the parity tests (max-abs 2e-2 on O, 2e-3 on LSE); the two entry points
    # run the same kernels, so in practice they agree far more closely than that.
    assert torch.isfinite(o2.float()).all()
    assert (o1.float() - o2.float()).abs().max().item() <= 2e-2
    assert (o1.float() - o2.float()).abs().mean().item() <= 2e-3
    assert (l1 - l2).abs().max().item() <= 2e-3


def test_static_entry_matches_workspace_entry_twice_in_a_row():
    # First call: the paper-shaped head layout (64/8 heads, B_k=128, k=64): about 1 MiB of
    # partials per query, so the 64 MiB array serves it in several passes.
    cfg = CONFIGS["c3"].scaled(name="na-1", T=4096 + 50)
    x = make_prefill_inputs(cfg, DEV, sharp=True)
    _, _, I = api.prefill_forward(cfg, x)
    _assert_same(*_both(cfg, x, I, 0, cfg.T))
    assert B.check_async_status()[0] == 0

    # Second call right after it, other shape and a query range in the middle of the
    # sequence: must not see anything of the first call in the shared array.
    cfg2 = CONFIGS["c2"].scaled(name="na-2", T=3000, seed=11)
    x2 = make_prefill_inputs(cfg2, DEV, sharp=True)
    _, _, I2 = api.prefill_forward(cfg2, x2)
    _assert_same(*_both(cfg2, x2, I2, 1000, 1500))
    assert B.check_async_status()[0] == 0


def test_static_entry_refuses_what_the_fixed_array_cannot_serve():
    # G = 16 with k = 128: 4 MiB of partials per query, so fewer than 16 queries fit 64 MiB.
    cfg = CONFIGS["c3"].scaled(name="na-big", T=2048, n_q_heads=128, n_kv_heads=8, top_k=128)
    shape = B.shape_of(cfg)
    x = make_prefill_inputs(cfg, DEV)
    I = torch.full((cfg.T, cfg.n_kv_heads, cfg.top_k), -1, dtype=torch.int32, device=DEV)
    out = torch.empty_like(x["q"])
    with pytest.raises(B.MsaError) as e:
        B.msa_sparse_attn_prefill_static(shape, x["q"], x["k"], x["v"], I, 0, cfg.T, cfg.T, out, None)
    assert e.value.code == 3  # MSA_ERR_WORKSPACE: reported before anything is launched
