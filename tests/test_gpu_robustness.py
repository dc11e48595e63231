"""Error paths and memory discipline of the CUDA library, exercised without faulting the GPU.

* Guard bands: every output and workspace is embedded in a larger buffer whose margins hold a
  known byte pattern; after the calls the margins must be untouched (a stand-in for a memory
  checker: a write outside a buffer the caller passed would land there first).
* Bounded waits: with a short wait limit and a copy-issuing warp that is merely late (both set
  through the library's test hook), a device-side wait runs out; the kernel must unwind and
  return, the status word must say "timeout", and the next call must be clean and correct.
  Nothing here traps, reads out of bounds or waits without a limit.
"""

import numpy as np
import pytest
import torch

import oracle
from paper_2606_13392_b200 import api
from paper_2606_13392_b200 import binding as B
from paper_2606_13392_b200.inputs import CONFIGS, make_decode_inputs, make_prefill_inputs, sample_positions, to_bits
from parity_utils import check_attn, check_scores

pytestmark = pytest.mark.gpu
DEV = "cuda"
GUARD = 4096          # bytes on either side
PATTERN = 0xCD


class Guarded:
    """A tensor of `shape`/`dtype` in the middle of a byte buffer filled with PATTERN."""

    def __init__(self, shape, dtype):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.n = n
        self.raw = torch.full((GUARD + n + GUARD,), PATTERN, dtype=torch.uint8, device=DEV)
        self.t = self.raw[GUARD:GUARD + n].view(dtype).view(*shape)

    def intact(self) -> bool:
        return bool((self.raw[:GUARD] == PATTERN).all()) and bool((self.raw[GUARD + self.n:] == PATTERN).all())


@pytest.mark.parametrize("name,T,ws", [("c1", 2048, "preferred"), ("c3", 12288 + 5, "preferred"),
                                       ("c3", 6144 + 77, "minimum"), ("c2", 4096 + 37, "minimum")])
def test_prefill_calls_write_inside_their_buffers_only(name, T, ws):
    cfg = CONFIGS[name].scaled(name=name + "-guard", T=T)
    shape = B.shape_of(cfg)
    x = make_prefill_inputs(cfg, DEV, sharp=True)
    mn, pf = B.msa_prefill_forward_workspace_bytes(shape, T)
    out = Guarded((T, cfg.n_q_heads, cfg.head_dim), torch.bfloat16)
    lse = Guarded((T, cfg.n_q_heads), torch.float32)
    bidx = Guarded((T, cfg.n_kv_heads, cfg.top_k), torch.int32)
    wsp = Guarded((pf if ws == "preferred" else mn,), torch.uint8)
    B.msa_prefill_forward(shape, x["q"], x["k"], x["v"], x["q_idx"], x["k_idx"], T, out.t, lse.t, bidx.t, wsp.t)
    # the stage calls on their own: scores with a pitch wider than B, a range inside the sequence
    q0, qc = T // 3, T - T // 3
    ld = B.score_ld(T, cfg.block_size) + 8
    sc = Guarded((qc, cfg.n_kv_heads, ld), torch.float32)
    B.msa_index_scores(shape, x["q_idx"][q0:], x["k_idx"], q0, qc, T, sc.t, ld)
    bidx2 = Guarded((qc, cfg.n_kv_heads, cfg.top_k), torch.int32)
    B.msa_topk_select(shape, sc.t, ld, q0, qc, T, bidx2.t)
    torch.cuda.synchronize()
    assert B.check_async_status()[0] == 0
    for g, what in ((out, "out"), (lse, "lse"), (bidx, "block_idx"), (wsp, "workspace"), (sc, "scores"),
                    (bidx2, "block_idx of the range")):
        assert g.intact(), "bytes outside %s were written" % what
    # columns [B, ld) of a scores row are not the call's to write
    nb = cfg.n_blocks
    assert bool((sc.t[:, :, nb:].contiguous().view(torch.uint8) == PATTERN).all())
    assert torch.equal(bidx2.t, bidx.t[q0:])


def test_decode_calls_write_inside_their_buffers_only():
    cfg = CONFIGS["c5"].scaled(name="c5-guard", seq_lens=(1, 127, 4000, 8200, 20000))
    shape = B.shape_of(cfg)
    x = make_decode_inputs(cfg, DEV, sharp=True)
    batch, max_len = len(cfg.seq_lens), max(cfg.seq_lens)
    ld = B.score_ld(max_len, cfg.block_size)
    sc = Guarded((batch, cfg.n_kv_heads, ld), torch.float32)
    bidx = Guarded((batch, cfg.n_kv_heads, cfg.top_k), torch.int32)
    out = Guarded((batch, cfg.n_q_heads, cfg.head_dim), torch.bfloat16)
    lse = Guarded((batch, cfg.n_q_heads), torch.float32)
    wsp = Guarded((B.msa_sparse_attn_decode_workspace_bytes(shape, batch),), torch.uint8)
    B.msa_decode_forward(shape, x["q"], x["q_idx"], x["k_cache"], x["v_cache"], x["k_idx_cache"],
                         x["k_cache"].shape[0], x["seq_offsets"], x["seq_lens"], batch, max_len, sc.t, ld, bidx.t,
                         out.t, lse.t, wsp.t)
    torch.cuda.synchronize()
    assert B.check_async_status()[0] == 0
    for g, what in ((sc, "scores"), (bidx, "block_idx"), (out, "out"), (lse, "lse"), (wsp, "workspace")):
        assert g.intact(), "bytes outside %s were written" % what
    want = api.decode_forward(cfg, x)
    assert torch.equal(out.t, want[0]) and torch.equal(bidx.t, want[2])


@pytest.fixture
def short_waits():
    """A wait limit of 2e5 cycles (about 0.1 ms) and copy-issuing warps that start 3e6 cycles
    (about 1.5 ms) late; the production values are restored afterwards, whatever happens."""
    B.msa_debug_set_wait(200_000, 3_000_000)
    try:
        yield
    finally:
        B.msa_debug_set_wait(0, 0)
        torch.cuda.synchronize()
        B.check_async_status()


def test_index_scoring_wait_runs_out_and_the_next_call_is_clean(short_waits):
    cfg = CONFIGS["c3"].scaled(name="c3-late", T=4096 + 19)
    x = make_prefill_inputs(cfg, DEV, sharp=True)
    assert B.msa_index_scores_plan(B.shape_of(cfg), cfg.T, cfg.T)[0]   # the tensor-core kernel
    api.index_scores(cfg, x["q_idx"], x["k_idx"], 0, cfg.T)
    torch.cuda.synchronize()   # the kernel has returned: no hang, no fault
    code, detail = B.check_async_status()
    assert code == 5, (code, detail)              # MSA_ERR_TIMEOUT
    assert 0x100 <= detail < 0x200, hex(detail)   # a wait of the index-scoring kernel
    assert B.check_async_status()[0] == 0         # reading cleared it
    # production limits again: the same call gives the oracle's scores
    B.msa_debug_set_wait(0, 0)
    M = api.index_scores(cfg, x["q_idx"], x["k_idx"], 0, cfg.T)
    torch.cuda.synchronize()
    assert B.check_async_status()[0] == 0
    pos = np.arange(cfg.T - 200, cfg.T)
    M_ref = oracle.index_scores(to_bits(x["q_idx"][cfg.T - 200:]), to_bits(x["k_idx"]), pos, cfg.block_size)
    check_scores(M[cfg.T - 200:, :, :cfg.n_blocks].cpu().numpy(), M_ref, pos, cfg.block_size)


def test_attention_wait_runs_out_and_the_next_call_is_clean(short_waits):
    cfg = CONFIGS["c3"].scaled(name="c3-late", T=4096 + 19)
    shape = B.shape_of(cfg)
    x = make_prefill_inputs(cfg, DEV, sharp=True)
    B.msa_debug_set_wait(0, 0)
    out0, lse0, I = api.prefill_forward(cfg, x)
    torch.cuda.synchronize()
    B.msa_debug_set_wait(200_000, 3_000_000)
    mn, pf = B.msa_sparse_attn_prefill_workspace_bytes(shape, cfg.T, cfg.T)
    ws = torch.zeros(pf, dtype=torch.uint8, device=DEV)   # partials that are never written read as zeros
    out = torch.zeros_like(x["q"])
    lse = torch.zeros((cfg.T, cfg.n_q_heads), dtype=torch.float32, device=DEV)
    B.msa_sparse_attn_prefill(shape, x["q"], x["k"], x["v"], I, 0, cfg.T, cfg.T, out, lse, ws)
    torch.cuda.synchronize()
    code, detail = B.check_async_status()
    assert code == 5, (code, detail)
    assert 0x300 <= detail < 0x400, hex(detail)   # a wait of the prefill attention kernel
    assert torch.isfinite(out.float()).all()
    B.msa_debug_set_wait(0, 0)
    B.msa_sparse_attn_prefill(shape, x["q"], x["k"], x["v"], I, 0, cfg.T, cfg.T, out, lse, ws)
    torch.cuda.synchronize()
    assert B.check_async_status()[0] == 0
    assert torch.equal(out, out0) and torch.equal(lse, lse0)
    pos = sample_positions(cfg.T, cfg.block_size, cfg.top_k, 48, 2)
    pos_t = torch.from_numpy(pos).to(DEV)
    O_ref, LSE_ref = oracle.sparse_attn(to_bits(x["q"][pos_t]), to_bits(x["k"]), to_bits(x["v"]),
                                        I[pos_t].cpu().numpy(), pos, cfg.block_size)
    check_attn(out[pos_t].float().cpu().numpy(), lse[pos_t].cpu().numpy(), O_ref, LSE_ref, "after a timeout")
