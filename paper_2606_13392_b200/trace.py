"""Per-role timelines of the prefill attention kernel and of the index-scoring kernel (a
development aid, not part of the path).

    python -m paper_2606_13392_b200.build --trace      # library with clock stamps compiled in
    python -m paper_2606_13392_b200.trace [workload]   # attention; default c3; cycles relative to the first stamp
    python -m paper_2606_13392_b200.trace index [workload]   # index scoring alone; default c3-40k
    python -m paper_2606_13392_b200.build              # back to the production build

CTA 0 stamps clock64() at fixed points of its roles for 16 consecutive items in steady state
(items 1000..1015 of its share).  Columns: when the softmax warps of the item's context saw S
(s_ok), wrote P (p_done), saw O (o_ok) and handed the partial to the copy engine (done); when the
MMA issuer was ready to issue S and had issued it, likewise for O = P V; when the producer found
the Q buffer free and had issued the item's gathers.

Index scoring: CTA 0 stamps 16 consecutive (key tile, head) units.  Columns: when the MMA issuer
had the unit's accumulator back (M:waited), started issuing (M:go) and had committed the unit
(M:issued); when epilogue warp 0 saw the accumulator full (E0:full); when each of the eight
epilogue warps had its part in registers and released the accumulator (rel0..rel7; warps 3 and 7
of these share a scheduler partition with the issuing warp).
"""

from __future__ import annotations

import ctypes
import sys

import numpy as np
import torch

from . import api, binding as B
from .inputs import CONFIGS, make_prefill_inputs

COLS = [(0, "s_ok"), (3, "p_done"), (5, "o_ok"), (7, "done"), (8, "S_go"), (9, "S_issued"), (10, "PV_go"),
        (11, "PV_issued"), (12, "q_free"), (13, "q_issued")]


IDX_COLS = [(10, "M:waited"), (0, "M:go"), (1, "M:issued"), (11, "E0:full")] + [(2 + i, "rel%d" % i) for i in range(8)]


def read_trace(lib) -> np.ndarray:
    buf = (ctypes.c_longlong * 256)()
    if lib.msa_debug_read_trace(buf) != 0:
        raise SystemExit("reading the trace failed")
    return np.array(buf[:], dtype=np.int64).reshape(16, 16)


def index_main(lib, name: str) -> None:
    cfg = CONFIGS[name]
    x = make_prefill_inputs(cfg, "cuda")
    tc, nh = B.msa_index_scores_plan(B.shape_of(cfg), cfg.T, cfg.T)
    print("%s: tensor-core kernel %d, heads per CTA %d" % (name, tc, nh))
    api.index_scores(cfg, x["q_idx"], x["k_idx"], 0, cfg.T)
    torch.cuda.synchronize()
    a = read_trace(lib)
    t0 = a[0, 10]
    print("unit " + " ".join("%9s" % n for _, n in IDX_COLS))
    for i in range(16):
        print("%4d " % i + " ".join("%9d" % (a[i, c] - t0) for c, _ in IDX_COLS))
    print("cycles per unit: %.0f (%d at the tensor pipe's nominal rate)"
          % (float(a[15, 0] - a[1, 0]) / 14.0, 128 * cfg.idx_dim // 16))


def main() -> None:
    lib = B.lib()
    if not hasattr(lib, "msa_debug_read_trace"):
        raise SystemExit("the library was built without -DMSA_TRACE: python -m paper_2606_13392_b200.build --trace")
    if len(sys.argv) > 1 and sys.argv[1] == "index":
        index_main(lib, sys.argv[2] if len(sys.argv) > 2 else "c3-40k")
        return
    cfg = CONFIGS[sys.argv[1] if len(sys.argv) > 1 else "c3"]
    x = make_prefill_inputs(cfg, "cuda")
    api.prefill_forward(cfg, x)
    torch.cuda.synchronize()
    a = read_trace(lib)
    t0 = a[0, 0]
    print("item " + " ".join("%10s" % n for _, n in COLS))
    for i in range(16):
        print("%4d " % i + " ".join("%10d" % (a[i, c] - t0) for c, _ in COLS))
    print("cycles per item (s_ok to s_ok, this context handles every other item): %.0f"
          % (float(a[14, 0] - a[0, 0]) / 14.0))


if __name__ == "__main__":
    main()
