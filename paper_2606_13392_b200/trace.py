"""Per-role timeline of the prefill attention kernel (a development aid, not part of the path).

    python -m paper_2606_13392_b200.build --trace      # library with clock stamps compiled in
    python -m paper_2606_13392_b200.trace [workload]   # default c3; prints cycles relative to the first stamp
    python -m paper_2606_13392_b200.build              # back to the production build

CTA 0 stamps clock64() at fixed points of its roles for 16 consecutive items in steady state
(items 1000..1015 of its share).  Columns: when the softmax warps of the item's context saw S
(s_ok), wrote P (p_done), saw O (o_ok) and handed the partial to the copy engine (done); when the
MMA issuer was ready to issue S and had issued it, likewise for O = P V; when the producer found
the Q buffer free and had issued the item's gathers.
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


def main() -> None:
    cfg = CONFIGS[sys.argv[1] if len(sys.argv) > 1 else "c3"]
    lib = B.lib()
    if not hasattr(lib, "msa_debug_read_trace"):
        raise SystemExit("the library was built without -DMSA_TRACE: python -m paper_2606_13392_b200.build --trace")
    x = make_prefill_inputs(cfg, "cuda")
    api.prefill_forward(cfg, x)
    torch.cuda.synchronize()
    buf = (ctypes.c_longlong * 256)()
    if lib.msa_debug_read_trace(buf) != 0:
        raise SystemExit("reading the trace failed")
    a = np.array(buf[:], dtype=np.int64).reshape(16, 16)
    t0 = a[0, 0]
    print("item " + " ".join("%10s" % n for _, n in COLS))
    for i in range(16):
        print("%4d " % i + " ".join("%10d" % (a[i, c] - t0) for c, _ in COLS))
    print("cycles per item (s_ok to s_ok, this context handles every other item): %.0f"
          % (float(a[14, 0] - a[0, 0]) / 14.0))


if __name__ == "__main__":
    main()
