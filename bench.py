#!/usr/bin/env python
"""Benchmark of the MSA forward hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3|c4|c5|...] [--impl reference]

One step = one pass of the whole path (index scoring -> Top-k -> block-sparse attention) over
one synthetic workload resident in HBM.  Prints ONE JSON line (rank 0).  With N > 1 (torchrun)
every rank runs its own independent sequence (the path needs no exchange): weak scaling.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""

from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2606_13392_b200.inputs import (CONFIGS, MSAConfig, make_decode_inputs,  # noqa: E402
                                          make_prefill_inputs, to_bits)

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


# ----------------------------------------------------------------------------- algorithmic work
def prefill_work(cfg: MSAConfig):
    """Algorithmic FLOPs/bytes of one prefill pass (formulas: Section 3.3 and Section 4.2)."""
    T, Bk, k = cfg.T, cfg.block_size, cfg.top_k
    lens = cfg.seq_lens if cfg.seq_lens else (T,)  # packed sequences: positions restart in each
    i = np.concatenate([np.arange(n, dtype=np.int64) for n in lens])
    loc = i // Bk
    n_sel = np.minimum(k, loc + 1)
    tokens = (n_sel - 1) * Bk + (i % Bk) + 1          # visible tokens of the selected blocks
    pairs = int(n_sel.sum()) * cfg.n_kv_heads          # (query, group, block) pairs
    gd2 = 2 * cfg.group * cfg.head_dim                 # bytes of one (query, group) bf16 row set
    q_el = 1.0 if cfg.q_fp8 else 2.0                   # bytes per gathered Q element
    kv_el = 1.0 if (cfg.q_fp8 and cfg.kv_fp8) else 2.0  # (fp8 K/V with bf16 Q are widened to bf16 first)
    return {
        "index_flops": float(cfg.n_kv_heads) * cfg.idx_dim * float(sum(float(n) * (n + 1) for n in lens)),
        "attn_flops": 4.0 * cfg.n_q_heads * cfg.head_dim * float(tokens.sum()),
        "topk_bytes": 4.0 * cfg.n_kv_heads * float((loc + 1).sum()) + 4.0 * T * cfg.n_kv_heads * k,
        # KV-outer with bf16 partials: K+V once, per pair Q gather + partial write, final O
        "attn_bytes": kv_el * 2 * T * cfg.n_kv_heads * cfg.head_dim
                      + pairs * (q_el / 2.0 * gd2 + gd2 + 4 * cfg.group) + 2.0 * T * cfg.n_q_heads * cfg.head_dim,
        # combine: reads every partial (+ its LSE) once, writes O and LSE
        "combine_bytes": pairs * (gd2 + 4.0 * cfg.group) + T * cfg.n_q_heads * (2.0 * cfg.head_dim + 4),
        "pairs": pairs,
    }


def decode_work(cfg: MSAConfig):
    Bk, k = cfg.block_size, cfg.top_k
    lens = np.array(cfg.seq_lens, dtype=np.int64)
    loc = (lens - 1) // Bk
    n_sel = np.minimum(k, loc + 1)
    tokens = (n_sel - 1) * Bk + ((lens - 1) % Bk) + 1
    return {
        "index_bytes": (1.0 if cfg.idx_fp8 else 2.0) * cfg.idx_dim * float(lens.sum()),
        "index_flops": 2.0 * cfg.n_kv_heads * cfg.idx_dim * float(lens.sum()),
        "attn_bytes": (1.0 if cfg.kv_fp8 else 2.0) * 2 * cfg.n_kv_heads * cfg.head_dim * float(tokens.sum()),
        "attn_flops": 4.0 * cfg.n_q_heads * cfg.head_dim * float(tokens.sum()),
    }


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "100"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            pass

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            parts = [t.strip() for t in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); pw.append(float(parts[2]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            # "under load": samples drawing more than half of the highest power seen
            hi = max(pw)
            load = [s for s, w in zip(sm, pw) if w >= 0.5 * hi] or sm
            out.update(sm_mhz=statistics.median(load), sm_max_mhz=max(mx), reasons=sorted(reasons),
                       samples=len(sm), power_w_max=hi)
        return out


# ----------------------------------------------------------------------------- oracle leg
def oracle_sample_prefill(cfg: MSAConfig, x_bits, n: int, seed: int = 123):
    """Times the CPU oracle (as it stands) on n uniformly drawn query positions."""
    import oracle
    rng = np.random.default_rng(seed)
    pos = np.sort(rng.choice(cfg.T, size=min(n, cfg.T), replace=False)).astype(np.int64)
    q, qi = x_bits["q"][pos], x_bits["q_idx"][pos]
    t0 = time.perf_counter()
    oracle.msa_forward(q, x_bits["k"], x_bits["v"], qi, x_bits["k_idx"], pos, cfg.block_size, cfg.top_k)
    dt = time.perf_counter() - t0
    return len(pos), dt


def oracle_sample_decode(cfg: MSAConfig, xd, seqs):
    import oracle
    offs = xd["seq_offsets"].cpu().numpy()
    prepared = []
    for s in seqs:
        L = cfg.seq_lens[s]
        sl = slice(int(offs[s]), int(offs[s]) + L)
        prepared.append((to_bits(xd["q"][s:s + 1]), to_bits(xd["k_cache"][sl]), to_bits(xd["v_cache"][sl]),
                         to_bits(xd["q_idx"][s:s + 1]), to_bits(xd["k_idx_cache"][sl]), np.array([L - 1])))
    t0 = time.perf_counter()
    for (q, k, v, qi, ki, pos) in prepared:
        oracle.msa_forward(q, k, v, qi, ki, pos, cfg.block_size, cfg.top_k)
    return len(seqs), time.perf_counter() - t0


def oracle_sample_size(cfg: MSAConfig) -> int:
    """Query positions that take the oracle roughly 10-30 s on ~8-16 host cores."""
    per_q = cfg.n_kv_heads * cfg.idx_dim * cfg.T / 2 + \
        cfg.n_q_heads * cfg.head_dim * 2 * min(cfg.T / 2, cfg.top_k * cfg.block_size)
    return int(max(16, min(cfg.T, 2.0e11 / per_q)))


# ----------------------------------------------------------------------------- main
# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the stage kernels, from
# ncu captures.  Every entry says what was captured (workload, kernel form) and how it was brought
# to a full launch of the benchmarked workload: "scale" multiplies the captured bytes by the ratio
# of the units the two launches process (traffic grows in proportion to them).  An entry goes
# stale when its kernel changes; `kernel` names the form that was captured so that this shows.
NCU_TRAFFIC = {
    ("c4", "index_scores"): {"bytes": 17.79e9, "captured": "c4, one 131072-query chunk",
                             "kernel": "index_scores_tc_kernel<128,8,1,2,0,0,1> (scores in run order)", "scale": 1.0},
    ("c4", "topk_select"): {"bytes": 18.06e9, "captured": "c4, one 131072-query chunk",
                            "kernel": "topk_select_kernel<2>", "scale": 1.0},
    # attention: 18.5 GB read + 33.7 GB written per query range; half of the Q gathers hit L2
    ("c4", "attn_prefill"): {"bytes": 52.2e9, "captured": "c4, one query range",
                             "kernel": "attn_prefill_tc_kernel<128,8>, one CTA per SM (before the packed-batch row "
                                       "indirection and the fp8 template flag were added; same memory accesses)",
                             "scale": 1.0},
    ("c4", "combine"): {"bytes": 34.30e9, "captured": "c4, one query range", "kernel": "combine_kernel<128,8>",
                        "scale": 1.0},
    ("c3", "attn_prefill"): {"bytes": 39.96e9, "captured": "c3, one query range",
                             "kernel": "attn_prefill_tc_kernel<128,8>, one CTA per SM", "scale": 1.0},
    ("c3", "combine"): {"bytes": 27.55e9, "captured": "c3, one query range", "kernel": "combine_kernel<128,8>",
                        "scale": 1.0},
    ("c5", "attn_decode"): {"bytes": 1.106e9, "captured": "c5-small (8 x 32K + 8 x 128K tokens)",
                            "kernel": "attn_decode_kernel<128,8>", "scale": "selected K/V bytes streamed, c5 / c5-small"},
    ("c5", "index_scores_decode"): {"bytes": 2.47e9, "captured": "c5-small", "kernel": "index_scores_decode_kernel<8,2>",
                                    "scale": "cached index keys streamed, c5 / c5-small"},
}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=None,
                    help="c1..c5 (default: c4 as the headline, plus short c3, c5, c2 and c1 runs reported under 'others')")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-others", action="store_true")
    ap.add_argument("--topk-table", action="store_true",
                    help="time Top-k alone on the four (rows, scores per row, k) shapes of the paper's Top-k "
                         "latency table (Section 4.1, Table 1) and print one JSON line; not the headline metric")
    ap.add_argument("--index-lse", action="store_true",
                    help="prefill: also time the index-branch log-sum-exp (Section 4.3) on the step's selection; "
                         "reported beside the step, not part of it")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    primary = args.workload or "c4"
    extras = [] if (args.workload or args.no_others) else ["c3", "c5", "c2", "c1"]
    cfg = CONFIGS[primary]
    if args.impl == "reference":
        if rank == 0:
            run_reference(cfg, args)
        return

    import torch.distributed as dist
    from paper_2606_13392_b200 import binding as B
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if args.topk_table:
        if rank == 0:
            topk_table(B, dev, load_peaks())
        return
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    peaks = load_peaks()
    packed = cfg.mode == "prefill" and bool(cfg.seq_lens)  # no host-buffer call and no oracle leg for packed batches
    line = measure(cfg, args, rank, world, dev, B, peaks, dist, e2e=not args.no_e2e and not packed,
                   cpu=(world == 1 and not args.no_cpu_baseline and not packed))
    others = {}
    for name in extras:
        torch.cuda.empty_cache()
        res = measure(CONFIGS[name], args, rank, world, dev, B, peaks, dist, e2e=not args.no_e2e, cpu=False)
        if rank == 0:
            others[name] = {k: res[k] for k in ("metric", "value", "unit", "ms_per_step", "gpu_launches",
                                                 "roofline", "kernels", "e2e", "cuda_graph", "config") if k in res}
    if rank == 0:
        if others:
            line["others"] = others
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def topk_table(B, dev, peaks):
    """Top-k alone on N independent rows of n_scores fp32 block scores, k selected (Table 1's shapes).

    A row is a decode row whose local block is block n_scores: the n_scores blocks before it are
    ranked and k of them selected (top_k = k + 1 with the forced local block).  The paper's figures
    (another GPU) are printed beside ours as context.
    """
    shapes = [(131072, 1024, 16, 779.0), (131072, 2048, 32, 1991.0), (524288, 4096, 16, 7880.0),
              (524288, 8192, 32, 21326.0)]
    H_kv, Bk = 8, 128
    out = []
    for n_rows, n_scores, k, paper_us in shapes:
        cfg = MSAConfig("topk-table", "decode", 0, 64, H_kv, Bk, k + 1)
        shape = B.shape_of(cfg)
        batch = n_rows // H_kv
        ld = B.score_ld((n_scores + 1) * Bk, Bk)
        g = torch.Generator(device=dev).manual_seed(n_scores)
        scores = torch.empty((batch, H_kv, ld), dtype=torch.float32, device=dev)
        for b0 in range(0, batch, 4096):  # drawn in pieces: the largest matrix is 17 GB
            scores[b0:b0 + 4096].normal_(generator=g)
        seq_lens = torch.full((batch,), n_scores * Bk + 1, dtype=torch.int32, device=dev)
        idx = torch.empty((batch, H_kv, k + 1), dtype=torch.int32, device=dev)
        stream = torch.cuda.current_stream()
        max_len = n_scores * Bk + 1
        for _ in range(3):
            B.msa_topk_select_decode(shape, scores, ld, seq_lens, batch, max_len, idx)
        torch.cuda.synchronize()
        reps = 10
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            B.msa_topk_select_decode(shape, scores, ld, seq_lens, batch, max_len, idx)
        e1.record(stream)
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) / reps * 1e3
        gbs = n_rows * n_scores * 4.0 / (us * 1e-6) / 1e9
        assert bool((idx[:, :, k] == n_scores).all()) and bool((idx[:, :, :k] >= 0).all())
        out.append({"rows": n_rows, "scores_per_row": n_scores, "k": k, "us": us, "GB/s": gbs,
                    "frac_of_hbm": gbs / peaks["hbm_gbs"], "paper_us_other_gpu": paper_us})
        del scores, idx
        torch.cuda.empty_cache()
    print(json.dumps({"metric": "topk_latency_us", "unit": "us", "higher_is_better": False, "dtype": "f32",
                      "data": "synthetic", "l2": "inputs larger than L2 (126 MB)", "shapes": out,
                      "peak_source": "of " + peaks["_source"]}))


def rank_seed(seed: int, rank: int) -> int:
    """Every rank draws its own independent sequence: no data is shared between ranks."""
    return seed + 7919 * rank


def aggregate(ms_total_local: float, steps: int, units: int, world: int, device, dist):
    """MAX over ranks of the timed duration -> (ms per step, whole-job units per second)."""
    t = torch.tensor([ms_total_local], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_step = float(t.item()) / steps
    return ms_step, world * units / (ms_step * 1e-3)


def base_line(cfg: MSAConfig, args, n_gpus: int):
    metric = "msa_prefill_tokens_per_s" if cfg.mode == "prefill" else "msa_decode_tokens_per_s"
    conf = {"workload": "%s: %s" % (cfg.name, describe(cfg)), "l2": "inputs larger than L2 (126 MB)",
            "sharding": "one independent sequence (decode: batch) per rank, no collective"}
    return {"metric": metric, "unit": "tokens/s", "n_gpus": n_gpus, "steps": args.steps,
            "warmup": args.warmup, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic", "config": conf}


def describe(cfg: MSAConfig) -> str:
    f8 = (", index operands fp8 E4M3" if cfg.idx_fp8 else "") + \
        (", Q, K, V fp8 E4M3" if cfg.q_fp8 else (", K/V caches fp8 E4M3" if cfg.kv_fp8 else ""))
    if cfg.mode == "prefill" and cfg.seq_lens:
        return ("prefill fwd, %d packed sequences of %s tokens (%d in all), causal, %d q heads / %d kv heads, d_h=%d, "
                "d_idx=%d, B_k=%d, k=%d%s"
                % (len(cfg.seq_lens), "/".join(str(n) for n in cfg.seq_lens), cfg.T, cfg.n_q_heads, cfg.n_kv_heads,
                   cfg.head_dim, cfg.idx_dim, cfg.block_size, cfg.top_k, f8))
    if cfg.mode == "prefill":
        return ("prefill fwd, batch 1, T=%d causal, %d q heads / %d kv heads, d_h=%d, d_idx=%d, B_k=%d, k=%d%s"
                % (cfg.T, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.idx_dim, cfg.block_size, cfg.top_k, f8))
    return ("decode, batch %d (lens %s), %d q heads / %d kv heads, d_h=%d, d_idx=%d, B_k=%d, k=%d%s"
            % (len(cfg.seq_lens), sorted(set(cfg.seq_lens)), cfg.n_q_heads, cfg.n_kv_heads,
               cfg.head_dim, cfg.idx_dim, cfg.block_size, cfg.top_k, f8))


def run_reference(cfg: MSAConfig, args):
    import oracle
    line = base_line(cfg, args, 1)
    steps, warm = max(1, args.steps), args.warmup
    if cfg.mode == "prefill":
        x = make_prefill_inputs(cfg, "cpu")
        xb = {n: to_bits(t) for n, t in x.items()}
        n = max(8, oracle_sample_size(cfg) // (steps + min(warm, 1)))
        for _ in range(min(warm, 1)):
            oracle_sample_prefill(cfg, xb, n, 1)
        tot_n, tot_t = 0, 0.0
        for s in range(steps):
            m, dt = oracle_sample_prefill(cfg, xb, n, 100 + s)
            tot_n += m; tot_t += dt
        sample = "%d uniformly drawn query positions per step, all heads" % n
    else:
        small = cfg.scaled(seq_lens=tuple(sorted(set(cfg.seq_lens))))
        xd = make_decode_inputs(small, "cpu")
        tot_n, tot_t = 0, 0.0
        for s in range(steps):
            m, dt = oracle_sample_decode(small, xd, list(range(len(small.seq_lens))))
            tot_n += m; tot_t += dt
        sample = "one sequence of each cache length per step"
    val = tot_n / tot_t
    line.update(impl="reference", value=val, ms_per_step=1e3 * tot_t / steps, dtype="f64",
                cpu_baseline={"value": val, "unit": "tokens/s", "cores": oracle.n_threads(),
                              "kind": "oracle", "sample": sample},
                e2e={"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                gpu_launches=0)
    print(json.dumps(line))


def measure(cfg: MSAConfig, args, rank, world, dev, B, peaks, dist, e2e: bool, cpu: bool):
    """One workload: warm-up, timed steps, per-stage rooflines, optional e2e and oracle legs."""
    shape = B.shape_of(cfg)
    mycfg = cfg.scaled(seed=rank_seed(cfg.seed, rank))
    stream = torch.cuda.current_stream()

    if cfg.mode == "prefill":
        x = make_prefill_inputs(mycfg, dev)
        T = cfg.T
        out = torch.empty(x["q"].shape, dtype=torch.bfloat16, device=dev)
        lse = torch.empty((T, cfg.n_q_heads), dtype=torch.float32, device=dev)
        block_idx = torch.empty((T, cfg.n_kv_heads, cfg.top_k), dtype=torch.int32, device=dev)
        mn, pf = B.msa_prefill_forward_workspace_bytes(shape, T)
        ws = B.alloc_workspace(pf, dev)
        units = T

        if cfg.seq_lens:  # packed sequences of these lengths (they sum to T)
            assert sum(cfg.seq_lens) == T
            cu = np.concatenate([[0], np.cumsum(cfg.seq_lens)]).tolist()
            mn, pf = B.msa_prefill_forward_varlen_workspace_bytes(shape, cu)
            ws = B.alloc_workspace(pf, dev)

            def step():
                B.msa_prefill_forward_varlen(shape, x["q"], x["k"], x["v"], x["q_idx"], x["k_idx"], cu, out, lse,
                                             block_idx, ws)
        else:
            def step():
                B.msa_prefill_forward(shape, x["q"], x["k"], x["v"], x["q_idx"], x["k_idx"], T, out, lse,
                                      block_idx, ws)
    else:
        x = make_decode_inputs(mycfg, dev)
        batch = len(cfg.seq_lens)
        max_len = int(max(cfg.seq_lens))
        ld = B.score_ld(max_len, cfg.block_size)
        scores = torch.empty((batch, cfg.n_kv_heads, ld), dtype=torch.float32, device=dev)
        block_idx = torch.empty((batch, cfg.n_kv_heads, cfg.top_k), dtype=torch.int32, device=dev)
        out = torch.empty_like(x["q"])
        lse = torch.empty((batch, cfg.n_q_heads), dtype=torch.float32, device=dev)
        ws = B.alloc_workspace(B.msa_sparse_attn_decode_workspace_bytes(shape, batch), dev)
        units = batch
        cache_tokens = x["k_cache"].shape[0]

        def step():
            B.msa_decode_forward(shape, x["q"], x["q_idx"], x["k_cache"], x["v_cache"], x["k_idx_cache"],
                                 cache_tokens, x["seq_offsets"], x["seq_lens"], batch, max_len, scores,
                                 ld, block_idx, out, lse, ws)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    steps = args.steps if cfg.mode == "prefill" else max(args.steps, 20)  # decode steps are ~1 ms
    for _ in range(max(args.warmup, 0)):
        step()
    barrier()

    sampler = ClockSampler(dev.index or 0) if rank == 0 else None
    n_before = B.launch_count()
    B.profile_begin()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        step()
    e1.record(stream)
    barrier()
    ms_total = e0.elapsed_time(e1)
    stages = B.profile_end()
    launches = B.launch_count() - n_before
    clocks = sampler.stop() if sampler else None
    code, detail = B.check_async_status()
    if code != 0:
        raise RuntimeError("device status %d (detail %d) after the timed region" % (code, detail))

    ms_step, value = aggregate(ms_total, steps, units, world, dev, dist)
    if rank != 0:
        return {}

    line = base_line(cfg, args, world)
    line["steps"] = steps
    line.update(value=value, ms_per_step=ms_step, gpu_launches=int(launches), clocks=clocks)

    # ---- per-kernel figures and the roofline of the dominant kernel
    hbm, tf_b, tf_s = peaks["hbm_gbs"], peaks["bf16_tflops"], peaks["bf16_tflops_sustained"]
    src = "of " + peaks["_source"]
    kern = {}
    if cfg.mode == "prefill":
        w = prefill_work(cfg)
        spec = {"index_scores": ("tensor", w["index_flops"]), "topk_select": ("hbm", w["topk_bytes"]),
                "attn_prefill": ("hbm", w["attn_bytes"]), "combine": ("hbm", w["combine_bytes"])}
    else:
        w = decode_work(cfg)
        spec = {"index_scores_decode": ("hbm", w["index_bytes"]), "attn_decode": ("hbm", w["attn_bytes"])}
    for name, (ms, n) in stages.items():
        if n == 0:
            continue
        per_step_ms = ms / steps
        ent = {"ms_per_step": per_step_ms, "launches_per_step": n / steps, "share": ms / max(ms_total, 1e-9)}
        if name in spec and spec[name][1] > 0:
            bound, work = spec[name]
            if bound == "tensor":
                ach = work / (per_step_ms * 1e-3) / 1e12
                # an fp8 contraction: the measured bf16 peaks times the nominal fp8 / bf16 ratio of 2
                mul = 2.0 if (cfg.idx_fp8 and name == "index_scores") else 1.0
                ent.update(bound="tensor", achieved=ach, unit="TFLOP/s", peak=tf_s * mul, frac=ach / (tf_s * mul),
                           frac_of_burst_peak=ach / (tf_b * mul))
                if mul != 1.0:
                    ent["peak_dtype"] = "fp8 = measured bf16 x 2 (nominal ratio)"
            else:
                ach = work / (per_step_ms * 1e-3) / 1e9
                ent.update(bound="hbm", achieved=ach, unit="GB/s", peak=hbm, frac=ach / hbm)
            tr = NCU_TRAFFIC.get((cfg.name, name))
            ent["traffic"] = tr["bytes"] if tr else None
            if tr:
                ent["traffic_source"] = {k: v for k, v in tr.items() if k != "bytes"}
                # measured DRAM bytes over the measured time: the fraction of the copy bandwidth the
                # kernel really draws (the algorithmic figure above counts bytes that L2 may serve)
                per_launch_ms = per_step_ms / max(n / steps, 1e-9)
                ent["dram_gbs"] = tr["bytes"] / (per_launch_ms * 1e-3) / 1e9
                ent["dram_frac"] = ent["dram_gbs"] / hbm
            if ent["frac"] > 1.0:
                ent["note"] = ("above 1.0: the numerator is algorithmic work; part of it is served from L2, and the "
                               "denominator is a measured copy / cuBLAS rate, not a hardware limit")
        kern[name] = ent
    if cfg.mode == "prefill" and "attn_prefill" in kern:
        kern["attn_prefill"]["tensor_tflops"] = w["attn_flops"] / (kern["attn_prefill"]["ms_per_step"] * 1e-3) / 1e12
        kern["attn_prefill"]["tensor_frac_of_sustained_peak"] = kern["attn_prefill"]["tensor_tflops"] / tf_s
        kern["attn_prefill"]["tensor_frac_of_burst_peak"] = kern["attn_prefill"]["tensor_tflops"] / tf_b
        if "combine" in kern:  # Eq. 8 end to end: the partials' pass and their merge as one stage
            both = kern["attn_prefill"]["ms_per_step"] + kern["combine"]["ms_per_step"]
            tfl = w["attn_flops"] / (both * 1e-3) / 1e12
            kern["attn_plus_combine"] = {"ms_per_step": both, "tensor_tflops": tfl,
                                         "tensor_frac_of_sustained_peak": tfl / tf_s,
                                         "tensor_frac_of_burst_peak": tfl / tf_b}
    dom = max((n for n in kern if "bound" in kern[n]), key=lambda n: kern[n]["ms_per_step"], default=None)
    if dom is not None:
        d = kern[dom]
        per_launch = d["launches_per_step"]
        line["roofline"] = {"kernel": dom, "bound": d["bound"], "achieved": d["achieved"], "peak": d["peak"],
                            "unit": d["unit"], "frac": d["frac"], "traffic": d.get("traffic"),
                            "launches_per_step": per_launch,
                            "peak_source": (src + ", sustained bf16 (kernel timed inside a long step)")
                            if d["bound"] == "tensor" else src}
    line["kernels"] = kern
    line["peaks"] = {"hbm_gbs": hbm, "bf16_tflops_burst": tf_b, "bf16_tflops_sustained": tf_s,
                     "source": peaks["_source"]}
    if cfg.mode == "prefill":
        line["tflops_total"] = (w["index_flops"] + w["attn_flops"]) / (ms_step * 1e-3) / 1e12

    # ---- the same decode step replayed from a CUDA graph (serving loops capture it once)
    if cfg.mode == "decode":
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(stream)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                step()
            for _ in range(3):
                g.replay()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            g0.record(side)
            for _ in range(steps):
                g.replay()
            g1.record(side)
        torch.cuda.synchronize()
        g_ms = g0.elapsed_time(g1) / steps
        line["cuda_graph"] = {"ms_per_step": g_ms, "value": world * units / (g_ms * 1e-3), "unit": line["unit"],
                              "note": "this rank's step captured once and replayed; not max over ranks"}
        del g

    # ---- training-side forward output, timed on its own (Section 4.3)
    if getattr(args, "index_lse", False) and cfg.mode == "prefill":
        mn_l, pf_l = B.msa_index_lse_prefill_workspace_bytes(shape, T, T)
        ws_l = B.alloc_workspace(pf_l, dev)
        lse_idx = torch.empty((T, cfg.n_kv_heads), dtype=torch.float32, device=dev)

        def lse_step():
            B.msa_index_lse_prefill(shape, x["q_idx"], x["k_idx"], block_idx, 0, T, T, lse_idx, ws_l)
        for _ in range(2):
            lse_step()
        torch.cuda.synchronize()
        n_rep = min(steps, 3)
        e0.record(stream)
        for _ in range(n_rep):
            lse_step()
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / n_rep
        w = prefill_work(cfg)
        # one dot product of d_idx per (query, index head, visible token of a selected block)
        flops = w["attn_flops"] / (4.0 * cfg.n_q_heads * cfg.head_dim) * 2.0 * cfg.n_kv_heads * cfg.idx_dim
        # Bound by the exponential unit, one exp2 per score: 16 per clock and SM (4 sub-partitions x 4 lanes)
        # x 148 SMs x 1.965 GHz = 4.65e12 per second; the 2*d_idx FLOPs per score need 5-10 % of the tensor peak.
        n_exp = flops / (2.0 * cfg.idx_dim)
        xu_peak = 16 * 148 * 1.965e9
        line["index_lse"] = {"ms": ms, "bound": "alu", "achieved": n_exp / (ms * 1e-3) / 1e9, "unit": "Gexp/s",
                             "peak": xu_peak / 1e9, "frac": n_exp / (ms * 1e-3) / xu_peak,
                             "peak_source": "derived: 16 exp2 per clock and SM x 148 SMs x 1.965 GHz",
                             "tensor_tflops": flops / (ms * 1e-3) / 1e12,
                             "includes": "reverse index, the per-item kernel and the slot reduction"}
        del ws_l, lse_idx

    # ---- end to end from host buffers (copies inside the timed region)
    if e2e:
        del out, lse, ws
        torch.cuda.empty_cache()
        line["e2e"] = run_e2e(cfg, shape, x, B, dev, max(5, min(steps, 10)), world)

    # ---- the oracle on this machine's host cores (bounded sample)
    if cpu:
        import oracle
        if cfg.mode == "prefill":
            xb = {n: to_bits(tn) for n, tn in x.items() if n != "q" and n != "q_idx"}
            n = oracle_sample_size(cfg)
            rng = np.random.default_rng(123)
            pos = np.sort(rng.choice(cfg.T, size=min(n, cfg.T), replace=False)).astype(np.int64)
            pt = torch.from_numpy(pos).to(dev)
            qb = to_bits(x["q"][pt])
            qib = (x["q_idx"].view(torch.uint8)[pt].cpu().numpy() if cfg.idx_fp8 else to_bits(x["q_idx"][pt]))
            t0 = time.perf_counter()
            oracle.msa_forward(qb, xb["k"], xb["v"], qib, xb["k_idx"], pos, cfg.block_size, cfg.top_k)
            dt = time.perf_counter() - t0
            m = len(pos)
            sample = "%d uniformly drawn query positions of the same inputs, all heads" % m
        else:
            seqs = [0, len(cfg.seq_lens) - 1]
            m, dt = oracle_sample_decode(cfg, x, seqs)
            sample = "sequences %s of the same batch (one of each cache length)" % seqs
        line["cpu_baseline"] = {"value": m / dt, "unit": "tokens/s", "cores": oracle.n_threads(),
                                "kind": "oracle", "sample": sample, "seconds": dt}
    return line


def run_e2e(cfg, shape, x, B, dev, steps, world):
    stream = torch.cuda.current_stream()
    if cfg.mode == "prefill":
        T = cfg.T
        host = {n: t.cpu().pin_memory() for n, t in x.items()}
        out_h = torch.empty(x["q"].shape, dtype=torch.bfloat16).pin_memory()
        mn, pf = B.msa_prefill_forward_host_workspace_bytes(shape, T)
        ws = B.alloc_workspace(pf, dev)
        h2d = sum(t.numel() * t.element_size() for t in host.values())
        d2h = out_h.numel() * 2

        def step():
            B.msa_prefill_forward_host(shape, host["q"], host["k"], host["v"], host["q_idx"],
                                       host["k_idx"], T, out_h, None, None, ws)
        units = T
    else:
        batch = len(cfg.seq_lens)
        max_len = int(max(cfg.seq_lens))
        ld = B.score_ld(max_len, cfg.block_size)
        qh, qih = x["q"].cpu().pin_memory(), x["q_idx"].cpu().pin_memory()
        out_h = torch.empty(x["q"].shape, dtype=torch.bfloat16).pin_memory()
        qd, qid, od = torch.empty_like(x["q"]), torch.empty_like(x["q_idx"]), torch.empty_like(x["q"])
        scores = torch.empty((batch, cfg.n_kv_heads, ld), dtype=torch.float32, device=dev)
        bi = torch.empty((batch, cfg.n_kv_heads, cfg.top_k), dtype=torch.int32, device=dev)
        ws = B.alloc_workspace(B.msa_sparse_attn_decode_workspace_bytes(shape, batch), dev)
        h2d = qh.numel() * 2 + qih.numel() * 2
        d2h = out_h.numel() * 2

        def step():
            B.msa_decode_forward_host(shape, qh, qih, qd, qid, x["k_cache"], x["v_cache"], x["k_idx_cache"],
                                      x["k_cache"].shape[0], x["seq_offsets"], x["seq_lens"], batch, max_len,
                                      scores, ld, bi, od, out_h, ws)
        units = batch
    step()  # warm-up (page-locks are already in place)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    return {"value": world * units / (ms * 1e-3), "unit": "tokens/s", "ms_per_step": ms,
            "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": steps}


if __name__ == "__main__":
    main()
