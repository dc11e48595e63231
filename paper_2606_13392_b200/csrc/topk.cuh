// Eq. 7 + Local Block rule: exp-free Top-k over raw block scores, one warp per row.
//
// Ranking order is "score descending, then block index ascending".  The kernel works in two
// passes over the row (the second one hits L2/L1):
//   pass 1  finds the VALUE of the (k-1)-th best score.  The warp streams the row with
//           coalesced 16-byte loads and filters on the fp32 score against the current
//           (k-1)-th best; survivors are turned into order-preserving 32-bit keys, compacted
//           into a shared staging buffer with a ballot, and merged 32 at a time into the
//           sorted kept set (registers, bitonic networks on 32-bit keys).
//   pass 2  takes every block whose key beats the threshold plus, among the blocks that tie
//           with it, the first ones in index order until k-1 are taken.  It reads the log of
//           pass-1 survivors (shared memory, in block order), which contains every selected
//           block; only rows with more survivors than the log holds are walked a second time.
//           Index order makes the output list ascending with no final sort; the local block
//           is appended by construction (never ranked).
#pragma once

#include "common.cuh"
#include "generic.cuh"

namespace msa {

// Order-preserving 32-bit image of an fp32 score (-0 and +0 map to the same key).
__device__ __forceinline__ uint32_t topk_key(float s) {
    s += 0.0f;
    const uint32_t u = __float_as_uint(s);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ float topk_key_score(uint32_t u) {
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u);
}

// One compare-exchange stage of a bitonic network over elements e = slot*32 + lane.
template <int R>
__device__ __forceinline__ void bitonic_stage(uint32_t (&v)[R], int lane, int size, int stride) {
    if (stride < 32) {
#pragma unroll
        for (int s = 0; s < R; ++s) {
            const int e = s * 32 + lane;
            const uint32_t o = __shfl_xor_sync(0xffffffffu, v[s], stride);
            const bool desc = (e & size) == 0;
            const bool lower = (e & stride) == 0;
            v[s] = (lower == desc) ? max(v[s], o) : min(v[s], o);
        }
    } else {
        const int ss = stride >> 5;
#pragma unroll
        for (int s = 0; s < R; ++s) {
            if ((s & ss) == 0) {
                const int p = s | ss;
                const bool desc = ((s * 32) & size) == 0;
                const uint32_t mx = max(v[s], v[p]), mn = min(v[s], v[p]);
                v[s] = desc ? mx : mn;
                v[p] = desc ? mn : mx;
            }
        }
    }
}

// Sorts the 32 keys held one per lane, descending.
__device__ __forceinline__ uint32_t sort32_desc(uint32_t v, int lane) {
    uint32_t a[1] = {v};
#pragma unroll
    for (int size = 2; size <= 32; size <<= 1) {
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) bitonic_stage<1>(a, lane, size, stride);
    }
    return a[0];
}

// kept: 32*R keys sorted descending; nw: 32 keys sorted descending (one per lane).
// kept <- the 32*R largest of the union, sorted descending.
template <int R>
__device__ __forceinline__ void merge_top32(uint32_t (&kept)[R], uint32_t nw, int lane) {
    const uint32_t o = __shfl_sync(0xffffffffu, nw, 31 - lane);
    kept[R - 1] = max(kept[R - 1], o);  // the sequence is now bitonic (down, then up)
#pragma unroll
    for (int stride = 16 * R; stride > 0; stride >>= 1) bitonic_stage<R>(kept, lane, 32 * R, stride);
}

template <int R>
__device__ __forceinline__ uint32_t element_at(const uint32_t (&v)[R], int e) {
    uint32_t t = 0;
#pragma unroll
    for (int s = 0; s < R; ++s)
        if (s == (e >> 5)) t = v[s];
    return __shfl_sync(0xffffffffu, t, e & 31);
}

__device__ __forceinline__ int warp_excl_scan(int v, int lane) {
    int x = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, x, o);
        if (lane >= o) x += y;
    }
    return x - v;
}

constexpr int kTopkWarps = 4;
#ifndef MSA_TOPK_LOADS
#define MSA_TOPK_LOADS 8
#endif
constexpr int kTopkLoads = MSA_TOPK_LOADS;            // coalesced 32-wide loads per round
constexpr int kTopkRound = 32 * kTopkLoads;           // blocks covered by one round
constexpr int kTopkStage = 32 + kTopkRound;           // flush threshold (32) + one round of pushes
constexpr int kTopkLog = 768;    // survivors remembered per row for the index pass

template <int R>
__global__ void __launch_bounds__(kTopkWarps * 32)
topk_select_kernel(const float* __restrict__ scores, int64_t ld_scores, RowMap rows,
                   int64_t n_rows, int H_kv, int B_k, int top_k, int32_t* __restrict__ block_idx) {
    __shared__ uint32_t stg_all[kTopkWarps][kTopkStage];
    __shared__ uint2 log_all[kTopkWarps][kTopkLog];   // (key, block) of every survivor, in index order
    __shared__ int32_t out_all[kTopkWarps][32 * R];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * kTopkWarps + warp;
    if (row >= n_rows) return;
    int64_t pos, len, base;
    rows.get(row / H_kv, pos, len, base);
    const int64_t loc = pos / B_k;
    int32_t* orow = block_idx + row * (int64_t)top_k;

    if (loc <= top_k - 1) {  // every visible block is selected
        for (int e = lane; e < top_k; e += 32) orow[e] = (e <= loc) ? e : -1;
        return;
    }
    const int m = top_k - 1;  // ranked entries; candidates are blocks [0, loc)
    if (m == 0) {
        for (int e = lane; e < top_k; e += 32) orow[e] = (e == 0) ? (int32_t)loc : -1;
        return;
    }
    const float* srow = scores + row * ld_scores;
    uint32_t* stg = stg_all[warp];
    uint2* logb = log_all[warp];
    int32_t* outb = out_all[warp];
    const unsigned lt_mask = (1u << lane) - 1u;

    // ------------------------------------------------------------------ pass 1: threshold value
    // A round covers kTopkRound consecutive blocks as coalesced 32-wide loads, so that compacting
    // the loads one after the other keeps the survivors in block order.
    uint32_t kept[R];
#pragma unroll
    for (int s = 0; s < R; ++s) kept[s] = 0;  // 0 is below every real key
    float tau_f = -INFINITY;                   // score of the current m-th best (strict filter)
    int cnt = 0, n_log = 0;
    bool log_ok = true;

    auto flush = [&](bool all) {
        __syncwarp();
        int done = 0;
        while (cnt - done >= 32 || (all && cnt - done > 0)) {
            const int e = done + lane;
            uint32_t nw = (e < cnt) ? stg[e] : 0u;
            nw = sort32_desc(nw, lane);
            merge_top32<R>(kept, nw, lane);
            done += 32;
        }
        // move the remainder (< 32 keys) to the front
        const int rem = cnt > done ? cnt - done : 0;
        uint32_t carry = 0;
        if (lane < rem) carry = stg[done + lane];
        __syncwarp();
        if (lane < rem) stg[lane] = carry;
        cnt = rem;
        const uint32_t tau = element_at<R>(kept, m - 1);
        tau_f = tau != 0u ? topk_key_score(tau) : -INFINITY;
        __syncwarp();
    };

    {
        constexpr int C = kTopkLoads;
        const int n = (int)loc;  // candidates are blocks [0, n); n < 2^31
        float nxt[C];
#pragma unroll
        for (int c = 0; c < C; ++c) {
            const int i = c * 32 + lane;
            nxt[c] = i < n ? __ldg(srow + i) : -INFINITY;
        }
        for (int i0 = 0; i0 < n; i0 += kTopkRound) {
            float x[C];
#pragma unroll
            for (int c = 0; c < C; ++c) x[c] = nxt[c];
#pragma unroll
            for (int c = 0; c < C; ++c) {  // next round's loads are in flight while this one is ranked
                const int i = i0 + kTopkRound + c * 32 + lane;
                nxt[c] = i < n ? __ldg(srow + i) : -INFINITY;
            }
            // While fewer than m keys are kept everything passes; afterwards only strictly better
            // scores can change the m-th best value.  (Out-of-range lanes hold -inf.)
            unsigned mk[C];
            unsigned any = 0u;
            if (tau_f == -INFINITY) {
#pragma unroll
                for (int c = 0; c < C; ++c) mk[c] = __ballot_sync(0xffffffffu, i0 + c * 32 + lane < n);
            } else {
#pragma unroll
                for (int c = 0; c < C; ++c) mk[c] = __ballot_sync(0xffffffffu, x[c] > tau_f);
            }
#pragma unroll
            for (int c = 0; c < C; ++c) any |= mk[c];
            if (any == 0u) continue;
            // survivors keep block order: component 0's lanes first, then component 1's, ...
            int off[C + 1];
            off[0] = 0;
#pragma unroll
            for (int c = 0; c < C; ++c) off[c + 1] = off[c] + __popc(mk[c]);
            const int tot = off[C];
            if (log_ok && n_log + tot > kTopkLog) log_ok = false;
#pragma unroll
            for (int c = 0; c < C; ++c) {
                if (mk[c] & (1u << lane)) {
                    const int rnk = off[c] + __popc(mk[c] & lt_mask);
                    const uint32_t key = topk_key(x[c]);
                    stg[cnt + rnk] = key;
                    if (log_ok) logb[n_log + rnk] = make_uint2(key, (uint32_t)(i0 + c * 32 + lane));
                }
            }
            cnt += tot;
            n_log += tot;
            if (cnt >= 32) flush(false);
        }
        flush(true);
    }
    const uint32_t tau = element_at<R>(kept, m - 1);  // key of the m-th best score (loc > m, so it exists)
    int n_gt = 0;                                      // kept keys strictly above the threshold
#pragma unroll
    for (int s = 0; s < R; ++s) n_gt += __popc(__ballot_sync(0xffffffffu, (s * 32 + lane) < m && kept[s] > tau));
    const int need_ties = m - n_gt;                    // blocks equal to the threshold still to take

    // ------------------------------------------------------------------ pass 2: indices, ascending
    // Every selected block survived the filter when it was seen (its score beat the threshold
    // of that moment), so the log holds them all, in block order; ties with the final threshold
    // are taken first come, first served.  Only a row with more survivors than the log holds
    // is walked a second time.
    int out_cnt = 0, ties_seen = 0;
    auto take_in_order = [&](uint32_t key, uint32_t blk, bool in) {
        const bool gt = in && key > tau, eq = in && key == tau;
        const unsigned eqm = __ballot_sync(0xffffffffu, eq);
        bool take = gt;
        if (eqm != 0u) {
            take = take || (eq && (ties_seen + __popc(eqm & lt_mask)) < need_ties);
            ties_seen += __popc(eqm);
        }
        const unsigned tm = __ballot_sync(0xffffffffu, take);
        if (take) {
            const int w = out_cnt + __popc(tm & lt_mask);
            if (w < m) outb[w] = (int32_t)blk;
        }
        out_cnt += __popc(tm);
    };
    if (log_ok) {
        for (int e0 = 0; e0 < n_log && out_cnt < m; e0 += 32) {
            const int e = e0 + lane;
            uint2 kv = make_uint2(0u, 0u);
            if (e < n_log) kv = logb[e];
            take_in_order(kv.x, kv.y, e < n_log);
        }
    } else {
        for (int64_t i0 = 0; i0 < loc && out_cnt < m; i0 += 32) {
            const int64_t i = i0 + lane;
            const float x = i < loc ? __ldg(srow + i) : 0.f;
            take_in_order(topk_key(x), (uint32_t)i, i < loc);
        }
    }
    __syncwarp();
    for (int e = lane; e < top_k; e += 32) orow[e] = e < m ? outb[e] : (e == m ? (int32_t)loc : -1);
}

}  // namespace msa
