// Eq. 7 + Local Block rule: exp-free Top-k over raw block scores, one warp per row.
//
// Ranking order is "score descending, then block index ascending".  The kernel works in two
// passes over the row (the second one hits L2/L1):
//   pass 1  finds the VALUE of the (k-1)-th best score.  The warp streams the row with
//           coalesced 16-byte loads and filters on the fp32 score against the current
//           (k-1)-th best; survivors are turned into order-preserving 32-bit keys, compacted
//           into a shared staging buffer with a ballot, and merged 32 at a time into the
//           sorted kept set (registers, bitonic networks on 32-bit keys).
//   pass 2  walks the row again in index order and takes every block whose key beats the
//           threshold plus, among the blocks that tie with it, the first ones in index order
//           until k-1 are taken.  Walking in index order makes the output list ascending with
//           no final sort; the local block is appended by construction (never ranked).
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

constexpr int kTopkWarps = 8;
constexpr int kTopkStage = 160;  // flush threshold (32) + one round of four pushes (4 x 32)

template <int R>
__global__ void __launch_bounds__(kTopkWarps * 32)
topk_select_kernel(const float* __restrict__ scores, int64_t ld_scores, RowMap rows,
                   int64_t n_rows, int H_kv, int B_k, int top_k, int32_t* __restrict__ block_idx) {
    __shared__ uint32_t stg_all[kTopkWarps][kTopkStage];
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
    int32_t* outb = out_all[warp];
    const unsigned lt_mask = (1u << lane) - 1u;
    const int64_t n4 = loc >> 2;
    const float4* srow4 = reinterpret_cast<const float4*>(srow);

    // ------------------------------------------------------------------ pass 1: threshold value
    uint32_t kept[R];
#pragma unroll
    for (int s = 0; s < R; ++s) kept[s] = 0;  // 0 is below every real key
    float tau_f = -INFINITY;                   // score of the current m-th best (strict filter)
    int cnt = 0;

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
    auto push = [&](float x, bool pass) {
        const unsigned mask = __ballot_sync(0xffffffffu, pass);
        if (pass) stg[cnt + __popc(mask & lt_mask)] = topk_key(x);
        cnt += __popc(mask);
    };

    {
        float4 nxt = make_float4(0.f, 0.f, 0.f, 0.f);
        if (lane < n4) nxt = __ldg(srow4 + lane);
        for (int64_t v0 = 0; v0 < n4; v0 += 32) {
            const int64_t vi = v0 + lane;
            const bool in = vi < n4;
            const float4 x = nxt;
            if (vi + 32 < n4) nxt = __ldg(srow4 + vi + 32);  // next round's load is in flight meanwhile
            // While fewer than m keys are kept everything passes; afterwards only strictly better
            // scores can change the m-th best value.
            const bool warm = tau_f == -INFINITY;
            const bool p0 = in && (warm || x.x > tau_f), p1 = in && (warm || x.y > tau_f);
            const bool p2 = in && (warm || x.z > tau_f), p3 = in && (warm || x.w > tau_f);
            if (__ballot_sync(0xffffffffu, p0 | p1 | p2 | p3) == 0u) continue;
            push(x.x, p0);
            push(x.y, p1);
            push(x.z, p2);
            push(x.w, p3);
            if (cnt >= 32) flush(false);
        }
        const int64_t idx = (n4 << 2) + lane;  // scalar tail (< 4 elements)
        const bool in = idx < loc;
        const float x = in ? __ldg(srow + idx) : 0.f;
        push(x, in && (tau_f == -INFINITY || x > tau_f));
        flush(true);
    }
    const uint32_t tau = element_at<R>(kept, m - 1);  // key of the m-th best score (loc > m, so it exists)
    int n_gt = 0;                                      // kept keys strictly above the threshold
#pragma unroll
    for (int s = 0; s < R; ++s) n_gt += __popc(__ballot_sync(0xffffffffu, (s * 32 + lane) < m && kept[s] > tau));
    const int need_ties = m - n_gt;                    // blocks equal to the threshold still to take

    // ------------------------------------------------------------------ pass 2: indices, ascending
    int out_cnt = 0, ties_seen = 0;
    for (int64_t v0 = 0; v0 < n4 + 1 && out_cnt < m; v0 += 32) {
        const int64_t vi = v0 + lane;
        float xs[4] = {0.f, 0.f, 0.f, 0.f};
        int n_in = 0;  // valid components of this lane
        if (vi < n4) {
            const float4 x = __ldg(srow4 + vi);
            xs[0] = x.x; xs[1] = x.y; xs[2] = x.z; xs[3] = x.w;
            n_in = 4;
        } else if (vi == n4) {  // the < 4 tail elements
            n_in = (int)(loc - (n4 << 2));
#pragma unroll
            for (int c = 0; c < 3; ++c)
                if (c < n_in) xs[c] = __ldg(srow + (n4 << 2) + c);
        }
        unsigned gt = 0, eq = 0;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const uint32_t key = topk_key(xs[c]);
            if (c < n_in && key > tau) gt |= 1u << c;
            if (c < n_in && key == tau) eq |= 1u << c;
        }
        if (__ballot_sync(0xffffffffu, (gt | eq) != 0u) == 0u) continue;
        unsigned take = gt;
        if (__ballot_sync(0xffffffffu, eq != 0u) != 0u) {  // ties: first ones in index order
            const int ne = __popc(eq);
            int rank = ties_seen + warp_excl_scan(ne, lane);
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (eq & (1u << c)) {
                    if (rank < need_ties) take |= 1u << c;
                    ++rank;
                }
            ties_seen = __shfl_sync(0xffffffffu, rank, 31);  // lane 31 ends at the running total
        }
        const int nt = __popc(take);
        int w = out_cnt + warp_excl_scan(nt, lane);
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (take & (1u << c)) {
                if (w < m) outb[w] = (int32_t)((vi << 2) + c);
                ++w;
            }
        out_cnt = __shfl_sync(0xffffffffu, w, 31);
    }
    __syncwarp();
    for (int e = lane; e < top_k; e += 32) orow[e] = e < m ? outb[e] : (e == m ? (int32_t)loc : -1);
}

}  // namespace msa
