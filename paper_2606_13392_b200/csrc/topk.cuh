// Eq. 7 + Local Block rule: exp-free Top-k over raw block scores, one warp per row.
//
// Ranking key = (order-preserving image of the fp32 score) << 32 | ~block, so one 64-bit
// compare realises "score descending, then block index ascending" and keys are unique.
// The warp streams the row with coalesced 16-byte loads, keeps the best k-1 keys sorted
// across its registers, and filters new elements against the current (k-1)-th best key;
// survivors are compacted into a shared-memory staging buffer with a ballot and merged in
// batches by a register bitonic network.  The local block is never ranked: it is appended
// by construction.  The final list is sorted by block index and written with one
// coalesced store per row.
#pragma once

#include "common.cuh"
#include "generic.cuh"

namespace msa {

__device__ __forceinline__ uint64_t topk_key(float s, uint32_t block) {
    s += 0.0f;  // -0 -> +0 so that equal scores compare equal
    uint32_t u = __float_as_uint(s);
    u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    return ((uint64_t)u << 32) | (uint32_t)(~block);
}

// Score part of a key, back as a float (inverse of the order-preserving image).
__device__ __forceinline__ float topk_key_score(uint64_t key) {
    const uint32_t u = (uint32_t)(key >> 32);
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u);
}

__device__ __forceinline__ uint64_t shfl_xor_u64(uint64_t v, int m) {
    return __shfl_xor_sync(0xffffffffu, v, m);
}

// One compare-exchange stage of a bitonic network over elements e = slot*32 + lane.
template <int R>
__device__ __forceinline__ void bitonic_stage(uint64_t (&v)[R], int lane, int size, int stride) {
    if (stride < 32) {
#pragma unroll
        for (int s = 0; s < R; ++s) {
            const int e = s * 32 + lane;
            const uint64_t o = shfl_xor_u64(v[s], stride);
            const bool desc = (e & size) == 0;
            const bool lower = (e & stride) == 0;
            const bool gt = v[s] > o;
            const uint64_t mx = gt ? v[s] : o, mn = gt ? o : v[s];
            v[s] = (lower == desc) ? mx : mn;
        }
    } else {
        const int ss = stride >> 5;
#pragma unroll
        for (int s = 0; s < R; ++s) {
            if ((s & ss) == 0) {
                const int p = s | ss;
                const bool desc = ((s * 32) & size) == 0;
                const bool gt = v[s] > v[p];
                const uint64_t mx = gt ? v[s] : v[p], mn = gt ? v[p] : v[s];
                v[s] = desc ? mx : mn;
                v[p] = desc ? mn : mx;
            }
        }
    }
}

template <int R>
__device__ __forceinline__ void bitonic_sort_desc(uint64_t (&v)[R], int lane) {
#pragma unroll
    for (int size = 2; size <= 32 * R; size <<= 1) {
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) bitonic_stage<R>(v, lane, size, stride);
    }
}

// kept, nw: both sorted descending.  kept <- the 32*R largest of the union, sorted descending.
template <int R>
__device__ __forceinline__ void merge_top(uint64_t (&kept)[R], const uint64_t (&nw)[R], int lane) {
#pragma unroll
    for (int s = 0; s < R; ++s) {
        const uint64_t o = __shfl_sync(0xffffffffu, nw[R - 1 - s], 31 - lane);
        kept[s] = kept[s] > o ? kept[s] : o;
    }
#pragma unroll
    for (int stride = 16 * R; stride > 0; stride >>= 1) bitonic_stage<R>(kept, lane, 32 * R, stride);
}

template <int R>
__device__ __forceinline__ uint64_t element_at(const uint64_t (&v)[R], int e) {
    uint64_t t = 0;
#pragma unroll
    for (int s = 0; s < R; ++s)
        if (s == (e >> 5)) t = v[s];
    return __shfl_sync(0xffffffffu, t, e & 31);
}

constexpr int kTopkWarps = 8;

template <int R>
__global__ void __launch_bounds__(kTopkWarps * 32)
topk_select_kernel(const float* __restrict__ scores, int64_t ld_scores, RowMap rows,
                   int64_t n_rows, int H_kv, int B_k, int top_k, int32_t* __restrict__ block_idx) {
    constexpr int KCAP = 32 * R;
    constexpr int STG = 160;  // flush threshold (32) + one round of four pushes (4 x 32)
    __shared__ uint64_t stg_all[kTopkWarps][STG];
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
    const float* srow = scores + row * ld_scores;
    uint64_t* stg = stg_all[warp];
    const unsigned lt_mask = (1u << lane) - 1u;

    uint64_t kept[R];
#pragma unroll
    for (int s = 0; s < R; ++s) kept[s] = 0;  // 0 is below every real key
    // The stream is filtered on the fp32 score alone (score >= score of the current (k-1)-th
    // best, -inf while fewer than k-1 are kept); the 64-bit key is only built for survivors and
    // the exact order, ties included, is settled in the merges.
    float tau_f = -INFINITY;
    int cnt = 0;

    auto flush = [&]() {
        __syncwarp();
        for (int b0 = 0; b0 < cnt; b0 += KCAP) {
            uint64_t nw[R];
#pragma unroll
            for (int s = 0; s < R; ++s) {
                const int e = b0 + s * 32 + lane;
                nw[s] = (e < cnt) ? stg[e] : 0;
            }
            bitonic_sort_desc<R>(nw, lane);
            merge_top<R>(kept, nw, lane);
        }
        cnt = 0;
        const uint64_t tau = element_at<R>(kept, m - 1);
        tau_f = tau != 0 ? topk_key_score(tau) : -INFINITY;
        __syncwarp();
    };
    // Appends the passing lanes' keys to the staging buffer (no flush inside: the buffer has
    // room for a whole round of four pushes beyond the flush threshold).
    auto push = [&](float x, uint32_t block, bool pass) {
        const unsigned mask = __ballot_sync(0xffffffffu, pass);
        if (pass) stg[cnt + __popc(mask & lt_mask)] = topk_key(x, block);
        cnt += __popc(mask);
    };

    const int64_t n4 = loc >> 2;
    const float4* srow4 = reinterpret_cast<const float4*>(srow);
    float4 nxt = make_float4(0.f, 0.f, 0.f, 0.f);
    if (lane < n4) nxt = __ldg(srow4 + lane);
    for (int64_t v0 = 0; v0 < n4; v0 += 32) {
        const int64_t vi = v0 + lane;
        const bool in = vi < n4;
        const float4 x = nxt;
        if (vi + 32 < n4) nxt = __ldg(srow4 + vi + 32);  // next round's load is in flight while this one is ranked
        const bool p0 = in && x.x >= tau_f, p1 = in && x.y >= tau_f;
        const bool p2 = in && x.z >= tau_f, p3 = in && x.w >= tau_f;
        if (__ballot_sync(0xffffffffu, p0 | p1 | p2 | p3) == 0u) continue;
        const uint32_t b0 = (uint32_t)(vi << 2);
        push(x.x, b0, p0);
        push(x.y, b0 + 1, p1);
        push(x.z, b0 + 2, p2);
        push(x.w, b0 + 3, p3);
        if (cnt > 32) flush();
    }
    {
        const int64_t idx = (n4 << 2) + lane;  // scalar tail (< 4 elements)
        const bool in = idx < loc;
        const float x = in ? __ldg(srow + idx) : 0.f;
        push(x, (uint32_t)idx, in && x >= tau_f);
    }
    if (cnt > 0) flush();

    // kept[0..m) are the winners.  Re-key by block index, add the local block, sort ascending.
    uint64_t fin[R];
#pragma unroll
    for (int s = 0; s < R; ++s) {
        const int e = s * 32 + lane;
        const uint32_t inv_block = (uint32_t)kept[s];
        fin[s] = (e < m) ? (uint64_t)inv_block : (e == m ? (uint64_t)(uint32_t)(~(uint32_t)loc) : 0ull);
    }
    bitonic_sort_desc<R>(fin, lane);
#pragma unroll
    for (int s = 0; s < R; ++s) {
        const int e = s * 32 + lane;
        if (e < top_k) orow[e] = (int32_t)(~(uint32_t)fin[s]);
    }
}

}  // namespace msa
