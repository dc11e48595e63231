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
// Both passes are written over a "stream" (elements in ascending block order); long rows run them
// twice, on the maxima of runs of 8 blocks and then on the blocks of the runs that matter (see
// "two-level selection" below).
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
// The kernel waits for memory more than for anything else: nine CTAs per SM (56 registers, 14 KB of shared
// memory each, which also leaves the SM most of its array as L1 for the second look at the candidate runs).
constexpr int kTopkMinCtas = 9;
#ifndef MSA_TOPK_LOADS
#define MSA_TOPK_LOADS 4
#endif
constexpr int kTopkLoads = MSA_TOPK_LOADS;            // coalesced 32-wide loads per round
constexpr int kTopkRound = 32 * kTopkLoads;           // blocks covered by one round
constexpr int kTopkStage = 32 + kTopkRound;           // flush threshold (32) + one round of pushes
constexpr int kTopkLog = 256;    // survivors remembered per row for the index pass (a row with more is walked a second time)    // survivors remembered per row for the index pass
constexpr int kTopkRunBlocks = 8;       // two-level selection: blocks per run
#ifndef MSA_TOPK_RUNLOADS
#define MSA_TOPK_RUNLOADS 4
#endif
constexpr int kTopkRunLoads = MSA_TOPK_RUNLOADS;  // two-level selection: runs per lane and round of the run-maxima pass
constexpr int kTopkTau0Slack = 4;       // two-level selection: candidate runs accepted beyond the m needed
constexpr int kTopkMaxRuns = 1024;     // two-level selection: rows of up to 8192 blocks (their run maxima wait in shared memory)
// Candidate runs listed per row (a row with more - ties by the hundred - takes one level).  The list is kept
// short on purpose: with room for all kTopkMaxRuns runs the kernel needed 28 KB of shared memory per CTA and 71
// registers, seven CTAs per SM; with this list it is 22 KB and 64 registers, eight CTAs, and 0.219 instead of
// 0.280 ms on 8192 rows of up to 8192 scores.
constexpr int kTopkMaxCand = 254;

// A row as the selection sees it: element i of n has a score and a block index; the elements come
// in ascending block order.
struct TopkPlainStream {            // blocks [0, n) of a score row
    const float* srow;
    int n;
    int lnb;
    __device__ __forceinline__ float score(int i) const { return i < n ? __ldg(srow + score_slot(i, lnb)) : -INFINITY; }
    __device__ __forceinline__ bool in(int i) const { return i < n; }
    __device__ __forceinline__ uint32_t block(int i) const { return (uint32_t)i; }
};

// Per-warp scratch of the selection.
struct TopkScratch {
    uint32_t* stg;   // [kTopkStage] survivors waiting to be merged
    uint2* logb;     // [log_cap] (key, block) of every survivor, in block order
    int log_cap;
};

// Pass 1: the sorted keys of the m best scores of the stream (kept), a log of every element that
// passed the filter when it was seen (all selected blocks are among them), its length, and
// whether the log holds them all.  floor_f: a score strictly below every score that may be
// selected (-inf if none is known); only elements above it are looked at.
template <int R, class Stream>
__device__ __forceinline__ void topk_pass1(const Stream& st, int m, float floor_f, const TopkScratch& sc,
                                           uint32_t (&kept)[R], int& n_log, bool& log_ok, int lane) {
    const unsigned lt_mask = (1u << lane) - 1u;
    uint32_t* stg = sc.stg;
    uint2* logb = sc.logb;
#pragma unroll
    for (int s = 0; s < R; ++s) kept[s] = 0;  // 0 is below every real key
    float tau_f = floor_f;                     // strict filter: the current m-th best, or the floor
    int cnt = 0;
    n_log = 0;
    log_ok = true;

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
        const float t_kept = tau != 0u ? topk_key_score(tau) : -INFINITY;
        tau_f = fmaxf(t_kept, floor_f);
        __syncwarp();
    };

    constexpr int C = kTopkLoads;
    const int n = st.n;
    float nxt[C];
#pragma unroll
    for (int c = 0; c < C; ++c) nxt[c] = st.score(c * 32 + lane);
    // A round covers kTopkRound consecutive elements as coalesced 32-wide loads, so that compacting
    // the loads one after the other keeps the survivors in block order.
    for (int i0 = 0; i0 < n; i0 += kTopkRound) {
        float x[C];
#pragma unroll
        for (int c = 0; c < C; ++c) x[c] = nxt[c];
#pragma unroll
        for (int c = 0; c < C; ++c)  // next round's loads are in flight while this one is ranked
            nxt[c] = st.score(i0 + kTopkRound + c * 32 + lane);
        // While fewer than m keys are kept (and no floor is known) everything passes; afterwards
        // only strictly better scores can change the m-th best value.
        unsigned mk[C];
        unsigned any = 0u;
        if (tau_f == -INFINITY) {
#pragma unroll
            for (int c = 0; c < C; ++c) mk[c] = __ballot_sync(0xffffffffu, st.in(i0 + c * 32 + lane));
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
        if (log_ok && n_log + tot > sc.log_cap) log_ok = false;
#pragma unroll
        for (int c = 0; c < C; ++c) {
            if (mk[c] & (1u << lane)) {
                const int rnk = off[c] + __popc(mk[c] & lt_mask);
                const uint32_t key = topk_key(x[c]);
                stg[cnt + rnk] = key;
                if (log_ok) logb[n_log + rnk] = make_uint2(key, st.block(i0 + c * 32 + lane));
            }
        }
        cnt += tot;
        n_log += tot;
        if (cnt >= 32) flush(false);
    }
    flush(true);
}

// Pass 2: every block whose key beats the threshold plus, among the blocks that tie with it, the
// first ones in block order until m are taken; written ascending to outb[0..m).  Every selected
// block survived the filter when it was seen (its score beat the threshold of that moment), so
// the log holds them all, in block order; only a row with more survivors than the log holds is
// walked a second time.
template <int R, class Stream>
__device__ __forceinline__ void topk_pass2(const Stream& st, int m, const TopkScratch& sc,
                                           const uint32_t (&kept)[R], int n_log, bool log_ok, int32_t* outb,
                                           int lane) {
    const unsigned lt_mask = (1u << lane) - 1u;
    const uint32_t tau = element_at<R>(kept, m - 1);  // key of the m-th best score (the stream has more than m elements)
    int n_gt = 0;                                      // kept keys strictly above the threshold
#pragma unroll
    for (int s = 0; s < R; ++s) n_gt += __popc(__ballot_sync(0xffffffffu, (s * 32 + lane) < m && kept[s] > tau));
    const int need_ties = m - n_gt;                    // blocks equal to the threshold still to take
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
            if (e < n_log) kv = sc.logb[e];
            take_in_order(kv.x, kv.y, e < n_log);
        }
    } else {
        for (int i0 = 0; i0 < st.n && out_cnt < m; i0 += 32) {
            const int i = i0 + lane;
            const bool in = st.in(i);
            const float x = in ? st.score(i) : 0.f;
            take_in_order(topk_key(x), st.block(i), in);
        }
    }
    __syncwarp();
}

// The selection once the threshold key is known: from a list of (key, block) in block order that
// holds every block that can be selected, the blocks above the threshold and the first need_ties
// blocks that equal it, written ascending to outb[0..m).
__device__ __forceinline__ void topk_take_listed(const uint2* lst, int n_lst, uint32_t tau, int need_ties, int m,
                                                 int32_t* outb, int lane) {
    const unsigned lt_mask = (1u << lane) - 1u;
    int out_cnt = 0, ties_seen = 0;
    for (int e0 = 0; e0 < n_lst && out_cnt < m; e0 += 32) {
        const int e = e0 + lane;
        uint2 kv = make_uint2(0u, 0u);
        if (e < n_lst) kv = lst[e];
        const bool gt = e < n_lst && kv.x > tau, eq = e < n_lst && kv.x == tau;
        const unsigned eqm = __ballot_sync(0xffffffffu, eq);
        bool take = gt;
        if (eqm != 0u) {
            take = take || (eq && (ties_seen + __popc(eqm & lt_mask)) < need_ties);
            ties_seen += __popc(eqm);
        }
        const unsigned tm = __ballot_sync(0xffffffffu, take);
        if (take) {
            const int w = out_cnt + __popc(tm & lt_mask);
            if (w < m) outb[w] = (int32_t)kv.y;
        }
        out_cnt += __popc(tm);
    }
    __syncwarp();
}

// Step 3 of the two-level selection when few blocks reach tau0 (the usual case: the m run maxima
// that define tau0 and a handful of second-best blocks).  Every lane loads whole candidate runs
// (32 bytes each), the blocks that reach tau0 are listed in block order, and the threshold - the
// m-th largest of the n listed keys - is found by taking away the n - m smallest, one warp-wide
// minimum at a time.  Returns false (nothing written) when more than kTopkListMax blocks reach
// tau0 or more than kTopkDropMax would have to go; the caller then ranks the candidates' blocks
// with the two general passes.  LNB: the order of the blocks inside a run (score_slot).
constexpr int kTopkListMax = 128;
constexpr int kTopkDropMax = 32;

template <int LNB>
__device__ __forceinline__ bool topk_few_above(const float* srow, const uint16_t* run, int n_run, int loc, float tau0,
                                               int m, uint2* lst, int32_t* outb, int lane) {
    int n_lst = 0;
    for (int c0 = 0; c0 < n_run; c0 += 32) {
        const int c = c0 + lane;
        const bool have = c < n_run;
        const int g = have ? (int)run[c] : 0;
        float x[8];
        {
            const float4* p = reinterpret_cast<const float4*>(srow) + 2 * g;
            const float4 a = have ? __ldg(p) : make_float4(0.f, 0.f, 0.f, 0.f);
            const float4 b = have ? __ldg(p + 1) : make_float4(0.f, 0.f, 0.f, 0.f);
            const float y[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
            for (int w = 0; w < 8; ++w) x[w] = y[score_slot(w, LNB)];  // block order
        }
        unsigned mine = 0u;  // bit w: block 8 g + w reaches tau0 and may rank (it lies before the local block)
#pragma unroll
        for (int w = 0; w < 8; ++w)
            if (have && g * kTopkRunBlocks + w < loc && x[w] >= tau0) mine |= 1u << w;
        const int cnt = __popc(mine);
        const int before = warp_excl_scan(cnt, lane);
        const int total = __shfl_sync(0xffffffffu, before + cnt, 31);
        if (n_lst + total > kTopkListMax) return false;
        int at = n_lst + before;
#pragma unroll
        for (int w = 0; w < 8; ++w)
            if (mine & (1u << w)) lst[at++] = make_uint2(topk_key(x[w]), (uint32_t)(g * kTopkRunBlocks + w));
        n_lst += total;
    }
    const int drop = n_lst - m;  // >= 0: m different runs reach tau0
    if (drop > kTopkDropMax || drop < 0) return false;
    __syncwarp();
    uint32_t sv[kTopkListMax / 32];
#pragma unroll
    for (int j = 0; j < kTopkListMax / 32; ++j) sv[j] = (j * 32 + lane < n_lst) ? lst[j * 32 + lane].x : 0xFFFFFFFFu;
    uint32_t tau = 0u;
    for (int it = 0; it <= drop; ++it) {
        uint32_t lmin = sv[0];
#pragma unroll
        for (int j = 1; j < kTopkListMax / 32; ++j) lmin = min(lmin, sv[j]);
        const uint32_t wmin = __reduce_min_sync(0xffffffffu, lmin);
        tau = wmin;
        if (it == drop) break;
        const unsigned holders = __ballot_sync(0xffffffffu, lmin == wmin);
        if (lane == __ffs(holders) - 1) {  // one copy of the minimum goes
            bool gone = false;
#pragma unroll
            for (int j = 0; j < kTopkListMax / 32; ++j)
                if (!gone && sv[j] == wmin) { sv[j] = 0xFFFFFFFFu; gone = true; }
        }
    }
    // tau is the m-th largest key; what is left in sv besides the removed ones is >= tau
    int n_gt = 0;
#pragma unroll
    for (int j = 0; j < kTopkListMax / 32; ++j)
        n_gt += __popc(__ballot_sync(0xffffffffu, sv[j] != 0xFFFFFFFFu && sv[j] > tau));
    topk_take_listed(lst, n_lst, tau, m - n_gt, m, outb, lane);
    return true;
}

// Rows with at most top_k visible blocks, or top_k = 1: no ranking.  Returns true if the row is done.
__device__ __forceinline__ bool topk_trivial_row(int64_t loc, int top_k, int32_t* orow, int lane) {
    if (loc <= top_k - 1) {  // every visible block is selected
        for (int e = lane; e < top_k; e += 32) orow[e] = (e <= loc) ? e : -1;
        return true;
    }
    if (top_k == 1) {
        for (int e = lane; e < top_k; e += 32) orow[e] = (e == 0) ? (int32_t)loc : -1;
        return true;
    }
    return false;
}

// ------------------------------------------------------------------ two-level selection (long rows)
// A long row is selected in three steps, the last two of which touch a fraction of it:
//   1. tau0 = a value that the maxima of at least m runs of kTopkRunBlocks consecutive blocks reach
//      (runs that lie wholly before the local block): m different blocks score at least tau0, so
//      the m-th best block score is at least tau0 (one streaming pass, 8 scores per lane and load
//      pair, no merge networks);
//   2. the candidate runs - those whose maximum reaches tau0, plus the run that holds the local
//      block - are listed in ascending order (every selected block is in one of them);
//   3. the blocks of the candidate runs form a stream in block order, and the two passes above
//      select from it exactly what they would select from the whole row, ties included.
// The merge networks, which dominate a one-level selection, then run on about a third of the
// survivors (run maxima first, then the few blocks above tau0).

struct TopkRunMaxStream {  // element i: maximum of blocks [8i, 8i+8), in either order of a run; rows are 16-byte aligned
    const float* srow;
    int n;
    __device__ __forceinline__ float score(int i) const {
        if (i >= n) return -INFINITY;
        const float4* p = reinterpret_cast<const float4*>(srow) + 2 * i;
        const float4 a = __ldg(p), b = __ldg(p + 1);
        return max3(max3(a.x, a.y, a.z), max3(a.w, b.x, b.y), fmaxf(b.z, b.w));
    }
    __device__ __forceinline__ bool in(int i) const { return i < n; }
    __device__ __forceinline__ uint32_t block(int i) const { return (uint32_t)i; }
};

struct TopkGatherStream {  // element i: block i % 8 of candidate run i / 8; blocks from loc on do not rank
    const float* srow;
    const uint16_t* run;   // candidate runs, ascending
    int n;                 // 8 * number of candidate runs
    int loc;
    int lnb;
    __device__ __forceinline__ uint32_t block(int i) const {
        return (uint32_t)run[i >> 3] * kTopkRunBlocks + (uint32_t)(i & 7);
    }
    __device__ __forceinline__ bool in(int i) const { return i < n && (int)block(i) < loc; }
    __device__ __forceinline__ float score(int i) const { return in(i) ? __ldg(srow + score_slot((int)block(i), lnb)) : -INFINITY; }
};

template <int R>
__global__ void __launch_bounds__(kTopkWarps * 32, kTopkMinCtas)
topk_select_kernel(const float* __restrict__ scores, int64_t ld_scores, RowMap rows,
                   int64_t n_rows, int H_kv, int B_k, int top_k, int32_t* __restrict__ block_idx, int* status,
                   int lnb) {
    __shared__ uint32_t stg_all[kTopkWarps][kTopkStage];
    __shared__ uint2 log_all[kTopkWarps][kTopkLog];   // (key, block) of every survivor, in index order
    __shared__ uint16_t run_all[kTopkWarps][kTopkMaxCand + 2];
    __shared__ int32_t out_all[kTopkWarps][32 * R];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * kTopkWarps + warp;
    if (row >= n_rows) return;
    int64_t pos, len, base;
    rows.get(row / H_kv, pos, len, base);
    const int64_t loc = pos / B_k;
    int32_t* orow = block_idx + row * (int64_t)top_k;
    if (loc >= ld_scores) {  // a decode row whose length (a device value) exceeds the score pitch: nothing is read
        if (lane == 0) report_async(status, kAsyncBadIndex, 0x201);
        for (int e = lane; e < top_k; e += 32) orow[e] = -1;
        return;
    }
    if (topk_trivial_row(loc, top_k, orow, lane)) return;
    const int m = top_k - 1;  // ranked entries; candidates are blocks [0, loc), loc < 2^31
    const float* srow = scores + row * ld_scores;
    const TopkScratch sc{stg_all[warp], log_all[warp], kTopkLog};
    int32_t* outb = out_all[warp];
    uint32_t kept[R];
    int n_log;
    bool log_ok;
    const int64_t n_full = loc / kTopkRunBlocks;  // runs wholly before the local block
    // Rows of fewer than 2 m runs can still take two levels when their runs are split into halves or
    // quarters for the threshold (4 or 2 blocks each): 2 m such groups make the threshold tight enough.
    const int sub = n_full >= 2 * m ? 1 : (2 * n_full >= 2 * m ? 2 : (4 * n_full >= 2 * m ? 4 : 0));
    auto one_level = [&]() {
        const TopkPlainStream st{srow, (int)loc, lnb};
        topk_pass1<R>(st, m, -INFINITY, sc, kept, n_log, log_ok, lane);
        topk_pass2<R>(st, m, sc, kept, n_log, log_ok, outb, lane);
    };
    if (sub == 0 || n_full > kTopkMaxRuns) {  // short row (or one beyond the run-maxima array): one level
        one_level();
    } else {
        // 1. A threshold from the run maxima.  Any value that m run maxima reach will do, so no exact
        // selection: every lane keeps the S = 2R largest of the maxima it sees (sorted registers, no
        // branches), and tau0 is a value that m to m + kTopkTau0Slack of the 32 S kept values - maxima
        // of different runs - reach, found by bisection (close to the m-th largest run maximum unless
        // one lane saw more than S of the m largest, and then a little lower).
        const TopkRunMaxStream rs{srow, (int)n_full};
        constexpr int S = 2 * R;
        float top[S];
#pragma unroll
        for (int i = 0; i < S; ++i) top[i] = -INFINITY;
        // The run maxima wait for step 2 in shared memory rounded UP to bf16 (half the room): step 2 only asks
        // whether a run can hold a block that reaches tau0, and a run listed in vain adds no block to step 3.
        __nv_bfloat16* runmax = reinterpret_cast<__nv_bfloat16*>(log_all[warp]);  // the log is not in use before step 3
        static_assert(kTopkLog * sizeof(uint2) >= kTopkMaxRuns * sizeof(__nv_bfloat16), "run maxima share the log");
        auto keep = [&](float v) {  // top[] <- the S largest of top[] and v, sorted
#pragma unroll
            for (int i = 0; i < S; ++i) {
                const float hi = fmaxf(top[i], v);
                v = fminf(top[i], v);
                top[i] = hi;
            }
        };
        if (sub != 1) {
            // fewer than 2 m <= 64 R runs, i.e. at most 2 R per lane: all loads first, then the maxima of the
            // runs (for step 2) and of their halves or quarters (for the threshold)
            float4 a[2 * R], b[2 * R];
#pragma unroll
            for (int u = 0; u < 2 * R; ++u) {
                const int g = u * 32 + lane;
                const float4* pr = reinterpret_cast<const float4*>(srow) + 2 * g;
                a[u] = g < (int)n_full ? __ldg(pr) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
                b[u] = g < (int)n_full ? __ldg(pr + 1) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
            }
#pragma unroll
            for (int u = 0; u < 2 * R; ++u) {
                const int g = u * 32 + lane;
                const float a0 = fmaxf(a[u].x, a[u].y), a1 = fmaxf(a[u].z, a[u].w);
                const float b0 = fmaxf(b[u].x, b[u].y), b1 = fmaxf(b[u].z, b[u].w);
                if (g < (int)n_full) runmax[g] = __float2bfloat16_ru(fmaxf(fmaxf(a0, a1), fmaxf(b0, b1)));
                if (sub == 2) {
                    keep(fmaxf(a0, a1)); keep(fmaxf(b0, b1));
                } else {
                    keep(a0); keep(a1); keep(b0); keep(b1);
                }
            }
        }
        float nx[kTopkRunLoads];
#pragma unroll
        for (int u = 0; u < kTopkRunLoads; ++u) nx[u] = sub == 1 ? rs.score(u * 32 + lane) : -INFINITY;  // -inf beyond n_full
        for (int g0 = 0; sub == 1 && g0 < (int)n_full; g0 += 32 * kTopkRunLoads) {
            float x[kTopkRunLoads];
#pragma unroll
            for (int u = 0; u < kTopkRunLoads; ++u) x[u] = nx[u];
#pragma unroll
            for (int u = 0; u < kTopkRunLoads; ++u) nx[u] = rs.score(g0 + 32 * kTopkRunLoads + u * 32 + lane);  // in flight during the inserts
#pragma unroll
            for (int u = 0; u < kTopkRunLoads; ++u) {
                if (g0 + u * 32 + lane < (int)n_full) runmax[g0 + u * 32 + lane] = __float2bfloat16_ru(x[u]);
                keep(x[u]);
            }
        }
        uint32_t tk[S];
#pragma unroll
        for (int i = 0; i < S; ++i) tk[i] = topk_key(top[i]);
        // Bisection on the key: the largest value found that at least m of the 32 S kept maxima reach
        // (there are at least 2 m real ones), stopping as soon as no more than m + kTopkTau0Slack do.
        uint32_t lo = __reduce_min_sync(0xffffffffu, tk[S - 1]);      // every kept maximum reaches it
        uint32_t hi = __reduce_max_sync(0xffffffffu, tk[0]) + 1u;     // none reaches it (keys stay below 2^32 - 1)
        for (int it = 0; it < 32 && hi - lo > 1u; ++it) {
            const uint32_t mid = lo + ((hi - lo) >> 1);
            int c = 0;
#pragma unroll
            for (int i = 0; i < S; ++i) c += tk[i] >= mid ? 1 : 0;
            c = __reduce_add_sync(0xffffffffu, c);
            if (c >= m) {
                lo = mid;
                if (c <= m + kTopkTau0Slack) break;
            } else {
                hi = mid;
            }
        }
        const float tau0 = topk_key_score(lo);  // finite: lo lies between two kept maxima
        // 2. candidate runs, ascending (their maxima wait in shared memory)
        uint16_t* run = run_all[warp];
        const unsigned lt_mask = (1u << lane) - 1u;
        int n_run = 0;
        __syncwarp();
        for (int g0 = 0; g0 < (int)n_full; g0 += 32) {
            const int g = g0 + lane;
            const bool c = g < (int)n_full && __bfloat162float(runmax[g]) >= tau0;
            const unsigned cm = __ballot_sync(0xffffffffu, c);
            if (c && n_run + __popc(cm & lt_mask) < kTopkMaxCand) run[n_run + __popc(cm & lt_mask)] = (uint16_t)g;
            n_run += __popc(cm);
        }
        if (n_full * kTopkRunBlocks < loc) {  // the run that holds the local block
            if (lane == 0 && n_run < kTopkMaxCand + 1) run[n_run] = (uint16_t)n_full;
            ++n_run;
        }
        __syncwarp();
        if (n_run > kTopkMaxCand + 1) {  // ties by the hundred: the list does not hold the candidates
            one_level();
        } else {
        // 3. select among the candidates' blocks; scores below tau0 cannot be selected.  The floor
        // only has to lie below tau0: a hair below it, whatever its sign or size.
        const bool few = lnb == 0   ? topk_few_above<0>(srow, run, n_run, (int)loc, tau0, m, log_all[warp], outb, lane)
                         : lnb == 1 ? topk_few_above<1>(srow, run, n_run, (int)loc, tau0, m, log_all[warp], outb, lane)
                                    : topk_few_above<2>(srow, run, n_run, (int)loc, tau0, m, log_all[warp], outb, lane);
        if (!few) {
            __syncwarp();
            const float floor_f = tau0 - fmaxf(fabsf(tau0) * 1e-6f, 1e-30f);
            const TopkGatherStream gs{srow, run, n_run * kTopkRunBlocks, (int)loc, lnb};
            topk_pass1<R>(gs, m, floor_f, sc, kept, n_log, log_ok, lane);
            topk_pass2<R>(gs, m, sc, kept, n_log, log_ok, outb, lane);
        }
        }
    }
    // Block order makes the list ascending with no final sort; the local block is appended by
    // construction (never ranked).
    for (int e = lane; e < top_k; e += 32) orow[e] = e < m ? outb[e] : (e == m ? (int32_t)loc : -1);
}

}  // namespace msa
