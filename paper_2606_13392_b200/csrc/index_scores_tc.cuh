// Eq. 6 on the 5th-gen tensor cores (d_idx in {64,128}, B_k in {64,128}).
//
// One CTA per (tile of 128 queries, NH consecutive index heads).  It streams the visible
// prefix of K_idx in tiles of 256 keys through a TMA ring and multiplies every key tile
// against the NH resident 128x64 query tiles, one after the other, with tcgen05.mma (M=128,
// N=256, four K=16 steps), alternating between two 256-column TMEM accumulators; eight
// epilogue warps reduce a finished accumulator to per-block row maxima (TMEM lane = query
// row, so the maximum over a block's columns is thread-local) while the next head's product
// runs.  Sharing one key tile among NH heads matters: with one head per CTA every 512 MMA
// cycles need a fresh 32 KB tile from L2, about 9 TB/s over the chip, and the kernel is
// L2-bound at 60 % tensor duty.  Only the tile that crosses the diagonal applies the causal
// mask.  In block order (RUNL = false) every thread stores its maxima one (tile, head) unit late
// and blocks beyond a query's local block are filled with -inf at the end; in run order (RUNL = true,
// see score_slot) a thread's maxima of a run of eight blocks wait in shared memory and leave as one
// 16-byte store, and nothing is written beyond the run of the local block.
#pragma once

#include "tc_common.cuh"

namespace msa {

constexpr int kIdxTileQ = 128;
constexpr int kIdxTileK = 256;
constexpr int kIdxThreads = 320;  // warp 0: TMA, warp 1: MMA, warps 2-9: epilogue

// NH heads per CTA, DI = d_idx / 64 swizzle atoms along the contraction, ST key-tile stages.
// RUNL: room for the block maxima of one run of eight blocks (four per epilogue thread and head).
template <int NH, int DI, int ST, bool RUNL = false>
struct IdxSmem {
    alignas(1024) uint8_t a[NH][DI][kIdxTileQ * 128];           // per head and atom: 128 query rows x 64 bf16
    alignas(1024) uint8_t b[ST][DI][kIdxTileK * 128];           // per stage and atom: 256 key rows x 64 bf16
    alignas(16) float run[RUNL ? NH * 4 : 1][256];              // [head][slot of the run][epilogue thread]
    alignas(8) uint64_t full[ST];
    uint64_t empty[ST];
    uint64_t a_full;
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint64_t drain;
    uint32_t tmem_base;
    int abort;
};

// FK = 0: the block maxima are written to `scores` (Eq. 6).  FK > 0 (fused Eq. 6 + Eq. 7 for
// top_k <= FK + 1, NH <= 2): nothing is written to `scores`; every epilogue thread keeps the FK best
// earlier blocks of its (row, head) among the blocks it sees (its half of every key tile) in
// registers, sorted by (score descending, block ascending); at the end the two halves of a row
// are merged through the shared memory the key tiles no longer need and the index list goes to
// block_idx, ascending, the local block last, padded with -1: the same list msa_topk_select
// writes, since both rank the same scaled fp32 maxima with the same tie rule.
constexpr int kIdxFuseKeep = 15;

// A packed batch (several sequences token-major in one tensor): the query tiles of all sequences in
// the order the grid takes them (longest key prefix first).  A tile never straddles two sequences.
struct IdxPackedTile {
    int32_t row0;  // packed row of the sequence's first token
    int32_t len;   // tokens of the sequence
    int32_t qt;    // query tile inside the sequence
};

//
// F8: the operands are fp8 E4M3 (Section 4.2), d_idx = 128 bytes = one swizzle atom (DI = 1).
// The tiles are the same bytes in the same places as 64 bf16 per row, so the tensor maps, the
// shared-memory layout and the descriptor walk are unchanged; only the MMA kind differs (32
// contraction elements per 32-byte step instead of 16).
template <int BK, int NH, int DI, int ST, int FK = 0, bool F8 = false, bool RUNL = false>
__global__ void __launch_bounds__(kIdxThreads, 1)
index_scores_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       int64_t q_begin, int64_t q_count, int H_kv, float scale,
                       float* __restrict__ scores, int64_t ld_scores, int64_t n_cols, int* status,
                       int32_t* __restrict__ block_idx = nullptr, int top_k = 0,
                       const IdxPackedTile* __restrict__ packed = nullptr, int64_t score_row0 = 0) {
    static_assert(FK == 0 || NH <= 2, "the fused form keeps its candidates in registers");
    static_assert(!F8 || DI == 1, "fp8 index vectors are one 128-byte atom");
    static_assert(!RUNL || FK == 0, "the run order is a layout of the score matrix");
    extern __shared__ uint8_t smem_raw[];
    IdxSmem<NH, DI, ST, RUNL>& sm =
        *reinterpret_cast<IdxSmem<NH, DI, ST, RUNL>*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_hg = H_kv / NH;  // head groups
    const int r0 = (int)(blockIdx.x % n_hg) * NH;
    // Longest items first: the last query tile sees the most keys.  In a packed batch the tile list
    // says which sequence (rows row0 .. row0 + q_count of every tensor) and which of its tiles.
    int64_t qt, row0 = 0;
    if (packed != nullptr) {
        const IdxPackedTile t = packed[blockIdx.x / n_hg];
        row0 = t.row0; q_count = t.len; qt = t.qt;
    } else {
        qt = (q_count + kIdxTileQ - 1) / kIdxTileQ - 1 - (int64_t)(blockIdx.x / n_hg);
    }
    const int64_t q0 = qt * kIdxTileQ;
    int64_t q_hi = q0 + kIdxTileQ - 1;
    if (q_hi > q_count - 1) q_hi = q_count - 1;
    const int n_tiles = (int)((q_begin + q_hi) / kIdxTileK) + 1;
    volatile int* abort = &sm.abort;

    if (threadIdx.x == 0) {
        for (int s = 0; s < ST; ++s) { mbar_init(&sm.full[s], 1); mbar_init(&sm.empty[s], 1); }
        mbar_init(&sm.a_full, 1);
        mbar_init(&sm.drain, 1);
        for (int b = 0; b < 2; ++b) { mbar_init(&sm.acc_full[b], 1); mbar_init(&sm.acc_empty[b], 8); }
        sm.abort = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
    }
    if (warp == 1) tmem_alloc(&sm.tmem_base, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            if (const long long late = g_debug_producer_delay; late > 0) spin_cycles(late);  // tests only
            mbar_arrive_expect_tx(&sm.a_full, NH * DI * kIdxTileQ * 128);
            for (int h = 0; h < NH; ++h)
                for (int a = 0; a < DI; ++a) tma_load_3d(sm.a[h][a], &tm_q, a * 64, r0 + h, (int)(row0 + q0), &sm.a_full);
            for (int t = 0; t < n_tiles; ++t) {
                const int s = t % ST;
                if (!mbar_wait(&sm.empty[s], ((t / ST) & 1) ^ 1, abort)) {
                    report_async(status, kAsyncTimeout, 0x101);
                    break;
                }
                mbar_arrive_expect_tx(&sm.full[s], DI * kIdxTileK * 128);
                for (int a = 0; a < DI; ++a)
                    tma_load_2d(sm.b[s][a], &tm_k, a * 64, (int)row0 + t * kIdxTileK, &sm.full[s]);
            }
            if (*abort != 0) spin_cycles(200000);  // let copies already in flight land
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc =
                F8 ? make_idesc_e4m3(kIdxTileQ, kIdxTileK) : make_idesc_bf16(kIdxTileQ, kIdxTileK, false, false);
            bool ok = mbar_wait(&sm.a_full, 0, abort);
            if (!ok) report_async(status, kAsyncTimeout, 0x102);
            // The tensor pipe takes an MMA from this thread only about as fast as it executes them, so
            // whatever the thread does between the last MMA of one (tile, head) unit and the first of the
            // next leaves the pipe idle: the head loop is unrolled and the operand descriptors are built
            // once, so that a unit costs a barrier test, the MMAs and a commit.
            uint64_t a_desc[NH][DI], b_desc[ST][DI];
#pragma unroll
            for (int h = 0; h < NH; ++h)
#pragma unroll
                for (int a = 0; a < DI; ++a) a_desc[h][a] = make_smem_desc(smem_u32(sm.a[h][a]), 16, 1024);
#pragma unroll
            for (int s = 0; s < ST; ++s)
#pragma unroll
                for (int a = 0; a < DI; ++a) b_desc[s][a] = make_smem_desc(smem_u32(sm.b[s][a]), 16, 1024);
            int s = 0;
            uint32_t full_par = 0;  // parity of the ring's current lap
            for (int t = 0; ok && t < n_tiles; ++t) {
                if (!mbar_wait(&sm.full[s], full_par, abort)) {
                    report_async(status, kAsyncTimeout, 0x104);
                    break;
                }
                uint64_t bd[DI];
#pragma unroll
                for (int a = 0; a < DI; ++a) {
                    bd[a] = b_desc[0][a];
#pragma unroll
                    for (int ss = 1; ss < ST; ++ss)
                        if (ss == s) bd[a] = b_desc[ss][a];
                }
#pragma unroll
                for (int h = 0; h < NH; ++h) {
                    const int u = t * NH + h, buf = u & 1;  // accumulators alternate over (tile, head)
                    if (!mbar_wait(&sm.acc_empty[buf], ((u >> 1) & 1) ^ 1, abort)) {
                        report_async(status, kAsyncTimeout, 0x103);
                        ok = false;
                        break;
                    }
                    MSA_STAMP(u, 10);
                    tc_fence_after();
                    MSA_STAMP(u, 0);
#pragma unroll
                    for (int a = 0; a < DI; ++a) {
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) {  // 32 bytes (16 bf16 or 32 fp8) = 2 descriptor units per K step
                            if constexpr (F8)
                                mma_e4m3_ss(tmem + buf * kIdxTileK, a_desc[h][a] + 2 * kk, bd[a] + 2 * kk, idesc, kk > 0);
                            else
                                mma_bf16_ss(tmem + buf * kIdxTileK, a_desc[h][a] + 2 * kk, bd[a] + 2 * kk, idesc, (a | kk) > 0);
                        }
                    }
                    mma_commit(&sm.acc_full[buf]);
                    MSA_STAMP(u, 1);
                }
                mma_commit(&sm.empty[s]);
                if (++s == ST) { s = 0; full_par ^= 1; }
            }
            if (*abort != 0) {  // unwinding: wait for the MMAs already issued before TMEM is freed
                mma_commit(&sm.drain);
                mbar_wait_quiet(&sm.drain, 0, 20000000);
            }
        }
    } else {
        const int ew = warp - 2;            // 0..7
        const int quarter = warp & 3;       // TMEM lanes this warp may read
        const int half = ew >> 2;           // which 128 columns of the 256-column tile
        const int row = quarter * 32 + lane;
        const int64_t q = q0 + row;
        const int64_t pos = q_begin + q;
        const bool valid_row = q < q_count;
        const int64_t loc = pos / BK;
        bool live = true;
        constexpr int FKN = FK > 0 ? FK : 1;
        float ts[NH][FKN];   // fused form: best earlier blocks seen by this thread, per head
        int32_t tb[NH][FKN];
        if constexpr (FK > 0) {
#pragma unroll
            for (int h = 0; h < NH; ++h)
#pragma unroll
                for (int i = 0; i < FK; ++i) { ts[h][i] = -INFINITY; tb[h][i] = -1; }
        }
        // Scores leave one unit late: a unit's maxima are stored right after the next unit's accumulator
        // has been released, ahead of that unit's reductions, so that the store and its address
        // arithmetic sit neither in front of an accumulator's release nor in front of the wait for the
        // next one.
        constexpr int NBP = 128 / BK;
        float pend[NBP];
        float* pend_ptr = nullptr;
        int pend_n = 0;
        // Run order (RUNL): the thread's maxima of one run of eight blocks - the NBP blocks of its half
        // of every key tile, over TPR tiles - wait in shared memory (the thread's own words) and leave
        // as one 16-byte store per head and run.
        constexpr int TPR = 4 / NBP;
        const int et = ew * 32 + lane;
        float4 pend4 = make_float4(0.f, 0.f, 0.f, 0.f);
        bool pend4_on = false;
        // (a packed batch scored group by group: the score matrix starts at packed row score_row0)
        float* const row_base = FK == 0 ? scores + ((row0 + q - score_row0) * H_kv + r0) * ld_scores : nullptr;
        for (int t = 0; live && t < n_tiles; ++t) {
            const int64_t key0 = (int64_t)t * kIdxTileK + half * 128;
            const bool need_mask = key0 + 127 > pos;
            const int lim = (int)(pos - key0);  // columns 0..lim are visible (may be negative)
#pragma unroll(FK > 0 ? NH : 1)
            for (int h = 0; h < NH; ++h) {
                if (FK > 0 && !live) break;
                const int u = t * NH + h, buf = u & 1;
                if (!mbar_wait(&sm.acc_full[buf], (u >> 1) & 1, abort)) {
                    report_async(status, kAsyncTimeout, 0x105);
                    live = false;
                    break;
                }
                tc_fence_after();
                if (lane == 0 && ew == 0) MSA_STAMP(u, 11);
                const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + buf * kIdxTileK + half * 128;
                constexpr int NB = 128 / BK;  // blocks in this thread's 128 columns
                float best[NB];
#pragma unroll
                for (int i = 0; i < NB; ++i) best[i] = -INFINITY;
                if constexpr (FK > 0) {
                    // 32 columns at a time: the candidate lists need the registers
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t v[32];
                        tmem_ld_32x32(taddr + c * 32, v);
                        tmem_wait_ld();
                        if (c == 3) {
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&sm.acc_empty[buf]);
                        }
                        if (need_mask) {
#pragma unroll
                            for (int e = 0; e < 32; ++e)
                                if (c * 32 + e > lim) v[e] = 0xFF800000u;  // -inf
                        }
                        best[(c * 32) / BK] = fmaxf(best[(c * 32) / BK], tree_max32(v));
                    }
                } else {
                    uint32_t v[4][32];
#pragma unroll
                    for (int c = 0; c < 4; ++c) tmem_ld_32x32(taddr + c * 32, v[c]);
                    tmem_wait_ld();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm.acc_empty[buf]);
                    if (lane == 0) MSA_STAMP(u, 2 + ew);
                    if constexpr (RUNL) {
                        if (pend4_on) *reinterpret_cast<float4*>(pend_ptr) = pend4;
                        pend4_on = false;
                    } else {
#pragma unroll
                        for (int i = 0; i < NB; ++i)
                            if (i < pend_n) pend_ptr[i] = pend[i];
                        pend_n = 0;
                    }
                    if (need_mask) {
#pragma unroll
                        for (int c = 0; c < 4; ++c)
#pragma unroll
                            for (int e = 0; e < 32; ++e)
                                if (c * 32 + e > lim) v[c][e] = 0xFF800000u;  // -inf
                    }
#pragma unroll
                    for (int c = 0; c < 4; ++c) best[(c * 32) / BK] = fmaxf(best[(c * 32) / BK], tree_max32(v[c]));
                }
                if constexpr (FK > 0) {
#pragma unroll
                    for (int i = 0; i < NB; ++i) {
                        const int64_t b = key0 / BK + i;
                        const float x = best[i] * scale;
                        // ranked: earlier blocks only; a later equal score never passes an earlier one
                        if (valid_row && b < loc && x > ts[h][FK - 1]) {
                            ts[h][FK - 1] = x; tb[h][FK - 1] = (int32_t)b;
#pragma unroll
                            for (int e = FK - 1; e > 0; --e) {
                                if (ts[h][e] > ts[h][e - 1]) {
                                    const float fs = ts[h][e]; ts[h][e] = ts[h][e - 1]; ts[h][e - 1] = fs;
                                    const int32_t fb = tb[h][e]; tb[h][e] = tb[h][e - 1]; tb[h][e - 1] = fb;
                                }
                            }
                        }
                    }
                } else if constexpr (RUNL) {
                    const int ti = t % TPR;
                    if (ti == TPR - 1 || t == n_tiles - 1) {
                        // (the key tiles may end inside the run: its other blocks are visible to no row of the tile)
                        float x[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            x[j] = -INFINITY;
                            if (j / NB < ti) x[j] = sm.run[RUNL ? h * 4 + j : 0][et];
                        }
#pragma unroll
                        for (int j = 0; j < 4; ++j)
#pragma unroll
                            for (int i = 0; i < NB; ++i)
                                if (j == ti * NB + i) x[j] = best[i] * scale;
                        const int64_t run = t / TPR;
                        pend4 = make_float4(x[0], x[1], x[2], x[3]);
                        pend_ptr = row_base + h * ld_scores + run * 8 + half * 4;
                        pend4_on = valid_row && run * 8 <= loc;
                    } else {
#pragma unroll
                        for (int i = 0; i < NB; ++i) sm.run[RUNL ? h * 4 + ti * NB + i : 0][et] = best[i] * scale;
                    }
                } else if (valid_row) {
                    const int64_t b0 = key0 / BK;  // this thread's blocks b0 .. b0 + NB - 1; those up to loc are visible
                    pend_ptr = row_base + h * ld_scores + b0;
#pragma unroll
                    for (int i = 0; i < NB; ++i) pend[i] = best[i] * scale;
                    const int64_t vis = loc - b0 + 1;
                    pend_n = vis >= NB ? NB : (vis > 0 ? (int)vis : 0);
                }
            }
        }
        if constexpr (RUNL) {
            if (pend4_on) *reinterpret_cast<float4*>(pend_ptr) = pend4;
        } else if constexpr (FK == 0) {
#pragma unroll
            for (int i = 0; i < NBP; ++i)
                if (i < pend_n) pend_ptr[i] = pend[i];
        }
        if constexpr (FK > 0) {
            // Merge the two halves of every row.  All MMAs have completed (the last accumulator was
            // read), so the key-tile stages are free: [half][row][head][FK] scores, then blocks.
            float* xs = reinterpret_cast<float*>(&sm.b[0][0][0]);
            int32_t* xb = reinterpret_cast<int32_t*>(xs + 2 * kIdxTileQ * NH * FK);
            static_assert(sizeof(sm.b) >= 2 * kIdxTileQ * NH * FK * 8 + kIdxTileQ * NH * 16 * 4, "exchange area");
            int32_t* xo = xb + 2 * kIdxTileQ * NH * FK;  // [row][head][16] merged picks
            asm volatile("bar.sync 1, 256;" ::: "memory");
#pragma unroll
            for (int h = 0; h < NH; ++h)
#pragma unroll
                for (int i = 0; i < FK; ++i) {
                    xs[((half * kIdxTileQ + row) * NH + h) * FK + i] = ts[h][i];
                    xb[((half * kIdxTileQ + row) * NH + h) * FK + i] = tb[h][i];
                }
            asm volatile("bar.sync 1, 256;" ::: "memory");
            // thread (row, half) finishes head `half` (and, with one head per CTA, half 0 does it)
            const int m = top_k - 1;
            for (int h = half; h < NH; h += 2) {
                if (!valid_row || !live) break;
                const float* sa = xs + ((0 * kIdxTileQ + row) * NH + h) * FK;
                const float* sb = xs + ((1 * kIdxTileQ + row) * NH + h) * FK;
                const int32_t* ba = xb + ((0 * kIdxTileQ + row) * NH + h) * FK;
                const int32_t* bb = xb + ((1 * kIdxTileQ + row) * NH + h) * FK;
                int32_t* pick = xo + (row * NH + h) * 16;
                int ia = 0, ib = 0, c = 0;
                while (c < m) {  // best first; equal scores: the lower block
                    const bool ha = ia < FK && ba[ia] >= 0, hb = ib < FK && bb[ib] >= 0;
                    if (!ha && !hb) break;
                    const bool take_a = ha && (!hb || sa[ia] > sb[ib] || (sa[ia] == sb[ib] && ba[ia] < bb[ib]));
                    pick[c++] = take_a ? ba[ia++] : bb[ib++];
                }
                for (int i = 1; i < c; ++i) {  // ascending block order
                    const int32_t v = pick[i];
                    int j2 = i - 1;
                    while (j2 >= 0 && pick[j2] > v) { pick[j2 + 1] = pick[j2]; --j2; }
                    pick[j2 + 1] = v;
                }
                int32_t* orow = block_idx + ((row0 + q) * H_kv + r0 + h) * (int64_t)top_k;
                for (int i = 0; i < top_k; ++i) orow[i] = i < c ? pick[i] : (i == c ? (int32_t)loc : -1);
            }
        }
        // Blocks with no visible token: -inf (Eq. 6).  Warp ew fills rows ew, ew+8, ...
        for (int rr = ew; FK == 0 && !RUNL && rr < kIdxTileQ; rr += 8) {
            const int64_t qq = q0 + rr;
            if (qq >= q_count) break;
            for (int h = 0; h < NH; ++h) {
                float* orow = scores + ((row0 + qq - score_row0) * H_kv + r0 + h) * ld_scores;
                for (int64_t b = (q_begin + qq) / BK + 1 + lane; b < n_cols; b += 32) orow[b] = -INFINITY;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, 512);
    }
}

}  // namespace msa
