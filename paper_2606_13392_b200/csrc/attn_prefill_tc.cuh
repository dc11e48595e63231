// Eq. 8 for prefill in KV-outer order (Section 4.2) on tcgen05/TMEM (d_h = 128,
// B_k in {64,128}, G in {8,16}).
//
// For one range of queries:
//   1. reverse index: count, per (KV block, KV head) tile, the queries that selected it;
//      exclusive scan; scatter 32-bit handles (query << 8 | slot), slot = position of the
//      block in the query's ascending list, so every partial has its own place and no
//      atomics touch the outputs;
//   2. attention: a tile's handles are cut into items of 128/G queries; an item stacks those
//      queries' G heads into one 128-row operand (query concatenation), computes
//      S = Q K_b^T into TMEM, a row softmax local to the item (one block = one S tile),
//      P (bf16) back into TMEM, O = P V_b into TMEM, and writes the locally normalised
//      partial and its log-sum-exp to the workspace;
//   3. combine: LSE-weighted merge of each query's partials (Section 4.2, two-phase forward).
#pragma once

#include "tc_common.cuh"

namespace msa {

struct RangeParams {
    int64_t q_begin;   // absolute position of the first query of the call
    int64_t q_first;   // first query of this range, relative to the call
    int32_t q_count;   // queries in this range
    int32_t n_blocks;  // KV blocks visible to the range: ceil((q_begin+q_first+q_count)/B_k)
    int32_t H_kv, top_k;
    // A packed batch (several sequences token-major in one tensor, q_begin = 0): blocks are numbered
    // through the batch, sequence after sequence, and n_blocks counts them all.  Null for one sequence.
    const int32_t* row_pos;   // [rows]   position of a packed row inside its own sequence
    const int32_t* row_blk0;  // [rows]   number of blocks of the sequences before the row's
    const int32_t* blk_row0;  // [blocks] packed row of the block's first key
};

// Position of query `qrow` (a row of the call) inside its sequence, and the batch-wide number of its block 0.
__device__ __forceinline__ int64_t query_pos(const RangeParams& p, int64_t qrow) {
    return p.row_pos != nullptr ? (int64_t)p.row_pos[qrow] : p.q_begin + qrow;
}
__device__ __forceinline__ int query_blk0(const RangeParams& p, int64_t qrow) {
    return p.row_blk0 != nullptr ? p.row_blk0[qrow] : 0;
}

// Fills the three arrays of a packed batch from the row offsets cu [n_seqs+1] and the block offsets
// blk_cum [n_seqs+1] of its sequences (one thread per row, then per block; binary searches).
__global__ void __launch_bounds__(256)
packed_map_kernel(const int64_t* __restrict__ cu, const int32_t* __restrict__ blk_cum, int n_seqs, int B_k,
                  int32_t* __restrict__ row_pos, int32_t* __restrict__ row_blk0, int32_t* __restrict__ blk_row0) {
    const int64_t rows = cu[n_seqs] - cu[0];
    const int64_t n_blk = blk_cum[n_seqs];
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < rows + n_blk;
         i += (int64_t)gridDim.x * blockDim.x) {
        int lo = 0, hi = n_seqs;  // last sequence that starts at or before the row (the block)
        if (i < rows) {
            const int64_t row = cu[0] + i;
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (cu[mid] <= row) lo = mid; else hi = mid;
            }
            row_pos[i] = (int32_t)(row - cu[lo]);
            row_blk0[i] = blk_cum[lo];
        } else {
            const int32_t b = (int32_t)(i - rows);
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (blk_cum[mid] <= b) lo = mid; else hi = mid;
            }
            blk_row0[b] = (int32_t)(cu[lo] - cu[0]) + (b - blk_cum[lo]) * B_k;
        }
    }
}

// Tiles are numbered head after head: the whole grid works on one KV head at a time, so the
// Q rows of (range, head) - gathered top_k times each - are the only hot lines in L2.
__device__ __forceinline__ int tile_id(int b, int r, const RangeParams& p) {
    return r * p.n_blocks + b;
}
__device__ __forceinline__ int n_phases(const RangeParams& p) { return p.H_kv; }
// First partial row (slot 0) of (query ql of the range, KV head r): the partial buffers are
// laid out [head][query][slot], so one head phase writes one contiguous part of them.
__device__ __forceinline__ int64_t partial_base(int64_t ql, int r, const RangeParams& p) {
    return ((int64_t)r * p.q_count + ql) * (int64_t)p.top_k;
}
// Items of phase ph dealt to this CTA: a contiguous share of the phase's item list.
__device__ __forceinline__ void phase_items(const int32_t* __restrict__ item_off, const RangeParams& p, int ph,
                                            int& lo, int& hi) {
    const int a = item_off[ph * p.n_blocks], b = item_off[(ph + 1) * p.n_blocks];
    const int per = (b - a + (int)gridDim.x - 1) / (int)gridDim.x;
    lo = min(b, a + (int)blockIdx.x * per);
    hi = min(b, lo + per);
}

// ---------------------------------------------------------------- 1. reverse index
// One warp per (query, group) row of the index list.  Pass 0 counts the queries of every
// (block, head) tile and remembers each entry's arrival rank within its tile; pass 1 (after
// the scan) writes the handle to tile_off[tile] + rank without touching the counters again.
template <int BK>
__global__ void __launch_bounds__(256)
revidx_kernel(const int32_t* __restrict__ block_idx, RangeParams p, int pass, int32_t* __restrict__ cnt,
              const int32_t* __restrict__ tile_off, uint32_t* __restrict__ rank,
              uint32_t* __restrict__ handles, int* status) {
    const int row = (int)((blockIdx.x * (unsigned)blockDim.x + threadIdx.x) >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= p.q_count * p.H_kv) return;
    const int ql = row / p.H_kv, r = row - ql * p.H_kv;
    const int64_t loc = query_pos(p, p.q_first + ql) / BK;
    const int blk0 = query_blk0(p, p.q_first + ql);
    const int32_t* sel = block_idx + ((p.q_first + ql) * (int64_t)p.H_kv + r) * p.top_k;
    for (int s = lane; s < p.top_k; s += 32) {
        const int32_t b = sel[s];
        if (b < 0 || (int64_t)b > loc) {
            if (b != -1 && pass == 0) report_async(status, kAsyncBadIndex, 0x301);
            continue;
        }
        const int tile = tile_id(blk0 + b, r, p);
        const int64_t e = (int64_t)row * p.top_k + s;
        if (pass == 0)
            rank[e] = (uint32_t)atomicAdd(&cnt[tile], 1);
        else
            handles[tile_off[tile] + rank[e]] = ((uint32_t)ql << 8) | (uint32_t)s;
    }
}

// Single-CTA exclusive scan of the tile counts -> pair offsets and item offsets.
__global__ void __launch_bounds__(1024)
revidx_scan_kernel(int32_t* __restrict__ cnt, int n_tiles, int qpi, int32_t* __restrict__ tile_off,
                   int32_t* __restrict__ item_off) {
    __shared__ int s_pairs[1024], s_items[1024];
    const int t = threadIdx.x;
    const int per = (n_tiles + 1023) / 1024;
    const int lo = t * per, hi = min(n_tiles, lo + per);
    int pairs = 0, items = 0;
    for (int i = lo; i < hi; ++i) { pairs += cnt[i]; items += (cnt[i] + qpi - 1) / qpi; }
    s_pairs[t] = pairs; s_items[t] = items;
    __syncthreads();
    for (int off = 1; off < 1024; off <<= 1) {
        const int a = t >= off ? s_pairs[t - off] : 0, b = t >= off ? s_items[t - off] : 0;
        __syncthreads();
        s_pairs[t] += a; s_items[t] += b;
        __syncthreads();
    }
    int po = s_pairs[t] - pairs, io = s_items[t] - items;
    for (int i = lo; i < hi; ++i) {
        const int c = cnt[i];
        tile_off[i] = po; item_off[i] = io;
        po += c; io += (c + qpi - 1) / qpi;
    }
    if (t == 1023) { tile_off[n_tiles] = s_pairs[1023]; item_off[n_tiles] = s_items[1023]; }
}

// ---------------------------------------------------------------- 2. attention
constexpr int kAttnInfoRing = 8;  // item descriptors; deeper than the furthest reader lags

struct AttnItemInfo {
    int32_t kv_row0, r, nq;  // row of the tile's first key in the K/V tensors; KV head; queries in the item
    int32_t kb, vb;        // K and V buffers of this item's tile
    int32_t new_tile;      // first item of its tile in this CTA: wait for the K/V loads
    int32_t last_of_tile;  // last item of its tile in this CTA: release the K/V buffers
    int32_t pad;
    uint32_t handle[16];
};

template <int BK>
struct AttnSmem {
    alignas(1024) uint8_t q[2][128 * 256];     // [context][query][head group of 8][d half][8 heads][64 bf16]
    alignas(1024) uint8_t kv[3][2][BK * 128];  // three tile buffers [d half][key][64 bf16]; roles rotate (see below)
    alignas(1024) uint8_t ostage[2][128 * 256];  // [context][query][16-byte chunk of d][head]: partials on their way out
    alignas(8) uint64_t q_full[2], q_empty[2];
    uint64_t kv_full[3], kv_empty[3];
    uint64_t s_full[2], p_full[2], o_full[2];
    uint64_t drain;
    uint32_t tmem_base;
    int abort;
    AttnItemInfo info[kAttnInfoRing];
};

// K and V tiles rotate through three buffers: the t-th tile a CTA touches keeps K in buffer
// (2t) mod 3 and V in buffer (2t+1) mod 3.  The next tile's K goes to the third buffer (free since
// the tile before), its V to this tile's K buffer, which is free as soon as this tile's last
// S = Q K^T has run, about one softmax before the first O = P V of the next tile needs it: tiles
// change without a bubble on 1.5x the memory of one tile pair.  Every buffer is used twice per
// three tiles, so the phase parity of a use depends only on the buffer and the role.
__device__ __forceinline__ int kv_k_buf(int t) { return (2 * t) % 3; }
__device__ __forceinline__ int kv_v_buf(int t) { return (2 * t + 1) % 3; }
__device__ __forceinline__ int kv_k_parity(int kb) { return kb == 1 ? 1 : 0; }   // second use of buffer 1
__device__ __forceinline__ int kv_v_parity(int vb) { return vb != 1 ? 1 : 0; }   // second use of buffers 0, 2

// One CTA per SM, eleven warps, two items in flight (contexts j = n mod 2, each with its own Q
// buffer, S/P and O columns in TMEM, softmax group and staging buffer):
//   warps 0, 10  producers: both walk the CTA's share of the item list head phase after head phase;
//             per item one TMA box per query into the context's Q buffer (free once S(n-2) has read
//             it), warp 0 the first half of the queries and warp 10 the second (a warp spends about
//             a hundred cycles per box it issues); per new tile warp 0 loads K and V.
//   warp 1    MMA issuer: S_j = Q(n) K^T as soon as Q(n) has landed, then O_j' = P(n-1) V once
//             P(n-1) is written.  MMAs execute in issue order, which is what lets S(n+2) reuse
//             the columns that hold P(n).
//   warps 2-5 / 6-9  softmax groups: read the S row from TMEM, exp2 with the scale folded in,
//             write P (bf16 pairs) over the S columns; then O row / ell as bf16 into the
//             context's staging buffer and one bulk copy per query to the partial buffer.  The
//             copies drain in the background: an SM moves about 32 bytes of stores per clock, and
//             as 16-byte stores issued by the softmax warps they stalled those warps for a third
//             of an item's time.
constexpr int kAttnThreads = 352;

//
// F8 (Section 4.2: the kernels also support fp8): Q, K and V are stored in fp8 E4M3.  A row of 128
// fp8 is one 128-byte swizzle row, so a Q tile is 16 KB (a query's G heads are one box of G rows)
// and a K tile BK x 128 bytes; S = Q K^T runs as kind::f8f6f4 MMAs (32 elements per step, four
// steps), whose products and fp32 sums are those of the decoded values.  The fp8 V tile lands in
// the half of the K buffer that an fp8 K tile leaves free and is widened once per tile (exactly:
// every E4M3 value is a bf16 value) by the first producer warp into the V buffer, in the layout a
// bf16 TMA load would have produced; P stays bf16 and O = P V is the bf16 path unchanged.  The
// kernel therefore computes what the bf16 kernel computes on the decoded operands, with half the
// bytes per gathered query and per K/V tile.
template <int BK, int G, bool F8 = false>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_prefill_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       const __grid_constant__ CUtensorMap tm_v, RangeParams p,
                       const int32_t* __restrict__ tile_off, const int32_t* __restrict__ item_off,
                       const uint32_t* __restrict__ handles, float scale_log2e,
                       __nv_bfloat16* __restrict__ o_buf, float* __restrict__ lse_buf, int* status) {
    constexpr int QPI = 128 / G;            // queries per item
    constexpr int TMEM_COLS = 512;          // context j: S/P at j*256, O at j*256 + 128
    constexpr uint32_t Q_BYTES = F8 ? G * 128 : G * 256;  // one query's G heads in the Q tile
    constexpr uint32_t O_BYTES = G * 256;   // one query's G heads of a bf16 partial
    constexpr uint32_t KV_HALF = BK * 128;  // one d half of a bf16 K or V tile = a whole fp8 tile
    extern __shared__ uint8_t smem_raw[];
    AttnSmem<BK>& sm =
        *reinterpret_cast<AttnSmem<BK>*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abort = &sm.abort;

    const int n_tiles = p.n_blocks * p.H_kv;
    const int phases = n_phases(p);
    int n_items = 0;  // items of this CTA over all phases (every role walks the same sequence)
    for (int ph = 0; ph < phases; ++ph) {
        int lo, hi;
        phase_items(item_off, p, ph, lo, hi);
        n_items += max(hi - lo, 0);
    }

    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sm.q_full[i], 2); mbar_init(&sm.q_empty[i], 1);
            mbar_init(&sm.s_full[i], 1); mbar_init(&sm.p_full[i], 4); mbar_init(&sm.o_full[i], 1);
        }
        for (int i = 0; i < 3; ++i) { mbar_init(&sm.kv_full[i], 1); mbar_init(&sm.kv_empty[i], 1); }
        mbar_init(&sm.drain, 1);
        sm.abort = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
    }
    if (warp == 1) tmem_alloc(&sm.tmem_base, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;

    if (warp == 0 || warp == 10) {
        // ---------------- producers
        const int half = warp == 10 ? 1 : 0;  // warp 10: the second half of the queries
        // Tile metadata lives in registers and is refreshed only when the walk crosses into the
        // next tile; an item's handles follow the previous item's in memory (the handle array is
        // laid out tile after tile), so the next item's handles are fetched one item ahead.
        const int handles_end = tile_off[n_tiles];
        // Q rows are gathered top_k times each, K/V tiles go by once.
        const uint64_t pol_q = l2_policy_evict_last(), pol_kv = l2_policy_evict_first();
        int loaded_tile = -1, tile_seq = -1, n = 0, kv_row0 = 0;
        bool ok = true;
        if (const long long late = g_debug_producer_delay; late > 0) spin_cycles(late);  // tests only
        for (int ph = 0; ph < phases && ok; ++ph) {
            int it_lo, it_hi;
            phase_items(item_off, p, ph, it_lo, it_hi);
            if (it_lo >= it_hi) continue;
            int tile;
            {   // last tile of the phase whose first item is <= it_lo (skips empty tiles)
                int lo = ph * p.n_blocks, hi = (ph + 1) * p.n_blocks;
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (item_off[mid] <= it_lo) lo = mid; else hi = mid;
                }
                tile = lo;
            }
            int i_next = item_off[tile + 1], p_end = tile_off[tile + 1];
            int first = tile_off[tile] + (it_lo - item_off[tile]) * QPI;
            uint32_t h_next = first + lane < handles_end ? handles[first + lane] : 0u;
            for (int it = it_lo; it < it_hi; ++it, ++n) {
                while (i_next <= it) {  // crossed into the next non-empty tile
                    ++tile;
                    i_next = item_off[tile + 1];
                    p_end = tile_off[tile + 1];
                }
                const int r = ph, b = tile - ph * p.n_blocks;
                const int nq = min(QPI, p_end - first);
                const bool new_tile = tile != loaded_tile;
                if (new_tile) kv_row0 = p.blk_row0 != nullptr ? p.blk_row0[b] : b * BK;
                const bool last_of_tile = (it + 1 == it_hi) || (i_next <= it + 1);
                if (new_tile) ++tile_seq;
                const int kb = kv_k_buf(tile_seq), vb = kv_v_buf(tile_seq);
                const uint32_t h = lane < nq ? h_next : 0u;
                {
                    const int nf = first + nq;  // the next item's handles start where this item's end
                    h_next = (it + 1 < it_hi && nf + lane < handles_end) ? handles[nf + lane] : 0u;
                }
                const int j = n & 1;
                // The context's Q buffer is free once S(n-2) has read it.
                if (n >= 2 && !mbar_wait(&sm.q_empty[j], ((n >> 1) - 1) & 1, abort)) {
                    if (lane == 0) report_async(status, kAsyncTimeout, 0x311);
                    ok = false;
                    break;
                }
                if (threadIdx.x == 0) MSA_STAMP(n, 12);
                // Slot n mod 8 was last read by the epilogue of item n-8, long before S(n-2) ran.
                AttnItemInfo& inf = sm.info[n % kAttnInfoRing];
                if (lane < QPI && half == 0) inf.handle[lane] = h;
                if (lane == 0 && half == 0) {
                    inf.kv_row0 = kv_row0; inf.r = r; inf.nq = nq; inf.kb = kb; inf.vb = vb;
                    inf.new_tile = new_tile ? 1 : 0; inf.last_of_tile = last_of_tile ? 1 : 0;
                }
                __syncwarp();
                const int q_lo = half * (QPI / 2), q_hi = min(nq, q_lo + QPI / 2);
                if (lane == 0) mbar_arrive_expect_tx(&sm.q_full[j], (uint32_t)max(q_hi - q_lo, 0) * Q_BYTES);
                __syncwarp();
                // One box per query: its G heads x 128 d, one contiguous read of G*256 bytes, laid
                // down as [8 heads][d half][8 heads][64 d] so that every 1 KB is one operand atom.
                if (lane >= q_lo && lane < q_hi) {
                    if constexpr (F8)  // (128 bytes, the group's G heads, one query): G swizzle rows
                        tma_load_3d_hint(sm.q[j] + lane * Q_BYTES, &tm_q, 0, r * G, (int)(p.q_first + (h >> 8)),
                                         &sm.q_full[j], pol_q);
                    else
                        tma_load_5d_hint(sm.q[j] + lane * Q_BYTES, &tm_q, 0, 0, 0, r * (G / 8),
                                         (int)(p.q_first + (h >> 8)), &sm.q_full[j], pol_q);
                }
                if (threadIdx.x == 0) MSA_STAMP(n, 13);
                if (new_tile) {
                    // K: the buffer was the V buffer of the tile before last (or the K buffer three
                    // tiles back); V: this buffer held the previous tile's K.  One warp does all the
                    // waiting on a buffer's barrier: a parity wait is only right for a waiter that
                    // has seen every earlier phase complete, and a second warp waiting for every
                    // other phase could be two phases behind and be let through a phase early.
                    const bool k_wait = tile_seq >= 3 || kv_k_parity(kb) == 1;
                    const bool v_wait = tile_seq >= 3 || kv_v_parity(vb) == 1;
                    if (half == 0 && k_wait && !mbar_wait(&sm.kv_empty[kb], kv_k_parity(kb) ^ 1, abort)) {
                        if (lane == 0) report_async(status, kAsyncTimeout, 0x312);
                        ok = false;
                        break;
                    }
                    if (lane == 0 && half == 0) {
                        mbar_arrive_expect_tx(&sm.kv_full[kb], 2 * KV_HALF);
                        if constexpr (F8) {  // the fp8 K tile, and the fp8 V tile on its way to being widened
                            tma_load_3d_hint(sm.kv[kb][0], &tm_k, 0, r, kv_row0, &sm.kv_full[kb], pol_kv);
                            tma_load_3d_hint(sm.kv[kb][1], &tm_v, 0, r, kv_row0, &sm.kv_full[kb], pol_kv);
                        } else {
                            tma_load_3d_hint(sm.kv[kb][0], &tm_k, 0, r, kv_row0, &sm.kv_full[kb], pol_kv);
                            tma_load_3d_hint(sm.kv[kb][1], &tm_k, 64, r, kv_row0, &sm.kv_full[kb], pol_kv);
                        }
                    }
                    if (half == 0 && v_wait && !mbar_wait(&sm.kv_empty[vb], kv_v_parity(vb) ^ 1, abort)) {
                        if (lane == 0) report_async(status, kAsyncTimeout, 0x313);
                        ok = false;
                        break;
                    }
                    if constexpr (F8) {
                        if (half == 0) {
                            // The fp8 V tile has landed behind the K tile: widen it into the V buffer.
                            // Source row = key, 128 fp8 in eight 16-byte chunks, chunk c stored at
                            // c ^ (key & 7); 16 fp8 become two chunks of the bf16 tile [d half][key][64].
                            if (!mbar_wait(&sm.kv_full[kb], kv_k_parity(kb), abort)) {
                                if (lane == 0) report_async(status, kAsyncTimeout, 0x314);
                                ok = false;
                                break;
                            }
                            const uint32_t src = smem_u32(sm.kv[kb][1]), dst = smem_u32(sm.kv[vb][0]);
                            for (int i = lane; i < BK * 8; i += 32) {
                                const int key = i >> 3, c = i & 7, sw = key & 7;
                                uint32_t w[4], o[8];
                                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                                             : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3])
                                             : "r"(src + key * 128 + ((c ^ sw) << 4)));
                                e4m3x16_to_bf16x16(w, o);
                                const uint32_t row = dst + (c >> 2) * KV_HALF + key * 128;
                                const int cc = 2 * (c & 3);
                                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row + ((cc ^ sw) << 4)),
                                             "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]) : "memory");
                                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row + (((cc + 1) ^ sw) << 4)),
                                             "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]) : "memory");
                            }
                            fence_proxy_async_smem();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&sm.kv_full[vb]);
                        }
                    } else if (lane == 0 && half == 0) {
                        mbar_arrive_expect_tx(&sm.kv_full[vb], 2 * KV_HALF);
                        tma_load_3d_hint(sm.kv[vb][0], &tm_v, 0, r, kv_row0, &sm.kv_full[vb], pol_kv);
                        tma_load_3d_hint(sm.kv[vb][1], &tm_v, 64, r, kv_row0, &sm.kv_full[vb], pol_kv);
                    }
                    loaded_tile = tile;
                }
                first += nq;
            }
        }
        if (*abort != 0) spin_cycles(200000);
    } else if (warp == 1) {
        // ---------------- MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_s = F8 ? make_idesc_e4m3(128, BK) : make_idesc_bf16(128, BK, false, false);
            constexpr uint32_t idesc_o = make_idesc_bf16(128, 128, false, true);
            int prev_vb = 0, prev_last = 0, prev_new = 0;
            for (int n = 0; n <= n_items; ++n) {
                int vb = 0, last = 0, nw = 0;
                if (n < n_items) {
                    const int j = n & 1;
                    if (!mbar_wait(&sm.q_full[j], (n >> 1) & 1, abort)) {
                        report_async(status, kAsyncTimeout, 0x321);
                        break;
                    }
                    const AttnItemInfo& inf = sm.info[n % kAttnInfoRing];
                    const int kb = inf.kb;
                    vb = inf.vb; last = inf.last_of_tile; nw = inf.new_tile;
                    if (nw && !mbar_wait(&sm.kv_full[kb], kv_k_parity(kb), abort)) {
                        report_async(status, kAsyncTimeout, 0x322);
                        break;
                    }
                    tc_fence_after();
                    MSA_STAMP(n, 8);
                    const uint32_t ts = tmem + j * 256;
                    if constexpr (F8) {
                        // rows of 128 fp8: dense 1 KB atoms of 8 rows, 32 bytes (32 elements) per step
                        const uint64_t qd = make_smem_desc(smem_u32(sm.q[j]), 16, 1024);
                        const uint64_t kd = make_smem_desc(smem_u32(sm.kv[kb][0]), 16, 1024);
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) mma_e4m3_ss(ts, qd + 2 * kk, kd + 2 * kk, idesc_s, kk > 0);
                    } else {
                        // Q atoms (8 rows x 64 d) of one d half are 2 KB apart; the other half sits 1 KB further.
                        const uint64_t qd0 = make_smem_desc(smem_u32(sm.q[j]), 16, 2048);
                        const uint64_t qd1 = make_smem_desc(smem_u32(sm.q[j]) + 1024, 16, 2048);
                        const uint64_t kd0 = make_smem_desc(smem_u32(sm.kv[kb][0]), 16, 1024);
                        const uint64_t kd1 = make_smem_desc(smem_u32(sm.kv[kb][1]), 16, 1024);
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) mma_bf16_ss(ts, qd0 + 2 * kk, kd0 + 2 * kk, idesc_s, kk > 0);
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) mma_bf16_ss(ts, qd1 + 2 * kk, kd1 + 2 * kk, idesc_s, true);
                    }
                    mma_commit(&sm.q_empty[j]);
                    mma_commit(&sm.s_full[j]);
                    if (last) mma_commit(&sm.kv_empty[kb]);
                    MSA_STAMP(n, 9);
                }
                if (n >= 1) {
                    const int m = n - 1, jm = m & 1;
                    if (!mbar_wait(&sm.p_full[jm], (m >> 1) & 1, abort)) {
                        report_async(status, kAsyncTimeout, 0x323);
                        break;
                    }
                    if (prev_new && !mbar_wait(&sm.kv_full[prev_vb], kv_v_parity(prev_vb), abort)) {
                        report_async(status, kAsyncTimeout, 0x324);
                        break;
                    }
                    tc_fence_after();
                    MSA_STAMP(m, 10);
                    const uint32_t ts = tmem + jm * 256, to = ts + 128;
                    // V as the MN-major B operand: next 64 columns of d are BK*128 bytes away.
                    const uint64_t vd = make_smem_desc(smem_u32(sm.kv[prev_vb][0]), BK * 128, 1024);
#pragma unroll
                    for (int kk = 0; kk < BK / 16; ++kk)  // P: 8 packed columns per 16 keys; V: 2048 bytes per 16 keys
                        mma_bf16_ts(to, ts + kk * 8, vd + (uint64_t)(kk * 2048 / 16), idesc_o, kk > 0);
                    mma_commit(&sm.o_full[jm]);
                    if (prev_last) mma_commit(&sm.kv_empty[prev_vb]);
                    MSA_STAMP(m, 11);
                }
                prev_vb = vb; prev_last = last; prev_new = nw;
            }
            if (*abort != 0) {
                mma_commit(&sm.drain);
                mbar_wait_quiet(&sm.drain, 0, 20000000);
            }
        }
    } else {
        // ---------------- softmax + epilogue: thread = row of the 128-row operand
        const int j = (warp - 2) >> 2;  // context: items n = j (mod 2)
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const int qi = row / G, g = row % G;
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        const uint32_t tmem_s = tmem + j * 256, tmem_o = tmem_s + 128;
        constexpr int QPW = 32 / G;  // queries per warp
        // staging: this thread's row goes to [query][chunk][head]; lanes < QPW copy one query each
        uint8_t* stg_row = sm.ostage[j] + (size_t)qi * O_BYTES + g * 16;
        const uint8_t* stg_query = sm.ostage[j] + (size_t)(quarter * QPW + lane) * O_BYTES;
        for (int n = j; n < n_items; n += 2) {
            if (!mbar_wait(&sm.s_full[j], (n >> 1) & 1, abort)) { report_async(status, kAsyncTimeout, 0x331); break; }
            tc_fence_after();
            if (lane == 0 && quarter == 0) MSA_STAMP(n, 0);
            const AttnItemInfo& inf = sm.info[n % kAttnInfoRing];
            const int kv_row0 = inf.kv_row0, r = inf.r, nq = inf.nq;
            const uint32_t h = inf.handle[qi];
            // handle of the query whose partial this lane hands to the bulk-copy engine
            const uint32_t h_copy = inf.handle[(quarter * QPW + lane) & 15];
            const bool valid = qi < nq;
            const int64_t ql = h >> 8;
            // Row of the query in the K/V tensors (its own position for one sequence starting at row 0, its
            // packed row in a batch); the keys of the tile at rows kv_row0.. up to that row are visible.
            const int64_t pos = p.q_begin + p.q_first + ql;
            // visible columns of this block for this query: 0..lim
            const int64_t lim64 = pos - (int64_t)kv_row0;
            const int lim = valid ? (int)(lim64 > BK - 1 ? BK - 1 : lim64) : BK - 1;

            uint32_t sv[BK / 32][32];
#pragma unroll
            for (int c = 0; c < BK / 32; ++c) tmem_ld_32x32(tmem_s + lane_base + c * 32, sv[c]);
            tmem_wait_ld();
            if (lim != BK - 1) {
#pragma unroll
                for (int c = 0; c < BK / 32; ++c)
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (c * 32 + e > lim) sv[c][e] = 0xFF800000u;  // -inf
            }
            float mx = tree_max32(sv[0]);
#pragma unroll
            for (int c = 1; c < BK / 32; ++c) mx = fmaxf(mx, tree_max32(sv[c]));
            const float mc = mx * scale_log2e;
            float ell4[4] = {0.f, 0.f, 0.f, 0.f};
            // P row (bf16 pairs) back into the first BK/2 columns of the S region.
#pragma unroll
            for (int c2 = 0; c2 < BK / 64; ++c2) {
                uint32_t pk[32];
#pragma unroll
                for (int w = 0; w < 32; ++w) {
                    const int col = c2 * 64 + 2 * w;
                    const float p0 = ex2_approx(fmaf(__uint_as_float(sv[col >> 5][col & 31]), scale_log2e, -mc));
                    const float p1 = ex2_approx(fmaf(__uint_as_float(sv[col >> 5][(col & 31) + 1]), scale_log2e, -mc));
                    ell4[w & 3] += p0 + p1;
                    const __nv_bfloat162 pb = __floats2bfloat162_rn(p0, p1);
                    pk[w] = *reinterpret_cast<const uint32_t*>(&pb);
                }
                tmem_st_32x32(tmem_s + lane_base + c2 * 32, pk);
            }
            const float ell = (ell4[0] + ell4[1]) + (ell4[2] + ell4[3]);
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.p_full[j]);
            if (lane == 0 && quarter == 0) MSA_STAMP(n, 3);

            // ---- epilogue: O row / ell -> bf16 partial (via the staging buffer), LSE partial
            // The copies of the context's previous item have read the staging buffer long ago;
            // the wait makes that certain.
            if (lane < QPW) bulk_wait_read_all();
            if (!mbar_wait(&sm.o_full[j], (n >> 1) & 1, abort)) { report_async(status, kAsyncTimeout, 0x332); break; }
            tc_fence_after();
            if (lane == 0 && quarter == 0) MSA_STAMP(n, 5);
            const float inv = 1.0f / ell;
            const float2 inv2 = make_float2(inv, inv);
            __syncwarp();
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t ov[32];
                tmem_ld_32x32(tmem_o + lane_base + c * 32, ov);
                tmem_wait_ld();
#pragma unroll
                for (int j4 = 0; j4 < 4; ++j4) {
                    uint32_t pk[4];
#pragma unroll
                    for (int w = 0; w < 4; ++w) {  // packed two-float multiply: half the instructions
                        const float2 o2 = __fmul2_rn(make_float2(__uint_as_float(ov[j4 * 8 + 2 * w]),
                                                                 __uint_as_float(ov[j4 * 8 + 2 * w + 1])), inv2);
                        const __nv_bfloat162 ob = __floats2bfloat162_rn(o2.x, o2.y);
                        pk[w] = *reinterpret_cast<const uint32_t*>(&ob);
                    }
                    *reinterpret_cast<uint4*>(stg_row + (c * 4 + j4) * (G * 16)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
            }
            tc_fence_before();
            fence_proxy_async_smem();
            __syncwarp();
            // Partial of (query, group, slot): G*256 contiguous bytes, [16-byte chunk of d][head].
            if (lane < QPW) {
                if (quarter * QPW + lane < nq) {
                    const int64_t pr = partial_base((int64_t)(h_copy >> 8), r, p) + (h_copy & 0xFF);
                    bulk_store(o_buf + pr * (G * 128), stg_query, O_BYTES);
                }
                bulk_commit();
            }
            if (valid)
                lse_buf[(partial_base(ql, r, p) + (h & 0xFF)) * G + g] = (mc + log2f(ell)) * 0.6931471805599453f;
            if (lane == 0 && quarter == 0) MSA_STAMP(n, 7);
        }
        if (lane < QPW) bulk_wait_all();  // partials still on their way out
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, TMEM_COLS);
    }
}

// ---------------------------------------------------------------- 3. combine
// One CTA per (query, KV head), G*16 threads.  Partials are stored as [16-byte chunk of d][head]
// inside each (query, group, slot) region, so thread t reads chunk t/G of head t%G and a warp
// reads 512 contiguous bytes per slot.
//   a = max_s LSE_s, LSE = a + log sum_s exp(LSE_s - a), w_s = exp(LSE_s - LSE), O = sum_s w_s O_s.
template <int BK, int G>
__global__ void __launch_bounds__(G * 16)
combine_kernel(const int32_t* __restrict__ block_idx, RangeParams p, const __nv_bfloat16* __restrict__ o_buf,
               const float* __restrict__ lse_buf, __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
    __shared__ float w_s[128][G];   // top_k <= 128
    __shared__ int valid_s[128];
    __shared__ uint4 o_s[G][16];    // final rows, [head][chunk], for a coalesced store
    const int ql = blockIdx.x / p.H_kv, r = blockIdx.x % p.H_kv;
    const int t = threadIdx.x;
    const int64_t q = p.q_first + ql;
    const int64_t loc = query_pos(p, q) / BK;
    const int32_t* sel = block_idx + (q * p.H_kv + r) * (int64_t)p.top_k;
    const int64_t pbase = partial_base(ql, r, p);
    for (int s = t; s < p.top_k; s += G * 16) {
        const int32_t b = sel[s];
        valid_s[s] = (b >= 0 && (int64_t)b <= loc) ? 1 : 0;
    }
    __syncthreads();
    {   // weights: 16 threads per head, thread j of a head owns slots j, j+16, ...
        const int g = t >> 4, j = t & 15;
        float lv[8];
        float a = -INFINITY;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int s = j + 16 * u;
            lv[u] = (s < p.top_k && valid_s[s]) ? lse_buf[(pbase + s) * G + g] : -INFINITY;
            a = fmaxf(a, lv[u]);
        }
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
        float sum = 0.f;
#pragma unroll
        for (int u = 0; u < 8; ++u) sum += (lv[u] > -INFINITY) ? expf(lv[u] - a) : 0.f;
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        const float L = a + logf(sum);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int s = j + 16 * u;
            if (s < p.top_k) w_s[s][g] = (lv[u] > -INFINITY) ? expf(lv[u] - L) : 0.f;
        }
        if (j == 0 && lse != nullptr) lse[q * (int64_t)(p.H_kv * G) + r * G + g] = L;
    }
    __syncthreads();
    const int g = t % G, ch = t / G;  // head, 16-byte chunk of d
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
    const uint4* src = reinterpret_cast<const uint4*>(o_buf + pbase * (G * 128)) + t;
#pragma unroll 8
    for (int s = 0; s < p.top_k; ++s) {
        if (!valid_s[s]) continue;
        const uint4 x = __ldg(src + (int64_t)s * (G * 16));
        const float w = w_s[s][g];
        const float2 a0 = bf16x2_to_float2(x.x), a1 = bf16x2_to_float2(x.y);
        const float2 a2 = bf16x2_to_float2(x.z), a3 = bf16x2_to_float2(x.w);
        acc[0] = fmaf(w, a0.x, acc[0]); acc[1] = fmaf(w, a0.y, acc[1]);
        acc[2] = fmaf(w, a1.x, acc[2]); acc[3] = fmaf(w, a1.y, acc[3]);
        acc[4] = fmaf(w, a2.x, acc[4]); acc[5] = fmaf(w, a2.y, acc[5]);
        acc[6] = fmaf(w, a3.x, acc[6]); acc[7] = fmaf(w, a3.y, acc[7]);
    }
    uint32_t pk[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat162 ob = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
        pk[i] = *reinterpret_cast<const uint32_t*>(&ob);
    }
    o_s[g][ch] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
    __syncthreads();
    // out[q, r*G + head, :]: the G rows are contiguous, G*256 bytes = G*16 chunks in order
    reinterpret_cast<uint4*>(out + (q * (int64_t)(p.H_kv * G) + r * G) * 128)[t] = o_s[t >> 4][t & 15];
}

}  // namespace msa
