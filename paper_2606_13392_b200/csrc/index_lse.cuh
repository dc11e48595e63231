// Section 4.3 ("LSE fusion"): the index branch's log-sum-exp over the selected blocks,
//   LSE_idx[i,r] = log sum_{b in I[i,r]} sum_{j in block b, j <= i} exp(<Q_idx[i,r], K_idx[j]> * scale),
// as a forward output for the sparse-KL backward.  Computed after Top-k, for the selected blocks
// only (per-block log-sum-exps inside the scoring kernel would cost four times that kernel's time
// on the exponential unit), in KV-outer order like the attention: the reverse index gives, per
// (block, head) tile, the (query, slot) pairs that selected it; an item is up to 128 of them; the
// item's 128 x B_k scores come from tcgen05 MMAs (the pass is 1.6 % of the scoring FLOPs, its cost
// is the B_k exponentials per row), each row's masked log-sum-exp goes to its (query, head, slot)
// place, and a second kernel reduces a row's slots.
#pragma once

#include "attn_prefill_tc.cuh"

namespace msa {

constexpr int kLseItemQueries = 128;
constexpr int kLseThreads = 256;  // all gather; the first four warps (thread = row) take the exponentials

// Byte offset of 16-byte chunk `ch` (0 .. DIDX/8) of row `row` in an operand tile of ROWS rows kept as
// 64-element atoms [atom][row][128 bytes] with the 128-byte swizzle the tensor-core descriptors expect.
template <int ROWS>
__device__ __forceinline__ uint32_t lse_tile_off(int row, int ch) {
    return (uint32_t)((ch >> 3) * (ROWS * 128) + row * 128 + (((ch & 7) ^ (row & 7)) << 4));
}

// One CTA walks a contiguous share of the items.  q_idx: rows of the call [q_count, H_kv, DIDX]; k_idx: [kv_len, DIDX].
// part: [range query][head][slot] natural-log partials.
// Per item: the 128 query rows are gathered into a swizzled operand tile with asynchronous 16-byte
// copies (the next item's gather runs while this item is computed), one thread issues
// S = Q_idx K_idx^T as tcgen05 MMAs (M = 128, N = B_k) into the CTA's tensor-memory columns, and the
// first four warps - thread = row - read their row back in chunks of 32 columns, once for the
// masked maximum and once for the sum of exponentials.  Several CTAs share an SM (B_k TMEM columns
// each), which is what overlaps one CTA's MMAs with another's exponentials.
template <int BK, int DIDX>
__global__ void __launch_bounds__(kLseThreads)
index_lse_kernel(const __nv_bfloat16* __restrict__ q_idx, const __nv_bfloat16* __restrict__ k_idx,
                 RangeParams p, int64_t kv_len, const int32_t* __restrict__ tile_off,
                 const int32_t* __restrict__ item_off, const uint32_t* __restrict__ handles,
                 float scale_log2e, float* __restrict__ part, int* status) {
    constexpr int CH = DIDX / 8;     // 16-byte chunks per row
    constexpr int ATOMS = DIDX / 64;
    constexpr int NCH = kLseItemQueries * CH / kLseThreads;  // chunks of a query tile gathered by one thread
    constexpr int K_BYTES = ATOMS * BK * 128, Q_BYTES = ATOMS * kLseItemQueries * 128;
    extern __shared__ uint8_t lse_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(lse_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* Ks = base;                       // key block
    uint8_t* Qs0 = Ks + K_BYTES;              // [2]: this item's and the next one's queries
    uint32_t* hs0 = reinterpret_cast<uint32_t*>(Qs0 + 2 * Q_BYTES);  // [2][128] handles
    __shared__ alignas(8) uint64_t done_bar;
    __shared__ uint32_t tmem_holder;
    __shared__ int abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = p.n_blocks * p.H_kv;
    const int total_items = item_off[n_tiles];

    // a contiguous share of the item list per CTA: consecutive items mostly share their key block
    const int per_cta = (total_items + (int)gridDim.x - 1) / (int)gridDim.x;
    const int it_lo = min(total_items, (int)blockIdx.x * per_cta), it_hi = min(total_items, it_lo + per_cta);
    if (it_lo >= it_hi) return;
    if (threadIdx.x == 0) {
        mbar_init(&done_bar, 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0) tmem_alloc(&tmem_holder, BK);  // B_k columns: at most four CTAs per SM fit in 512
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_holder;
    volatile int* abort = &abort_flag;
    // Every thread walks the tile list for the item being fetched (uniform loads): a search for the
    // first item, then steps.
    int w_tile, w_next;
    {   // last tile whose first item is <= it_lo (skips empty tiles)
        int lo = 0, hi = n_tiles;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (item_off[mid] <= it_lo) lo = mid; else hi = mid;
        }
        w_tile = lo;
        w_next = item_off[lo + 1];
    }
    auto fetch = [&](int it, int buf, int& tile, int& nq) {
        while (w_next <= it) {  // crossed into the next non-empty tile
            ++w_tile;
            w_next = item_off[w_tile + 1];
        }
        tile = w_tile;
        const int first = tile_off[w_tile] + (it - item_off[w_tile]) * kLseItemQueries;
        nq = min(kLseItemQueries, tile_off[w_tile + 1] - first);
        const int r = tile / p.n_blocks;
        uint8_t* Qs = Qs0 + buf * Q_BYTES;
        uint32_t* hs = hs0 + buf * kLseItemQueries;
        uint32_t hh[NCH];
#pragma unroll
        for (int j = 0; j < NCH; ++j) {
            const int row = ((int)threadIdx.x + j * kLseThreads) / CH;
            hh[j] = row < nq ? __ldg(handles + first + row) : 0u;
        }
#pragma unroll
        for (int j = 0; j < NCH; ++j) {
            const int e = (int)threadIdx.x + j * kLseThreads, row = e / CH, ch = e % CH;
            if (ch == 0) hs[row] = hh[j];
            if (row < nq) {  // rows past nq keep stale data: their scores are never written back
                const int64_t ql = hh[j] >> 8;
                const __nv_bfloat16* src = q_idx + ((p.q_first + ql) * p.H_kv + r) * DIDX + ch * 8;
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(
                                 smem_u32(Qs + lse_tile_off<kLseItemQueries>(row, ch))), "l"(src)
                             : "memory");
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    int loaded_tile = -1;
    int tile, nq;
    fetch(it_lo, 0, tile, nq);
    for (int it = it_lo; it < it_hi; ++it) {
        const int n = it - it_lo, buf = n & 1;
        int tile_n = 0, nq_n = 0;
        if (it + 1 < it_hi) fetch(it + 1, buf ^ 1, tile_n, nq_n);
        const int r = tile / p.n_blocks, b = tile - r * p.n_blocks;  // tiles are numbered head after head
        // K_idx block: BK rows of DIDX bf16, 16-byte chunks; rows past the sequence are zero (masked below)
        for (int e = threadIdx.x; tile != loaded_tile && e < BK * CH; e += kLseThreads) {
            const int row = e / CH, ch = e % CH;
            const int64_t j = (int64_t)b * BK + row;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (j < kv_len) v = __ldg(reinterpret_cast<const uint4*>(k_idx + j * DIDX) + ch);
            *reinterpret_cast<uint4*>(Ks + lse_tile_off<BK>(row, ch)) = v;
        }
        if (it + 1 < it_hi) asm volatile("cp.async.wait_group 1;" ::: "memory");
        else asm volatile("cp.async.wait_group 0;" ::: "memory");
        fence_proxy_async_smem();  // the tiles were written through the generic proxy; the MMAs read them through the async one
        __syncthreads();           // this item's queries and handles, and the key block, are in shared memory
        const uint8_t* Qs = Qs0 + buf * Q_BYTES;
        const uint32_t* hs = hs0 + buf * kLseItemQueries;
        if (threadIdx.x == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(kLseItemQueries, BK, false, false);
            tc_fence_after();
#pragma unroll
            for (int a = 0; a < ATOMS; ++a) {
                const uint64_t a_desc = make_smem_desc(smem_u32(Qs) + a * (kLseItemQueries * 128), 16, 1024);
                const uint64_t b_desc = make_smem_desc(smem_u32(Ks) + a * (BK * 128), 16, 1024);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)  // 16 bf16 = 32 bytes = 2 descriptor units per K step
                    mma_bf16_ss(tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (a | kk) > 0);
            }
            mma_commit(&done_bar);
        }
        if (warp < 4) {  // thread = row of the item (TMEM lane)
            const int row = threadIdx.x;
            const uint32_t h = hs[row];
            const int64_t pos = p.q_begin + p.q_first + (int64_t)(h >> 8);
            const int64_t lim64 = pos - (int64_t)b * BK;  // visible columns 0..lim
            const int lim = (int)(lim64 > BK - 1 ? BK - 1 : lim64);
            const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16);
            if (!mbar_wait(&done_bar, n & 1, abort)) {
                if (lane == 0) report_async(status, kAsyncTimeout, 0x161);
            } else {
                tc_fence_after();
                // Two passes over the row in chunks of 32 columns (maximum, then the sum of exponentials):
                // 64 registers per thread keep four CTAs on an SM, which a one-pass form with two
                // chunks in flight does not (measured slower).
                float mx = -INFINITY;
#pragma unroll
                for (int c = 0; c < BK / 32; ++c) {
                    uint32_t v[32];
                    tmem_ld_32x32(taddr + c * 32, v);
                    tmem_wait_ld();
                    if (lim < c * 32 + 31) {
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (c * 32 + e > lim) v[e] = 0xFF800000u;  // -inf
                    }
                    mx = fmaxf(mx, tree_max32(v));
                }
                const float mc = mx * scale_log2e;
                float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int c = 0; c < BK / 32; ++c) {
                    uint32_t v[32];
                    tmem_ld_32x32(taddr + c * 32, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const float x = c * 32 + e <= lim ? ex2_approx(fmaf(__uint_as_float(v[e]), scale_log2e, -mc)) : 0.f;
                        s4[e & 3] += x;
                    }
                }
                const float sum = (s4[0] + s4[1]) + (s4[2] + s4[3]);
                if (row < nq)
                    part[((int64_t)(h >> 8) * p.H_kv + r) * p.top_k + (h & 0xFF)] = (mc + log2f(sum)) * 0.6931471805599453f;
            }
            tc_fence_before();
        }
        loaded_tile = tile;
        __syncthreads();  // TMEM, this buffer and the key block are free for the next items
        if (*abort != 0) break;
        tile = tile_n;
        nq = nq_n;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, BK);
    }
}

// One warp per (query, head) row: log-sum-exp of the row's valid slots.
template <int BK>
__global__ void __launch_bounds__(256)
index_lse_reduce_kernel(const int32_t* __restrict__ block_idx, RangeParams p, const float* __restrict__ part,
                        float* __restrict__ lse_idx) {
    const int row = (int)((blockIdx.x * (unsigned)blockDim.x + threadIdx.x) >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= p.q_count * p.H_kv) return;
    const int ql = row / p.H_kv;
    const int64_t q = p.q_first + ql;
    const int64_t loc = (p.q_begin + q) / BK;
    const int32_t* sel = block_idx + (q * p.H_kv + (row - ql * p.H_kv)) * (int64_t)p.top_k;
    float v[4];
    float mx = -INFINITY;
#pragma unroll
    for (int u = 0; u < 4; ++u) {  // top_k <= 128
        const int s = lane + 32 * u;
        v[u] = -INFINITY;
        if (s < p.top_k) {
            const int32_t b = sel[s];
            if (b >= 0 && (int64_t)b <= loc) v[u] = part[(int64_t)row * p.top_k + s];
        }
        mx = fmaxf(mx, v[u]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float sum = 0.f;
#pragma unroll
    for (int u = 0; u < 4; ++u) sum += v[u] > -INFINITY ? expf(v[u] - mx) : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0) lse_idx[q * p.H_kv + (row - ql * p.H_kv)] = mx > -INFINITY ? mx + logf(sum) : -INFINITY;
}

// Any shape (no tensor cores, no reuse of key blocks between queries): one warp per (query,
// head) row walks its selected blocks; lanes take keys, the row's sum is kept online.
template <bool F8>
__global__ void __launch_bounds__(256)
index_lse_generic_kernel(const void* __restrict__ q_idx, const void* __restrict__ k_idx,
                         const int32_t* __restrict__ block_idx, int64_t q_begin, int64_t q_count, int64_t kv_len,
                         int H_kv, int d_idx, int B_k, int top_k, float scale, float* __restrict__ lse_idx) {
    const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (row >= q_count * H_kv) return;
    const int64_t q = row / H_kv;
    const int64_t pos = q_begin + q, loc = pos / B_k;
    constexpr int ELT = F8 ? 1 : 2;
    const char* qrow = static_cast<const char*>(q_idx) + row * d_idx * ELT;
    const int32_t* sel = block_idx + row * top_k;
    float mx = -INFINITY, sum = 0.f;
    for (int s = 0; s < top_k; ++s) {
        const int32_t b = sel[s];
        if (b < 0 || (int64_t)b > loc) continue;
        for (int t = lane; t < B_k; t += 32) {
            const int64_t j = (int64_t)b * B_k + t;
            if (j > pos || j >= kv_len) continue;
            const char* krow = static_cast<const char*>(k_idx) + j * d_idx * ELT;
            float dot = 0.f;
            for (int c = 0; c < d_idx; ++c) dot = fmaf(idx_elem<F8>(qrow, c), idx_elem<F8>(krow, c), dot);
            const float x = dot * scale;
            if (x > mx) { sum = sum * expf(mx - x) + 1.f; mx = x; }
            else sum += expf(x - mx);
        }
    }
    // merge the lanes' (max, sum) pairs
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, mx, o), s2 = __shfl_xor_sync(0xffffffffu, sum, o);
        const float m = fmaxf(mx, m2);
        sum = (mx > -INFINITY ? sum * expf(mx - m) : 0.f) + (m2 > -INFINITY ? s2 * expf(m2 - m) : 0.f);
        mx = m;
    }
    if (lane == 0) lse_idx[row] = mx > -INFINITY ? mx + logf(sum) : -INFINITY;
}

}  // namespace msa
