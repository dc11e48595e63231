// Section 4.3 ("LSE fusion"): the index branch's log-sum-exp over the selected blocks,
//   LSE_idx[i,r] = log sum_{b in I[i,r]} sum_{j in block b, j <= i} exp(<Q_idx[i,r], K_idx[j]> * scale),
// as a forward output for the sparse-KL backward.  Computed after Top-k, for the selected blocks
// only (per-block log-sum-exps inside the scoring kernel would cost four times that kernel's time
// on the exponential unit), in KV-outer order like the attention: the reverse index gives, per
// (block, head) tile, the (query, slot) pairs that selected it; an item is up to 128 of them; the
// item's 128 x B_k scores come from warp-level tensor-core MMAs (the pass is 1.6 % of the scoring
// FLOPs), each row's masked log-sum-exp goes to its (query, head, slot) place, and a second kernel
// reduces a row's slots.
#pragma once

#include "attn_prefill_tc.cuh"

namespace msa {

constexpr int kLseItemQueries = 128;
constexpr int kLseThreads = 256;  // 8 warps x 16 queries

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* smem_row) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(smem_u32(smem_row)));
}
__device__ __forceinline__ void ldmatrix_x2(uint32_t (&r)[2], const void* smem_row) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];"
                 : "=r"(r[0]), "=r"(r[1])
                 : "r"(smem_u32(smem_row)));
}
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, "
                 "{%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// One CTA walks a contiguous share of the items.  q_idx: rows of the call [q_count, H_kv, DIDX]; k_idx: [kv_len, DIDX].
// part: [range query][head][slot] natural-log partials.
template <int BK, int DIDX>
__global__ void __launch_bounds__(kLseThreads)
index_lse_kernel(const __nv_bfloat16* __restrict__ q_idx, const __nv_bfloat16* __restrict__ k_idx,
                 RangeParams p, int64_t kv_len, const int32_t* __restrict__ tile_off,
                 const int32_t* __restrict__ item_off, const uint32_t* __restrict__ handles,
                 float scale_log2e, float* __restrict__ part) {
    constexpr int LD = DIDX + 8;  // padded row (bf16): conflict-free ldmatrix
    constexpr int CH = DIDX / 8;  // 16-byte chunks per row
    constexpr int NCH = kLseItemQueries * CH / kLseThreads;  // chunks of a query tile gathered by one thread
    extern __shared__ __align__(16) uint8_t lse_smem[];
    __nv_bfloat16* Ks = reinterpret_cast<__nv_bfloat16*>(lse_smem);        // [BK][LD]
    __nv_bfloat16* Qs0 = Ks + BK * LD;                                     // [2][128][LD]: this item's and the next one's queries
    uint32_t* hs0 = reinterpret_cast<uint32_t*>(Qs0 + 2 * kLseItemQueries * LD);  // [2][128] handles
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = p.n_blocks * p.H_kv;
    const int total_items = item_off[n_tiles];

    // a contiguous share of the item list per CTA: consecutive items mostly share their key block
    const int per_cta = (total_items + (int)gridDim.x - 1) / (int)gridDim.x;
    const int it_lo = min(total_items, (int)blockIdx.x * per_cta), it_hi = min(total_items, it_lo + per_cta);
    if (it_lo >= it_hi) return;
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
    // The gather of item `it` into buffer `buf`: per row its handle, then DIDX*2 bytes of its index
    // vector as asynchronous 16-byte copies; the next item's gather is in flight while this item's
    // scores are computed.
    auto fetch = [&](int it, int buf, int& tile, int& nq) {
        while (w_next <= it) {  // crossed into the next non-empty tile
            ++w_tile;
            w_next = item_off[w_tile + 1];
        }
        tile = w_tile;
        const int first = tile_off[w_tile] + (it - item_off[w_tile]) * kLseItemQueries;
        nq = min(kLseItemQueries, tile_off[w_tile + 1] - first);
        const int r = tile / p.n_blocks;
        __nv_bfloat16* Qs = Qs0 + buf * (kLseItemQueries * LD);
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
            if (row < nq) {  // rows past nq keep stale (finite or not, never written back) data
                const int64_t ql = hh[j] >> 8;
                const __nv_bfloat16* src = q_idx + ((p.q_first + ql) * p.H_kv + r) * DIDX + ch * 8;
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(Qs + row * LD + ch * 8)), "l"(src)
                             : "memory");
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    int loaded_tile = -1;
    int tile, nq;
    fetch(it_lo, 0, tile, nq);
    for (int it = it_lo; it < it_hi; ++it) {
        const int buf = (it - it_lo) & 1;
        int tile_n = 0, nq_n = 0;
        if (it + 1 < it_hi) fetch(it + 1, buf ^ 1, tile_n, nq_n);
        const int r = tile / p.n_blocks, b = tile - r * p.n_blocks;  // tiles are numbered head after head
        // K_idx block: BK rows of DIDX bf16, 16-byte chunks; rows past the sequence are zero (masked below)
        for (int e = threadIdx.x; tile != loaded_tile && e < BK * CH; e += kLseThreads) {
            const int row = e / CH, ch = e % CH;
            const int64_t j = (int64_t)b * BK + row;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (j < kv_len) v = __ldg(reinterpret_cast<const uint4*>(k_idx + j * DIDX) + ch);
            *reinterpret_cast<uint4*>(Ks + row * LD + ch * 8) = v;
        }
        if (it + 1 < it_hi) asm volatile("cp.async.wait_group 1;" ::: "memory");
        else asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();  // this item's queries and handles, and the key block, are in shared memory
        const __nv_bfloat16* Qs = Qs0 + buf * (kLseItemQueries * LD);
        const uint32_t* hs = hs0 + buf * kLseItemQueries;

        // scores of 16 queries (this warp) x BK keys
        float acc[BK / 8][4];
#pragma unroll
        for (int nt = 0; nt < BK / 8; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < DIDX / 16; ++ks) {
            uint32_t a[4];
            ldmatrix_x4(a, Qs + (warp * 16 + (lane & 15)) * LD + ks * 16 + (lane >> 4) * 8);
#pragma unroll
            for (int nt = 0; nt < BK / 8; ++nt) {
                uint32_t bb[2];
                ldmatrix_x2(bb, Ks + (nt * 8 + (lane & 7)) * LD + ks * 16 + ((lane >> 3) & 1) * 8);
                mma_16816(acc[nt], a, bb);
            }
        }
        // rows lane/4 and lane/4 + 8 of the warp's 16; columns nt*8 + (lane%4)*2 + {0,1}
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int row = warp * 16 + (lane >> 2) + half * 8;
            const uint32_t h = hs[row];
            const int64_t pos = p.q_begin + p.q_first + (int64_t)(h >> 8);
            const int64_t lim = pos - (int64_t)b * BK;  // visible columns 0..lim
            float mx = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < BK / 8; ++nt)
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const int col = nt * 8 + (lane & 3) * 2 + c;
                    float& x = acc[nt][half * 2 + c];
                    x = col <= lim ? x * scale_log2e : -INFINITY;
                    mx = fmaxf(mx, x);
                }
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            float sum = 0.f;
#pragma unroll
            for (int nt = 0; nt < BK / 8; ++nt)
#pragma unroll
                for (int c = 0; c < 2; ++c) sum += exp2f(acc[nt][half * 2 + c] - mx);
            sum += __shfl_xor_sync(0xffffffffu, sum, 1);
            sum += __shfl_xor_sync(0xffffffffu, sum, 2);
            if ((lane & 3) == 0 && row < nq)
                part[((int64_t)(h >> 8) * p.H_kv + r) * p.top_k + (h & 0xFF)] = (mx + log2f(sum)) * 0.6931471805599453f;
        }
        loaded_tile = tile;
        __syncthreads();  // this buffer and the key block are free for the gathers and loads of later items
        tile = tile_n;
        nq = nq_n;
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
