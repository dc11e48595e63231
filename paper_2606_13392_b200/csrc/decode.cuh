// Decode path (one query per cached sequence): HBM-bound streaming kernels.
//
//   index_scores_decode_kernel : Eq. 6 for the last token of every sequence.  One warp per key
//       block streams the block's K_idx rows straight from global memory into mma.sync
//       B fragments (no shared memory) and keeps the per-group running maximum.
//   attn_decode_kernel         : Eq. 8.  Persistent CTAs; a producer warp streams the selected
//       K/V blocks through a TMA ring in shared memory, four consumer warps each own 32 keys
//       of every block (S = Q K^T with mma.sync, online softmax in registers, O^T += V^T P^T).
//   attn_decode_combine_kernel : merges the per-warp partials of a sequence (Section 4.2
//       combine).
#pragma once

#include "tc_common.cuh"

namespace msa {

__device__ __forceinline__ void mma_m16n8k16_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                                  uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// fp8 E4M3 operands, 32 contraction elements: the same register roles as m16n8k16 with four
// fp8 per register instead of two bf16.
__device__ __forceinline__ void mma_m16n8k32_e4m3(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                                  uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.f32.e4m3.e4m3.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t smem_addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(smem_addr));
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t smem_addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(smem_addr));
}

__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// ------------------------------------------------------------------ stage 1, decode
// d_idx = 32*NSEG (64 or 128), H_kv <= 8, any B_k.  A = Q_idx padded to 16 rows.
// The contraction index is permuted identically in A and B so that a lane's B fragment for
// two consecutive k-steps is one 16-byte load: within a 32-wide segment of d, lane quad
// position t owns d[8t..8t+7]; k-step 0 uses d[8t..8t+3], k-step 1 uses d[8t+4..8t+7].
// F8: rows of 64*NSEG fp8 E4M3 occupy the same bytes as 32*NSEG bf16, and the fp8 MMA takes 32
// contraction elements from the registers that hold 16 bf16, so the same loads feed it: within a
// 64-wide segment of d, lane quad position t owns d[16t..16t+15].
constexpr int kIdxDecWarps = 8;

template <int UNROLL, int NSEG, bool F8 = false>
__global__ void __launch_bounds__(kIdxDecWarps * 32)
index_scores_decode_kernel(const __nv_bfloat16* __restrict__ q_idx, const __nv_bfloat16* __restrict__ k_idx,
                           const int64_t* __restrict__ seq_offsets, const int32_t* __restrict__ seq_lens,
                           int batch, int H_kv, int B_k, float scale, float* __restrict__ scores,
                           int64_t ld_scores, int64_t n_cols) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    // Global list of (sequence, block) work items, including the -inf tail blocks of short
    // sequences; dealt to warps round-robin, so neighbouring warps stream neighbouring blocks.
    const int64_t total = (int64_t)batch * n_cols;
    const int64_t n_warps = (int64_t)gridDim.x * kIdxDecWarps;
    int64_t it = (int64_t)blockIdx.x * kIdxDecWarps + warp;
    const int64_t it_end = total;
    int cur_seq = -1;
    constexpr int D = 32 * NSEG;
    uint32_t qa[4 * NSEG];  // A fragments of the current sequence's query: [segment][k-step][lo/hi]
    int64_t len = 0, base = 0;
    for (; it < it_end; it += n_warps) {
        const int s = (int)(it / n_cols);
        const int64_t b = it - (int64_t)s * n_cols;
        if (s != cur_seq) {
            cur_seq = s;
            len = seq_lens[s];
            base = seq_offsets[s];
#pragma unroll
            for (int i = 0; i < 4 * NSEG; ++i) qa[i] = 0u;
            if (g < H_kv) {
                const uint4* qrow = reinterpret_cast<const uint4*>(q_idx + ((int64_t)s * H_kv + g) * D);
#pragma unroll
                for (int seg = 0; seg < NSEG; ++seg) {
                    const uint4 v = __ldg(qrow + seg * 4 + t);
                    qa[seg * 4 + 0] = v.x; qa[seg * 4 + 1] = v.y;  // k-step 0: a0a1, a4a5
                    qa[seg * 4 + 2] = v.z; qa[seg * 4 + 3] = v.w;  // k-step 1
                }
            }
        }
        float* out = scores + ((int64_t)s * H_kv) * ld_scores + b;
        const int64_t j0 = b * B_k;
        if (j0 >= len) {  // block beyond this sequence: -inf (Eq. 6)
            if (lane < H_kv) out[(int64_t)lane * ld_scores] = -INFINITY;
            continue;
        }
        const int64_t pos = len - 1;
        int n_vis = (int)((pos - j0 + 1) < B_k ? (pos - j0 + 1) : B_k);
        const int n_nt = (n_vis + 7) >> 3;  // 8-key tiles that hold a visible key
        float best0 = -INFINITY, best1 = -INFINITY;
        const __nv_bfloat16* kb = k_idx + (base + j0) * D;
        for (int nt0 = 0; nt0 < n_nt; nt0 += UNROLL) {
            uint4 kv[UNROLL][NSEG];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int nt = nt0 + u;
                // rows past the visible range are clamped (loaded but masked below)
                int row = nt * 8 + g;
                if (row > n_vis - 1) row = n_vis - 1;
                const uint4* krow = reinterpret_cast<const uint4*>(kb + (int64_t)row * D);
#pragma unroll
                for (int seg = 0; seg < NSEG; ++seg) kv[u][seg] = ldg_stream(krow + seg * 4 + t);
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int nt = nt0 + u;
                if (nt < n_nt) {
                    float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int seg = 0; seg < NSEG; ++seg) {
                        if constexpr (F8) {
                            mma_m16n8k32_e4m3(c, qa[seg * 4], 0u, qa[seg * 4 + 1], 0u, kv[u][seg].x, kv[u][seg].y);
                            mma_m16n8k32_e4m3(c, qa[seg * 4 + 2], 0u, qa[seg * 4 + 3], 0u, kv[u][seg].z, kv[u][seg].w);
                        } else {
                            mma_m16n8k16_bf16(c, qa[seg * 4], 0u, qa[seg * 4 + 1], 0u, kv[u][seg].x, kv[u][seg].y);
                            mma_m16n8k16_bf16(c, qa[seg * 4 + 2], 0u, qa[seg * 4 + 3], 0u, kv[u][seg].z, kv[u][seg].w);
                        }
                    }
                    // c[0], c[1]: group g, keys nt*8 + 2t, +1
                    const int key = nt * 8 + 2 * t;
                    if (key < n_vis) best0 = fmaxf(best0, c[0]);
                    if (key + 1 < n_vis) best1 = fmaxf(best1, c[1]);
                }
            }
        }
        float best = fmaxf(best0, best1);
        best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, 1));
        best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, 2));
        if (t == 0 && g < H_kv) out[(int64_t)g * ld_scores] = best * scale;
    }
}

// ------------------------------------------------------------------ stage 3, decode
constexpr int kDecStages = 3;         // 96 KB of tiles at B_k = 128: two CTAs per SM (measured a little ahead of one CTA with six)
constexpr int kDecThreads = 160;      // warp 0: TMA producer, warps 1-4: consumers
constexpr int kDecBlocksPerItem = 8;  // selected blocks streamed by one work item
constexpr int kDecPartsPerItem = 4;   // one partial per consumer warp

template <int BK>
struct DecSmem {
    alignas(1024) uint8_t tile[kDecStages][2][BK * 128];  // [stage][d half][key][64 bf16], 128-byte swizzle
    alignas(8) uint64_t full[kDecStages];
    uint64_t empty[kDecStages];
    int abort;
};

struct DecParams {
    const __nv_bfloat16* q;         // [batch, H_q, 128]
    const int32_t* block_idx;       // [batch, H_kv, top_k]
    const int64_t* seq_offsets;
    const int32_t* seq_lens;
    float* part_o;                  // [items*4, G, 128]
    float* part_ml;                 // [items*4, 2, G]  (running max in log2 units, sum)
    int batch, H_kv, top_k, n_split;
    float scale_log2e;
};

// A register of a transposed V fragment holds one d of two consecutive keys (`key` in the low
// half, `key + 1` in the high half).  Keys past `lim` are not part of the sequence: their P is
// exactly 0, but the cache rows there may be uninitialised (NaN or Inf), and 0 * NaN is NaN, so
// their V values are replaced with zeros.
__device__ __forceinline__ uint32_t keep_visible_pair(uint32_t v, int key, int lim) {
    return (key <= lim ? (v & 0x0000FFFFu) : 0u) | (key + 1 <= lim ? (v & 0xFFFF0000u) : 0u);
}

// 16-byte chunk `chunk` (0..15 over d) of key row `key` inside a swizzled K or V tile.
template <int BK>
__device__ __forceinline__ uint32_t dec_tile_addr(uint32_t tile_base, int key, int chunk) {
    return tile_base + (uint32_t)((chunk >> 3) * (BK * 128) + key * 128 + (((chunk & 7) ^ (key & 7)) << 4));
}

template <int BK, int G>
__global__ void __launch_bounds__(kDecThreads, 2)
attn_decode_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                   DecParams p, int* status) {
    constexpr int KPW = BK / 4;    // keys per consumer warp
    constexpr int NT = KPW / 8;    // 8-key score tiles per warp
    constexpr int KS = KPW / 16;   // 16-key steps of the second product
    constexpr uint32_t TILE_BYTES = 2 * BK * 128;
    extern __shared__ uint8_t smem_raw[];
    DecSmem<BK>& sm = *reinterpret_cast<DecSmem<BK>*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abort = &sm.abort;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kDecStages; ++s) { mbar_init(&sm.full[s], 1); mbar_init(&sm.empty[s], 4); }
        sm.abort = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
    }
    __syncthreads();
    const int n_items = p.batch * p.H_kv * p.n_split;
    constexpr int HG = G / 8;  // half-groups of 8 heads: rows 0-7 and 8-15 of the 16-row MMA
    const int H_q = p.H_kv * G;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t sc = 0;  // tiles issued so far
            bool ok = true;
            for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
                const int u = item / p.n_split, sp = item - u * p.n_split;
                const int seq = u / p.H_kv, r = u - seq * p.H_kv;
                const int64_t len = p.seq_lens[seq], base = p.seq_offsets[seq];
                const int64_t loc = (len - 1) / BK;
                const int32_t* sel = p.block_idx + (int64_t)u * p.top_k;
                for (int e = sp * kDecBlocksPerItem; ok && e < min(p.top_k, (sp + 1) * kDecBlocksPerItem); ++e) {
                    const int32_t b = sel[e];
                    if (b < 0 || (int64_t)b > loc) {
                        if (b != -1) report_async(status, kAsyncBadIndex, 0x401);
                        continue;
                    }
                    const int tok = (int)(base + (int64_t)b * BK);
                    for (int kv = 0; kv < 2; ++kv, ++sc) {
                        const int st = sc % kDecStages;
                        if (!mbar_wait(&sm.empty[st], ((sc / kDecStages) & 1) ^ 1, abort)) {
                            report_async(status, kAsyncTimeout, 0x402);
                            ok = false;
                            break;
                        }
                        mbar_arrive_expect_tx(&sm.full[st], TILE_BYTES);
                        const CUtensorMap* tm = kv == 0 ? &tm_k : &tm_v;
                        tma_load_3d(sm.tile[st][0], tm, 0, r, tok, &sm.full[st]);
                        tma_load_3d(sm.tile[st][1], tm, 64, r, tok, &sm.full[st]);
                    }
                }
            }
            if (*abort != 0) spin_cycles(200000);
        }
    } else {
        const int w = warp - 1;
        const int g = lane >> 2, t = lane & 3;
        uint32_t sc = 0;
        bool ok = true;
        for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
            const int u = item / p.n_split, sp = item - u * p.n_split;
            const int seq = u / p.H_kv, r = u - seq * p.H_kv;
            const int64_t len = p.seq_lens[seq];
            const int64_t pos = len - 1, loc = pos / BK;
            const int32_t* sel = p.block_idx + (int64_t)u * p.top_k;
            // A fragments of Q: rows 0-7 = heads 0-7 of the group, rows 8-15 = heads 8-15 (G = 16)
            // or zero padding (G = 8)
            uint32_t qa[8][4];
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) qa[ks][0] = qa[ks][1] = qa[ks][2] = qa[ks][3] = 0u;
#pragma unroll
            for (int hg = 0; hg < HG; ++hg) {
                const __nv_bfloat16* qrow = p.q + ((int64_t)seq * H_q + r * G + hg * 8 + g) * 128;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    qa[ks][hg] = *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 2 * t);
                    qa[ks][2 + hg] = *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8 + 2 * t);
                }
            }
            float m_run[HG], l_part[HG];
            float acc[HG][8][4];
#pragma unroll
            for (int hg = 0; hg < HG; ++hg) {
                m_run[hg] = -INFINITY; l_part[hg] = 0.f;
#pragma unroll
                for (int mt = 0; mt < 8; ++mt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[hg][mt][i] = 0.f;
            }

            for (int e = sp * kDecBlocksPerItem; ok && e < min(p.top_k, (sp + 1) * kDecBlocksPerItem); ++e) {
                const int32_t b = sel[e];
                if (b < 0 || (int64_t)b > loc) continue;
                // ---- K tile: S[head][keys of this warp]; c[.][0,1] = head g, c[.][2,3] = head 8+g
                int st = sc % kDecStages;
                if (!mbar_wait(&sm.full[st], (sc / kDecStages) & 1, abort)) {
                    if (lane == 0) report_async(status, kAsyncTimeout, 0x411);
                    ok = false;
                    break;
                }
                uint32_t tb = smem_u32(sm.tile[st][0]);
                float c[NT][4];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0.f;
                    const int key = w * KPW + nt * 8 + (lane & 7);
#pragma unroll
                    for (int kc = 0; kc < 4; ++kc) {
                        uint32_t r4[4];
                        ldmatrix_x4(r4, dec_tile_addr<BK>(tb, key, kc * 4 + (lane >> 3)));
                        mma_m16n8k16_bf16(c[nt], qa[2 * kc][0], qa[2 * kc][1], qa[2 * kc][2], qa[2 * kc][3], r4[0], r4[1]);
                        mma_m16n8k16_bf16(c[nt], qa[2 * kc + 1][0], qa[2 * kc + 1][1], qa[2 * kc + 1][2],
                                          qa[2 * kc + 1][3], r4[2], r4[3]);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.empty[st]);
                ++sc;
                // ---- online softmax per head over this warp's keys (values in log2 units)
                const int lim = (int)(pos - (int64_t)b * BK);  // keys 0..lim of the block are visible
                uint32_t pb[HG][KS][2];
#pragma unroll
                for (int hg = 0; hg < HG; ++hg) {
                    float mx = -INFINITY;
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const int key = w * KPW + nt * 8 + 2 * t;
                        c[nt][2 * hg] = key <= lim ? c[nt][2 * hg] * p.scale_log2e : -INFINITY;
                        c[nt][2 * hg + 1] = key + 1 <= lim ? c[nt][2 * hg + 1] * p.scale_log2e : -INFINITY;
                        mx = fmaxf(mx, fmaxf(c[nt][2 * hg], c[nt][2 * hg + 1]));
                    }
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                    const float m_new = fmaxf(m_run[hg], mx);
                    const float m_use = m_new == -INFINITY ? 0.f : m_new;   // slice fully masked so far
                    const float corr = ex2_approx(m_run[hg] - m_use);        // 0 when m_run = -inf
                    float psum = 0.f;
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const float p0 = ex2_approx(c[nt][2 * hg] - m_use), p1 = ex2_approx(c[nt][2 * hg + 1] - m_use);
                        psum += p0 + p1;
                        const __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
                        pb[hg][nt >> 1][nt & 1] = *reinterpret_cast<const uint32_t*>(&pk);
                    }
                    l_part[hg] = l_part[hg] * corr + psum;
                    m_run[hg] = m_new;
                    // O^T columns of this lane are heads 2t, 2t+1 of the half-group: fetch their factors
                    const float corr0 = __shfl_sync(0xffffffffu, corr, (2 * t) * 4);
                    const float corr1 = __shfl_sync(0xffffffffu, corr, (2 * t + 1) * 4);
#pragma unroll
                    for (int mt = 0; mt < 8; ++mt) {
                        acc[hg][mt][0] *= corr0; acc[hg][mt][1] *= corr1;
                        acc[hg][mt][2] *= corr0; acc[hg][mt][3] *= corr1;
                    }
                }
                // ---- V tile: O^T[d][head] += V^T[d][key] P^T[key][head]
                st = sc % kDecStages;
                if (!mbar_wait(&sm.full[st], (sc / kDecStages) & 1, abort)) {
                    if (lane == 0) report_async(status, kAsyncTimeout, 0x412);
                    ok = false;
                    break;
                }
                tb = smem_u32(sm.tile[st][0]);
#pragma unroll
                for (int mt = 0; mt < 8; ++mt) {
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        const int i = lane >> 3;
                        const int key = w * KPW + ks * 16 + (i >> 1) * 8 + (lane & 7);
                        uint32_t r4[4];
                        ldmatrix_x4_trans(r4, dec_tile_addr<BK>(tb, key, mt * 2 + (i & 1)));
                        if (lim < BK - 1) {  // local block: rows past the sequence's end may hold anything
                            const int k0 = w * KPW + ks * 16 + 2 * t;
                            r4[0] = keep_visible_pair(r4[0], k0, lim); r4[1] = keep_visible_pair(r4[1], k0, lim);
                            r4[2] = keep_visible_pair(r4[2], k0 + 8, lim); r4[3] = keep_visible_pair(r4[3], k0 + 8, lim);
                        }
#pragma unroll
                        for (int hg = 0; hg < HG; ++hg)
                            mma_m16n8k16_bf16(acc[hg][mt], r4[0], r4[1], r4[2], r4[3], pb[hg][ks][0], pb[hg][ks][1]);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.empty[st]);
                ++sc;
            }
            // ---- partial of this warp: O^T (unnormalised), running max, sum
            const int64_t pidx = (int64_t)item * kDecPartsPerItem + w;
            float* po = p.part_o + pidx * (G * 128);
#pragma unroll
            for (int hg = 0; hg < HG; ++hg) {
                float l = l_part[hg];
                l += __shfl_xor_sync(0xffffffffu, l, 1);
                l += __shfl_xor_sync(0xffffffffu, l, 2);
#pragma unroll
                for (int mt = 0; mt < 8; ++mt) {
                    const int d0 = mt * 16 + g;
                    po[(hg * 8 + 2 * t) * 128 + d0] = acc[hg][mt][0];
                    po[(hg * 8 + 2 * t + 1) * 128 + d0] = acc[hg][mt][1];
                    po[(hg * 8 + 2 * t) * 128 + d0 + 8] = acc[hg][mt][2];
                    po[(hg * 8 + 2 * t + 1) * 128 + d0 + 8] = acc[hg][mt][3];
                }
                if (t == 0) {
                    p.part_ml[pidx * (2 * G) + hg * 8 + g] = m_run[hg];
                    p.part_ml[pidx * (2 * G) + G + hg * 8 + g] = l;
                }
            }
        }
    }
}

// One warp per (sequence, head): merges the n_split*4 partials of its (sequence, KV head).
__global__ void __launch_bounds__(128)
attn_decode_combine_kernel(const float* __restrict__ part_o, const float* __restrict__ part_ml, int batch, int H_kv,
                           int G, int n_split, __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
    const int row = blockIdx.x * 4 + (threadIdx.x >> 5);  // (seq, head)
    const int lane = threadIdx.x & 31;
    const int H_q = H_kv * G;
    if (row >= batch * H_q) return;
    const int seq = row / H_q, h = row - seq * H_q;
    const int r = h / G, g = h - r * G;
    const int n_parts = n_split * kDecPartsPerItem;
    const int64_t p0 = ((int64_t)seq * H_kv + r) * n_parts;
    // Lane i holds the weight of parts i, i + 32, ... (the maxima and sums are read once, in parallel);
    // the partial rows are then accumulated four at a time, their loads independent of one another.
    constexpr int kMaxSlots = 4;  // n_parts <= 128: top_k <= 128 -> n_split <= 16, four parts each = 64
    float wv[kMaxSlots], M = -INFINITY;
#pragma unroll
    for (int u = 0; u < kMaxSlots; ++u) {
        const int i = lane + 32 * u;
        wv[u] = i < n_parts ? part_ml[(p0 + i) * (2 * G) + g] : -INFINITY;
        M = fmaxf(M, wv[u]);
    }
    M = warp_max(M);
    float L = 0.f;
#pragma unroll
    for (int u = 0; u < kMaxSlots; ++u) {
        const int i = lane + 32 * u;
        wv[u] = wv[u] > -INFINITY ? exp2f(wv[u] - M) : 0.f;  // a part with no visible key weighs nothing
        if (i < n_parts && wv[u] > 0.f) L += wv[u] * part_ml[(p0 + i) * (2 * G) + G + g];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    const float* orow = part_o + (p0 * G + g) * 128 + lane * 4;
    for (int i0 = 0; i0 < n_parts; i0 += 4) {
        float4 o[4];
        float w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int i = i0 + j;
            float wi = 0.f;
#pragma unroll
            for (int u = 0; u < kMaxSlots; ++u)
                if (u == (i >> 5)) wi = wv[u];
            w[j] = __shfl_sync(0xffffffffu, wi, i & 31);
            o[j] = i < n_parts ? *reinterpret_cast<const float4*>(orow + (int64_t)i * G * 128) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (w[j] > 0.f) {  // (an unweighted part may hold anything)
                acc[0] = fmaf(w[j], o[j].x, acc[0]); acc[1] = fmaf(w[j], o[j].y, acc[1]);
                acc[2] = fmaf(w[j], o[j].z, acc[2]); acc[3] = fmaf(w[j], o[j].w, acc[3]);
            }
        }
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
    const __nv_bfloat162 o01 = __floats2bfloat162_rn(acc[0] * inv, acc[1] * inv);
    const __nv_bfloat162 o23 = __floats2bfloat162_rn(acc[2] * inv, acc[3] * inv);
    uint2 pk;
    pk.x = *reinterpret_cast<const uint32_t*>(&o01);
    pk.y = *reinterpret_cast<const uint32_t*>(&o23);
    *reinterpret_cast<uint2*>(out + (int64_t)row * 128 + lane * 4) = pk;
    if (lse != nullptr && lane == 0) lse[row] = (M + log2f(L)) * 0.6931471805599453f;
}

}  // namespace msa
