// Decode attention on a K/V cache stored in fp8 E4M3 (Section 4.2: the kernels also support fp8).
//
// The structure of attn_decode_kernel - persistent CTAs, a producer warp streaming the selected
// blocks through a TMA ring, four consumer warps with 32 keys of every block each, online softmax
// in registers, per-warp partials - with tiles of half the bytes (a key row is one 128-byte swizzle
// atom), two CTAs per SM (six tiles of 16 KB each) and tensor maps with a 128-byte L2 promotion (a
// head's 128-byte row has other heads' rows as neighbours; a 256-byte promotion fetched them too).  K and V are dequantised in registers: E4M3 -> f16 is exact and one
// instruction per pair, so both products run as f16 MMAs with Q converted to f16 (exact for bf16
// values in f16's normal range) and P rounded to f16: the result differs from the bf16-cache
// kernel's only by the rounding of K and V to fp8.  The contraction index of Q K^T and the row
// index of O^T are permuted to the order in which 16-bit shared-memory matrix loads hand out fp8
// bytes (see the fragment comments).
#pragma once

#include <cuda_fp16.h>

#include "decode.cuh"

namespace msa {

constexpr int kDecKv8Stages = 6;  // 96 KB at B_k = 128: two CTAs per SM, eight consumer warps to hide the dequantisation

template <int BK>
struct DecKv8Smem {
    alignas(1024) uint8_t tile[kDecKv8Stages][BK * 128];  // [stage][key][128 fp8], 128-byte swizzle
    alignas(8) uint64_t full[kDecKv8Stages];
    uint64_t empty[kDecKv8Stages];
    int abort;
};

// 16-byte chunk `chunk` (0..7: d = 16 chunk .. 16 chunk + 15) of key row `key` inside a swizzled fp8 tile.
__device__ __forceinline__ uint32_t dec_kv8_addr(uint32_t tile_base, int key, int chunk) {
    return tile_base + (uint32_t)(key * 128 + ((chunk ^ (key & 7)) << 4));
}

__device__ __forceinline__ void mma_m16n8k16_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                 uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Two bf16 (lower half first) -> two f16, round to nearest.
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t two) {
    const float2 f = bf16x2_to_float2(two);
    const __half2 h = __floats2half2_rn(f.x, f.y);
    return *reinterpret_cast<const uint32_t*>(&h);
}

// fp8 E4M3 -> bf16, exact (every E4M3 value is a bf16 value): the prefill calls run on bf16 copies of
// fp8 K/V caches.  One thread per 16 elements; n16 = elements / 16.
__global__ void __launch_bounds__(256)
e4m3_to_bf16_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, int64_t n16) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (int64_t)gridDim.x * blockDim.x) {
        const uint4 in = __ldg(src + i);
        const uint32_t w[4] = {in.x, in.y, in.z, in.w};
        uint32_t o[8];
        e4m3x16_to_bf16x16(w, o);
        dst[2 * i] = make_uint4(o[0], o[1], o[2], o[3]);
        dst[2 * i + 1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
}

template <int BK, int G>
__global__ void __launch_bounds__(kDecThreads, 2)
attn_decode_kv8_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                   DecParams p, int* status) {
    constexpr int KPW = BK / 4;    // keys per consumer warp
    constexpr int NT = KPW / 8;    // 8-key score tiles per warp
    constexpr int KS = KPW / 16;   // 16-key steps of the second product
    constexpr uint32_t TILE_BYTES = BK * 128;  // BK keys x 128 fp8
    constexpr int kStages = kDecKv8Stages;
    extern __shared__ uint8_t smem_raw[];
    DecKv8Smem<BK>& sm = *reinterpret_cast<DecKv8Smem<BK>*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abort = &sm.abort;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&sm.full[s], 1); mbar_init(&sm.empty[s], 4); }
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
                        const int st = sc % kStages;
                        if (!mbar_wait(&sm.empty[st], ((sc / kStages) & 1) ^ 1, abort)) {
                            report_async(status, kAsyncTimeout, 0x402);
                            ok = false;
                            break;
                        }
                        mbar_arrive_expect_tx(&sm.full[st], TILE_BYTES);
                        const CUtensorMap* tm = kv == 0 ? &tm_k : &tm_v;
                        tma_load_3d(sm.tile[st], tm, 0, r, tok, &sm.full[st]);
                    }
                }
            }
            if (*abort != 0) spin_cycles(200000);
        }
    } else {
        const int w = warp - 1;
        const int g = lane >> 2, t = lane & 3;
        const float sl2 = p.scale_log2e;
        uint32_t sc = 0;
        bool ok = true;
        for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
            const int u = item / p.n_split, sp = item - u * p.n_split;
            const int seq = u / p.H_kv, r = u - seq * p.H_kv;
            const int64_t len = p.seq_lens[seq];
            const int64_t pos = len - 1, loc = pos / BK;
            const int32_t* sel = p.block_idx + (int64_t)u * p.top_k;
            // A fragments of Q (as f16: exact for bf16 values in f16's normal range): rows 0-7 = heads
            // 0-7 of the group, rows 8-15 = heads 8-15 (G = 16) or zero padding (G = 8).  The 16
            // contraction indices of step ks are d = 16 ks .. 16 ks + 15, permuted the way the fp8 K
            // fragments arrive: this lane's first pair is d = 16 ks + 4t, +1, its second d + 2, + 3.
            uint32_t qa[8][4];
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) qa[ks][0] = qa[ks][1] = qa[ks][2] = qa[ks][3] = 0u;
#pragma unroll
            for (int hg = 0; hg < HG; ++hg) {
                const __nv_bfloat16* qrow = p.q + ((int64_t)seq * H_q + r * G + hg * 8 + g) * 128;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint2 v = *reinterpret_cast<const uint2*>(qrow + ks * 16 + 4 * t);  // four bf16
                    qa[ks][hg] = bf16x2_to_f16x2(v.x);
                    qa[ks][2 + hg] = bf16x2_to_f16x2(v.y);
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
                int st = sc % kStages;
                if (!mbar_wait(&sm.full[st], (sc / kStages) & 1, abort)) {
                    if (lane == 0) report_async(status, kAsyncTimeout, 0x411);
                    ok = false;
                    break;
                }
                uint32_t tb = smem_u32(sm.tile[st]);
                float c[NT][4];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0.f;
                    const int key = w * KPW + nt * 8 + (lane & 7);
#pragma unroll
                    for (int q4 = 0; q4 < 2; ++q4) {  // four 16-byte chunks (64 d) per load
                        uint32_t r4[4];
                        ldmatrix_x4(r4, dec_kv8_addr(tb, key, q4 * 4 + (lane >> 3)));
#pragma unroll
                        for (int j = 0; j < 4; ++j) {  // chunk 4 q4 + j: this lane holds its bytes 4t .. 4t+3 of key g
                            const int ks = q4 * 4 + j;
                            uint32_t b0, b1;
                            e4m3x4_to_f16x2x2(r4[j], b0, b1);
                            mma_m16n8k16_f16(c[nt], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b0, b1);
                        }
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
                        c[nt][2 * hg] = key <= lim ? c[nt][2 * hg] * sl2 : -INFINITY;
                        c[nt][2 * hg + 1] = key + 1 <= lim ? c[nt][2 * hg + 1] * sl2 : -INFINITY;
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
                        const __half2 pk = __floats2half2_rn(p0, p1);
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
                st = sc % kStages;
                if (!mbar_wait(&sm.full[st], (sc / kStages) & 1, abort)) {
                    if (lane == 0) report_async(status, kAsyncTimeout, 0x412);
                    ok = false;
                    break;
                }
                tb = smem_u32(sm.tile[st]);
                // Output tile mt = the 16 d of chunk mt; row g of the tile is d = 16 mt + 2g, row g + 8 is
                // d = 16 mt + 2g + 1: a transposed 16-bit load hands this lane both d of a pair for two
                // consecutive keys, and two byte permutes split them into the two rows.
#pragma unroll
                for (int mp = 0; mp < 4; ++mp) {  // pairs of output tiles: chunks 2 mp, 2 mp + 1
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        const int i = lane >> 3;  // matrix: keys (i & 1) * 8 .., chunk 2 mp + (i >> 1)
                        const int key = w * KPW + ks * 16 + (i & 1) * 8 + (lane & 7);
                        uint32_t r4[4];
                        ldmatrix_x4_trans(r4, dec_kv8_addr(tb, key, mp * 2 + (i >> 1)));
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            uint32_t lo = r4[half * 2], hi = r4[half * 2 + 1];  // keys 2t, 2t+1 and 8 + 2t, 8 + 2t + 1
                            if (lim < BK - 1) {  // local block: bytes past the sequence's end may decode to NaN
                                const int k0 = w * KPW + ks * 16 + 2 * t;
                                lo = keep_visible_pair(lo, k0, lim);
                                hi = keep_visible_pair(hi, k0 + 8, lim);
                            }
                            // bytes (key 2t: d even, d odd; key 2t+1: d even, d odd) -> (d even: both keys; d odd: both keys)
                            uint32_t a0, a1, a2, a3;
                            e4m3x4_to_f16x2x2(__byte_perm(lo, 0u, 0x3120), a0, a1);
                            e4m3x4_to_f16x2x2(__byte_perm(hi, 0u, 0x3120), a2, a3);
#pragma unroll
                            for (int hg = 0; hg < HG; ++hg)
                                mma_m16n8k16_f16(acc[hg][mp * 2 + half], a0, a1, a2, a3, pb[hg][ks][0], pb[hg][ks][1]);
                        }
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
                    const int d0 = mt * 16 + 2 * g;  // rows g and g + 8 of the tile are d0 and d0 + 1
                    *reinterpret_cast<float2*>(po + (hg * 8 + 2 * t) * 128 + d0) = make_float2(acc[hg][mt][0], acc[hg][mt][2]);
                    *reinterpret_cast<float2*>(po + (hg * 8 + 2 * t + 1) * 128 + d0) = make_float2(acc[hg][mt][1], acc[hg][mt][3]);
                }
                if (t == 0) {
                    p.part_ml[pidx * (2 * G) + hg * 8 + g] = m_run[hg];
                    p.part_ml[pidx * (2 * G) + G + hg * 8 + g] = l;
                }
            }
        }
    }
}

}  // namespace msa
