// Generic (any-shape) kernels for Eq. 6 and Eq. 8.  They serve shapes the specialised
// tensor-core kernels do not cover (odd head sizes, tiny blocks); they are plain FMA code.
#pragma once

#include "common.cuh"

namespace msa {

// Row addressing shared by the prefill form (one sequence, rows q_begin..) and the decode
// form (row s = sequence s, query at its last token).
struct RowMap {
    int64_t q_begin;             // prefill: first query position of the range
    int64_t kv_len;              // prefill: sequence length
    const int64_t* seq_offsets;  // decode: token offset of each sequence (nullptr => prefill)
    const int32_t* seq_lens;     // decode: length of each sequence
    int64_t n_cols;              // score columns to write per row (>= this row's block count)
    const int32_t* row_pos = nullptr;  // packed prefill batch: position of every packed row in its own sequence;
                                       // row r of the call is packed row q_begin + r (stage 2 only)

    __device__ __forceinline__ void get(int64_t row, int64_t& pos, int64_t& len,
                                        int64_t& base) const {
        if (row_pos != nullptr) {
            pos = row_pos[q_begin + row];
            len = pos + 1;
            base = 0;
        } else if (seq_lens != nullptr) {
            len = seq_lens[row];
            pos = len - 1;
            base = seq_offsets != nullptr ? seq_offsets[row] : 0;
        } else {
            len = kv_len;
            pos = q_begin + row;
            base = 0;
        }
    }
};

// Eq. 6.  One warp per (query row, key block): lanes stride over the block's visible
// tokens, each lane scoring one K_idx row against all H_kv index query heads.
// F8: the operands are fp8 E4M3 instead of bf16 (Section 4.2).
template <int WARPS, bool F8>
__global__ void __launch_bounds__(WARPS * 32)
index_scores_generic_kernel(const void* __restrict__ q_idx, const void* __restrict__ k_idx, RowMap rows,
                            int64_t n_chunks, int H_kv, int d_idx, int B_k, float scale,
                            float* __restrict__ scores, int64_t ld_scores, int lnb) {
    extern __shared__ float q_s[];  // [H_kv][d_idx]
    const int64_t row = blockIdx.x / n_chunks;
    const int64_t chunk = blockIdx.x % n_chunks;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int64_t pos, len, base;
    rows.get(row, pos, len, base);

    constexpr int ELT = F8 ? 1 : 2;
    const char* qrow = static_cast<const char*>(q_idx) + row * (int64_t)H_kv * d_idx * ELT;
    for (int t = threadIdx.x; t < H_kv * d_idx; t += WARPS * 32) q_s[t] = idx_elem<F8>(qrow, t);
    __syncthreads();

    const int64_t b = chunk * WARPS + warp;
    if (b >= rows.n_cols) return;
    float* out = scores + row * (int64_t)H_kv * ld_scores + score_slot(b, lnb);
    const int64_t j0 = b * B_k;
    if (pos < 0 || j0 > pos) {  // no visible token in this block
        if (lane < H_kv) out[(int64_t)lane * ld_scores] = -INFINITY;
        return;
    }
    int64_t j_end = j0 + B_k;  // exclusive
    if (j_end > pos + 1) j_end = pos + 1;

    float best[kMaxKvHeadsGeneric];
#pragma unroll
    for (int r = 0; r < kMaxKvHeadsGeneric; ++r) best[r] = -INFINITY;

    for (int64_t j = j0 + lane; j < j_end; j += 32) {
        const char* krow = static_cast<const char*>(k_idx) + (base + j) * (int64_t)d_idx * ELT;
        float acc[kMaxKvHeadsGeneric];
#pragma unroll
        for (int r = 0; r < kMaxKvHeadsGeneric; ++r) acc[r] = 0.f;
        for (int c = 0; c < d_idx / 8; ++c) {
            float2 k0, k1, k2, k3;  // eight consecutive elements of the key row
            if constexpr (F8) {
                const uint2 kv = __ldg(reinterpret_cast<const uint2*>(krow) + c);
                k0 = make_float2(e4m3_to_float(kv.x & 0xFF), e4m3_to_float((kv.x >> 8) & 0xFF));
                k1 = make_float2(e4m3_to_float((kv.x >> 16) & 0xFF), e4m3_to_float(kv.x >> 24));
                k2 = make_float2(e4m3_to_float(kv.y & 0xFF), e4m3_to_float((kv.y >> 8) & 0xFF));
                k3 = make_float2(e4m3_to_float((kv.y >> 16) & 0xFF), e4m3_to_float(kv.y >> 24));
            } else {
                const uint4 kv = __ldg(reinterpret_cast<const uint4*>(krow) + c);
                k0 = bf16x2_to_float2(kv.x); k1 = bf16x2_to_float2(kv.y);
                k2 = bf16x2_to_float2(kv.z); k3 = bf16x2_to_float2(kv.w);
            }
#pragma unroll
            for (int r = 0; r < kMaxKvHeadsGeneric; ++r) {
                if (r < H_kv) {
                    const float* qq = q_s + r * d_idx + c * 8;
                    float a = acc[r];
                    a = fmaf(qq[0], k0.x, a); a = fmaf(qq[1], k0.y, a);
                    a = fmaf(qq[2], k1.x, a); a = fmaf(qq[3], k1.y, a);
                    a = fmaf(qq[4], k2.x, a); a = fmaf(qq[5], k2.y, a);
                    a = fmaf(qq[6], k3.x, a); a = fmaf(qq[7], k3.y, a);
                    acc[r] = a;
                }
            }
        }
#pragma unroll
        for (int r = 0; r < kMaxKvHeadsGeneric; ++r) best[r] = fmaxf(best[r], acc[r] * scale);
    }
#pragma unroll
    for (int r = 0; r < kMaxKvHeadsGeneric; ++r) {
        if (r < H_kv) {
            const float m = warp_max(best[r]);
            if (lane == r) out[(int64_t)r * ld_scores] = m;
        }
    }
}

// Eq. 8, query-outer.  One CTA per (query row, KV head), one warp per query head of the
// group; each warp walks the selected blocks with an online softmax in registers.
constexpr int kMaxDimsPerLane = 8;  // d_h <= 256

__global__ void sparse_attn_generic_kernel(const __nv_bfloat16* __restrict__ q,
                                           const __nv_bfloat16* __restrict__ k,
                                           const __nv_bfloat16* __restrict__ v,
                                           const int32_t* __restrict__ block_idx, RowMap rows,
                                           int H_q, int H_kv, int d, int B_k, int top_k,
                                           float scale, __nv_bfloat16* __restrict__ out,
                                           float* __restrict__ lse, int* status) {
    extern __shared__ float q_sh[];  // [G][d]
    const int G = H_q / H_kv;
    const int64_t row = blockIdx.x / H_kv;
    const int r = (int)(blockIdx.x % H_kv);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = r * G + warp;
    int64_t pos, len, base;
    rows.get(row, pos, len, base);
    const int64_t loc = pos / B_k;

    float* qs = q_sh + warp * d;
    const __nv_bfloat16* qrow = q + (row * H_q + h) * (int64_t)d;
    for (int c = lane; c < d; c += 32) qs[c] = __bfloat162float(qrow[c]);
    __syncwarp();

    float m = -INFINITY, ell = 0.f;
    float acc[kMaxDimsPerLane];
#pragma unroll
    for (int u = 0; u < kMaxDimsPerLane; ++u) acc[u] = 0.f;

    const int32_t* sel = block_idx + (row * H_kv + r) * (int64_t)top_k;
    for (int s = 0; s < top_k; ++s) {
        const int32_t b = sel[s];
        if (b < 0) {
            if (b != -1 && lane == 0) report_async(status, kAsyncBadIndex, 1);
            continue;
        }
        if (b > loc) {
            if (lane == 0) report_async(status, kAsyncBadIndex, 2);
            continue;
        }
        const int64_t j0 = (int64_t)b * B_k;
        int64_t nvis = pos - j0 + 1;
        if (nvis > B_k) nvis = B_k;
        for (int64_t t0 = 0; t0 < nvis; t0 += 32) {
            const int64_t j = j0 + t0 + lane;
            const bool valid = (t0 + lane) < nvis;
            float z = -INFINITY;
            if (valid) {
                const uint4* krow =
                    reinterpret_cast<const uint4*>(k + ((base + j) * H_kv + r) * (int64_t)d);
                float a = 0.f;
                for (int c = 0; c < d / 8; ++c) {
                    const uint4 kv = __ldg(krow + c);
                    const float2 k0 = bf16x2_to_float2(kv.x), k1 = bf16x2_to_float2(kv.y);
                    const float2 k2 = bf16x2_to_float2(kv.z), k3 = bf16x2_to_float2(kv.w);
                    const float* qq = qs + c * 8;
                    a = fmaf(qq[0], k0.x, a); a = fmaf(qq[1], k0.y, a);
                    a = fmaf(qq[2], k1.x, a); a = fmaf(qq[3], k1.y, a);
                    a = fmaf(qq[4], k2.x, a); a = fmaf(qq[5], k2.y, a);
                    a = fmaf(qq[6], k3.x, a); a = fmaf(qq[7], k3.y, a);
                }
                z = a * scale;
            }
            const float m_new = fmaxf(m, warp_max(z));
            const float p = valid ? expf(z - m_new) : 0.f;
            const float corr = (m == -INFINITY) ? 0.f : expf(m - m_new);
            ell = ell * corr + warp_sum(p);
            m = m_new;
#pragma unroll
            for (int u = 0; u < kMaxDimsPerLane; ++u) acc[u] *= corr;
            const int cnt = (int)((nvis - t0) < 32 ? (nvis - t0) : 32);
            for (int tt = 0; tt < cnt; ++tt) {
                const float pj = __shfl_sync(0xffffffffu, p, tt);
                const __nv_bfloat16* vrow = v + ((base + j0 + t0 + tt) * H_kv + r) * (int64_t)d;
#pragma unroll
                for (int u = 0; u < kMaxDimsPerLane; ++u) {
                    const int c = lane + 32 * u;
                    if (c < d) acc[u] = fmaf(pj, __bfloat162float(vrow[c]), acc[u]);
                }
            }
        }
    }
    __nv_bfloat16* orow = out + (row * H_q + h) * (int64_t)d;
    const float inv = ell > 0.f ? 1.f / ell : 0.f;
#pragma unroll
    for (int u = 0; u < kMaxDimsPerLane; ++u) {
        const int c = lane + 32 * u;
        if (c < d) orow[c] = __float2bfloat16(acc[u] * inv);
    }
    if (lse != nullptr && lane == 0) lse[row * H_q + h] = m + logf(ell);
}

}  // namespace msa
