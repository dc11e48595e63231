// Shared device/host helpers of the MSA CUDA library (not used by the CPU oracle).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/msa.h"

namespace msa {

constexpr int kMaxKvHeadsGeneric = 16;
constexpr int kWarp = 32;

// Device status word: 0 = ok, otherwise (code << 24) | detail.  Kernels receive its
// address as an argument; the first non-zero value wins.
enum AsyncCode : int { kAsyncOk = 0, kAsyncTimeout = 1, kAsyncBadIndex = 2 };

__device__ __forceinline__ void report_async(int* status, int code, int detail) {
    atomicCAS(status, 0, (code << 24) | (detail & 0xFFFFFF));
}

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) {
    return __uint_as_float(((uint32_t)b) << 16);
}

// Two packed bf16 (low half first) -> two floats.
__device__ __forceinline__ float2 bf16x2_to_float2(uint32_t u) {
    return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xFFFF0000u));
}

// fp8 E4M3 ("fn": bias 7, no infinities, 0x7F / 0xFF are NaN) to fp32; exact.
__device__ __forceinline__ float e4m3_to_float(uint8_t b) {
    const __half_raw h = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)b, __NV_E4M3);
    return __half2float(__half(h));
}

// Four fp8 E4M3 (bytes x0 .. x3 of a register) -> two registers of two f16 each, (x0, x1) and (x2, x3);
// exact.  (Integer bit moves instead of the conversion instruction - sign and the seven other bits
// shifted to their f16 places, a factor 2^8 folded into the scales - were measured at the same speed.)
__device__ __forceinline__ void e4m3x4_to_f16x2x2(uint32_t four, uint32_t& lo, uint32_t& hi) {
    asm("{\n\t.reg .b16 a, b;\n\t"
        "mov.b32 {a, b}, %2;\n\t"
        "cvt.rn.f16x2.e4m3x2 %0, a;\n\t"
        "cvt.rn.f16x2.e4m3x2 %1, b;\n\t}"
        : "=r"(lo), "=r"(hi)
        : "r"(four));
}

// Sixteen fp8 E4M3 (four registers) -> sixteen bf16 (eight registers), in order; exact, since every
// E4M3 value is a bf16 value.
__device__ __forceinline__ void e4m3x16_to_bf16x16(const uint32_t (&w)[4], uint32_t (&o)[8]) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        uint32_t lo, hi;
        e4m3x4_to_f16x2x2(w[j], lo, hi);
        const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&lo));
        const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&hi));
        const __nv_bfloat162 ab = __floats2bfloat162_rn(a.x, a.y), bb = __floats2bfloat162_rn(b.x, b.y);
        o[2 * j] = *reinterpret_cast<const uint32_t*>(&ab);
        o[2 * j + 1] = *reinterpret_cast<const uint32_t*>(&bb);
    }
}

// Element c of an index-branch row stored as fp8 E4M3 (F8) or bf16.
template <bool F8>
__device__ __forceinline__ float idx_elem(const void* row, int c) {
    if constexpr (F8) return e4m3_to_float(static_cast<const uint8_t*>(row)[c]);
    else return __bfloat162float(static_cast<const __nv_bfloat16*>(row)[c]);
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

inline int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }

int* async_status_ptr();  // device address of the status word of the current device

// Stages of the path, for launch counting and the optional per-stage timing.
enum Stage : int {
    kStageIndex = 0,      // Eq. 6, prefill
    kStageTopk = 1,       // Eq. 7
    kStageSchedule = 2,   // reverse index + work list (KV-outer prefill)
    kStageAttn = 3,       // Eq. 8, prefill partials
    kStageCombine = 4,    // LSE-weighted merge
    kStageIndexDecode = 5,
    kStageAttnDecode = 6,
    kStageCombineDecode = 7,
    kStageIndexLse = 8,   // Section 4.3: index-branch log-sum-exp over the selected blocks
    kNumStages = 9
};

// Wraps one kernel launch: counts it and, while profiling is on, brackets it with CUDA
// events on the launching stream.
class StageScope {
public:
    StageScope(int stage, cudaStream_t st);
    ~StageScope();
private:
    int slot_;
    cudaStream_t st_;
};

// Three-input maximum (one instruction on sm_100).
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// Where block b of a score row sits.  Block order (what msa_index_scores documents): at b.  Run
// order (the tensor-core scoring kernel writes a thread's four blocks of a run of eight as one
// 16-byte store): a run's eight blocks stay in the run's 32 bytes, those of the first half of every
// key tile first; with nb = 2^lnb blocks per thread and tile, block w = b mod 8 is block (w mod nb)
// of half ((w / nb) mod 2) of tile w / (2 nb) and sits at 4 half + nb tile + block.  lnb = 2 is the
// identity (block order).
template <class I>
__device__ __forceinline__ I score_slot(I b, int lnb) {
    const int w = (int)(b & 7);
    return (b & ~(I)7) | (I)((((w >> lnb) & 1) << 2) | ((w >> (lnb + 1)) << lnb) | (w & ((1 << lnb) - 1)));
}

}  // namespace msa
