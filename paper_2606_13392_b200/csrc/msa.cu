// C ABI of the MSA forward path (see include/msa.h): argument validation, workspace
// planning and kernel dispatch.  All arithmetic is in the kernels included below.
#include <atomic>
#include <cstdio>
#include <cstring>
#include <cstdlib>

#include "common.cuh"
#include "generic.cuh"
#include "topk.cuh"
#include "index_scores_tc.cuh"
#include "attn_prefill_tc.cuh"
#include "index_lse.cuh"
#include "decode.cuh"
#include "decode_kv8.cuh"

namespace msa {

static std::atomic<int64_t> g_launches{0};

// Optional per-stage timing: a fixed pool of event pairs, created by msa_profile_begin().
constexpr int kProfSlots = 16384;
static bool g_prof_on = false;
static int g_prof_used = 0;
static cudaEvent_t g_prof_ev[kProfSlots][2];
static int g_prof_stage[kProfSlots];
static bool g_prof_created = false;

StageScope::StageScope(int stage, cudaStream_t st) : slot_(-1), st_(st) {
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (g_prof_on && g_prof_used < kProfSlots) {
        slot_ = g_prof_used++;
        g_prof_stage[slot_] = stage;
        cudaEventRecord(g_prof_ev[slot_][0], st_);
    }
}
StageScope::~StageScope() {
    if (slot_ >= 0) cudaEventRecord(g_prof_ev[slot_][1], st_);
}

__device__ int g_async_status = 0;

int* async_status_ptr() {
    // One address per device; looked up on each call (cheap, no allocation).
    int* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_async_status) != cudaSuccess) return nullptr;
    return p;
}

struct Resolved {
    int H_q, H_kv, G, d, d_idx, B_k, k;
    float softmax_scale, index_scale;
    bool kv_fp8;                                         // the K and V caches are fp8 E4M3 (else bf16)
    size_t kv_elt() const { return kv_fp8 ? 1 : 2; }    // bytes per K/V element
    bool q_fp8;                                          // prefill: Q is fp8 E4M3 as well (needs kv_fp8)
    size_t q_elt() const { return q_fp8 ? 1 : 2; }      // bytes per Q element
    bool score_runs;                                     // score rows between the stage-1 and stage-2 calls are in run order
    bool idx_fp8;                                        // index-branch operands are fp8 E4M3 (else bf16)
    size_t idx_elt() const { return idx_fp8 ? 1 : 2; }  // bytes per index-branch element
};

static msa_status_t resolve(const msa_shape_t* s, Resolved& r) {
    if (s == nullptr) return MSA_ERR_INVALID_ARG;
    if (s->n_q_heads <= 0 || s->n_kv_heads <= 0 || s->head_dim <= 0 || s->idx_dim <= 0 ||
        s->block_size <= 0 || s->top_k <= 0)
        return MSA_ERR_INVALID_ARG;
    if (s->n_q_heads % s->n_kv_heads != 0) return MSA_ERR_INVALID_ARG;
    r.H_q = s->n_q_heads; r.H_kv = s->n_kv_heads; r.G = r.H_q / r.H_kv;
    r.d = s->head_dim; r.d_idx = s->idx_dim; r.B_k = s->block_size; r.k = s->top_k;
    if (r.k > 128) return MSA_ERR_UNSUPPORTED;
    if (r.d % 8 != 0 || r.d > 256 || r.d_idx % 8 != 0 || r.d_idx > 128) return MSA_ERR_UNSUPPORTED;
    if (r.H_kv > kMaxKvHeadsGeneric || r.G > 32) return MSA_ERR_UNSUPPORTED;
    if (!(s->softmax_scale >= 0.f) || !(s->index_scale >= 0.f)) return MSA_ERR_INVALID_ARG;
    r.softmax_scale = s->softmax_scale > 0.f ? s->softmax_scale : 1.0f / sqrtf((float)r.d);
    r.index_scale = s->index_scale > 0.f ? s->index_scale : 1.0f / sqrtf((float)r.d_idx);
    if (s->idx_fp8 != 0 && s->idx_fp8 != 1) return MSA_ERR_INVALID_ARG;
    r.idx_fp8 = s->idx_fp8 == 1;
    if (r.idx_fp8 && r.d_idx % 16 != 0) return MSA_ERR_UNSUPPORTED;  // 16-byte rows
    if (s->kv_fp8 != 0 && s->kv_fp8 != 1) return MSA_ERR_INVALID_ARG;
    r.kv_fp8 = s->kv_fp8 == 1;
    if (s->q_fp8 != 0 && s->q_fp8 != 1) return MSA_ERR_INVALID_ARG;
    r.q_fp8 = s->q_fp8 == 1;
    if (r.q_fp8 && !r.kv_fp8) return MSA_ERR_UNSUPPORTED;  // fp8 Q comes with fp8 K and V
    if (s->score_runs != 0 && s->score_runs != 1) return MSA_ERR_INVALID_ARG;
    r.score_runs = s->score_runs == 1;
    if (r.score_runs && r.B_k != 64 && r.B_k != 128) return MSA_ERR_UNSUPPORTED;
    return MSA_OK;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static msa_status_t check_range(int64_t q_begin, int64_t q_count, int64_t kv_len) {
    if (q_begin < 0 || q_count < 0 || kv_len < 0 || q_begin + q_count > kv_len)
        return MSA_ERR_INVALID_ARG;
    return MSA_OK;
}

static int sm_count();
static int current_device();

static msa_status_t launch_status() {
    return cudaPeekAtLastError() == cudaSuccess ? MSA_OK : MSA_ERR_CUDA;
}

// ---------------------------------------------------------------------- tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    // Looked up through the runtime so that the library does not link against libcuda.
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &p, 12000, cudaEnableDefault, &qres) ==
                cudaSuccess && qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// promote_128: rows of 128 bytes whose neighbours in memory belong to other CTAs (fp8 K/V rows of one
// head): a 256-byte L2 promotion would fetch the neighbour's row from DRAM as well.
bool encode_tmap_bf16(CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                      const uint64_t* strides_bytes, const uint32_t* box, bool promote_128) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    cuuint64_t gdim[5], gstr[5];
    cuuint32_t bx[5], es[5];
    for (int i = 0; i < rank; ++i) { gdim[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
    for (int i = 0; i + 1 < rank; ++i) gstr[i] = strides_bytes[i];
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstr, bx, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              promote_128 ? CU_TENSOR_MAP_L2_PROMOTION_L2_128B : CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// ---------------------------------------------------------------------- stage 1
// log2 of the blocks one epilogue thread of the tensor-core scoring kernel holds per key tile, the
// parameter of the run order of a score row (score_slot); 2 = block order.
static int score_lnb(const Resolved& r, bool runs) { return !runs ? 2 : (r.B_k == 128 ? 0 : 1); }

// F8: fp8 E4M3 operands with d_idx = 128; the bytes of a row are laid out like 64 bf16, so the
// tensor maps below (bf16 element type, used only to move bytes) serve both.
template <int BK, int NH, int DI, int FK = 0, bool F8 = false, bool RUNL = false>
static msa_status_t launch_index_tc(const Resolved& r, const void* q_idx, const void* k_idx, int64_t q_begin,
                                    int64_t q_count, int64_t kv_len, float* scores, int64_t ld_scores,
                                    int64_t n_cols, cudaStream_t st, int32_t* block_idx = nullptr,
                                    const IdxPackedTile* packed = nullptr, int64_t n_packed = 0,
                                    int64_t score_row0 = 0) {
    // key-tile stages: what fits beside the NH*DI query atoms in 227 KB of shared memory (at most 3)
    constexpr int RUN_KB = RUNL ? NH * 4 : 0;  // block maxima of a run of eight, waiting for their 16-byte store
    constexpr int ST = (NH * DI * 16 + 3 * DI * 32 + RUN_KB <= 224) ? 3 : 2;
    static_assert(NH * DI * 16 + ST * DI * 32 + RUN_KB <= 224, "shared memory budget");
    CUtensorMap tm_q, tm_k;
    const uint64_t row_b = (uint64_t)DI * 128;  // bytes of one index vector
    const uint64_t qd[3] = {(uint64_t)DI * 64, (uint64_t)r.H_kv, (uint64_t)q_count};
    const uint64_t qs[2] = {row_b, (uint64_t)r.H_kv * row_b};
    const uint32_t qb[3] = {64, 1, kIdxTileQ};
    const uint64_t kd[2] = {(uint64_t)DI * 64, (uint64_t)kv_len};
    const uint64_t ks[1] = {row_b};
    const uint32_t kb[2] = {64, kIdxTileK};
    if (!encode_tmap_bf16(&tm_q, q_idx, 3, qd, qs, qb) || !encode_tmap_bf16(&tm_k, k_idx, 2, kd, ks, kb))
        return MSA_ERR_CUDA;
    int* status = async_status_ptr();
    if (status == nullptr) return MSA_ERR_CUDA;
    const size_t smem = sizeof(IdxSmem<NH, DI, ST, RUNL>) + 1024;
    static bool attr_set_dev[64] = {false};  // the attribute is per device
    const int dev_id = current_device();
    if (!attr_set_dev[dev_id]) {
        if (cudaFuncSetAttribute(index_scores_tc_kernel<BK, NH, DI, ST, FK, F8, RUNL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem) != cudaSuccess)
            return MSA_ERR_CUDA;
        attr_set_dev[dev_id] = true;
    }
    // (a packed batch: q_count and kv_len are the batch's rows, for the tensor maps; the grid follows the tile list)
    const int64_t grid = (packed != nullptr ? n_packed : ceil_div64(q_count, kIdxTileQ)) * (r.H_kv / NH);
    if (grid > 2147483647LL) return MSA_ERR_UNSUPPORTED;
    {
        StageScope sc(kStageIndex, st);
        index_scores_tc_kernel<BK, NH, DI, ST, FK, F8, RUNL><<<(unsigned)grid, kIdxThreads, smem, st>>>(
            tm_q, tm_k, q_begin, q_count, r.H_kv, r.index_scale, scores, ld_scores, n_cols, status, block_idx, r.k,
            packed, score_row0);
    }
    return launch_status();
}

// Heads sharing one key tile per CTA: the most (8, 4, 2, 1; at most 2 when d_idx = 128, for
// shared memory) that divide H_kv and still leave at least two CTAs per SM, so that short
// chunks keep the machine full.
static int index_heads_for_tiles(const Resolved& r, int64_t n_qtiles);
static int index_heads_per_cta(const Resolved& r, int64_t q_count) {
    return index_heads_for_tiles(r, ceil_div64(q_count, kIdxTileQ));
}
static int index_heads_for_tiles(const Resolved& r, int64_t n_qtiles) {
    const bool one_atom = r.idx_fp8 || r.d_idx == 64;  // the index vector is one 128-byte atom
    for (int cand = one_atom ? 8 : 2; cand > 1; cand >>= 1)
        if (r.H_kv % cand == 0 && n_qtiles * (r.H_kv / cand) >= 2 * sm_count()) return cand;
    return 1;
}

// packed != null: a group of sequences of a packed batch (q_count = kv_len = the batch's rows), its query
// tiles listed in `packed`; the score matrix starts at packed row score_row0.
template <int BK, int DI, bool F8, bool RUNL>
static msa_status_t launch_index_tc_nh(const Resolved& r, const void* q_idx, const void* k_idx, int64_t q_begin,
                                       int64_t q_count, int64_t kv_len, float* scores, int64_t ld_scores,
                                       int64_t n_cols, cudaStream_t st, const IdxPackedTile* packed = nullptr,
                                       int64_t n_packed = 0, int64_t score_row0 = 0) {
    const int nh = packed != nullptr ? index_heads_for_tiles(r, n_packed) : index_heads_per_cta(r, q_count);
    if constexpr (DI == 1) {
        if (nh == 8) return launch_index_tc<BK, 8, DI, 0, F8, RUNL>(r, q_idx, k_idx, q_begin, q_count, kv_len, scores, ld_scores, n_cols, st, nullptr, packed, n_packed, score_row0);
        if (nh == 4) return launch_index_tc<BK, 4, DI, 0, F8, RUNL>(r, q_idx, k_idx, q_begin, q_count, kv_len, scores, ld_scores, n_cols, st, nullptr, packed, n_packed, score_row0);
    }
    if (nh == 2) return launch_index_tc<BK, 2, DI, 0, F8, RUNL>(r, q_idx, k_idx, q_begin, q_count, kv_len, scores, ld_scores, n_cols, st, nullptr, packed, n_packed, score_row0);
    return launch_index_tc<BK, 1, DI, 0, F8, RUNL>(r, q_idx, k_idx, q_begin, q_count, kv_len, scores, ld_scores, n_cols, st, nullptr, packed, n_packed, score_row0);
}

// runs: the score rows are written in run order (score_slot) instead of block order.
template <int BK, int DI, bool F8 = false>
static msa_status_t launch_index_tc_bk(const Resolved& r, const void* q_idx, const void* k_idx, int64_t q_begin,
                                       int64_t q_count, int64_t kv_len, float* scores, int64_t ld_scores,
                                       int64_t n_cols, cudaStream_t st, bool runs) {
    if (runs) return launch_index_tc_nh<BK, DI, F8, true>(r, q_idx, k_idx, q_begin, q_count, kv_len, scores, ld_scores, n_cols, st);
    return launch_index_tc_nh<BK, DI, F8, false>(r, q_idx, k_idx, q_begin, q_count, kv_len, scores, ld_scores, n_cols, st);
}


// Shapes of the tensor-core index kernel: one or two 128-byte atoms per index vector.
static bool index_tc_ok(const Resolved& r) {
    return (r.idx_fp8 ? r.d_idx == 128 : (r.d_idx == 64 || r.d_idx == 128)) && (r.B_k == 64 || r.B_k == 128);
}

// Eq. 6 and Eq. 7 in one kernel, no score matrix (top_k <= 16 on the tensor-core path).
static bool index_topk_fused_ok(const Resolved& r, int64_t q_count, int64_t kv_len) {
    return r.k <= kIdxFuseKeep + 1 && index_tc_ok(r) && kv_len < 2147483647LL && q_count >= 32;
}

template <int BK, int DI, bool F8 = false>
static msa_status_t launch_index_fused_bk(const Resolved& r, const void* q_idx, const void* k_idx, int64_t q_begin,
                                          int64_t q_count, int64_t kv_len, int32_t* block_idx, cudaStream_t st,
                                          const IdxPackedTile* packed, int64_t n_packed) {
    if (r.H_kv % 2 == 0)
        return launch_index_tc<BK, 2, DI, kIdxFuseKeep, F8>(r, q_idx, k_idx, q_begin, q_count, kv_len, nullptr, 0, 0, st,
                                                        block_idx, packed, n_packed);
    return launch_index_tc<BK, 1, DI, kIdxFuseKeep, F8>(r, q_idx, k_idx, q_begin, q_count, kv_len, nullptr, 0, 0, st,
                                                    block_idx, packed, n_packed);
}

// packed != null: a packed batch of q_count = kv_len rows in all, its query tiles listed in `packed`.
static msa_status_t run_index_topk_fused(const Resolved& r, const void* q_idx, const void* k_idx, int64_t q_begin,
                                         int64_t q_count, int64_t kv_len, int32_t* block_idx, cudaStream_t st,
                                         const IdxPackedTile* packed = nullptr, int64_t n_packed = 0) {
    if (r.idx_fp8) {
        if (r.B_k == 64) return launch_index_fused_bk<64, 1, true>(r, q_idx, k_idx, q_begin, q_count, kv_len, block_idx, st, packed, n_packed);
        return launch_index_fused_bk<128, 1, true>(r, q_idx, k_idx, q_begin, q_count, kv_len, block_idx, st, packed, n_packed);
    }
    if (r.d_idx == 64) {
        if (r.B_k == 64) return launch_index_fused_bk<64, 1>(r, q_idx, k_idx, q_begin, q_count, kv_len, block_idx, st, packed, n_packed);
        return launch_index_fused_bk<128, 1>(r, q_idx, k_idx, q_begin, q_count, kv_len, block_idx, st, packed, n_packed);
    }
    if (r.B_k == 64) return launch_index_fused_bk<64, 2>(r, q_idx, k_idx, q_begin, q_count, kv_len, block_idx, st, packed, n_packed);
    return launch_index_fused_bk<128, 2>(r, q_idx, k_idx, q_begin, q_count, kv_len, block_idx, st, packed, n_packed);
}

// Prefill ranges of at least 32 rows run on the tensor cores; shorter ones (and decode rows of
// shapes without a streaming kernel) take the generic kernel.
static bool index_scores_on_tc(const Resolved& r, int64_t n_rows, int64_t kv_len) {
    return index_tc_ok(r) && kv_len < 2147483647LL && n_rows >= 32;
}

static msa_status_t run_index_scores(const Resolved& r, const void* q_idx, const void* k_idx,
                                     const RowMap& rows, int64_t n_rows, float* scores,
                                     int64_t ld_scores, cudaStream_t st, bool runs = false) {
    if (n_rows == 0 || rows.n_cols == 0) return MSA_OK;
    if (rows.seq_lens == nullptr && index_scores_on_tc(r, n_rows, rows.kv_len)) {
        const int64_t qb = rows.q_begin, kl = rows.kv_len, nc = rows.n_cols;
        if (r.idx_fp8) {
            if (r.B_k == 64) return launch_index_tc_bk<64, 1, true>(r, q_idx, k_idx, qb, n_rows, kl, scores, ld_scores, nc, st, runs);
            return launch_index_tc_bk<128, 1, true>(r, q_idx, k_idx, qb, n_rows, kl, scores, ld_scores, nc, st, runs);
        }
        if (r.d_idx == 64) {
            if (r.B_k == 64) return launch_index_tc_bk<64, 1>(r, q_idx, k_idx, qb, n_rows, kl, scores, ld_scores, nc, st, runs);
            return launch_index_tc_bk<128, 1>(r, q_idx, k_idx, qb, n_rows, kl, scores, ld_scores, nc, st, runs);
        }
        if (r.B_k == 64) return launch_index_tc_bk<64, 2>(r, q_idx, k_idx, qb, n_rows, kl, scores, ld_scores, nc, st, runs);
        return launch_index_tc_bk<128, 2>(r, q_idx, k_idx, qb, n_rows, kl, scores, ld_scores, nc, st, runs);
    }
    constexpr int WARPS = 8;
    const int64_t n_chunks = ceil_div64(rows.n_cols, WARPS);
    const int64_t grid = n_rows * n_chunks;
    if (grid > 2147483647LL) return MSA_ERR_UNSUPPORTED;
    const size_t smem = sizeof(float) * (size_t)r.H_kv * r.d_idx;
    {
        StageScope sc(rows.seq_lens ? kStageIndexDecode : kStageIndex, st);
        if (r.idx_fp8)
            index_scores_generic_kernel<WARPS, true><<<(unsigned)grid, WARPS * 32, smem, st>>>(
                q_idx, k_idx, rows, n_chunks, r.H_kv, r.d_idx, r.B_k, r.index_scale, scores, ld_scores, score_lnb(r, runs));
        else
            index_scores_generic_kernel<WARPS, false><<<(unsigned)grid, WARPS * 32, smem, st>>>(
                q_idx, k_idx, rows, n_chunks, r.H_kv, r.d_idx, r.B_k, r.index_scale, scores, ld_scores, score_lnb(r, runs));
    }
    return launch_status();
}

// Eq. 6 for a group of sequences of a packed batch in one launch (tensor-core shapes only): the
// group's query tiles are listed in `tiles`; scores [group rows, H_kv, ld] in run order, row 0 =
// packed row score_row0.
static msa_status_t run_index_scores_packed(const Resolved& r, const void* q_idx, const void* k_idx, int64_t batch_rows,
                                            float* scores, int64_t ld, cudaStream_t st, const IdxPackedTile* tiles,
                                            int64_t n_tiles, int64_t score_row0) {
    if (n_tiles == 0) return MSA_OK;
    if (r.idx_fp8) {
        if (r.B_k == 64) return launch_index_tc_nh<64, 1, true, true>(r, q_idx, k_idx, 0, batch_rows, batch_rows, scores, ld, ld, st, tiles, n_tiles, score_row0);
        return launch_index_tc_nh<128, 1, true, true>(r, q_idx, k_idx, 0, batch_rows, batch_rows, scores, ld, ld, st, tiles, n_tiles, score_row0);
    }
    if (r.d_idx == 64) {
        if (r.B_k == 64) return launch_index_tc_nh<64, 1, false, true>(r, q_idx, k_idx, 0, batch_rows, batch_rows, scores, ld, ld, st, tiles, n_tiles, score_row0);
        return launch_index_tc_nh<128, 1, false, true>(r, q_idx, k_idx, 0, batch_rows, batch_rows, scores, ld, ld, st, tiles, n_tiles, score_row0);
    }
    if (r.B_k == 64) return launch_index_tc_nh<64, 2, false, true>(r, q_idx, k_idx, 0, batch_rows, batch_rows, scores, ld, ld, st, tiles, n_tiles, score_row0);
    return launch_index_tc_nh<128, 2, false, true>(r, q_idx, k_idx, 0, batch_rows, batch_rows, scores, ld, ld, st, tiles, n_tiles, score_row0);
}

// ---------------------------------------------------------------------- stage 2
static msa_status_t run_topk(const Resolved& r, const float* scores, int64_t ld_scores,
                             const RowMap& rows, int64_t n_q, int32_t* block_idx,
                             cudaStream_t st, bool runs = false) {
    const int64_t n_rows = n_q * r.H_kv;
    const int lnb = score_lnb(r, runs);
    if (n_rows == 0) return MSA_OK;
    const int64_t grid = ceil_div64(n_rows, kTopkWarps);
    if (grid > 2147483647LL) return MSA_ERR_UNSUPPORTED;
    const dim3 g((unsigned)grid), b(kTopkWarps * 32);
    int* status = async_status_ptr();
    if (status == nullptr) return MSA_ERR_CUDA;
    StageScope sc(kStageTopk, st);
    if (r.k <= 32)
        topk_select_kernel<1><<<g, b, 0, st>>>(scores, ld_scores, rows, n_rows, r.H_kv, r.B_k, r.k, block_idx, status, lnb);
    else if (r.k <= 64)
        topk_select_kernel<2><<<g, b, 0, st>>>(scores, ld_scores, rows, n_rows, r.H_kv, r.B_k, r.k, block_idx, status, lnb);
    else
        topk_select_kernel<4><<<g, b, 0, st>>>(scores, ld_scores, rows, n_rows, r.H_kv, r.B_k, r.k, block_idx, status, lnb);
    return launch_status();
}

// ---------------------------------------------------------------------- stage 3 (generic)
static msa_status_t run_attn_generic(const Resolved& r, const void* q, const void* k, const void* v,
                                     const int32_t* block_idx, const RowMap& rows, int64_t n_q,
                                     void* out, float* lse, cudaStream_t st) {
    if (n_q == 0) return MSA_OK;
    const int64_t grid = n_q * r.H_kv;
    if (grid > 2147483647LL) return MSA_ERR_UNSUPPORTED;
    int* status = async_status_ptr();
    if (status == nullptr) return MSA_ERR_CUDA;
    const size_t smem = sizeof(float) * (size_t)r.G * r.d;
    {
        StageScope sc(rows.seq_lens ? kStageAttnDecode : kStageAttn, st);
        sparse_attn_generic_kernel<<<(unsigned)grid, r.G * 32, smem, st>>>(
            (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, block_idx, rows,
            r.H_q, r.H_kv, r.d, r.B_k, r.k, r.softmax_scale, (__nv_bfloat16*)out, lse, status);
    }
    return launch_status();
}

static RowMap prefill_rows(int64_t q_begin, int64_t kv_len, int B_k) {
    RowMap m;
    m.q_begin = q_begin; m.kv_len = kv_len; m.seq_offsets = nullptr; m.seq_lens = nullptr;
    m.n_cols = ceil_div64(kv_len, B_k);
    return m;
}

static RowMap decode_rows(const int64_t* seq_offsets, const int32_t* seq_lens, int64_t max_len,
                          int B_k) {
    RowMap m;
    m.q_begin = 0; m.kv_len = 0; m.seq_offsets = seq_offsets; m.seq_lens = seq_lens;
    m.n_cols = ceil_div64(max_len, B_k);
    return m;
}

constexpr size_t kAlign = 256;
static size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// ---------------------------------------------------------------------- stage 3 (KV-outer, tcgen05)
static bool attn_tc_supported(const Resolved& r) {
    return r.d == 128 && (r.B_k == 64 || r.B_k == 128) && (r.G == 8 || r.G == 16);
}

// Workspace of the KV-outer path for ranges of R queries:
//   [cnt | tile_off | item_off] int32 per (block, head) tile, handles, LSE_buf, O_buf.
struct AttnPlan {
    int64_t R;
    size_t off_cnt, off_tile_off, off_item_off, off_handles, off_rank, off_lse, off_obuf, total;
};

static size_t attn_per_query_bytes(const Resolved& r) {
    return (size_t)r.H_q * r.k * r.d * 2 + (size_t)r.H_q * r.k * 4 + (size_t)r.H_kv * r.k * 8;
}

// n_blocks: KV blocks of the sequence (of all sequences of a packed batch).
static AttnPlan attn_plan_blocks(const Resolved& r, int64_t n_blocks, int64_t R) {
    AttnPlan p;
    p.R = R;
    const size_t n_tiles = (size_t)n_blocks * r.H_kv + 1;
    size_t o = 0;
    p.off_cnt = o; o += align_up(n_tiles * 4);
    p.off_tile_off = o; o += align_up(n_tiles * 4);
    p.off_item_off = o; o += align_up(n_tiles * 4);
    p.off_handles = o; o += align_up((size_t)R * r.H_kv * r.k * 4);
    p.off_rank = o; o += align_up((size_t)R * r.H_kv * r.k * 4);
    p.off_lse = o; o += align_up((size_t)R * r.H_q * r.k * 4);
    p.off_obuf = o; o += align_up((size_t)R * r.H_q * r.k * r.d * 2);
    p.total = o;
    return p;
}

static AttnPlan attn_plan(const Resolved& r, int64_t kv_len, int64_t R) {
    return attn_plan_blocks(r, ceil_div64(kv_len, r.B_k), R);
}

static int64_t attn_range_for_blocks(const Resolved& r, int64_t q_count, int64_t n_blocks, size_t ws_bytes) {
    const size_t fixed = attn_plan_blocks(r, n_blocks, 0).total + 4 * kAlign;
    if (ws_bytes <= fixed) return 0;
    int64_t R = (int64_t)((ws_bytes - fixed) / attn_per_query_bytes(r));
    if (R > q_count) R = q_count;
    if (R > (1 << 23)) R = 1 << 23;  // handles keep the query in 24 bits
    if (R >= 128) R = R / 128 * 128;
    return R;
}

static int64_t attn_range_for(const Resolved& r, int64_t q_count, int64_t kv_len, size_t ws_bytes) {
    return attn_range_for_blocks(r, q_count, ceil_div64(kv_len, r.B_k), ws_bytes);
}

static int current_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
    return dev;
}

static int sm_count() {
    static int n[64] = {0};  // per device
    const int dev = current_device();
    if (n[dev] == 0 && cudaDeviceGetAttribute(&n[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        n[dev] = 148;
    return n[dev];
}

// Copy-out hook used by msa_prefill_forward_host: after each query range is combined, its
// rows of O (and LSE) are copied to host memory on a second stream while the next range runs.
struct HostOutHook {
    bool on = false;
    cudaStream_t copy = nullptr;
    char* out_host = nullptr;
    float* lse_host = nullptr;
    int64_t rows_copied = 0;
};
static HostOutHook g_out_hook;

// Copy-in hook of the same call: Q is uploaded in pieces on the copy stream, an event after each;
// a query range's attention waits only for the piece that holds its last row (its reverse index
// and the ranges before it run while later pieces are still on their way).
struct HostInHook {
    bool on = false;
    int64_t piece_rows = 0;
    int n_pieces = 0;
    cudaEvent_t ev[256];            // the hook's own events (not drawn from the shared ring, whose
    int created[64] = {0};          // cursor may wrap during a long call); created per device
    cudaEvent_t own[64][256];
};
static cudaEvent_t next_sync_event();
static HostInHook g_in_hook;      // Q rows, waited for by the attention of each query range
static HostInHook g_in_idx_hook;  // Q_idx rows, waited for by the scoring of each query chunk

static msa_status_t wait_rows(const HostInHook& h, int64_t last_row, cudaStream_t st) {
    if (!h.on) return MSA_OK;
    int piece = (int)(last_row / h.piece_rows);
    if (piece >= h.n_pieces) piece = h.n_pieces - 1;
    return cudaStreamWaitEvent(st, h.ev[piece], 0) == cudaSuccess ? MSA_OK : MSA_ERR_CUDA;
}
// Uploads `rows` rows of `row_bytes` each in pieces on the copy stream, an event after each piece.
static msa_status_t upload_in_pieces(HostInHook& h, char* dst, const void* src, int64_t rows, size_t row_bytes,
                                     int64_t piece, cudaStream_t copy) {
    while (ceil_div64(rows, piece) > 256) piece *= 2;
    h.piece_rows = piece;
    h.n_pieces = (int)ceil_div64(rows, piece);
    const int dev = current_device();
    for (int i = 0; i < h.n_pieces; ++i) {
        const int64_t r0 = (int64_t)i * piece, n = (rows - r0) < piece ? (rows - r0) : piece;
        if (i >= h.created[dev]) {
            if (cudaEventCreateWithFlags(&h.own[dev][i], cudaEventDisableTiming) != cudaSuccess) return MSA_ERR_CUDA;
            h.created[dev] = i + 1;
        }
        h.ev[i] = h.own[dev][i];
        if (
            cudaMemcpyAsync(dst + (size_t)r0 * row_bytes, (const char*)src + (size_t)r0 * row_bytes, (size_t)n * row_bytes,
                            cudaMemcpyHostToDevice, copy) != cudaSuccess ||
            cudaEventRecord(h.ev[i], copy) != cudaSuccess)
            return MSA_ERR_CUDA;
    }
    return MSA_OK;
}

// A ring of events per device for orderings that are consumed at once (record on one stream, wait on
// another, in the same call): an event may be re-recorded as soon as the wait has been enqueued.
static cudaEvent_t next_sync_event() {
    constexpr int kPool = 2048;
    static cudaEvent_t pool[64][kPool];
    static int created[64] = {0}, cursor[64] = {0};
    const int dev = current_device();
    if (created[dev] < kPool && cursor[dev] == created[dev]) {
        if (cudaEventCreateWithFlags(&pool[dev][created[dev]], cudaEventDisableTiming) != cudaSuccess) return nullptr;
        ++created[dev];
    }
    cudaEvent_t e = pool[dev][cursor[dev]];
    cursor[dev] = (cursor[dev] + 1) % kPool;
    return e;
}

static msa_status_t hook_copy_rows(const Resolved& r, const void* out, const float* lse, int64_t row0,
                                   int64_t rows, cudaStream_t st) {
    HostOutHook& h = g_out_hook;
    cudaEvent_t e = next_sync_event();
    if (e == nullptr || cudaEventRecord(e, st) != cudaSuccess || cudaStreamWaitEvent(h.copy, e, 0) != cudaSuccess)
        return MSA_ERR_CUDA;
    const size_t rb = (size_t)r.H_q * r.d * 2;
    if (cudaMemcpyAsync(h.out_host + (size_t)row0 * rb, (const char*)out + (size_t)row0 * rb, (size_t)rows * rb,
                        cudaMemcpyDeviceToHost, h.copy) != cudaSuccess)
        return MSA_ERR_CUDA;
    if (h.lse_host && lse &&
        cudaMemcpyAsync(h.lse_host + row0 * r.H_q, lse + row0 * r.H_q, (size_t)rows * r.H_q * 4,
                        cudaMemcpyDeviceToHost, h.copy) != cudaSuccess)
        return MSA_ERR_CUDA;
    h.rows_copied = row0 + rows;
    return MSA_OK;
}

// F8: Q, K and V hold fp8 E4M3; rows of 128 bytes are moved as 64 two-byte elements.
// The three device arrays of a packed batch (see RangeParams) and its number of blocks; all zero for one sequence.
struct PackedBatch {
    const int32_t* row_pos = nullptr;
    const int32_t* row_blk0 = nullptr;
    const int32_t* blk_row0 = nullptr;
    int64_t n_blocks = 0;
};

template <int BK, int G, bool F8 = false>
static msa_status_t run_attn_prefill_tc(const Resolved& r, const void* q, const void* k, const void* v,
                                        const int32_t* block_idx, int64_t q_begin, int64_t q_count,
                                        int64_t kv_len, void* out, float* lse, void* ws, size_t ws_bytes,
                                        cudaStream_t st, const PackedBatch& pk = PackedBatch()) {
    const bool packed = pk.row_pos != nullptr;
    const int64_t all_blocks = packed ? pk.n_blocks : ceil_div64(kv_len, BK);
    const int64_t R = attn_range_for_blocks(r, q_count, all_blocks, ws_bytes);
    if (R <= 0) return MSA_ERR_WORKSPACE;
    const AttnPlan pl = attn_plan_blocks(r, all_blocks, R);
    char* w = static_cast<char*>(ws);
    int32_t* cnt = (int32_t*)(w + pl.off_cnt);
    int32_t* tile_off = (int32_t*)(w + pl.off_tile_off);
    int32_t* item_off = (int32_t*)(w + pl.off_item_off);
    uint32_t* handles = (uint32_t*)(w + pl.off_handles);
    uint32_t* rank = (uint32_t*)(w + pl.off_rank);
    float* lse_buf = (float*)(w + pl.off_lse);
    __nv_bfloat16* o_buf = (__nv_bfloat16*)(w + pl.off_obuf);

    CUtensorMap tm_q, tm_k, tm_v;
    if constexpr (F8) {
        // Q as (128 bytes, head, query): one box is a query's G heads, G swizzle rows.
        const uint64_t qd[3] = {64, (uint64_t)r.H_q, (uint64_t)q_count};
        const uint64_t qs[2] = {128, (uint64_t)r.H_q * 128};
        const uint32_t qb[3] = {64, (uint32_t)G, 1};
        const uint64_t kd[3] = {64, (uint64_t)r.H_kv, (uint64_t)kv_len};
        const uint64_t ks[2] = {128, (uint64_t)r.H_kv * 128};
        const uint32_t kb[3] = {64, 1, (uint32_t)BK};
        // (128-byte rows whose neighbours in memory are other heads' rows: no 256-byte L2 promotion)
        if (!encode_tmap_bf16(&tm_q, q, 3, qd, qs, qb) || !encode_tmap_bf16(&tm_k, k, 3, kd, ks, kb, true) ||
            !encode_tmap_bf16(&tm_v, v, 3, kd, ks, kb, true))
            return MSA_ERR_CUDA;
    } else {
        // Q as (64 d, 8 heads, 2 d halves, H_q/8 head groups, query): one box is a query's G heads.
        const uint64_t qd[5] = {64, 8, 2, (uint64_t)r.H_q / 8, (uint64_t)q_count};
        const uint64_t qs[4] = {256, 128, 2048, (uint64_t)r.H_q * 256};
        const uint32_t qb[5] = {64, 8, 2, (uint32_t)G / 8, 1};
        const uint64_t kd[3] = {128, (uint64_t)r.H_kv, (uint64_t)kv_len};
        const uint64_t ks[2] = {256, (uint64_t)r.H_kv * 256};
        const uint32_t kb[3] = {64, 1, (uint32_t)BK};
        if (!encode_tmap_bf16(&tm_q, q, 5, qd, qs, qb) || !encode_tmap_bf16(&tm_k, k, 3, kd, ks, kb) ||
            !encode_tmap_bf16(&tm_v, v, 3, kd, ks, kb))
            return MSA_ERR_CUDA;
    }
    int* status = async_status_ptr();
    if (status == nullptr) return MSA_ERR_CUDA;
    const size_t smem = sizeof(AttnSmem<BK>) + 1024;
    static bool attr_set_dev[64] = {false};  // the attribute is per device
    const int dev_id = current_device();
    if (!attr_set_dev[dev_id]) {
        if (cudaFuncSetAttribute(attn_prefill_tc_kernel<BK, G, F8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem) != cudaSuccess)
            return MSA_ERR_CUDA;
        attr_set_dev[dev_id] = true;
    }
    const float scale_log2e = r.softmax_scale * 1.4426950408889634f;
    const int grid_attn = sm_count();  // one CTA per SM (all of its shared memory and TMEM)
    for (int64_t q_first = 0; q_first < q_count; q_first += R) {
        RangeParams p = {};
        p.q_begin = q_begin; p.q_first = q_first;
        p.q_count = (int32_t)((q_count - q_first) < R ? (q_count - q_first) : R);
        // one sequence: the blocks up to the range's last query; a packed batch: all of its blocks
        p.n_blocks = (int32_t)(packed ? all_blocks : ceil_div64(q_begin + q_first + p.q_count, BK));
        p.H_kv = r.H_kv; p.top_k = r.k;
        p.row_pos = pk.row_pos; p.row_blk0 = pk.row_blk0; p.blk_row0 = pk.blk_row0;
        const int n_tiles = p.n_blocks * r.H_kv;
        const unsigned eg = (unsigned)ceil_div64((int64_t)p.q_count * r.H_kv, 8);  // 8 warps (rows) per CTA
        if (cudaMemsetAsync(cnt, 0, (size_t)(n_tiles + 1) * 4, st) != cudaSuccess) return MSA_ERR_CUDA;
        {
            StageScope sc(kStageSchedule, st);
            revidx_kernel<BK><<<eg, 256, 0, st>>>(block_idx, p, 0, cnt, tile_off, rank, handles, status);
        }
        {
            StageScope sc(kStageSchedule, st);
            revidx_scan_kernel<<<1, 1024, 0, st>>>(cnt, n_tiles, 128 / G, tile_off, item_off);
        }
        {
            StageScope sc(kStageSchedule, st);
            revidx_kernel<BK><<<eg, 256, 0, st>>>(block_idx, p, 1, cnt, tile_off, rank, handles, status);
        }
        if (q_begin == 0 && wait_rows(g_in_hook, q_first + p.q_count - 1, st) != MSA_OK)  // the range's Q rows
            return MSA_ERR_CUDA;
        {
            StageScope sc(kStageAttn, st);
            attn_prefill_tc_kernel<BK, G, F8><<<grid_attn, kAttnThreads, smem, st>>>(
                tm_q, tm_k, tm_v, p, tile_off, item_off, handles, scale_log2e, o_buf, lse_buf, status);
        }
        {
            StageScope sc(kStageCombine, st);
            combine_kernel<BK, G><<<(unsigned)(p.q_count * r.H_kv), G * 16, 0, st>>>(
                block_idx, p, o_buf, lse_buf, (__nv_bfloat16*)out, lse);
        }
        if (cudaPeekAtLastError() != cudaSuccess) return MSA_ERR_CUDA;
        if (g_out_hook.on && q_begin == 0 && g_out_hook.rows_copied == q_first) {
            const msa_status_t hs = hook_copy_rows(r, out, lse, q_first, p.q_count, st);
            if (hs != MSA_OK) return hs;
        }
    }
    return MSA_OK;
}

// ---------------------------------------------------------------------- decode path
static bool index_decode_fast(const Resolved& r) {
    return (r.d_idx == 64 || r.d_idx == 128) && r.H_kv <= 8;
}

static msa_status_t run_index_decode(const Resolved& r, const void* q_idx, const void* k_idx_cache,
                                     const int64_t* seq_offsets, const int32_t* seq_lens, int batch,
                                     int64_t n_cols, float* scores, int64_t ld_scores, cudaStream_t st) {
    const int grid = sm_count() * 4;
    StageScope sc(kStageIndexDecode, st);
    if (r.idx_fp8 && r.d_idx == 64)  // 64 fp8 per row: one 64-byte segment
        index_scores_decode_kernel<16, 1, true><<<grid, kIdxDecWarps * 32, 0, st>>>(
            (const __nv_bfloat16*)q_idx, (const __nv_bfloat16*)k_idx_cache, seq_offsets, seq_lens, batch, r.H_kv,
            r.B_k, r.index_scale, scores, ld_scores, n_cols);
    else if (r.idx_fp8)  // 128 fp8 per row: the bytes of 64 bf16
        index_scores_decode_kernel<8, 2, true><<<grid, kIdxDecWarps * 32, 0, st>>>(
            (const __nv_bfloat16*)q_idx, (const __nv_bfloat16*)k_idx_cache, seq_offsets, seq_lens, batch, r.H_kv,
            r.B_k, r.index_scale, scores, ld_scores, n_cols);
    else if (r.d_idx == 64)
        index_scores_decode_kernel<8, 2><<<grid, kIdxDecWarps * 32, 0, st>>>(
            (const __nv_bfloat16*)q_idx, (const __nv_bfloat16*)k_idx_cache, seq_offsets, seq_lens, batch, r.H_kv,
            r.B_k, r.index_scale, scores, ld_scores, n_cols);
    else
        index_scores_decode_kernel<4, 4><<<grid, kIdxDecWarps * 32, 0, st>>>(
            (const __nv_bfloat16*)q_idx, (const __nv_bfloat16*)k_idx_cache, seq_offsets, seq_lens, batch, r.H_kv,
            r.B_k, r.index_scale, scores, ld_scores, n_cols);
    return launch_status();
}

static bool attn_decode_fast(const Resolved& r) {
    return r.d == 128 && (r.G == 8 || r.G == 16) && (r.B_k == 64 || r.B_k == 128);
}

static int decode_n_split(const Resolved& r) { return (r.k + kDecBlocksPerItem - 1) / kDecBlocksPerItem; }

static size_t decode_ws_bytes(const Resolved& r, int batch) {
    const size_t parts = (size_t)batch * r.H_kv * decode_n_split(r) * kDecPartsPerItem;
    return align_up(parts * r.G * 128 * 4) + align_up(parts * 2 * r.G * 4) + kAlign;
}

// KV8: the caches hold fp8 E4M3; a key row of 128 bytes is moved as 64 two-byte elements (one box per tile).
template <int BK, int G, bool KV8 = false>
static msa_status_t run_attn_decode_tc(const Resolved& r, const void* q, const void* k_cache, const void* v_cache,
                                       int64_t cache_tokens, const int64_t* seq_offsets, const int32_t* seq_lens,
                                       int batch, const int32_t* block_idx, void* out, float* lse, void* ws,
                                       cudaStream_t st) {
    CUtensorMap tm_k, tm_v;
    const uint64_t row_b = KV8 ? 128 : 256;  // bytes of one head's key or value vector
    const uint64_t kd[3] = {row_b / 2, (uint64_t)r.H_kv, (uint64_t)cache_tokens};
    const uint64_t ks[2] = {row_b, (uint64_t)r.H_kv * row_b};
    const uint32_t kb[3] = {64, 1, (uint32_t)BK};
    if (!encode_tmap_bf16(&tm_k, k_cache, 3, kd, ks, kb, KV8) || !encode_tmap_bf16(&tm_v, v_cache, 3, kd, ks, kb, KV8))
        return MSA_ERR_CUDA;
    int* status = async_status_ptr();
    if (status == nullptr) return MSA_ERR_CUDA;
    const size_t smem = (KV8 ? sizeof(DecKv8Smem<BK>) : sizeof(DecSmem<BK>)) + 1024;
    static bool attr_set_dev[64] = {false};  // the attribute is per device
    const int dev_id = current_device();
    if (!attr_set_dev[dev_id]) {
        const cudaError_t e =
            KV8 ? cudaFuncSetAttribute(attn_decode_kv8_kernel<BK, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
                : cudaFuncSetAttribute(attn_decode_kernel<BK, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return MSA_ERR_CUDA;
        attr_set_dev[dev_id] = true;
    }
    DecParams p;
    p.q = (const __nv_bfloat16*)q; p.block_idx = block_idx; p.seq_offsets = seq_offsets; p.seq_lens = seq_lens;
    p.batch = batch; p.H_kv = r.H_kv; p.top_k = r.k; p.n_split = decode_n_split(r);
    p.scale_log2e = r.softmax_scale * 1.4426950408889634f;
    const size_t parts = (size_t)batch * r.H_kv * p.n_split * kDecPartsPerItem;
    p.part_o = (float*)ws;
    p.part_ml = (float*)((char*)ws + align_up(parts * G * 128 * 4));
    const int n_items = batch * r.H_kv * p.n_split;
    const int ctas = sm_count() * 2;
    const int grid = n_items < ctas ? n_items : ctas;
    {
        StageScope sc(kStageAttnDecode, st);
        if constexpr (KV8)
            attn_decode_kv8_kernel<BK, G><<<grid, kDecThreads, smem, st>>>(tm_k, tm_v, p, status);
        else
            attn_decode_kernel<BK, G><<<grid, kDecThreads, smem, st>>>(tm_k, tm_v, p, status);
    }
    {
        StageScope sc(kStageCombineDecode, st);
        attn_decode_combine_kernel<<<(batch * r.H_q + 3) / 4, 128, 0, st>>>(p.part_o, p.part_ml, batch, r.H_kv, G,
                                                                             p.n_split, (__nv_bfloat16*)out, lse);
    }
    return launch_status();
}

// ---------------------------------------------------------------------- index-branch LSE (Section 4.3)
static bool index_lse_fast(const Resolved& r) {  // bf16 operands; fp8 takes the generic kernel
    return !r.idx_fp8 && (r.d_idx == 64 || r.d_idx == 128) && (r.B_k == 64 || r.B_k == 128);
}

// Workspace for ranges of R queries: [cnt | tile_off | item_off] per tile, handles, rank, partials.
struct LsePlan {
    size_t off_cnt, off_tile_off, off_item_off, off_handles, off_rank, off_part, total;
};

static LsePlan lse_plan(const Resolved& r, int64_t kv_len, int64_t R) {
    LsePlan p;
    const size_t n_tiles = (size_t)ceil_div64(kv_len, r.B_k) * r.H_kv + 1;
    const size_t pairs = (size_t)R * r.H_kv * r.k;
    size_t o = 0;
    p.off_cnt = o; o += align_up(n_tiles * 4);
    p.off_tile_off = o; o += align_up(n_tiles * 4);
    p.off_item_off = o; o += align_up(n_tiles * 4);
    p.off_handles = o; o += align_up(pairs * 4);
    p.off_rank = o; o += align_up(pairs * 4);
    p.off_part = o; o += align_up(pairs * 4);
    p.total = o;
    return p;
}

template <int BK, int DIDX>
static msa_status_t run_index_lse(const Resolved& r, const void* q_idx, const void* k_idx,
                                  const int32_t* block_idx, int64_t q_begin, int64_t q_count, int64_t kv_len,
                                  float* lse_idx, void* ws, size_t ws_bytes, cudaStream_t st) {
    const size_t fixed = lse_plan(r, kv_len, 0).total + 4 * kAlign;
    if (ws_bytes <= fixed) return MSA_ERR_WORKSPACE;
    int64_t R = (int64_t)((ws_bytes - fixed) / ((size_t)r.H_kv * r.k * 12));
    if (R > q_count) R = q_count;
    if (R > (1 << 23)) R = 1 << 23;  // handles keep the query in 24 bits
    if (R <= 0) return MSA_ERR_WORKSPACE;
    const LsePlan pl = lse_plan(r, kv_len, R);
    char* w = static_cast<char*>(ws);
    int32_t* cnt = (int32_t*)(w + pl.off_cnt);
    int32_t* tile_off = (int32_t*)(w + pl.off_tile_off);
    int32_t* item_off = (int32_t*)(w + pl.off_item_off);
    uint32_t* handles = (uint32_t*)(w + pl.off_handles);
    uint32_t* rank = (uint32_t*)(w + pl.off_rank);
    float* part = (float*)(w + pl.off_part);
    int* status = async_status_ptr();
    if (status == nullptr) return MSA_ERR_CUDA;
    const size_t smem = (size_t)(BK + 2 * kLseItemQueries) * DIDX * 2 + 2 * kLseItemQueries * 4 + 1024;
    static bool attr_set_dev[64] = {false};  // the attribute is per device
    const int dev_id = current_device();
    if (!attr_set_dev[dev_id]) {
        if (cudaFuncSetAttribute(index_lse_kernel<BK, DIDX>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
            cudaSuccess)
            return MSA_ERR_CUDA;
        attr_set_dev[dev_id] = true;
    }
    const float scale_log2e = r.index_scale * 1.4426950408889634f;
    int per_sm = (int)((227 * 1024) / (smem + 1024));  // resident CTAs by shared memory, at most 4
    if (per_sm > 4) per_sm = 4;
    const int grid = sm_count() * per_sm;
    for (int64_t q_first = 0; q_first < q_count; q_first += R) {
        RangeParams p = {};
        p.q_begin = q_begin; p.q_first = q_first;
        p.q_count = (int32_t)((q_count - q_first) < R ? (q_count - q_first) : R);
        p.n_blocks = (int32_t)ceil_div64(q_begin + q_first + p.q_count, BK);
        p.H_kv = r.H_kv; p.top_k = r.k;
        const int n_tiles = p.n_blocks * r.H_kv;
        const unsigned eg = (unsigned)ceil_div64((int64_t)p.q_count * r.H_kv, 8);  // 8 warps (rows) per CTA
        if (cudaMemsetAsync(cnt, 0, (size_t)(n_tiles + 1) * 4, st) != cudaSuccess) return MSA_ERR_CUDA;
        {
            StageScope sc(kStageSchedule, st);
            revidx_kernel<BK><<<eg, 256, 0, st>>>(block_idx, p, 0, cnt, tile_off, rank, handles, status);
        }
        {
            StageScope sc(kStageSchedule, st);
            revidx_scan_kernel<<<1, 1024, 0, st>>>(cnt, n_tiles, kLseItemQueries, tile_off, item_off);
        }
        {
            StageScope sc(kStageSchedule, st);
            revidx_kernel<BK><<<eg, 256, 0, st>>>(block_idx, p, 1, cnt, tile_off, rank, handles, status);
        }
        {
            StageScope sc(kStageIndexLse, st);
            index_lse_kernel<BK, DIDX><<<grid, kLseThreads, smem, st>>>(
                (const __nv_bfloat16*)q_idx, (const __nv_bfloat16*)k_idx, p, kv_len, tile_off, item_off, handles,
                scale_log2e, part, status);
        }
        {
            StageScope sc(kStageIndexLse, st);
            index_lse_reduce_kernel<BK><<<eg, 256, 0, st>>>(block_idx, p, part, lse_idx);
        }
        if (cudaPeekAtLastError() != cudaSuccess) return MSA_ERR_CUDA;
    }
    return MSA_OK;
}

}  // namespace msa

using namespace msa;

extern "C" {

const char* msa_status_string(msa_status_t s) {
    switch (s) {
        case MSA_OK: return "ok";
        case MSA_ERR_INVALID_ARG: return "invalid argument";
        case MSA_ERR_UNSUPPORTED: return "unsupported shape";
        case MSA_ERR_WORKSPACE: return "workspace too small";
        case MSA_ERR_CUDA: return "CUDA error";
        case MSA_ERR_TIMEOUT: return "device-side wait timed out";
        case MSA_ERR_BAD_INDEX: return "block index out of range";
    }
    return "unknown status";
}

int64_t msa_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

msa_status_t msa_profile_begin(void) {
    if (!g_prof_created) {
        for (int i = 0; i < kProfSlots; ++i)
            for (int j = 0; j < 2; ++j)
                if (cudaEventCreate(&g_prof_ev[i][j]) != cudaSuccess) return MSA_ERR_CUDA;
        g_prof_created = true;
    }
    g_prof_used = 0;
    g_prof_on = true;
    return MSA_OK;
}

msa_status_t msa_profile_end(float* stage_ms_host, int64_t* stage_launches_host) {
    g_prof_on = false;
    if (cudaDeviceSynchronize() != cudaSuccess) return MSA_ERR_CUDA;
    for (int i = 0; i < kNumStages; ++i) {
        if (stage_ms_host) stage_ms_host[i] = 0.f;
        if (stage_launches_host) stage_launches_host[i] = 0;
    }
    for (int i = 0; i < g_prof_used; ++i) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, g_prof_ev[i][0], g_prof_ev[i][1]) != cudaSuccess) return MSA_ERR_CUDA;
        if (stage_ms_host) stage_ms_host[g_prof_stage[i]] += ms;
        if (stage_launches_host) stage_launches_host[g_prof_stage[i]] += 1;
    }
    const bool overflow = g_prof_used >= kProfSlots;
    g_prof_used = 0;
    return overflow ? MSA_ERR_UNSUPPORTED : MSA_OK;
}

msa_status_t msa_check_async_status(int32_t* detail_host) {
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_async_status, sizeof(int)) != cudaSuccess) return MSA_ERR_CUDA;
    if (v != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(g_async_status, &zero, sizeof(int)) != cudaSuccess) return MSA_ERR_CUDA;
    }
    if (detail_host) *detail_host = v & 0xFFFFFF;
    const int code = v >> 24;
    if (code == kAsyncTimeout) return MSA_ERR_TIMEOUT;
    if (code == kAsyncBadIndex) return MSA_ERR_BAD_INDEX;
    return MSA_OK;
}

msa_status_t msa_index_scores(const msa_shape_t* shape, const void* q_idx, const void* k_idx,
                              int64_t q_begin, int64_t q_count, int64_t kv_len, float* scores,
                              int64_t ld_scores, msa_stream_t stream) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    if ((s = check_range(q_begin, q_count, kv_len)) != MSA_OK) return s;
    if (q_count == 0) return MSA_OK;
    if (!q_idx || !k_idx || !scores || !aligned16(q_idx) || !aligned16(k_idx) || !aligned16(scores))
        return MSA_ERR_INVALID_ARG;
    const int64_t B = ceil_div64(kv_len, r.B_k);
    if (ld_scores < B || ld_scores % 4 != 0) return MSA_ERR_INVALID_ARG;
    if (r.score_runs && (ld_scores < (B + 7) / 8 * 8 || ld_scores % 8 != 0)) return MSA_ERR_INVALID_ARG;
    return run_index_scores(r, q_idx, k_idx, prefill_rows(q_begin, kv_len, r.B_k), q_count, scores,
                            ld_scores, (cudaStream_t)stream, r.score_runs);
}

msa_status_t msa_index_scores_plan(const msa_shape_t* shape, int64_t q_count, int64_t kv_len,
                                   int32_t* tensor_core, int32_t* heads_per_cta) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    if (q_count < 0 || kv_len < 0 || q_count > kv_len) return MSA_ERR_INVALID_ARG;
    const bool tc = q_count > 0 && index_scores_on_tc(r, q_count, kv_len);
    if (tensor_core) *tensor_core = tc ? 1 : 0;
    if (heads_per_cta) *heads_per_cta = tc ? index_heads_per_cta(r, q_count) : 0;
    return MSA_OK;
}

#ifdef MSA_TRACE
// Development builds only (-DMSA_TRACE): the 16 x 16 clock stamps CTA 0 of the prefill attention kernel recorded.
extern "C" int msa_debug_read_trace(long long* host256) {
    return cudaMemcpyFromSymbol(host256, g_trace, sizeof(long long) * 256) == cudaSuccess ? 0 : 1;
}
#endif

msa_status_t msa_debug_set_wait(int64_t wait_limit_cycles, int64_t producer_delay_cycles) {
    if (wait_limit_cycles < 0 || producer_delay_cycles < 0) return MSA_ERR_INVALID_ARG;
    // Never longer than the production limit, and a delay well inside it: a test can shorten a
    // wait, it cannot turn a kernel into one that runs for long.
    const long long limit = (wait_limit_cycles == 0 || wait_limit_cycles > kWaitLimitCycles)
                                ? kWaitLimitCycles : (long long)wait_limit_cycles;
    if (producer_delay_cycles > 100000000LL) return MSA_ERR_INVALID_ARG;  // 50 ms
    const long long late = (long long)producer_delay_cycles;
    if (cudaMemcpyToSymbol(g_wait_limit_cycles, &limit, sizeof(limit)) != cudaSuccess ||
        cudaMemcpyToSymbol(g_debug_producer_delay, &late, sizeof(late)) != cudaSuccess)
        return MSA_ERR_CUDA;
    return MSA_OK;
}

msa_status_t msa_index_topk_fused(const msa_shape_t* shape, const void* q_idx, const void* k_idx,
                                  int64_t q_begin, int64_t q_count, int64_t kv_len, int32_t* block_idx,
                                  msa_stream_t stream) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    if ((s = check_range(q_begin, q_count, kv_len)) != MSA_OK) return s;
    if (q_count == 0) return MSA_OK;
    if (!q_idx || !k_idx || !block_idx || !aligned16(q_idx) || !aligned16(k_idx)) return MSA_ERR_INVALID_ARG;
    if (!index_topk_fused_ok(r, q_count, kv_len)) return MSA_ERR_UNSUPPORTED;
    return run_index_topk_fused(r, q_idx, k_idx, q_begin, q_count, kv_len, block_idx, (cudaStream_t)stream);
}

msa_status_t msa_index_scores_decode(const msa_shape_t* shape, const void* q_idx,
                                     const void* k_idx_cache, const int64_t* seq_offsets,
                                     const int32_t* seq_lens, int32_t batch, int64_t max_seq_len,
                                     float* scores, int64_t ld_scores, msa_stream_t stream) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    if (r.score_runs) return MSA_ERR_UNSUPPORTED;  // decode rows are in block order
    if (batch < 0 || max_seq_len < 0) return MSA_ERR_INVALID_ARG;
    if (batch == 0) return MSA_OK;
    if (!q_idx || !k_idx_cache || !seq_offsets || !seq_lens || !scores || !aligned16(q_idx) ||
        !aligned16(k_idx_cache) || !aligned16(scores))
        return MSA_ERR_INVALID_ARG;
    if (ld_scores < ceil_div64(max_seq_len, r.B_k) || ld_scores % 4 != 0) return MSA_ERR_INVALID_ARG;
    if (index_decode_fast(r))
        return run_index_decode(r, q_idx, k_idx_cache, seq_offsets, seq_lens, batch,
                                ceil_div64(max_seq_len, r.B_k), scores, ld_scores, (cudaStream_t)stream);
    return run_index_scores(r, q_idx, k_idx_cache, decode_rows(seq_offsets, seq_lens, max_seq_len, r.B_k),
                            batch, scores, ld_scores, (cudaStream_t)stream);
}

msa_status_t msa_topk_select(const msa_shape_t* shape, const float* scores, int64_t ld_scores,
                             int64_t q_begin, int64_t q_count, int64_t kv_len, int32_t* block_idx,
                             msa_stream_t stream) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    if ((s = check_range(q_begin, q_count, kv_len)) != MSA_OK) return s;
    if (q_count == 0) return MSA_OK;
    if (!scores || !block_idx || !aligned16(scores)) return MSA_ERR_INVALID_ARG;
    if (ld_scores < ceil_div64(kv_len, r.B_k) || ld_scores % 4 != 0) return MSA_ERR_INVALID_ARG;
    if (r.score_runs && (ld_scores < (ceil_div64(kv_len, r.B_k) + 7) / 8 * 8 || ld_scores % 8 != 0))
        return MSA_ERR_INVALID_ARG;
    return run_topk(r, scores, ld_scores, prefill_rows(q_begin, kv_len, r.B_k), q_count, block_idx,
                    (cudaStream_t)stream, r.score_runs);
}

msa_status_t msa_topk_select_decode(const msa_shape_t* shape, const float* scores, int64_t ld_scores,
                                    const int32_t* seq_lens, int32_t batch, int64_t max_seq_len,
                                    int32_t* block_idx, msa_stream_t stream) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    if (r.score_runs) return MSA_ERR_UNSUPPORTED;  // decode rows are in block order
    if (batch < 0 || max_seq_len < 0) return MSA_ERR_INVALID_ARG;
    if (batch == 0) return MSA_OK;
    if (!scores || !block_idx || !seq_lens || !aligned16(scores) || ld_scores % 4 != 0 || ld_scores <= 0)
        return MSA_ERR_INVALID_ARG;
    if (ld_scores < ceil_div64(max_seq_len, r.B_k)) return MSA_ERR_INVALID_ARG;
    RowMap rows = decode_rows(nullptr, seq_lens, 0, r.B_k);  // offsets are not needed for ranking
    return run_topk(r, scores, ld_scores, rows, batch, block_idx, (cudaStream_t)stream);
}

// A prefill call on fp8 K/V caches runs on bf16 copies of the rows it can see (E4M3 -> bf16 is
// exact): the caches are read once more per call, 3 bytes of traffic per element, against the
// partial buffers' hundreds of bytes per (query, head).
static size_t kv_copy_bytes(const Resolved& r, int64_t kv_len) {
    return align_up((size_t)kv_len * r.H_kv * r.d * 2);
}

// Q, K and V all in fp8 on a shape of the tensor-core kernel: the kernel reads the fp8 tensors itself.
static bool attn_fp8_direct(const Resolved& r, int64_t kv_len) {
    return r.q_fp8 && r.kv_fp8 && attn_tc_supported(r) && kv_len < 2147483647LL;
}

msa_status_t msa_sparse_attn_prefill_workspace_bytes(const msa_shape_t* shape, int64_t q_count,
                                                     int64_t kv_len, size_t* min_bytes,
                                                     size_t* preferred_bytes) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    if (q_count < 0 || kv_len < 0) return MSA_ERR_INVALID_ARG;
    size_t mn = kAlign, pf = kAlign;
    if (attn_tc_supported(r) && q_count > 0) {
        // at least 256 queries in flight; preferred: partial buffers of up to 32 GiB (larger ranges
        // mean fuller tiles and fewer K/V reloads; measured 498 / 484 / 473 ms at 8 / 16 / 32 GiB, T = 1M)
        const int64_t r_min = q_count < 256 ? q_count : 256;
        int64_t r_pref = (int64_t)((32ull << 30) / attn_per_query_bytes(r));
        if (r_pref > q_count) r_pref = q_count;
        if (r_pref < r_min) r_pref = r_min;
        mn = attn_plan(r, kv_len, r_min).total + 8 * kAlign;
        pf = attn_plan(r, kv_len, r_pref).total + 8 * kAlign;
    }
    if (r.kv_fp8 && !attn_fp8_direct(r, kv_len)) {  // bf16 copies of the visible K and V rows in front
        mn += 2 * kv_copy_bytes(r, kv_len);
        pf += 2 * kv_copy_bytes(r, kv_len);
    }
    if (min_bytes) *min_bytes = mn;
    if (preferred_bytes) *preferred_bytes = pf;
    return MSA_OK;
}

// The tensor-core attention for the shape's (B_k, G), bf16 or fp8 operands; pk: a packed batch or nothing.
static msa_status_t attn_prefill_tc_dispatch(const Resolved& r, bool f8, const void* q, const void* k, const void* v,
                                             const int32_t* block_idx, int64_t q_begin, int64_t q_count, int64_t kv_len,
                                             void* out, float* lse, void* ws, size_t ws_bytes, cudaStream_t st,
                                             const PackedBatch& pk = PackedBatch()) {
#define MSA_ATTN_CASE(BK_, G_)                                                                                              \
    if (r.B_k == BK_ && r.G == G_)                                                                                          \
        return f8 ? run_attn_prefill_tc<BK_, G_, true>(r, q, k, v, block_idx, q_begin, q_count, kv_len, out, lse, ws,      \
                                                        ws_bytes, st, pk)                                                    \
                  : run_attn_prefill_tc<BK_, G_, false>(r, q, k, v, block_idx, q_begin, q_count, kv_len, out, lse, ws,     \
                                                         ws_bytes, st, pk);
    MSA_ATTN_CASE(64, 8)
    MSA_ATTN_CASE(64, 16)
    MSA_ATTN_CASE(128, 8)
    MSA_ATTN_CASE(128, 16)
#undef MSA_ATTN_CASE
    return MSA_ERR_UNSUPPORTED;
}

// fp8 E4M3 -> bf16 copies of `rows` K and V rows into kb and vb (exact).
static msa_status_t widen_kv(const Resolved& r, const void* k, const void* v, int64_t rows, char* kb, char* vb,
                             cudaStream_t st) {
    if (r.d % 16 != 0) return MSA_ERR_UNSUPPORTED;  // the conversion moves 16 elements per thread
    const int64_t n16 = rows * r.H_kv * r.d / 16;
    const unsigned grid = (unsigned)(n16 < 148 * 8 * 256 ? ceil_div64(n16 > 0 ? n16 : 1, 256) : 148 * 8);
    {
        StageScope sc(kStageAttn, st);
        e4m3_to_bf16_kernel<<<grid, 256, 0, st>>>((const uint4*)k, (uint4*)kb, n16);
    }
    {
        StageScope sc(kStageAttn, st);
        e4m3_to_bf16_kernel<<<grid, 256, 0, st>>>((const uint4*)v, (uint4*)vb, n16);
    }
    return cudaPeekAtLastError() == cudaSuccess ? MSA_OK : MSA_ERR_CUDA;
}

msa_status_t msa_sparse_attn_prefill(const msa_shape_t* shape, const void* q, const void* k,
                                     const void* v, const int32_t* block_idx, int64_t q_begin,
                                     int64_t q_count, int64_t kv_len, void* out, float* lse,
                                     void* workspace, size_t workspace_bytes, msa_stream_t stream) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    if ((s = check_range(q_begin, q_count, kv_len)) != MSA_OK) return s;
    if (q_count == 0) return MSA_OK;
    if (!q || !k || !v || !block_idx || !out || !aligned16(q) || !aligned16(k) || !aligned16(v) ||
        !aligned16(out))
        return MSA_ERR_INVALID_ARG;
    size_t need = 0;
    msa_sparse_attn_prefill_workspace_bytes(shape, q_count, kv_len, &need, nullptr);
    if (workspace == nullptr || workspace_bytes < need || !aligned16(workspace)) return MSA_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    if (attn_fp8_direct(r, kv_len))
        return attn_prefill_tc_dispatch(r, true, q, k, v, block_idx, q_begin, q_count, kv_len, out, lse, workspace,
                                        workspace_bytes, st);
    if (r.q_fp8) return MSA_ERR_UNSUPPORTED;  // fp8 Q: the tensor-core kernel's shapes only
    if (r.kv_fp8) {  // bf16 copies of the visible rows, then the bf16 path on the rest of the workspace
        const size_t cb = kv_copy_bytes(r, kv_len);
        char* kb = (char*)workspace;
        char* vb = kb + cb;
        if ((s = widen_kv(r, k, v, kv_len, kb, vb, st)) != MSA_OK) return s;
        msa_shape_t wide = *shape;
        wide.kv_fp8 = 0;
        return msa_sparse_attn_prefill(&wide, q, kb, vb, block_idx, q_begin, q_count, kv_len, out, lse,
                                       (char*)workspace + 2 * cb, workspace_bytes - 2 * cb, stream);
    }
    if (attn_tc_supported(r) && kv_len < 2147483647LL)
        return attn_prefill_tc_dispatch(r, false, q, k, v, block_idx, q_begin, q_count, kv_len, out, lse, workspace,
                                        workspace_bytes, st);
    return run_attn_generic(r, q, k, v, block_idx, prefill_rows(q_begin, kv_len, r.B_k), q_count, out,
                            lse, st);
}

// ---------------------------------------------------------------------- index-branch LSE (Section 4.3)
msa_status_t msa_index_lse_prefill_workspace_bytes(const msa_shape_t* shape, int64_t q_count,
                                                   int64_t kv_len, size_t* min_bytes,
                                                   size_t* preferred_bytes) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    if (q_count < 0 || kv_len < 0) return MSA_ERR_INVALID_ARG;
    size_t mn = kAlign, pf = kAlign;
    if (index_lse_fast(r) && q_count > 0) {
        const int64_t r_min = q_count < 256 ? q_count : 256;
        const int64_t r_pref = q_count < 131072 ? q_count : 131072;
        mn = lse_plan(r, kv_len, r_min).total + 8 * kAlign;
        pf = lse_plan(r, kv_len, r_pref).total + 8 * kAlign;
    }
    if (min_bytes) *min_bytes = mn;
    if (preferred_bytes) *preferred_bytes = pf;
    return MSA_OK;
}

msa_status_t msa_index_lse_prefill(const msa_shape_t* shape, const void* q_idx, const void* k_idx,
                                   const int32_t* block_idx, int64_t q_begin, int64_t q_count,
                                   int64_t kv_len, float* lse_idx, void* workspace,
                                   size_t workspace_bytes, msa_stream_t stream) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    if ((s = check_range(q_begin, q_count, kv_len)) != MSA_OK) return s;
    if (q_count == 0) return MSA_OK;
    if (!q_idx || !k_idx || !block_idx || !lse_idx || !aligned16(q_idx) || !aligned16(k_idx))
        return MSA_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (index_lse_fast(r) && kv_len < 2147483647LL) {
        size_t need = 0;
        msa_index_lse_prefill_workspace_bytes(shape, q_count, kv_len, &need, nullptr);
        if (workspace == nullptr || workspace_bytes < need || !aligned16(workspace)) return MSA_ERR_WORKSPACE;
        if (r.B_k == 64 && r.d_idx == 64)
            return run_index_lse<64, 64>(r, q_idx, k_idx, block_idx, q_begin, q_count, kv_len, lse_idx, workspace, workspace_bytes, st);
        if (r.B_k == 64)
            return run_index_lse<64, 128>(r, q_idx, k_idx, block_idx, q_begin, q_count, kv_len, lse_idx, workspace, workspace_bytes, st);
        if (r.d_idx == 64)
            return run_index_lse<128, 64>(r, q_idx, k_idx, block_idx, q_begin, q_count, kv_len, lse_idx, workspace, workspace_bytes, st);
        return run_index_lse<128, 128>(r, q_idx, k_idx, block_idx, q_begin, q_count, kv_len, lse_idx, workspace, workspace_bytes, st);
    }
    const int64_t rows = q_count * r.H_kv;
    const int64_t grid = ceil_div64(rows, 8);
    if (grid > 2147483647LL) return MSA_ERR_UNSUPPORTED;
    {
        StageScope sc(kStageIndexLse, st);
        if (r.idx_fp8)
            index_lse_generic_kernel<true><<<(unsigned)grid, 256, 0, st>>>(
                q_idx, k_idx, block_idx, q_begin, q_count, kv_len, r.H_kv, r.d_idx, r.B_k, r.k, r.index_scale, lse_idx);
        else
            index_lse_generic_kernel<false><<<(unsigned)grid, 256, 0, st>>>(
                q_idx, k_idx, block_idx, q_begin, q_count, kv_len, r.H_kv, r.d_idx, r.B_k, r.k, r.index_scale, lse_idx);
    }
    return launch_status();
}

// Scratch of msa_sparse_attn_prefill_static: part of the library's device image, so no call
// ever allocates it.  In host code this name is only a handle for cudaGetSymbolAddress; it
// is not a device address and must never be passed to a kernel as is.
static __device__ __align__(256) unsigned char g_static_scratch[MSA_STATIC_SCRATCH_BYTES];

// Device address of g_static_scratch on the current device, looked up once per device.
static msa_status_t static_scratch_ptr(void** out) {
    constexpr int kMaxDevices = 64;
    static void* cached[kMaxDevices] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return MSA_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return MSA_ERR_UNSUPPORTED;
    if (cached[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return MSA_ERR_CUDA;
        cached[dev] = p;
    }
    *out = cached[dev];
    return MSA_OK;
}

msa_status_t msa_sparse_attn_prefill_static(const msa_shape_t* shape, const void* q, const void* k,
                                            const void* v, const int32_t* block_idx, int64_t q_begin,
                                            int64_t q_count, int64_t kv_len, void* out, float* lse,
                                            msa_stream_t stream) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    if (r.kv_fp8) return MSA_ERR_UNSUPPORTED;  // fp8 K/V caches: decode calls only
    if ((s = check_range(q_begin, q_count, kv_len)) != MSA_OK) return s;
    if (q_count == 0) return MSA_OK;
    if (!q || !k || !v || !block_idx || !out || !aligned16(q) || !aligned16(k) || !aligned16(v) ||
        !aligned16(out))
        return MSA_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (!attn_tc_supported(r) || kv_len >= 2147483647LL)  // the generic kernel needs no scratch at all
        return run_attn_generic(r, q, k, v, block_idx, prefill_rows(q_begin, kv_len, r.B_k), q_count, out,
                                lse, st);
    // Refuse sizes the fixed array cannot serve: fewer than min(q_count, 16) queries per pass.
    const int64_t fit = attn_range_for(r, q_count, kv_len, (size_t)MSA_STATIC_SCRATCH_BYTES);
    if (fit < (q_count < 16 ? q_count : 16)) return MSA_ERR_WORKSPACE;
    void* scratch = nullptr;
    if ((s = static_scratch_ptr(&scratch)) != MSA_OK) return s;
    const size_t bytes = (size_t)MSA_STATIC_SCRATCH_BYTES;
    if (r.B_k == 64 && r.G == 8)
        return run_attn_prefill_tc<64, 8>(r, q, k, v, block_idx, q_begin, q_count, kv_len, out, lse, scratch, bytes, st);
    if (r.B_k == 64 && r.G == 16)
        return run_attn_prefill_tc<64, 16>(r, q, k, v, block_idx, q_begin, q_count, kv_len, out, lse, scratch, bytes, st);
    if (r.B_k == 128 && r.G == 8)
        return run_attn_prefill_tc<128, 8>(r, q, k, v, block_idx, q_begin, q_count, kv_len, out, lse, scratch, bytes, st);
    return run_attn_prefill_tc<128, 16>(r, q, k, v, block_idx, q_begin, q_count, kv_len, out, lse, scratch, bytes, st);
}

msa_status_t msa_sparse_attn_decode_workspace_bytes(const msa_shape_t* shape, int32_t batch,
                                                    size_t* min_bytes) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    if (batch < 0) return MSA_ERR_INVALID_ARG;
    if (min_bytes) *min_bytes = attn_decode_fast(r) ? decode_ws_bytes(r, batch) : kAlign;
    return MSA_OK;
}

msa_status_t msa_sparse_attn_decode(const msa_shape_t* shape, const void* q, const void* k_cache,
                                    const void* v_cache, int64_t cache_tokens,
                                    const int64_t* seq_offsets, const int32_t* seq_lens,
                                    int32_t batch, const int32_t* block_idx, void* out, float* lse,
                                    void* workspace, size_t workspace_bytes, msa_stream_t stream) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    if (batch < 0 || cache_tokens < 0) return MSA_ERR_INVALID_ARG;
    if (r.q_fp8) return MSA_ERR_UNSUPPORTED;  // one bf16 query row per sequence: nothing to gain from fp8
    if (batch == 0) return MSA_OK;
    if (!q || !k_cache || !v_cache || !seq_offsets || !seq_lens || !block_idx || !out ||
        !aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(out))
        return MSA_ERR_INVALID_ARG;
    size_t need = 0;
    msa_sparse_attn_decode_workspace_bytes(shape, batch, &need);
    if (workspace == nullptr || workspace_bytes < need || !aligned16(workspace)) return MSA_ERR_WORKSPACE;
    if (r.kv_fp8) {  // fp8 caches: the streaming tensor-core kernel only
        if (!attn_decode_fast(r) || cache_tokens >= 2147483647LL) return MSA_ERR_UNSUPPORTED;
        cudaStream_t st = (cudaStream_t)stream;
        if (r.B_k == 64 && r.G == 8)
            return run_attn_decode_tc<64, 8, true>(r, q, k_cache, v_cache, cache_tokens, seq_offsets, seq_lens, batch, block_idx, out, lse, workspace, st);
        if (r.B_k == 64)
            return run_attn_decode_tc<64, 16, true>(r, q, k_cache, v_cache, cache_tokens, seq_offsets, seq_lens, batch, block_idx, out, lse, workspace, st);
        if (r.G == 8)
            return run_attn_decode_tc<128, 8, true>(r, q, k_cache, v_cache, cache_tokens, seq_offsets, seq_lens, batch, block_idx, out, lse, workspace, st);
        return run_attn_decode_tc<128, 16, true>(r, q, k_cache, v_cache, cache_tokens, seq_offsets, seq_lens, batch, block_idx, out, lse, workspace, st);
    }
    if (attn_decode_fast(r) && cache_tokens < 2147483647LL) {
        cudaStream_t st = (cudaStream_t)stream;
        if (r.B_k == 64 && r.G == 8)
            return run_attn_decode_tc<64, 8>(r, q, k_cache, v_cache, cache_tokens, seq_offsets, seq_lens, batch, block_idx, out, lse, workspace, st);
        if (r.B_k == 64)
            return run_attn_decode_tc<64, 16>(r, q, k_cache, v_cache, cache_tokens, seq_offsets, seq_lens, batch, block_idx, out, lse, workspace, st);
        if (r.G == 8)
            return run_attn_decode_tc<128, 8>(r, q, k_cache, v_cache, cache_tokens, seq_offsets, seq_lens, batch, block_idx, out, lse, workspace, st);
        return run_attn_decode_tc<128, 16>(r, q, k_cache, v_cache, cache_tokens, seq_offsets, seq_lens, batch, block_idx, out, lse, workspace, st);
    }
    return run_attn_generic(r, q, k_cache, v_cache, block_idx, decode_rows(seq_offsets, seq_lens, 0, r.B_k),
                            batch, out, lse, (cudaStream_t)stream);
}

// ---------------------------------------------------------------------- whole path
static int64_t score_ld(int64_t T, int B_k) { return (ceil_div64(T, B_k) + 7) / 8 * 8; }  // whole runs of eight blocks

static int64_t pick_score_chunk(const Resolved& r, int64_t T, size_t bytes_for_scores) {
    const size_t row_bytes = sizeof(float) * (size_t)r.H_kv * (size_t)score_ld(T, r.B_k);
    int64_t rows = (int64_t)(bytes_for_scores / row_bytes);
    if (rows > T) rows = T;
    if (rows >= 128) rows = rows / 128 * 128;
    return rows;
}

msa_status_t msa_prefill_forward_workspace_bytes(const msa_shape_t* shape, int64_t T,
                                                 size_t* min_bytes, size_t* preferred_bytes) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    if (T < 0) return MSA_ERR_INVALID_ARG;
    size_t a_min = 0, a_pref = 0;
    msa_sparse_attn_prefill_workspace_bytes(shape, T, T, &a_min, &a_pref);
    const size_t row_bytes = sizeof(float) * (size_t)r.H_kv * (size_t)score_ld(T, r.B_k);
    const int64_t rows_min = T < 128 ? T : 128;
    const int64_t rows_pref = T < 32768 ? T : 32768;
    const size_t s_min = align_up(row_bytes * (size_t)rows_min);
    const size_t s_pref = align_up(row_bytes * (size_t)rows_pref);
    // stages 1-2 finish before stage 3 starts, so the two regions overlap
    if (min_bytes) *min_bytes = (s_min > a_min ? s_min : a_min) + kAlign;
    if (preferred_bytes) *preferred_bytes = (s_pref > a_pref ? s_pref : a_pref) + kAlign;
    return MSA_OK;
}

static msa_status_t prefill_stages_1_2(const msa_shape_t* shape, const Resolved& r, const void* q_idx,
                                       const void* k_idx, int64_t T, int32_t* block_idx, void* workspace,
                                       size_t workspace_bytes, msa_stream_t stream);

msa_status_t msa_prefill_forward(const msa_shape_t* shape, const void* q, const void* k,
                                 const void* v, const void* q_idx, const void* k_idx, int64_t T,
                                 void* out, float* lse, int32_t* block_idx, void* workspace,
                                 size_t workspace_bytes, msa_stream_t stream) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    if (T < 0) return MSA_ERR_INVALID_ARG;
    if (T == 0) return MSA_OK;
    if (!q || !k || !v || !q_idx || !k_idx || !out || !block_idx) return MSA_ERR_INVALID_ARG;
    size_t need = 0;
    msa_prefill_forward_workspace_bytes(shape, T, &need, nullptr);
    if (workspace == nullptr || workspace_bytes < need || !aligned16(workspace)) return MSA_ERR_WORKSPACE;
    if ((s = prefill_stages_1_2(shape, r, q_idx, k_idx, T, block_idx, workspace, workspace_bytes, stream)) != MSA_OK)
        return s;
    return msa_sparse_attn_prefill(shape, q, k, v, block_idx, 0, T, T, out, lse, workspace,
                                   workspace_bytes, stream);
}

// Stages 1-2 over query chunks sized to the workspace (scores never exist for the whole sequence).
static msa_status_t prefill_stages_1_2(const msa_shape_t* shape, const Resolved& r, const void* q_idx,
                                       const void* k_idx, int64_t T, int32_t* block_idx, void* workspace,
                                       size_t workspace_bytes, msa_stream_t stream) {
    msa_status_t s = MSA_OK;
    if (index_topk_fused_ok(r, T, T)) {  // no score matrix, no chunks
        if (wait_rows(g_in_idx_hook, T - 1, (cudaStream_t)stream) != MSA_OK) return MSA_ERR_CUDA;
        return run_index_topk_fused(r, q_idx, k_idx, 0, T, T, block_idx, (cudaStream_t)stream);
    }
    const int64_t ld = score_ld(T, r.B_k);
    const int64_t chunk = pick_score_chunk(r, T, workspace_bytes);
    if (chunk <= 0) return MSA_ERR_WORKSPACE;
    float* scores = static_cast<float*>(workspace);
    const bool runs = r.B_k == 64 || r.B_k == 128;  // the workspace's score rows are in run order where one exists
    for (int64_t q0 = 0; q0 < T; q0 += chunk) {
        const int64_t qc = (T - q0) < chunk ? (T - q0) : chunk;
        const char* qi = static_cast<const char*>(q_idx) + (size_t)q0 * r.H_kv * r.d_idx * r.idx_elt();
        // Only keys up to the chunk's last query are visible, so score that prefix.
        const int64_t kv_vis = q0 + qc;
        if (wait_rows(g_in_idx_hook, q0 + qc - 1, (cudaStream_t)stream) != MSA_OK) return MSA_ERR_CUDA;
        s = run_index_scores(r, qi, k_idx, prefill_rows(q0, kv_vis, r.B_k), qc, scores, ld, (cudaStream_t)stream, runs);
        if (s != MSA_OK) return s;
        s = run_topk(r, scores, ld, prefill_rows(q0, kv_vis, r.B_k), qc, block_idx + (size_t)q0 * r.H_kv * r.k,
                     (cudaStream_t)stream, runs);
        if (s != MSA_OK) return s;
    }
    return MSA_OK;
}

static msa_status_t check_cu_seqlens(const int64_t* cu, int32_t n_seqs) {
    if (n_seqs < 0 || cu == nullptr || cu[0] < 0) return MSA_ERR_INVALID_ARG;
    for (int32_t i = 0; i < n_seqs; ++i)
        if (cu[i + 1] < cu[i]) return MSA_ERR_INVALID_ARG;
    return MSA_OK;
}

// ---------------------------------------------------------------------- packed batches
// A batch of sequences packed token-major runs as ONE problem per stage where the kernels allow:
// the fused index + Top-k kernel takes the query tiles of all sequences from one list (longest key
// prefix first), and the KV-outer attention numbers its blocks through the batch, so that one
// reverse index, one item list, one attention launch and one merge serve every sequence of a query
// range.  What the kernels need for that sits in front of the workspace: the row offsets, the block
// offsets, the tile list, and per row / per block the three arrays of RangeParams.
struct VarlenPlan {
    bool packed;            // the tensor-core attention runs once over the whole batch
    bool fused;             // Eq. 6 + Eq. 7 in one launch over the whole batch (top_k <= 16)
    int64_t rows, n_blocks, n_idx_tiles;
    size_t off_cu, off_blk_cum, off_tiles, off_row_pos, off_row_blk0, off_blk_row0, meta;  // bytes
    size_t copies;          // bf16 copies of fp8 K and V (bf16 Q), in all
    size_t stage_min, stage_pref;
};

static msa_status_t varlen_plan(const msa_shape_t* shape, const Resolved& r, const int64_t* cu, int32_t n_seqs,
                                VarlenPlan& vp) {
    vp = VarlenPlan();
    vp.rows = cu[n_seqs] - cu[0];
    for (int32_t i = 0; i < n_seqs; ++i) {
        const int64_t T = cu[i + 1] - cu[i];
        vp.n_blocks += ceil_div64(T, r.B_k);
        vp.n_idx_tiles += ceil_div64(T, kIdxTileQ);
    }
    vp.packed = n_seqs > 1 && attn_tc_supported(r) && vp.rows < 2147483647LL && vp.n_blocks < (1 << 24);
    vp.fused = vp.packed && index_topk_fused_ok(r, vp.rows, vp.rows);
    // stages 1-2 (and, unpacked, stage 3) sequence by sequence: what the largest sequence needs
    size_t seq_min = kAlign, seq_pref = kAlign;
    for (int32_t i = 0; i < n_seqs; ++i) {
        size_t a = 0, b = 0;
        const msa_status_t st = msa_prefill_forward_workspace_bytes(shape, cu[i + 1] - cu[i], &a, &b);
        if (st != MSA_OK) return st;
        if (a > seq_min) seq_min = a;
        if (b > seq_pref) seq_pref = b;
    }
    if (!vp.packed) {
        vp.stage_min = seq_min; vp.stage_pref = seq_pref;
        return MSA_OK;
    }
    size_t o = 0;
    vp.off_cu = o; o += align_up((size_t)(n_seqs + 1) * 8);
    vp.off_blk_cum = o; o += align_up((size_t)(n_seqs + 1) * 4);
    vp.off_tiles = o; o += align_up((size_t)vp.n_idx_tiles * sizeof(IdxPackedTile));
    vp.off_row_pos = o; o += align_up((size_t)vp.rows * 4);
    vp.off_row_blk0 = o; o += align_up((size_t)vp.rows * 4);
    vp.off_blk_row0 = o; o += align_up((size_t)vp.n_blocks * 4);
    vp.meta = o;
    vp.copies = (r.kv_fp8 && !r.q_fp8) ? 2 * kv_copy_bytes(r, vp.rows) : 0;
    const int64_t r_min = vp.rows < 256 ? vp.rows : 256;
    int64_t r_pref = (int64_t)((32ull << 30) / attn_per_query_bytes(r));
    if (r_pref > vp.rows) r_pref = vp.rows;
    if (r_pref < r_min) r_pref = r_min;
    size_t a_min = attn_plan_blocks(r, vp.n_blocks, r_min).total + 8 * kAlign;
    size_t a_pref = attn_plan_blocks(r, vp.n_blocks, r_pref).total + 8 * kAlign;
    if (!vp.fused) {  // score chunks of the longest sequence share the region with the attention's buffers
        if (seq_min > a_min) a_min = seq_min;
        if (seq_pref > a_pref) a_pref = seq_pref;
    }
    vp.stage_min = a_min; vp.stage_pref = a_pref;
    return MSA_OK;
}

msa_status_t msa_prefill_forward_varlen_workspace_bytes(const msa_shape_t* shape,
                                                        const int64_t* cu_seqlens, int32_t n_seqs,
                                                        size_t* min_bytes, size_t* preferred_bytes) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    if ((s = check_cu_seqlens(cu_seqlens, n_seqs)) != MSA_OK) return s;
    VarlenPlan vp;
    if ((s = varlen_plan(shape, r, cu_seqlens, n_seqs, vp)) != MSA_OK) return s;
    if (min_bytes) *min_bytes = vp.meta + vp.copies + vp.stage_min;
    if (preferred_bytes) *preferred_bytes = vp.meta + vp.copies + vp.stage_pref;
    return MSA_OK;
}

msa_status_t msa_prefill_forward_varlen(const msa_shape_t* shape, const void* q, const void* k,
                                        const void* v, const void* q_idx, const void* k_idx,
                                        const int64_t* cu_seqlens, int32_t n_seqs, void* out,
                                        float* lse, int32_t* block_idx, void* workspace,
                                        size_t workspace_bytes, msa_stream_t stream) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    if ((s = check_cu_seqlens(cu_seqlens, n_seqs)) != MSA_OK) return s;
    if (n_seqs == 0 || cu_seqlens[n_seqs] == cu_seqlens[0]) return MSA_OK;
    if (!q || !k || !v || !q_idx || !k_idx || !out || !block_idx) return MSA_ERR_INVALID_ARG;
    VarlenPlan vp;
    if ((s = varlen_plan(shape, r, cu_seqlens, n_seqs, vp)) != MSA_OK) return s;
    if (workspace == nullptr || workspace_bytes < vp.meta + vp.copies + vp.stage_min || !aligned16(workspace))
        return MSA_ERR_WORKSPACE;
    const size_t q_row = (size_t)r.H_q * r.d * r.q_elt(), o_row = (size_t)r.H_q * r.d * 2;
    const size_t kv_row = (size_t)r.H_kv * r.d * r.kv_elt();
    const size_t qi_row = (size_t)r.H_kv * r.d_idx * r.idx_elt(), ki_row = (size_t)r.d_idx * r.idx_elt();
    cudaStream_t st = (cudaStream_t)stream;
    const int64_t row0 = cu_seqlens[0];
    if (!vp.packed) {  // every sequence through the single-sequence path, one after the other
        for (int32_t i = 0; i < n_seqs; ++i) {
            const int64_t o = cu_seqlens[i], T = cu_seqlens[i + 1] - o;
            if (T == 0) continue;
            s = msa_prefill_forward(shape, (const char*)q + o * q_row, (const char*)k + o * kv_row,
                                    (const char*)v + o * kv_row, (const char*)q_idx + o * qi_row,
                                    (const char*)k_idx + o * ki_row, T, (char*)out + o * o_row,
                                    lse ? lse + o * r.H_q : nullptr, block_idx + o * (int64_t)r.H_kv * r.k, workspace,
                                    workspace_bytes, stream);
            if (s != MSA_OK) return s;
        }
        return MSA_OK;
    }
    // ---- the batch's maps: offsets and the tile list from the host, the per-row arrays by a kernel
    char* w = static_cast<char*>(workspace);
    int64_t* cu_dev = (int64_t*)(w + vp.off_cu);
    int32_t* blk_cum_dev = (int32_t*)(w + vp.off_blk_cum);
    IdxPackedTile* tiles_dev = (IdxPackedTile*)(w + vp.off_tiles);
    int32_t* row_pos = (int32_t*)(w + vp.off_row_pos);
    int32_t* row_blk0 = (int32_t*)(w + vp.off_row_blk0);
    int32_t* blk_row0 = (int32_t*)(w + vp.off_blk_row0);
    char* stage = w + vp.meta + vp.copies;
    const size_t stage_bytes = workspace_bytes - vp.meta - vp.copies;
    // top_k > 16 on the tensor-core shapes: stages 1-2 run on groups of consecutive sequences, as many
    // as the score matrix of the stage region holds rows for; one scoring launch and one Top-k launch
    // per group.  A sequence too long for the region alone takes the single-sequence path (in chunks).
    struct SeqGroup { int32_t seq_a, seq_b; int64_t row_a, row_b, tile_off, n_tiles; };
    const bool grouped = !vp.fused && index_tc_ok(r) && vp.rows >= 32;
    SeqGroup* groups = nullptr;
    int32_t n_groups = 0;
    int64_t group_ld = 0;
    {
        // (pageable host memory: the runtime has copied it out when the call returns)
        int32_t* blk_cum = (int32_t*)malloc((size_t)(n_seqs + 1) * 4);
        IdxPackedTile* tiles = (IdxPackedTile*)malloc((size_t)(vp.n_idx_tiles > 0 ? vp.n_idx_tiles : 1) * sizeof(IdxPackedTile));
        if (!blk_cum || !tiles) { free(blk_cum); free(tiles); return MSA_ERR_CUDA; }
        blk_cum[0] = 0;
        int64_t max_qt = 0;
        for (int32_t i = 0; i < n_seqs; ++i) {
            const int64_t T = cu_seqlens[i + 1] - cu_seqlens[i];
            blk_cum[i + 1] = blk_cum[i] + (int32_t)ceil_div64(T, r.B_k);
            if (ceil_div64(T, kIdxTileQ) > max_qt) max_qt = ceil_div64(T, kIdxTileQ);
        }
        // longest key prefix first: by tile number inside the sequence, descending
        int64_t n = 0;
        auto list_tiles = [&](int32_t seq_a, int32_t seq_b) {
            int64_t top_qt = 0;
            for (int32_t i = seq_a; i < seq_b; ++i)
                if (ceil_div64(cu_seqlens[i + 1] - cu_seqlens[i], kIdxTileQ) > top_qt)
                    top_qt = ceil_div64(cu_seqlens[i + 1] - cu_seqlens[i], kIdxTileQ);
            for (int64_t qt = top_qt - 1; qt >= 0; --qt)
                for (int32_t i = seq_a; i < seq_b; ++i) {
                    const int64_t T = cu_seqlens[i + 1] - cu_seqlens[i];
                    if (qt < ceil_div64(T, kIdxTileQ)) {
                        tiles[n].row0 = (int32_t)(cu_seqlens[i] - row0); tiles[n].len = (int32_t)T; tiles[n].qt = (int32_t)qt;
                        ++n;
                    }
                }
        };
        if (!grouped) {
            list_tiles(0, n_seqs);
        } else {
            groups = (SeqGroup*)malloc((size_t)n_seqs * sizeof(SeqGroup));
            if (!groups) { free(blk_cum); free(tiles); return MSA_ERR_CUDA; }
            group_ld = score_ld(max_qt * kIdxTileQ, r.B_k);
            const int64_t rows_cap = (int64_t)(stage_bytes / (sizeof(float) * (size_t)r.H_kv * (size_t)group_ld));
            int32_t a = 0;
            while (a < n_seqs) {
                int32_t b = a;
                int64_t rows_in = 0;
                while (b < n_seqs && rows_in + (cu_seqlens[b + 1] - cu_seqlens[b]) <= rows_cap) {
                    rows_in += cu_seqlens[b + 1] - cu_seqlens[b];
                    ++b;
                }
                SeqGroup g;
                g.seq_a = a; g.row_a = cu_seqlens[a] - row0; g.tile_off = n;
                if (b == a) {  // this sequence alone does not fit: n_tiles = -1 marks the single-sequence path
                    b = a + 1;
                    g.n_tiles = -1;
                } else {
                    list_tiles(a, b);
                    g.n_tiles = n - g.tile_off;
                }
                g.seq_b = b; g.row_b = cu_seqlens[b] - row0;
                groups[n_groups++] = g;
                a = b;
            }
        }
        bool ok = cudaMemcpyAsync(cu_dev, cu_seqlens, (size_t)(n_seqs + 1) * 8, cudaMemcpyHostToDevice, st) == cudaSuccess &&
                  cudaMemcpyAsync(blk_cum_dev, blk_cum, (size_t)(n_seqs + 1) * 4, cudaMemcpyHostToDevice, st) == cudaSuccess &&
                  (n == 0 || cudaMemcpyAsync(tiles_dev, tiles, (size_t)n * sizeof(IdxPackedTile), cudaMemcpyHostToDevice, st) == cudaSuccess);
        free(blk_cum);
        free(tiles);
        if (!ok) { free(groups); return MSA_ERR_CUDA; }
    }
    {
        const int64_t work = vp.rows + vp.n_blocks;
        const unsigned grid = (unsigned)(ceil_div64(work, 256) < 148 * 8 ? ceil_div64(work, 256) : 148 * 8);
        StageScope sc(kStageSchedule, st);
        packed_map_kernel<<<grid, 256, 0, st>>>(cu_dev, blk_cum_dev, n_seqs, r.B_k, row_pos, row_blk0, blk_row0);
    }
    if (cudaPeekAtLastError() != cudaSuccess) { free(groups); return MSA_ERR_CUDA; }
    // tensors of the batch start at its first row
    const char* qb = (const char*)q + row0 * q_row;
    const char* kb = (const char*)k + row0 * kv_row;
    const char* vb = (const char*)v + row0 * kv_row;
    const char* qib = (const char*)q_idx + row0 * qi_row;
    const char* kib = (const char*)k_idx + row0 * ki_row;
    int32_t* bi = block_idx + row0 * (int64_t)r.H_kv * r.k;
    // ---- stages 1-2
    if (vp.fused) {
        s = run_index_topk_fused(r, qib, kib, 0, vp.rows, vp.rows, bi, st, tiles_dev, vp.n_idx_tiles);
        if (s != MSA_OK) return s;
    } else if (grouped) {
        float* scores = reinterpret_cast<float*>(stage);
        for (int32_t gi = 0; gi < n_groups && s == MSA_OK; ++gi) {
            const SeqGroup& g = groups[gi];
            if (g.row_b == g.row_a) continue;
            if (g.n_tiles < 0) {
                const int64_t o = cu_seqlens[g.seq_a];
                s = prefill_stages_1_2(shape, r, (const char*)q_idx + o * qi_row, (const char*)k_idx + o * ki_row,
                                       cu_seqlens[g.seq_a + 1] - o, block_idx + o * (int64_t)r.H_kv * r.k, stage,
                                       stage_bytes, stream);
                continue;
            }
            s = run_index_scores_packed(r, qib, kib, vp.rows, scores, group_ld, st, tiles_dev + g.tile_off, g.n_tiles,
                                        g.row_a);
            if (s != MSA_OK) break;
            RowMap rows = prefill_rows(g.row_a, 0, r.B_k);
            rows.row_pos = row_pos;
            s = run_topk(r, scores, group_ld, rows, g.row_b - g.row_a, bi + g.row_a * (int64_t)r.H_kv * r.k, st, true);
        }
        free(groups);
        if (s != MSA_OK) return s;
    } else {
        for (int32_t i = 0; i < n_seqs; ++i) {
            const int64_t o = cu_seqlens[i], T = cu_seqlens[i + 1] - o;
            if (T == 0) continue;
            s = prefill_stages_1_2(shape, r, (const char*)q_idx + o * qi_row, (const char*)k_idx + o * ki_row, T,
                                   block_idx + o * (int64_t)r.H_kv * r.k, stage, stage_bytes, stream);
            if (s != MSA_OK) return s;
        }
    }
    // ---- stage 3, once over the batch
    PackedBatch pk;
    pk.row_pos = row_pos; pk.row_blk0 = row_blk0; pk.blk_row0 = blk_row0; pk.n_blocks = vp.n_blocks;
    const bool f8 = r.q_fp8 && r.kv_fp8;
    if (vp.copies) {  // fp8 K/V caches with bf16 Q: bf16 copies of all rows first
        char* kw = w + vp.meta;
        char* vw = kw + vp.copies / 2;
        if ((s = widen_kv(r, kb, vb, vp.rows, kw, vw, st)) != MSA_OK) return s;
        kb = kw; vb = vw;
    }
    return attn_prefill_tc_dispatch(r, f8, qb, kb, vb, bi, 0, vp.rows, vp.rows, (char*)out + row0 * o_row,
                                    lse ? lse + row0 * r.H_q : nullptr, stage, stage_bytes, st, pk);
}

static size_t host_staging_bytes(const Resolved& r, int64_t T, size_t off[8]) {
    size_t o = 0;
    off[0] = o; o += align_up((size_t)T * r.H_q * r.d * r.q_elt());  // q
    off[1] = o; o += align_up((size_t)T * r.H_kv * r.d * r.kv_elt());  // k
    off[2] = o; o += align_up((size_t)T * r.H_kv * r.d * r.kv_elt());  // v
    off[3] = o; o += align_up((size_t)T * r.H_kv * r.d_idx * r.idx_elt()); // q_idx
    off[4] = o; o += align_up((size_t)T * r.d_idx * r.idx_elt());          // k_idx
    off[5] = o; o += align_up((size_t)T * r.H_q * r.d * 2);      // out
    off[6] = o; o += align_up((size_t)T * r.H_q * 4);            // lse
    off[7] = o; o += align_up((size_t)T * r.H_kv * r.k * 4);     // block_idx
    return o;
}

msa_status_t msa_prefill_forward_host_workspace_bytes(const msa_shape_t* shape, int64_t T,
                                                      size_t* min_bytes, size_t* preferred_bytes) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    size_t mn = 0, pf = 0, off[8];
    if ((s = msa_prefill_forward_workspace_bytes(shape, T, &mn, &pf)) != MSA_OK) return s;
    const size_t stage = host_staging_bytes(r, T, off);
    if (min_bytes) *min_bytes = stage + mn;
    if (preferred_bytes) *preferred_bytes = stage + pf;
    return MSA_OK;
}

static msa_status_t prefill_forward_host_body(const msa_shape_t* shape, const void* q_host,
                                              const void* k_host, const void* v_host,
                                              const void* q_idx_host, const void* k_idx_host, int64_t T,
                                              void* out_host, float* lse_host, int32_t* block_idx_host,
                                              void* workspace, size_t workspace_bytes, msa_stream_t stream,
                                              cudaStream_t* copy_used);

msa_status_t msa_prefill_forward_host(const msa_shape_t* shape, const void* q_host,
                                      const void* k_host, const void* v_host,
                                      const void* q_idx_host, const void* k_idx_host, int64_t T,
                                      void* out_host, float* lse_host, int32_t* block_idx_host,
                                      void* workspace, size_t workspace_bytes, msa_stream_t stream) {
    cudaStream_t copy = nullptr;
    const msa_status_t s = prefill_forward_host_body(shape, q_host, k_host, v_host, q_idx_host, k_idx_host, T, out_host,
                                                     lse_host, block_idx_host, workspace, workspace_bytes, stream, &copy);
    g_in_idx_hook.on = false; g_in_hook.on = false; g_out_hook.on = false;
    if (s != MSA_OK && copy != nullptr) {
        // Copies from and to the caller's host buffers may be in flight: the buffers are the
        // caller's again only once both streams have drained.
        cudaStreamSynchronize((cudaStream_t)stream);
        cudaStreamSynchronize(copy);
    }
    return s;
}

static msa_status_t prefill_forward_host_body(const msa_shape_t* shape, const void* q_host,
                                              const void* k_host, const void* v_host,
                                              const void* q_idx_host, const void* k_idx_host, int64_t T,
                                              void* out_host, float* lse_host, int32_t* block_idx_host,
                                              void* workspace, size_t workspace_bytes, msa_stream_t stream,
                                              cudaStream_t* copy_used) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    if (T < 0) return MSA_ERR_INVALID_ARG;
    if (T == 0) return MSA_OK;
    if (!q_host || !k_host || !v_host || !q_idx_host || !k_idx_host || !out_host)
        return MSA_ERR_INVALID_ARG;
    size_t need = 0, off[8];
    if ((s = msa_prefill_forward_host_workspace_bytes(shape, T, &need, nullptr)) != MSA_OK) return s;
    if (workspace == nullptr || workspace_bytes < need || !aligned16(workspace)) return MSA_ERR_WORKSPACE;
    const size_t stage = host_staging_bytes(r, T, off);
    char* w = static_cast<char*>(workspace);
    cudaStream_t st = (cudaStream_t)stream;
    // A second stream carries the copies: the index inputs go first so that stages 1-2 start
    // while Q, K and V are still on their way; each finished query range of O is copied back
    // while the next one is computed.
    static cudaStream_t copy_dev[64] = {};
    cudaStream_t& copy = copy_dev[current_device()];
    if (copy == nullptr && cudaStreamCreateWithFlags(&copy, cudaStreamNonBlocking) != cudaSuccess) return MSA_ERR_CUDA;
    *copy_used = copy;
    cudaEvent_t e_in = next_sync_event(), e_idx = next_sync_event(), e_kv = next_sync_event();
    if (!e_in || !e_idx || !e_kv) return MSA_ERR_CUDA;
    if (cudaEventRecord(e_in, st) != cudaSuccess || cudaStreamWaitEvent(copy, e_in, 0) != cudaSuccess) return MSA_ERR_CUDA;
    const void* src[5] = {q_host, k_host, v_host, q_idx_host, k_idx_host};
    const size_t nbytes[5] = {(size_t)T * r.H_q * r.d * r.q_elt(), (size_t)T * r.H_kv * r.d * r.kv_elt(),
                              (size_t)T * r.H_kv * r.d * r.kv_elt(), (size_t)T * r.H_kv * r.d_idx * r.idx_elt(),
                              (size_t)T * r.d_idx * r.idx_elt()};
    // Order on the copy stream: K_idx, Q_idx, K, V, Q; Q_idx and Q go in pieces with an event after each,
    // so that every scoring chunk and every attention range waits only for its own rows.
    if (cudaMemcpyAsync(w + off[4], src[4], nbytes[4], cudaMemcpyHostToDevice, copy) != cudaSuccess) return MSA_ERR_CUDA;
    if (cudaEventRecord(e_idx, copy) != cudaSuccess) return MSA_ERR_CUDA;
    const size_t qi_rb = (size_t)r.H_kv * r.d_idx * r.idx_elt(), q_rb = (size_t)r.H_q * r.d * r.q_elt();
    if (upload_in_pieces(g_in_idx_hook, w + off[3], src[3], T, qi_rb, 65536, copy) != MSA_OK) return MSA_ERR_CUDA;
    for (int i = 1; i <= 2; ++i)
        if (cudaMemcpyAsync(w + off[i], src[i], nbytes[i], cudaMemcpyHostToDevice, copy) != cudaSuccess) return MSA_ERR_CUDA;
    if (cudaEventRecord(e_kv, copy) != cudaSuccess) return MSA_ERR_CUDA;
    if (upload_in_pieces(g_in_hook, w + off[0], src[0], T, q_rb, 16384, copy) != MSA_OK) return MSA_ERR_CUDA;
    float* lse_dev = lse_host ? (float*)(w + off[6]) : nullptr;
    int32_t* bi_dev = (int32_t*)(w + off[7]);
    if (cudaStreamWaitEvent(st, e_idx, 0) != cudaSuccess) return MSA_ERR_CUDA;
    g_in_idx_hook.on = true;
    s = prefill_stages_1_2(shape, r, w + off[3], w + off[4], T, bi_dev, w + stage, workspace_bytes - stage, stream);
    g_in_idx_hook.on = false;
    if (s != MSA_OK) return s;
    if (cudaStreamWaitEvent(st, e_kv, 0) != cudaSuccess) return MSA_ERR_CUDA;
    // The tensor-core path waits for Q range by range; any other path waits for all of it here.
    g_in_hook.on = attn_tc_supported(r) && T < 2147483647LL;
    if (!g_in_hook.on && cudaStreamWaitEvent(st, g_in_hook.ev[g_in_hook.n_pieces - 1], 0) != cudaSuccess)
        return MSA_ERR_CUDA;
    g_out_hook.on = true; g_out_hook.copy = copy; g_out_hook.out_host = (char*)out_host;
    g_out_hook.lse_host = lse_host; g_out_hook.rows_copied = 0;
    s = msa_sparse_attn_prefill(shape, w + off[0], w + off[1], w + off[2], bi_dev, 0, T, T, w + off[5], lse_dev,
                                w + stage, workspace_bytes - stage, stream);
    g_out_hook.on = false;
    g_in_hook.on = false;
    if (s != MSA_OK) return s;
    if (g_out_hook.rows_copied < T) {  // rows the per-range hook did not cover (generic kernel path)
        const msa_status_t hs = hook_copy_rows(r, w + off[5], lse_dev, g_out_hook.rows_copied,
                                               T - g_out_hook.rows_copied, st);
        if (hs != MSA_OK) return hs;
    }
    if (block_idx_host &&
        cudaMemcpyAsync(block_idx_host, bi_dev, (size_t)T * r.H_kv * r.k * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return MSA_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess || cudaStreamSynchronize(copy) != cudaSuccess) return MSA_ERR_CUDA;
    return MSA_OK;
}

msa_status_t msa_decode_forward(const msa_shape_t* shape, const void* q, const void* q_idx,
                                const void* k_cache, const void* v_cache, const void* k_idx_cache,
                                int64_t cache_tokens, const int64_t* seq_offsets,
                                const int32_t* seq_lens, int32_t batch, int64_t max_seq_len,
                                float* scores, int64_t ld_scores, int32_t* block_idx, void* out,
                                float* lse, void* workspace, size_t workspace_bytes,
                                msa_stream_t stream) {
    msa_status_t s = msa_index_scores_decode(shape, q_idx, k_idx_cache, seq_offsets, seq_lens, batch,
                                             max_seq_len, scores, ld_scores, stream);
    if (s != MSA_OK) return s;
    s = msa_topk_select_decode(shape, scores, ld_scores, seq_lens, batch, max_seq_len, block_idx, stream);
    if (s != MSA_OK) return s;
    return msa_sparse_attn_decode(shape, q, k_cache, v_cache, cache_tokens, seq_offsets, seq_lens,
                                  batch, block_idx, out, lse, workspace, workspace_bytes, stream);
}

msa_status_t msa_decode_forward_host(const msa_shape_t* shape, const void* q_host,
                                     const void* q_idx_host, void* q_dev, void* q_idx_dev,
                                     const void* k_cache, const void* v_cache,
                                     const void* k_idx_cache, int64_t cache_tokens,
                                     const int64_t* seq_offsets, const int32_t* seq_lens,
                                     int32_t batch, int64_t max_seq_len, float* scores,
                                     int64_t ld_scores, int32_t* block_idx, void* out_dev,
                                     void* out_host, void* workspace, size_t workspace_bytes,
                                     msa_stream_t stream) {
    Resolved r;
    msa_status_t s = resolve(shape, r);
    if (s != MSA_OK) return s;
    if (batch < 0) return MSA_ERR_INVALID_ARG;
    if (batch == 0) return MSA_OK;
    if (!q_host || !q_idx_host || !q_dev || !q_idx_dev || !out_dev || !out_host) return MSA_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t qb = (size_t)batch * r.H_q * r.d * 2, qib = (size_t)batch * r.H_kv * r.d_idx * r.idx_elt();
    if (cudaMemcpyAsync(q_dev, q_host, qb, cudaMemcpyHostToDevice, st) != cudaSuccess) return MSA_ERR_CUDA;
    if (cudaMemcpyAsync(q_idx_dev, q_idx_host, qib, cudaMemcpyHostToDevice, st) != cudaSuccess) return MSA_ERR_CUDA;
    s = msa_decode_forward(shape, q_dev, q_idx_dev, k_cache, v_cache, k_idx_cache, cache_tokens,
                           seq_offsets, seq_lens, batch, max_seq_len, scores, ld_scores, block_idx,
                           out_dev, nullptr, workspace, workspace_bytes, stream);
    if (s != MSA_OK) return s;
    if (cudaMemcpyAsync(out_host, out_dev, qb, cudaMemcpyDeviceToHost, st) != cudaSuccess) return MSA_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? MSA_OK : MSA_ERR_CUDA;
}

}  // extern "C"
