/*
 * msa.h - C ABI of the B200 (sm_100a) forward hot path of MiniMax Sparse Attention.
 *
 * The path is Algorithm 1, lines 3-5 of the paper:
 *   line 3  BlockMaxPool : index scoring + causal block max        (Eq. 6)  msa_index_scores
 *   line 4  TopK         : exp-free Top-k, local block forced in   (Eq. 7)  msa_topk_select
 *   line 5  TopKAttn     : block-sparse GQA softmax attention      (Eq. 8)  msa_sparse_attn_prefill
 *                                                                           msa_sparse_attn_decode
 *
 * Conventions common to every call
 *   - Every pointer is a DEVICE pointer unless its name ends in "_host".  The caller owns
 *     every buffer, including workspaces; the library allocates no device memory, never
 *     frees, and never synchronises the stream unless a call says so.
 *   - bf16 tensors are passed as `const void*`; all tensors are dense, token-major, last
 *     dimension contiguous:  Q [T,H_q,d_h], K,V [T,H_kv,d_h], Q_idx [T,H_kv,d_idx],
 *     K_idx [T,d_idx] (one index key head shared by all groups, Eq. 5).  Bases must be
 *     16-byte aligned.
 *   - Indices are 0-based: token j is in block j / B_k (Eq. 4); query head h is in GQA
 *     group r = h / G, G = H_q / H_kv (Section 2.1); B = ceil(kv_len / B_k).
 *   - A "query range" is rows [q_begin, q_begin + q_count) of one sequence of kv_len
 *     tokens; q_begin + q_count <= kv_len; row pointers point at row q_begin.
 *   - Calls return MSA_OK after enqueuing their work on `stream`.  Argument, shape,
 *     alignment and workspace errors are returned before anything is launched.  CUDA
 *     launch errors map to MSA_ERR_CUDA.  Device-side anomalies (a bounded wait that ran
 *     out, a block index out of range) never trap: they set a status word that
 *     msa_check_async_status() reads.
 *   - Fast kernels are specialised for d_h = 128, d_idx in {64,128}, B_k in {64,128},
 *     G in {8,16} (decode index scoring: H_kv <= 8); other shapes (d_h, d_idx multiples
 *     of 8, d_h <= 256, d_idx <= 128) run on generic kernels.  k is limited to 1..128.
 *   - State the library keeps: per device, a ring of CUDA events, the copy stream of the
 *     *_host calls, cached kernel
 *     attributes, and ONE async status word (a device global, not part of any workspace:
 *     two callers sharing a device cannot tell whose kernel set it; whoever reads it clears
 *     it); per process, the profiling hooks (their events belong to the device that was
 *     current at the first msa_profile_begin).  Calls from several host threads must be
 *     serialised by the caller; calls on different streams from one thread are fine, but
 *     two calls that are in flight at the same time must not share a workspace.
 *   - Beyond the four stage calls there are: whole-path calls (msa_prefill_forward,
 *     msa_prefill_forward_varlen, msa_decode_forward and their *_host forms), the fused
 *     Eq. 6 + Eq. 7 call msa_index_topk_fused (top_k <= 16), and the index branch's
 *     log-sum-exp msa_index_lse_prefill (Section 4.3).
 */
#ifndef MSA_H_
#define MSA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MSA_OK = 0,
    MSA_ERR_INVALID_ARG = 1, /* null pointer, negative size, misaligned base, bad range   */
    MSA_ERR_UNSUPPORTED = 2, /* shape outside what the kernels implement                   */
    MSA_ERR_WORKSPACE = 3,   /* workspace smaller than the *_workspace_bytes() minimum     */
    MSA_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed                        */
    MSA_ERR_TIMEOUT = 5,     /* a device-side bounded wait ran out (see async status)      */
    MSA_ERR_BAD_INDEX = 6    /* a block index outside [-1, B) was met on the device        */
} msa_status_t;

/* Shape of one MSA layer, in the paper's notation (Sections 2 and 3.1). */
typedef struct {
    int32_t n_q_heads;   /* H_q                                                   */
    int32_t n_kv_heads;  /* H_kv (= number of GQA groups = index query heads)     */
    int32_t head_dim;    /* d_h                                                   */
    int32_t idx_dim;     /* d_idx                                                 */
    int32_t block_size;  /* B_k                                                   */
    int32_t top_k;       /* k, blocks per (query, group) including the local one  */
    float softmax_scale; /* 0 => 1/sqrt(d_h)   (Eq. 1, Eq. 8)                     */
    float index_scale;   /* 0 => 1/sqrt(d_idx) (Eq. 6)                            */
    int32_t idx_fp8;     /* 0: q_idx / k_idx are bf16.  1: they are fp8 E4M3      */
                         /* (Section 4.2), one byte per element, d_idx % 16 == 0; */
                         /* every "bf16" below then reads "fp8" for those two     */
                         /* operands.  Codes 0x7F / 0xFF (NaN) must not occur.    */
                         /* Any other value: MSA_ERR_INVALID_ARG.                 */
    int32_t kv_fp8;      /* 0: K and V are bf16.  1: k / v (prefill) and k_cache / */
                         /* v_cache (decode) are fp8 E4M3 (Section 4.2), one byte  */
                         /* per element, dequantised exactly; Q stays bf16.        */
                         /* Decode: needs d_h = 128, G in {8,16}, B_k in {64,128}, */
                         /* and Q in the normal range of fp16 (it is multiplied as */
                         /* fp16).  Prefill (msa_sparse_attn_prefill,              */
                         /* msa_prefill_forward, msa_prefill_forward_varlen):      */
                         /* d_h % 16 == 0; the call widens the kv_len visible rows */
                         /* to bf16 in its workspace first (the *_workspace_bytes  */
                         /* results include 4 * kv_len * H_kv * d_h bytes for it)  */
                         /* and then computes as with bf16 K and V holding the     */
                         /* same values (msa_prefill_forward_host uploads the fp8  */
                         /* bytes and does the same).  The allocation-free prefill */
                         /* call returns MSA_ERR_UNSUPPORTED with the flag.  Other */
                         /* values: INVALID_ARG.                                   */
    int32_t q_fp8;       /* 0: Q is bf16.  1 (prefill only, needs kv_fp8 = 1, d_h = */
                         /* 128, G in {8,16}, B_k in {64,128}): q holds fp8 E4M3 as */
                         /* well (Section 4.2).  The attention kernel then reads    */
                         /* the fp8 tensors itself: S = Q K^T on fp8 tensor-core    */
                         /* MMAs (exact products, fp32 sums), V widened exactly to  */
                         /* bf16 once per K/V tile, P and O = P V as with bf16      */
                         /* operands; no bf16 copies, so no extra workspace.  out   */
                         /* stays bf16.  Other shapes, decode calls and the         */
                         /* allocation-free call: MSA_ERR_UNSUPPORTED.  Other       */
                         /* values: INVALID_ARG.                                    */
    int32_t score_runs;  /* Order of the blocks inside a score row, for the two     */
                         /* calls that exchange one (msa_index_scores writes it,    */
                         /* msa_topk_select reads it).  0: block order, column b =  */
                         /* block b.  1 (B_k in {64,128}, ld_scores % 8 == 0): run  */
                         /* order, the order in which the tensor-core kernel has    */
                         /* the maxima at hand - a thread's four blocks of a run of */
                         /* eight leave as one 16-byte store.  The eight blocks of  */
                         /* run j stay in columns [8j, 8j+8); with n = 128 / B_k,   */
                         /* block 8j + w sits in column 8j + 4*((w/n) mod 2) +      */
                         /* n*(w / (2n)) + (w mod n): the columns of a run hold its */
                         /* blocks 0 2 4 6 1 3 5 7 for B_k = 128 and 0 1 4 5 2 3 6  */
                         /* 7 for B_k = 64.  Columns of                             */
                         /* blocks after a query's local block are unspecified      */
                         /* (not read by msa_topk_select).  The whole-path calls    */
                         /* use run order in their workspace whatever this field    */
                         /* says; decode calls take 0 only (else UNSUPPORTED).      */
                         /* Other values: INVALID_ARG.  The paper has no            */
                         /* counterpart: Eq. 6 fixes the values, not their place.   */
} msa_shape_t;

typedef void* msa_stream_t; /* a cudaStream_t */

const char* msa_status_string(msa_status_t s);

/*
 * Reads and clears the device-side status word (synchronises the device).  Returns
 * MSA_OK, MSA_ERR_TIMEOUT or MSA_ERR_BAD_INDEX; *detail (optional, host) receives a code
 * naming the kernel and the wait or index that failed.
 */
msa_status_t msa_check_async_status(int32_t* detail_host);

/* ------------------------------------------------------------------------------------
 * Stage 1 - Eq. 6 (Algorithm 1, line 3; Section 6 appendix remark that inference needs
 * only the block-wise maximum of Q_idx K_idx^T).
 *   scores[q, r, b] = index_scale * max_{j in block b, j <= q_begin+q} <Q_idx[q,r,:], K_idx[j,:]>
 *   scores[q, r, b] = -inf for blocks with no visible token (b > (q_begin+q)/B_k).
 * q_idx  [q_count,H_kv,d_idx] bf16 (rows of the range), k_idx [kv_len,d_idx] bf16,
 * scores [q_count,H_kv,ld_scores] fp32, ld_scores >= B and a multiple of 4; columns
 * b in [0,B) of every row are written, columns [B, ld_scores) are left untouched.
 * With shape->score_runs = 1 the columns of a row are in run order (see msa_shape_t):
 * ld_scores >= B rounded up to 8 and a multiple of 8; the columns of blocks up to the
 * query's local block hold the Eq. 6 values, the others are unspecified.
 */
msa_status_t msa_index_scores(const msa_shape_t* shape, const void* q_idx, const void* k_idx,
                              int64_t q_begin, int64_t q_count, int64_t kv_len,
                              float* scores, int64_t ld_scores, msa_stream_t stream);

/*
 * Stage 1 for batched decode: sequence s has its K_idx rows at
 * k_idx_cache[seq_offsets[s] .. seq_offsets[s]+seq_lens[s]) and one query (its last
 * token, position seq_lens[s]-1, already appended to the cache).
 * q_idx [batch,H_kv,d_idx]; seq_offsets int64 [batch] (in tokens); seq_lens int32 [batch];
 * scores [batch,H_kv,ld_scores]: columns [0, ceil(seq_lens[s]/B_k)) are written with the
 * Eq. 6 values, columns up to ceil(max_seq_len/B_k) with -inf.
 */
/*
 * Which kernel msa_index_scores runs for a range of q_count rows of a kv_len-token sequence on
 * the current device (the paper has no counterpart: a query for tests and tuning).  *tensor_core
 * is 1 for the tcgen05 kernel (d_idx in {64,128}, B_k in {64,128}, at least 32 rows), 0 for the
 * generic kernel; *heads_per_cta is the number of index heads that share one key tile in a CTA of
 * the tensor-core kernel (8, 4, 2 or 1: the most that divides H_kv and still leaves two CTAs per
 * SM), 0 for the generic kernel.  Either pointer may be NULL.  Launches nothing.
 */
msa_status_t msa_index_scores_plan(const msa_shape_t* shape, int64_t q_count, int64_t kv_len,
                                   int32_t* tensor_core, int32_t* heads_per_cta);

msa_status_t msa_index_scores_decode(const msa_shape_t* shape, const void* q_idx,
                                     const void* k_idx_cache, const int64_t* seq_offsets,
                                     const int32_t* seq_lens, int32_t batch,
                                     int64_t max_seq_len, float* scores, int64_t ld_scores,
                                     msa_stream_t stream);

/* ------------------------------------------------------------------------------------
 * Stage 2 - Eq. 7 with the Local Block rule (Section 3.2) and exp-free ranking
 * (Section 4.1): for row (q, r), loc = (q_begin+q)/B_k is always selected and the
 * other min(k-1, loc) entries are the earlier blocks with the largest raw scores
 * (ties: lower block index wins).
 * block_idx [q_count,H_kv,k] int32: ascending block indices, padded with -1 when fewer
 * than k blocks are visible.  Only columns [0, loc] of a scores row are read.
 */
msa_status_t msa_topk_select(const msa_shape_t* shape, const float* scores, int64_t ld_scores,
                             int64_t q_begin, int64_t q_count, int64_t kv_len,
                             int32_t* block_idx, msa_stream_t stream);

/*
 * Stage 2 for batched decode: row (s, r) ranks blocks of sequence s, loc = (seq_lens[s]-1)/B_k.
 * max_seq_len bounds every seq_lens[s] (as in msa_index_scores_decode); ld_scores must hold
 * ceil(max_seq_len/B_k) columns, else MSA_ERR_INVALID_ARG.  A device-side seq_lens[s] beyond
 * ld_scores*B_k is not read past the row: its list is all -1 and the async status reports a bad index.
 */
msa_status_t msa_topk_select_decode(const msa_shape_t* shape, const float* scores,
                                    int64_t ld_scores, const int32_t* seq_lens, int32_t batch,
                                    int64_t max_seq_len, int32_t* block_idx, msa_stream_t stream);

/* ------------------------------------------------------------------------------------
 * Stage 3, prefill - Eq. 8 (Algorithm 1, line 5): for each query of the range and each
 * head h of group r, softmax attention over the causally visible tokens of the blocks
 * block_idx[q, r, :] (entries < 0 are skipped), using KV head r.
 *   out [q_count,H_q,d_h] bf16;  lse [q_count,H_q] fp32 or NULL:
 *   lse = log sum_j exp(softmax_scale * <q, k_j>) over the attended tokens (natural log).
 * The specialised path gathers, per (KV block, KV head), the queries that selected it
 * (KV-outer order, Section 4.2), writes locally normalised partials to the workspace
 * and merges them with the LSE-weighted combine of Section 4.2.  The workspace bounds
 * how many queries are in flight at once; a larger workspace means fewer passes.
 * A block index outside [-1, loc] is skipped and reported through the async status.
 */
msa_status_t msa_sparse_attn_prefill(const msa_shape_t* shape, const void* q, const void* k,
                                     const void* v, const int32_t* block_idx,
                                     int64_t q_begin, int64_t q_count, int64_t kv_len,
                                     void* out, float* lse, void* workspace,
                                     size_t workspace_bytes, msa_stream_t stream);

/*
 * Stage 3, prefill, for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a convenience of the library.)
 *
 * Some hosts of this library are not allowed to call cudaMalloc, or to ask their framework
 * for a buffer, at the point where they need attention: a plug-in running inside an engine
 * that owns all device memory, a callback that runs after the memory pool has been frozen,
 * a real-time loop where an allocation may stall on the driver.  msa_sparse_attn_prefill
 * needs a caller-provided workspace, so such callers cannot use it.  This variant takes the
 * same inputs and outputs and no workspace: its scratch (reverse index, partial outputs,
 * partial log-sum-exps) lives in one fixed array of MSA_STATIC_SCRATCH_BYTES inside the
 * library's device image.  Every GPU that loads the library holds that array until the
 * process exits.
 *
 * Limits and rules:
 *   - The query range is processed in passes of as many queries as fit the fixed array.
 *     If fewer than min(q_count, 16) queries fit (long sequences with many heads and a large
 *     k), the call returns MSA_ERR_WORKSPACE and launches nothing; use the workspace form.
 *   - The call allocates nothing: no cudaMalloc/cudaFree and no allocating library routine.
 *   - The first call on each device looks up the array's device address (with that device
 *     current) and sets a kernel attribute; make that first call outside any stream capture.
 *   - All calls share the one array, and it keeps the previous call's contents; the call
 *     clears the counters that must start at zero itself.  Two calls whose kernels overlap
 *     on the GPU (different streams, or different host threads) race on it: serialise them.
 *   - Results equal those of msa_sparse_attn_prefill on the same inputs.
 */
#define MSA_STATIC_SCRATCH_BYTES (64u << 20)
msa_status_t msa_sparse_attn_prefill_static(const msa_shape_t* shape, const void* q, const void* k,
                                            const void* v, const int32_t* block_idx,
                                            int64_t q_begin, int64_t q_count, int64_t kv_len,
                                            void* out, float* lse, msa_stream_t stream);

/* Minimum and preferred workspace for msa_sparse_attn_prefill (bytes; either may be NULL). */
msa_status_t msa_sparse_attn_prefill_workspace_bytes(const msa_shape_t* shape, int64_t q_count,
                                                     int64_t kv_len, size_t* min_bytes,
                                                     size_t* preferred_bytes);

/* ------------------------------------------------------------------------------------
 * Stage 3, decode - Eq. 8 for one query per cached sequence (position seq_lens[s]-1).
 * q [batch,H_q,d_h]; k_cache, v_cache [cache_tokens,H_kv,d_h] bf16 packed token-major,
 * sequence s at rows seq_offsets[s]..; block_idx [batch,H_kv,k]; out [batch,H_q,d_h]
 * bf16; lse [batch,H_q] fp32 or NULL.  The selected blocks of each (sequence, KV head)
 * are split over several CTAs; partials are merged with the Section 4.2 combine.
 */
msa_status_t msa_sparse_attn_decode(const msa_shape_t* shape, const void* q, const void* k_cache,
                                    const void* v_cache, int64_t cache_tokens,
                                    const int64_t* seq_offsets, const int32_t* seq_lens,
                                    int32_t batch, const int32_t* block_idx, void* out,
                                    float* lse, void* workspace, size_t workspace_bytes,
                                    msa_stream_t stream);

msa_status_t msa_sparse_attn_decode_workspace_bytes(const msa_shape_t* shape, int32_t batch,
                                                    size_t* min_bytes);

/* ------------------------------------------------------------------------------------
 * Eq. 6 and Eq. 7 in one kernel (the indexer only needs block-wise maxima, so the score
 * matrix M need not exist): block_idx [q_count,H_kv,k] int32 exactly as msa_index_scores
 * followed by msa_topk_select would write it (same scaled fp32 maxima, same tie rule, same
 * list format).  Every epilogue thread of the scoring kernel keeps the best 15 earlier blocks
 * of its row in registers, so this form exists for top_k <= 16, d_idx in {64,128}, B_k in
 * {64,128} and q_count >= 32; anything else returns MSA_ERR_UNSUPPORTED and the two separate
 * calls are the way.  msa_prefill_forward uses it whenever the shape allows.  No workspace.
 */
msa_status_t msa_index_topk_fused(const msa_shape_t* shape, const void* q_idx, const void* k_idx,
                                  int64_t q_begin, int64_t q_count, int64_t kv_len, int32_t* block_idx,
                                  msa_stream_t stream);

/* ------------------------------------------------------------------------------------
 * Index-branch log-sum-exp over the selected blocks (Section 4.3, "LSE fusion": the forward
 * emits LSE_idx so that the sparse-KL backward need not recompute it):
 *   lse_idx[i,r] = log sum over b in block_idx[i,r,:], j in block b, j <= q_begin+i of
 *                  exp(<q_idx[i,r,:], k_idx[j,:]> * index_scale)            (natural log)
 * q_idx [q_count,H_kv,d_idx] bf16 (rows of the range), k_idx [kv_len,d_idx] bf16, block_idx
 * [q_count,H_kv,k] int32 as written by msa_topk_select (entries < 0 are padding), lse_idx
 * [q_count,H_kv] float32 (out; -inf for a row with no valid entry).  Runs after Top-k, KV-outer
 * over the (block, head) tiles like the attention, on tcgen05 MMAs (items of 128 queries x one
 * key block) for d_idx in {64,128} and B_k in {64,128}; any other shape takes a plain kernel that needs no
 * workspace.  workspace >= msa_index_lse_prefill_workspace_bytes (device, 16-byte aligned).
 * Errors as msa_sparse_attn_prefill; a block index outside [-1, loc] sets the async status.
 */
msa_status_t msa_index_lse_prefill(const msa_shape_t* shape, const void* q_idx, const void* k_idx,
                                   const int32_t* block_idx, int64_t q_begin, int64_t q_count,
                                   int64_t kv_len, float* lse_idx, void* workspace,
                                   size_t workspace_bytes, msa_stream_t stream);

msa_status_t msa_index_lse_prefill_workspace_bytes(const msa_shape_t* shape, int64_t q_count,
                                                   int64_t kv_len, size_t* min_bytes,
                                                   size_t* preferred_bytes);

/* ------------------------------------------------------------------------------------
 * Whole path, prefill (Algorithm 1, lines 3-5) for one sequence of T tokens: runs stage 1
 * and 2 over query chunks sized to the workspace, then stage 3.  block_idx [T,H_kv,k] is
 * an output (required); lse may be NULL.  workspace >= msa_prefill_forward_workspace_bytes.
 */
msa_status_t msa_prefill_forward(const msa_shape_t* shape, const void* q, const void* k,
                                 const void* v, const void* q_idx, const void* k_idx, int64_t T,
                                 void* out, float* lse, int32_t* block_idx, void* workspace,
                                 size_t workspace_bytes, msa_stream_t stream);

msa_status_t msa_prefill_forward_workspace_bytes(const msa_shape_t* shape, int64_t T,
                                                 size_t* min_bytes, size_t* preferred_bytes);

/*
 * Whole path, prefill, for a batch of sequences of different lengths packed token-major
 * (Section 4.2 names variable-length sequences as a source of uneven tile work; blocks are
 * counted from each sequence's own first token, every sequence is causal on its own and no
 * quantity of Eq. 6-8 crosses a sequence boundary).  Sequence s owns rows
 * cu_seqlens[s] .. cu_seqlens[s+1]-1 of q, k, v, q_idx, k_idx, out, lse and block_idx;
 * cu_seqlens is a HOST array of n_seqs+1 non-decreasing row offsets (int64), cu_seqlens[0] >= 0.
 * block_idx holds block numbers relative to the row's own sequence.  Sequences of length 0 are
 * skipped.  On the shapes of the tensor-core attention kernel (d_h = 128, G in {8,16}, B_k in
 * {64,128}) a batch of two or more sequences runs as ONE problem per stage: Eq. 6 + Eq. 7 as a single
 * launch of the fused kernel over the query tiles of all sequences (top_k <= 16), or (larger top_k)
 * one scoring launch and one Top-k launch per group of consecutive sequences - as many sequences as
 * the workspace holds score rows for (a row takes 4 * H_kv * the block count of the batch's longest
 * sequence, rounded up to 8, bytes); a sequence too long for the region alone is scored by the
 * single-sequence path in chunks - and Eq. 8 with its blocks numbered through the batch, so that one
 * reverse index, one attention launch and one merge serve every sequence of a query range (ranges
 * span sequence boundaries).  Other shapes, and a batch of one, run the single-sequence call per
 * sequence on `stream`.  Results do not depend on which way a sequence ran.  The call copies
 * cu_seqlens and a tile list from host memory to the front of the workspace with cudaMemcpyAsync:
 * it must not be captured into a CUDA graph.  Everything runs on `stream`; the library owns no
 * stream here.
 * workspace >= msa_prefill_forward_varlen_workspace_bytes' minimum (the batch's maps - 8 bytes per
 * row, 4 per block - plus what the stages need).  Errors: MSA_ERR_INVALID_ARG for a NULL or decreasing
 * cu_seqlens or n_seqs < 0, otherwise as msa_prefill_forward.
 */
msa_status_t msa_prefill_forward_varlen(const msa_shape_t* shape, const void* q, const void* k,
                                        const void* v, const void* q_idx, const void* k_idx,
                                        const int64_t* cu_seqlens, int32_t n_seqs, void* out,
                                        float* lse, int32_t* block_idx, void* workspace,
                                        size_t workspace_bytes, msa_stream_t stream);

msa_status_t msa_prefill_forward_varlen_workspace_bytes(const msa_shape_t* shape,
                                                        const int64_t* cu_seqlens, int32_t n_seqs,
                                                        size_t* min_bytes, size_t* preferred_bytes);

/*
 * Same, from HOST buffers: copies q, k, v, q_idx, k_idx host->device into the staging
 * area at the front of `workspace`, runs the three stages, copies `out` (and lse,
 * block_idx when non-NULL) back, and synchronises before returning.  The copies run on a
 * second stream owned by the library (created on first use) and overlap the kernels: the
 * index inputs are uploaded first so that stages 1-2 start while Q, K and V are still in
 * flight; q_idx and q go up in pieces of rows, and a scoring chunk or the attention of a query
 * range waits only for the piece that holds its last row; each finished query range of the
 * output is copied back while the next one is computed.  Host buffers should be page-locked for the copies to run at full rate and to
 * overlap at all.
 * workspace >= msa_prefill_forward_host_workspace_bytes.
 */
msa_status_t msa_prefill_forward_host(const msa_shape_t* shape, const void* q_host,
                                      const void* k_host, const void* v_host,
                                      const void* q_idx_host, const void* k_idx_host, int64_t T,
                                      void* out_host, float* lse_host, int32_t* block_idx_host,
                                      void* workspace, size_t workspace_bytes,
                                      msa_stream_t stream);

msa_status_t msa_prefill_forward_host_workspace_bytes(const msa_shape_t* shape, int64_t T,
                                                      size_t* min_bytes,
                                                      size_t* preferred_bytes);

/*
 * Whole path, decode step (stages 1-3 for one new token per sequence).  scores
 * [batch,H_kv,ld_scores] and block_idx [batch,H_kv,k] are outputs kept for the caller.
 */
msa_status_t msa_decode_forward(const msa_shape_t* shape, const void* q, const void* q_idx,
                                const void* k_cache, const void* v_cache,
                                const void* k_idx_cache, int64_t cache_tokens,
                                const int64_t* seq_offsets, const int32_t* seq_lens,
                                int32_t batch, int64_t max_seq_len, float* scores,
                                int64_t ld_scores, int32_t* block_idx, void* out, float* lse,
                                void* workspace, size_t workspace_bytes, msa_stream_t stream);

/*
 * Same with the step's inputs and result in HOST memory: q_host [batch,H_q,d_h] and
 * q_idx_host [batch,H_kv,d_idx] are copied in, out_host [batch,H_q,d_h] is copied back;
 * the caches stay resident on the device.  q_dev/q_idx_dev/out_dev are device staging
 * buffers of the same sizes.  Synchronises `stream` before returning.
 */
msa_status_t msa_decode_forward_host(const msa_shape_t* shape, const void* q_host,
                                     const void* q_idx_host, void* q_dev, void* q_idx_dev,
                                     const void* k_cache, const void* v_cache,
                                     const void* k_idx_cache, int64_t cache_tokens,
                                     const int64_t* seq_offsets, const int32_t* seq_lens,
                                     int32_t batch, int64_t max_seq_len, float* scores,
                                     int64_t ld_scores, int32_t* block_idx, void* out_dev,
                                     void* out_host, void* workspace, size_t workspace_bytes,
                                     msa_stream_t stream);

/*
 * Test hook for the device-side bounded waits (the paper has no counterpart).  Every wait of a
 * kernel on an mbarrier gives up after a limit of SM cycles (about two seconds by default),
 * raises MSA_ERR_TIMEOUT in the async status and lets the kernel unwind and return.
 * wait_limit_cycles sets that limit for the kernels launched afterwards on the current device
 * (0 or anything above the default restores the default); producer_delay_cycles (at most 1e8)
 * makes the warp that issues the copies of the tensor-core prefill kernels (index scoring,
 * attention) sit out that many cycles before its first copy, so that a short limit runs out on a
 * role that is merely late.  Both values stay until changed; production code never calls this.
 */
msa_status_t msa_debug_set_wait(int64_t wait_limit_cycles, int64_t producer_delay_cycles);

/* Number of kernel launches the library has enqueued since the process started. */
int64_t msa_launch_count(void);

/*
 * Optional per-stage timing for benchmarks (the paper has no counterpart).  Between
 * msa_profile_begin() and msa_profile_end() every kernel launch of the library is
 * bracketed by CUDA events on its stream; msa_profile_end() synchronises the device and
 * returns, per stage, the summed device time in milliseconds and the number of launches
 * (arrays of 9: 0 index scoring, 1 top-k, 2 reverse index/schedule, 3 prefill attention,
 * 4 combine, 5 decode index scoring, 6 decode attention, 7 decode combine, 8 index-branch
 * log-sum-exp).  The first
 * msa_profile_begin() creates the event pool (16384 launches); MSA_ERR_UNSUPPORTED from
 * msa_profile_end() means the pool ran out and the sums are partial.  Not thread-safe.
 */
msa_status_t msa_profile_begin(void);
msa_status_t msa_profile_end(float* stage_ms_host, int64_t* stage_launches_host);

#ifdef __cplusplus
}
#endif
#endif /* MSA_H_ */
