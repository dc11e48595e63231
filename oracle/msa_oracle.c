/*
 * CPU oracle for the forward path of MiniMax Sparse Attention (MSA).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the path
 * computes, written from the paper's definitions.  It shares no code, header, table or
 * helper with the CUDA library and must never be called from the product path.
 *
 * All arithmetic is IEEE double.  Inputs are bf16 bit patterns (uint16_t) widened
 * exactly.  Positions, blocks and heads are 0-based here (the paper is 1-based):
 * token j belongs to block j / B_k (Eq. 4), query head h belongs to GQA group
 * r = h / G with G = H_q / H_kv ("G adjacent query heads", Section 2.1).
 *
 * Every function takes an explicit list of query positions pos[0..n), so the same code
 * serves full prefill (pos = 0..T-1), a sampled prefill and decode (pos = L-1).
 *
 * Conventions of this build where the paper is silent (each is a stated reading, not a
 * fact of the paper):
 *   - ties between equal block scores go to the lower block index;
 *   - when fewer than k blocks are visible all of them are selected and the list is
 *     padded with -1;
 *   - index lists are written in ascending block order.
 *
 * Parity pins: every function below is pinned by tests that run without a GPU
 * (invariants, special cases that reduce to library routines, brute force on tiny
 * inputs).  Unpinned by anything but choice: the tie-break direction and the list
 * format (ascending, -1 padded), which are conventions.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static inline double bf16_to_double(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/*
 * fp8 E4M3 ("fn" flavour: no infinities, S.1111.111 is NaN) widened exactly: 1 sign bit, 4
 * exponent bits with bias 7, 3 mantissa bits; exponent 0 is subnormal, m/8 * 2^-6.
 * (The paper states that its kernels also support fp8, Section 4.2; this build accepts the
 * index branch's operands in that format.)
 */
static inline double e4m3_to_double(uint8_t b) {
    const int sign = b >> 7, e = (b >> 3) & 15, m = b & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m / 8.0, -6);
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return sign ? -v : v;
}

/* element c of an index-branch row stored as bf16 (idx_fp8 = 0) or E4M3 (idx_fp8 = 1) */
/* Element e of a K or V tensor stored as fp8 E4M3 (Section 4.2: the kernels also support fp8) or bf16. */
static inline double kv_elem(const void* base, int64_t e, int kv_fp8) {
    return kv_fp8 ? e4m3_to_double(((const uint8_t*)base)[e]) : bf16_to_double(((const uint16_t*)base)[e]);
}

static inline double idx_elem(const void* row, int c, int idx_fp8) {
    return idx_fp8 ? e4m3_to_double(((const uint8_t*)row)[c]) : bf16_to_double(((const uint16_t*)row)[c]);
}

/*
 * Eq. 6: token-level index scores and their block-wise causal maximum.
 *   S[i,r,j] = <Q_idx[i,r,:], K_idx[j,:]> * scale           for j <= i
 *   M[i,r,b] = max over j in block b with j <= i of S[i,r,j]
 *   M[i,r,b] = -inf when block b holds no token j <= i.
 * q_idx: [n, H_kv, d_idx] rows for the listed positions; k_idx: [L, d_idx] (one shared
 * index key head, Eq. 5); M: [n, H_kv, B] with B = ceil(L / B_k).
 */
void msa_oracle_index_scores(const void* q_idx, const void* k_idx,
                             const int64_t* pos, int64_t n, int64_t L, int H_kv,
                             int d_idx, int B_k, double scale, double* M, int idx_fp8) {
    const int64_t B = (L + B_k - 1) / B_k;
    const int64_t eb = idx_fp8 ? 1 : 2;  /* bytes per index element */
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t a = 0; a < n * H_kv; ++a) {
        const int64_t qi = a / H_kv;
        const int r = (int)(a % H_kv);
        const int64_t i = pos[qi];
        const char* qrow = (const char*)q_idx + (qi * H_kv + r) * (int64_t)d_idx * eb;
        double* Mrow = M + (qi * H_kv + r) * B;
        for (int64_t b = 0; b < B; ++b) {
            double best = -INFINITY;
            const int64_t j0 = b * B_k;
            int64_t j1 = j0 + B_k;
            if (j1 > L) j1 = L;
            for (int64_t j = j0; j < j1 && j <= i; ++j) {
                const char* krow = (const char*)k_idx + j * (int64_t)d_idx * eb;
                double s = 0.0;
                for (int c = 0; c < d_idx; ++c)
                    s += idx_elem(qrow, c, idx_fp8) * idx_elem(krow, c, idx_fp8);
                s *= scale;
                if (s > best) best = s;
            }
            Mrow[b] = best;
        }
    }
}

/*
 * Section 4.3, "LSE fusion": the log-sum-exp of the index branch over the selected blocks,
 *   LSE_idx[i,r] = log sum over b in I[i,r], j in block b, j <= i of exp(S[i,r,j])
 * with S as in Eq. 6 (natural logarithm).  The paper obtains it by reducing per-block
 * log-sum-exps over the Top-k blocks; here it is the definition written out as one sum,
 * stabilised by the largest selected score.  Entries of I below 0 are padding.
 * q_idx: [n, H_kv, d_idx]; k_idx: [L, d_idx]; I: [n, H_kv, k]; out: [n, H_kv].
 */
void msa_oracle_index_lse(const void* q_idx, const void* k_idx, const int32_t* I,
                          const int64_t* pos, int64_t n, int64_t L, int H_kv, int d_idx,
                          int B_k, int k, double scale, double* out, int idx_fp8) {
    const int64_t eb = idx_fp8 ? 1 : 2;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t a = 0; a < n * H_kv; ++a) {
        const int64_t qi = a / H_kv;
        const int64_t i = pos[qi];
        const char* qrow = (const char*)q_idx + a * (int64_t)d_idx * eb;
        const int32_t* sel = I + a * (int64_t)k;
        double best = -INFINITY, sum = 0.0;
        for (int pass = 0; pass < 2; ++pass) {  /* pass 0: the largest score; pass 1: the sum */
            for (int t = 0; t < k; ++t) {
                if (sel[t] < 0) continue;
                const int64_t j0 = (int64_t)sel[t] * B_k;
                int64_t j1 = j0 + B_k;
                if (j1 > L) j1 = L;
                for (int64_t j = j0; j < j1 && j <= i; ++j) {
                    const char* krow = (const char*)k_idx + j * (int64_t)d_idx * eb;
                    double s = 0.0;
                    for (int c = 0; c < d_idx; ++c)
                        s += idx_elem(qrow, c, idx_fp8) * idx_elem(krow, c, idx_fp8);
                    s *= scale;
                    if (pass == 0) { if (s > best) best = s; }
                    else sum += exp(s - best);
                }
            }
        }
        out[a] = (best == -INFINITY) ? -INFINITY : best + log(sum);
    }
}

typedef struct {
    double score;
    int32_t block;
} cand_t;

/* Total order used for ranking: score descending, then block index ascending. */
static int cand_cmp(const void* pa, const void* pb) {
    const cand_t* a = (const cand_t*)pa;
    const cand_t* b = (const cand_t*)pb;
    if (a->score > b->score) return -1;
    if (a->score < b->score) return 1;
    return (a->block > b->block) - (a->block < b->block);
}

static int int32_cmp(const void* pa, const void* pb) {
    const int32_t a = *(const int32_t*)pa, b = *(const int32_t*)pb;
    return (a > b) - (a < b);
}

/*
 * Eq. 7 with the Local Block rule of Section 3.2: for query i of group r the local
 * block loc = i / B_k is always selected; the remaining min(k-1, loc) slots go to the
 * earlier blocks 0..loc-1 with the largest raw scores M (exp-free: no softmax is
 * applied before ranking, Section 4.1).  Blocks after loc are invisible (-inf) and never
 * selected.  I: [n, H_kv, k], ascending, padded with -1.
 */
void msa_oracle_topk_select(const double* M, const int64_t* pos, int64_t n, int64_t L,
                            int H_kv, int B_k, int k, int32_t* I) {
    const int64_t B = (L + B_k - 1) / B_k;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t a = 0; a < n * H_kv; ++a) {
        const int64_t qi = a / H_kv;
        const int64_t loc = pos[qi] / B_k;
        const double* Mrow = M + a * B;
        int32_t* out = I + a * (int64_t)k;
        cand_t* c = (cand_t*)malloc(sizeof(cand_t) * (size_t)(loc > 0 ? loc : 1));
        for (int64_t b = 0; b < loc; ++b) {
            c[b].score = Mrow[b];
            c[b].block = (int32_t)b;
        }
        qsort(c, (size_t)loc, sizeof(cand_t), cand_cmp);
        int m = k - 1;
        if ((int64_t)m > loc) m = (int)loc;
        int cnt = 0;
        for (int t = 0; t < m; ++t) out[cnt++] = c[t].block;
        out[cnt++] = (int32_t)loc;
        qsort(out, (size_t)cnt, sizeof(int32_t), int32_cmp);
        for (; cnt < k; ++cnt) out[cnt] = -1;
        free(c);
    }
}

/*
 * Eq. 8: for query i, head h of group r = h / G, softmax attention over the causally
 * visible tokens of the selected blocks I[i,r,:]:
 *   tokens   = { j : j <= i, j < L, j / B_k in I[i,r,:] }
 *   z[j]     = <Q[i,h,:], K[j,r,:]> * scale
 *   O[i,h,:] = sum_j softmax(z)[j] * V[j,r,:]
 *   LSE[i,h] = log sum_j exp(z[j])   (natural log)
 * q: [n,H_q,d]; K,V: [L,H_kv,d]; I: [n,H_kv,k] (entries < 0 are padding);
 * O: [n,H_q,d]; LSE: [n,H_q].
 * Operands stored in fp8 E4M3 (Section 4.2: the kernels also support fp8) are decoded exactly and
 * everything after the decoding is the arithmetic above, in double: the oracle models no rounding
 * of P or of partial results.
 */
void msa_oracle_sparse_attn(const void* q, const void* K, const void* V,
                            const int32_t* I, const int64_t* pos, int64_t n, int64_t L,
                            int H_q, int H_kv, int d, int B_k, int k, double scale,
                            double* O, double* LSE, int kv_fp8, int q_fp8) {
    const int G = H_q / H_kv;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t a = 0; a < n * H_q; ++a) {
        const int64_t qi = a / H_q;
        const int h = (int)(a % H_q);
        const int r = h / G;
        const int64_t i = pos[qi];
        const int64_t qrow = a * (int64_t)d;  /* element offset; Q holds bf16 or fp8 E4M3 like K and V */
        const int32_t* sel = I + (qi * H_kv + r) * (int64_t)k;
        double* z = (double*)malloc(sizeof(double) * (size_t)k * (size_t)B_k);
        int64_t* tok = (int64_t*)malloc(sizeof(int64_t) * (size_t)k * (size_t)B_k);
        int64_t nt = 0;
        for (int s = 0; s < k; ++s) {
            if (sel[s] < 0) continue;
            const int64_t j0 = (int64_t)sel[s] * B_k;
            for (int64_t j = j0; j < j0 + B_k && j < L && j <= i; ++j) {
                const int64_t krow = (j * H_kv + r) * (int64_t)d;  /* element offset; K, V hold bf16 or fp8 E4M3 */
                double acc = 0.0;
                for (int c = 0; c < d; ++c)
                    acc += kv_elem(q, qrow + c, q_fp8) * kv_elem(K, krow + c, kv_fp8);
                z[nt] = acc * scale;
                tok[nt] = j;
                ++nt;
            }
        }
        double mx = -INFINITY;
        for (int64_t t = 0; t < nt; ++t)
            if (z[t] > mx) mx = z[t];
        double ell = 0.0;
        for (int64_t t = 0; t < nt; ++t) ell += exp(z[t] - mx);
        double* orow = O + a * (int64_t)d;
        for (int c = 0; c < d; ++c) orow[c] = 0.0;
        for (int64_t t = 0; t < nt; ++t) {
            const double w = exp(z[t] - mx) / ell;
            const int64_t vrow = (tok[t] * H_kv + r) * (int64_t)d;
            for (int c = 0; c < d; ++c) orow[c] += w * kv_elem(V, vrow + c, kv_fp8);
        }
        LSE[a] = mx + log(ell);
        free(z);
        free(tok);
    }
}

/*
 * Eq. 1: dense causal GQA attention, the definition the sparse path must reduce to when
 * every visible block is selected.  Same layouts as msa_oracle_sparse_attn.
 */
void msa_oracle_dense_attn(const uint16_t* q, const uint16_t* K, const uint16_t* V,
                           const int64_t* pos, int64_t n, int64_t L, int H_q, int H_kv,
                           int d, double scale, double* O, double* LSE) {
    const int G = H_q / H_kv;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t a = 0; a < n * H_q; ++a) {
        const int64_t qi = a / H_q;
        const int h = (int)(a % H_q);
        const int r = h / G;
        const int64_t t = pos[qi];
        const uint16_t* qrow = q + a * (int64_t)d;
        double* z = (double*)malloc(sizeof(double) * (size_t)(t + 1));
        double mx = -INFINITY;
        for (int64_t i = 0; i <= t && i < L; ++i) {
            const uint16_t* krow = K + (i * H_kv + r) * (int64_t)d;
            double acc = 0.0;
            for (int c = 0; c < d; ++c)
                acc += bf16_to_double(qrow[c]) * bf16_to_double(krow[c]);
            z[i] = acc * scale;
            if (z[i] > mx) mx = z[i];
        }
        double den = 0.0;
        for (int64_t i = 0; i <= t && i < L; ++i) den += exp(z[i] - mx);
        double* orow = O + a * (int64_t)d;
        for (int c = 0; c < d; ++c) orow[c] = 0.0;
        for (int64_t i = 0; i <= t && i < L; ++i) {
            const double alpha = exp(z[i] - mx) / den;
            const uint16_t* vrow = V + (i * H_kv + r) * (int64_t)d;
            for (int c = 0; c < d; ++c) orow[c] += alpha * bf16_to_double(vrow[c]);
        }
        LSE[a] = mx + log(den);
        free(z);
    }
}

/*
 * Two-phase forward, combine step (Section 4.2): merge S locally normalised partial
 * outputs of one (query, head) with their log-sum-exps:
 *   a = max_s LSE_s;  LSE = a + log sum_s exp(LSE_s - a);  w_s = exp(LSE_s - LSE);
 *   O = sum_s w_s O_s.
 * O_parts: [S, d]; LSE_parts: [S]; a part with LSE = -inf is empty and contributes
 * nothing.  O_out: [d]; returns LSE.
 */
double msa_oracle_combine(const double* O_parts, const double* LSE_parts, int S, int d,
                          double* O_out) {
    double a = -INFINITY;
    for (int s = 0; s < S; ++s)
        if (LSE_parts[s] > a) a = LSE_parts[s];
    double sum = 0.0;
    for (int s = 0; s < S; ++s)
        if (LSE_parts[s] > -INFINITY) sum += exp(LSE_parts[s] - a);
    const double lse = a + log(sum);
    for (int c = 0; c < d; ++c) O_out[c] = 0.0;
    for (int s = 0; s < S; ++s) {
        if (!(LSE_parts[s] > -INFINITY)) continue;
        const double w = exp(LSE_parts[s] - lse);
        for (int c = 0; c < d; ++c) O_out[c] += w * O_parts[(int64_t)s * d + c];
    }
    return lse;
}
