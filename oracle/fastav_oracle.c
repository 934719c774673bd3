/*
 * CPU oracle for the FastAV prune step.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain definition that the CUDA library is checked
 * against.  It shares no code with the CUDA path, is never linked into it, and
 * may be used only by the tests, by the smoke check and by the benchmark's
 * CPU-baseline leg.  Nothing here is tuned: straight loops, double precision,
 * libm's exp().  The only concession to wall-clock time is an OpenMP
 * "parallel for" over query heads, which does not change any arithmetic
 * (each head writes its own buffer; the head sum is taken afterwards in
 * ascending head order).
 *
 * What it computes (paper, Section 2.2, "Fine pruning", Eq. 4):
 *     s = mean_h softmax(Q_last K^T)
 * generalised to R scored query rows instead
 * of one (mean over rows and heads), grouped-query attention (query head h
 * reads KV head h / G), an optional causal mask by token index, an explicit
 * softmax scale, and variable-length batches.  Then the bottom-P % rule of the
 * same paragraph, stated on the survivors: keep the k largest, ties to the lower
 * index, protected tokens always kept; survivors stay in their original order
 * and carry their rows of hidden states, position ids, K and V with them.
 *
 * Pins: tests/test_oracle_pins.py (brute-force full attention maps, hand-worked
 * examples under tests/golden/, closed forms, invariants, an independent
 * selector).  Eq. 4 on real model activations is "parity unpinned": the paper
 * prints no worked numeric example of it.
 *
 * All tensors are bf16 bit patterns (uint16_t) unless stated; strides are in
 * elements; the innermost (head_dim / hidden) dimension is contiguous.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_double(uint16_t bits) {
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Number of OpenMP threads the library will use (1 when built without OpenMP). */
int oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Eq. 4.  For sequence b with tokens [cu_seqlens[b], cu_seqlens[b+1]) and scored
 * rows [cu_qlens[b], cu_qlens[b+1]):
 *
 *   z[h][r][j] = scale * <q[r][h][:], k[j][h / G][:]>
 *   p[h][r][:] = softmax over the keys row r may see
 *                (all keys, or j <= q_idx[r] when causal != 0)
 *   s[j]       = (1 / (Hq * R_b)) * sum_r sum_h p[h][r][j]
 *
 * q_idx[r] is the sequence-local index of the token that scored row r belongs
 * to.  A row that sees no key contributes nothing (but still counts in R_b).
 * A sequence with R_b = 0 gets all-zero scores.
 *
 * nthreads <= 0 means "all the OpenMP runtime offers"; 1 forces a serial run.
 * Returns 0, or -1 when a scratch allocation fails.
 */
int oracle_score(int batch, const int32_t *cu_seqlens, const int32_t *cu_qlens, const int32_t *q_idx,
                 const uint16_t *q, int64_t q_stride_tok, int64_t q_stride_head,
                 const uint16_t *k, int64_t k_stride_tok, int64_t k_stride_head,
                 int num_q_heads, int num_kv_heads, int head_dim, double scale, int causal,
                 double *scores_out, int nthreads) {
    const int group = num_q_heads / num_kv_heads;
#ifdef _OPENMP
    if (nthreads <= 0) nthreads = omp_get_max_threads();
#else
    nthreads = 1;
#endif
    for (int b = 0; b < batch; ++b) {
        const int tok0 = cu_seqlens[b], n = cu_seqlens[b + 1] - tok0;
        const int row0 = cu_qlens[b], rows = cu_qlens[b + 1] - row0;
        if (n <= 0) continue;
        for (int j = 0; j < n; ++j) scores_out[tok0 + j] = 0.0;
        if (rows <= 0) continue;

        /* per_head[h][j] = sum over rows of softmax(row r, head h)[j] */
        double *per_head = (double *)calloc((size_t)num_q_heads * (size_t)n, sizeof(double));
        double *logit_buf = (double *)malloc((size_t)nthreads * (size_t)n * sizeof(double));
        if (!per_head || !logit_buf) {
            free(per_head);
            free(logit_buf);
            return -1;
        }
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) num_threads(nthreads)
#endif
        for (int h = 0; h < num_q_heads; ++h) {
#ifdef _OPENMP
            double *z = logit_buf + (size_t)omp_get_thread_num() * (size_t)n;
#else
            double *z = logit_buf;
#endif
            const int g = h / group;
            double *acc = per_head + (size_t)h * (size_t)n;
            for (int r = 0; r < rows; ++r) {
                int visible = n;
                if (causal) {
                    int last = q_idx[row0 + r];
                    visible = last + 1;
                    if (visible > n) visible = n;
                }
                if (visible <= 0) continue;
                const uint16_t *qv = q + (int64_t)(row0 + r) * q_stride_tok + (int64_t)h * q_stride_head;
                double zmax = -INFINITY;
                for (int j = 0; j < visible; ++j) {
                    const uint16_t *kv = k + (int64_t)(tok0 + j) * k_stride_tok + (int64_t)g * k_stride_head;
                    double dot = 0.0;
                    for (int c = 0; c < head_dim; ++c) dot += bf16_to_double(qv[c]) * bf16_to_double(kv[c]);
                    z[j] = scale * dot;
                    if (z[j] > zmax) zmax = z[j];
                }
                double denom = 0.0;
                for (int j = 0; j < visible; ++j) {
                    z[j] = exp(z[j] - zmax);
                    denom += z[j];
                }
                for (int j = 0; j < visible; ++j) acc[j] += z[j] / denom;
            }
        }
        const double inv = 1.0 / ((double)num_q_heads * (double)rows);
        for (int j = 0; j < n; ++j) {
            double total = 0.0;
            for (int h = 0; h < num_q_heads; ++h) total += per_head[(size_t)h * (size_t)n + j];
            scores_out[tok0 + j] = total * inv;
        }
        free(per_head);
        free(logit_buf);
    }
    return 0;
}

/* ---- selection ------------------------------------------------------------------- */

typedef struct {
    float key;      /* score, or +inf for a protected token */
    int32_t index;  /* sequence-local */
} ranked_token;

static int ranked_before(const void *pa, const void *pb) {
    const ranked_token *a = (const ranked_token *)pa, *b = (const ranked_token *)pb;
    if (a->key > b->key) return -1; /* larger score first */
    if (a->key < b->key) return 1;
    return (a->index > b->index) - (a->index < b->index); /* equal score: lower index first */
}

static int ascending_i32(const void *pa, const void *pb) {
    int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    return (a > b) - (a < b);
}

/*
 * The bottom-P % rule (Section 2.2, "Fine pruning"): per sequence keep the k_b
 * tokens that come first when tokens are ranked by (score descending, index
 * ascending); protected tokens rank as +infinity.  The decision is taken on
 * fp32 scores, the precision the CUDA selector works in.  k_b is clamped to
 * [0, n_b].  Survivors are written in ascending index order: sequence-local
 * indices, or indices into the packed batch when global_index != 0.
 *
 * protect_mask (one byte per token of the packed batch, non-zero = always keep)
 * may be NULL; protect_rows != 0 additionally protects the tokens q_idx names.
 */
int oracle_select(int batch, const int32_t *cu_seqlens, const float *scores, const int32_t *keep_counts,
                  const uint8_t *protect_mask, int protect_rows, const int32_t *q_idx, const int32_t *cu_qlens,
                  int global_index, int32_t *keep_idx_out, int32_t *cu_keep_out) {
    int32_t written = 0;
    cu_keep_out[0] = 0;
    for (int b = 0; b < batch; ++b) {
        const int tok0 = cu_seqlens[b], n = cu_seqlens[b + 1] - tok0;
        int keep = keep_counts[b];
        if (keep < 0) keep = 0;
        if (keep > n) keep = n;
        if (n > 0 && keep > 0) {
            ranked_token *rank = (ranked_token *)malloc((size_t)n * sizeof(ranked_token));
            if (!rank) return -1;
            for (int j = 0; j < n; ++j) {
                rank[j].key = scores[tok0 + j];
                rank[j].index = j;
                if (protect_mask && protect_mask[tok0 + j]) rank[j].key = INFINITY;
            }
            if (protect_rows) {
                for (int r = cu_qlens[b]; r < cu_qlens[b + 1]; ++r) {
                    int j = q_idx[r];
                    if (j >= 0 && j < n) rank[j].key = INFINITY;
                }
            }
            qsort(rank, (size_t)n, sizeof(ranked_token), ranked_before);
            for (int i = 0; i < keep; ++i) keep_idx_out[written + i] = rank[i].index;
            qsort(keep_idx_out + written, (size_t)keep, sizeof(int32_t), ascending_i32);
            if (global_index)
                for (int i = 0; i < keep; ++i) keep_idx_out[written + i] += tok0;
            free(rank);
            written += keep;
        }
        cu_keep_out[b + 1] = written;
    }
    return 0;
}

/* ---- compaction ------------------------------------------------------------------ */

/*
 * Survivor layout: output row cu_keep[b] + i is input row cu_seqlens[b] + keep[i]
 * (keep sequence-local, or already global when global_index != 0) of the hidden
 * states [N, hidden], the position ids [N], and K and V [N, Hkv, head_dim]
 * (token and head strides given, for inputs and outputs separately).  Any
 * in/out pair may be NULL and is then skipped.  Pure byte moves.
 */
void oracle_compact(int batch, const int32_t *cu_seqlens, const int32_t *keep_idx, const int32_t *cu_keep,
                    int global_index, int hidden, int num_kv_heads, int head_dim,
                    const uint16_t *hidden_in, uint16_t *hidden_out, const int32_t *pos_in, int32_t *pos_out,
                    const uint16_t *k_in, int64_t k_stride_tok, int64_t k_stride_head,
                    uint16_t *k_out, int64_t ko_stride_tok, int64_t ko_stride_head,
                    const uint16_t *v_in, int64_t v_stride_tok, int64_t v_stride_head,
                    uint16_t *v_out, int64_t vo_stride_tok, int64_t vo_stride_head) {
    for (int b = 0; b < batch; ++b) {
        for (int32_t i = cu_keep[b]; i < cu_keep[b + 1]; ++i) {
            const int64_t src = global_index ? (int64_t)keep_idx[i] : (int64_t)cu_seqlens[b] + keep_idx[i];
            if (hidden_in && hidden_out)
                memcpy(hidden_out + (int64_t)i * hidden, hidden_in + src * hidden, (size_t)hidden * sizeof(uint16_t));
            if (pos_in && pos_out) pos_out[i] = pos_in[src];
            for (int g = 0; g < num_kv_heads; ++g) {
                if (k_in && k_out)
                    memcpy(k_out + (int64_t)i * ko_stride_tok + (int64_t)g * ko_stride_head,
                           k_in + src * k_stride_tok + (int64_t)g * k_stride_head,
                           (size_t)head_dim * sizeof(uint16_t));
                if (v_in && v_out)
                    memcpy(v_out + (int64_t)i * vo_stride_tok + (int64_t)g * vo_stride_head,
                           v_in + src * v_stride_tok + (int64_t)g * v_stride_head,
                           (size_t)head_dim * sizeof(uint16_t));
            }
        }
    }
}
