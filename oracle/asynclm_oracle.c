/*
 * CPU oracle for one AsyncLM serving step: interrupt append + mixed attention over a paged KV pool.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA library is checked
 * against.  It shares no code, headers, tables or helpers with the CUDA path and must never be
 * called from it.
 *
 * What it follows.  The paper (Section 3.2, "Triggering Interrupts"; Section 5.3, "Interrupt
 * Manager") states that an interrupt block is inserted at the end of a sequence's token stream and
 * that those tokens are processed by the LLM in the next decoding step, while the other sequences
 * keep decoding; Section 5.5 describes the alternative that discards the session and recomputes
 * the whole context.  At the attention layer that means, for each sequence b with ctx_b tokens
 * already cached and q_b new tokens this step:
 *
 *   1. append:  new row i (0 <= i < q_b) is stored at position pos = ctx_b + i of the sequence,
 *               i.e. in physical page page_indices[page_indptr[b] + pos / P], slot pos % P;
 *   2. attend:  new row i sees keys 0 .. ctx_b + i (all prior context, causal inside the span):
 *               o = softmax(q . K^T / sqrt(d)) . V, per query head, with query heads
 *               [h*G, (h+1)*G) sharing kv head h.
 *
 * Everything is the textbook definition in fp64: two-pass softmax, no tiling, no online update, no
 * chunking.  bf16 inputs are widened exactly.
 *
 * Layouts (all row-major, bf16 as uint16 bit patterns):
 *   kv_pool [num_pages][2 (0=K,1=V)][Hkv][P][d]
 *   q       [T][Hq][d]        k_new, v_new [T][Hkv][d]
 *   out     [T][Hq][d] fp64   lse [T][Hq] fp64 (natural log)
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_f64(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* address of the d-element row of (page, K|V, kv head, slot) inside the pool */
static size_t pool_row(int64_t page, int which, int h, int slot, int Hkv, int P, int d)
{
    return ((((size_t)page * 2 + (size_t)which) * (size_t)Hkv + (size_t)h) * (size_t)P
            + (size_t)slot) * (size_t)d;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Step 1 (append).  Bit copy of every new K row and V row into its page slot.  Returns 0, or -1 if
 * a page index falls outside the sequence's page list or the pool.
 */
int oracle_kv_append(int Hkv, int d, int P, int64_t num_pages, int batch,
                     const int32_t *q_indptr, const int32_t *kv_len_before,
                     const int32_t *page_indptr, const int32_t *page_indices,
                     const uint16_t *k_new, const uint16_t *v_new, uint16_t *kv_pool)
{
    for (int b = 0; b < batch; ++b) {
        int q_b = q_indptr[b + 1] - q_indptr[b];
        for (int i = 0; i < q_b; ++i) {
            int pos = kv_len_before[b] + i;
            int lp = pos / P;
            if (page_indptr[b] + lp >= page_indptr[b + 1]) return -1;
            int64_t pg = page_indices[page_indptr[b] + lp];
            if (pg < 0 || pg >= num_pages) return -1;
            size_t r = (size_t)(q_indptr[b] + i);
            for (int h = 0; h < Hkv; ++h) {
                const uint16_t *ks = k_new + (r * (size_t)Hkv + (size_t)h) * (size_t)d;
                const uint16_t *vs = v_new + (r * (size_t)Hkv + (size_t)h) * (size_t)d;
                memcpy(kv_pool + pool_row(pg, 0, h, pos % P, Hkv, P, d), ks, (size_t)d * 2);
                memcpy(kv_pool + pool_row(pg, 1, h, pos % P, Hkv, P, d), vs, (size_t)d * 2);
            }
        }
    }
    return 0;
}

/*
 * Step 2 (attend) for one (token row, query head).  n keys are visible.  scores is scratch [n].
 */
static void attend_row(int Hkv, int d, int P, const int32_t *pages, const uint16_t *kv_pool,
                       const uint16_t *qrow, int hkv, int n, double scale, double *scores,
                       double *o, double *lse)
{
    double m = -INFINITY;
    for (int j = 0; j < n; ++j) {
        const uint16_t *krow = kv_pool + pool_row(pages[j / P], 0, hkv, j % P, Hkv, P, d);
        double s = 0.0;
        for (int t = 0; t < d; ++t) s += bf16_to_f64(qrow[t]) * bf16_to_f64(krow[t]);
        s *= scale;
        scores[j] = s;
        if (s > m) m = s;
    }
    double Z = 0.0;
    for (int j = 0; j < n; ++j) {
        scores[j] = exp(scores[j] - m);
        Z += scores[j];
    }
    for (int t = 0; t < d; ++t) o[t] = 0.0;
    for (int j = 0; j < n; ++j) {
        const uint16_t *vrow = kv_pool + pool_row(pages[j / P], 1, hkv, j % P, Hkv, P, d);
        double p = scores[j];
        for (int t = 0; t < d; ++t) o[t] += p * bf16_to_f64(vrow[t]);
    }
    for (int t = 0; t < d; ++t) o[t] /= Z;
    *lse = m + log(Z);
}

/*
 * Step 2 over a batch.  The pool must already hold the appended rows.  sm_scale <= 0 selects
 * 1/sqrt(d).  If n_sel > 0 only the token rows listed in sel_rows are computed (the others are left
 * untouched); otherwise all T rows.  Returns 0 on success.
 */
int oracle_attn_mixed(int Hq, int Hkv, int d, int P, int batch,
                      const int32_t *q_indptr, const int32_t *kv_len_before,
                      const int32_t *page_indptr, const int32_t *page_indices,
                      const uint16_t *q, const uint16_t *kv_pool, double sm_scale,
                      int n_sel, const int32_t *sel_rows, double *out, double *lse)
{
    const int G = Hq / Hkv;
    const int T = q_indptr[batch];
    const double scale = sm_scale > 0.0 ? sm_scale : 1.0 / sqrt((double)d);
    /* row -> sequence map */
    int32_t *row_seq = (int32_t *)malloc(sizeof(int32_t) * (size_t)(T > 0 ? T : 1));
    if (!row_seq) return -2;
    int max_n = 1;
    for (int b = 0; b < batch; ++b) {
        for (int r = q_indptr[b]; r < q_indptr[b + 1]; ++r) row_seq[r] = b;
        int n_b = kv_len_before[b] + (q_indptr[b + 1] - q_indptr[b]);
        if (n_b > max_n) max_n = n_b;
    }
    const long n_rows = n_sel > 0 ? n_sel : T;
    const long n_work = n_rows * Hq;
    int fail = 0;
#pragma omp parallel
    {
        double *scores = (double *)malloc(sizeof(double) * (size_t)max_n);
        if (!scores) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp for schedule(dynamic, 1)
        for (long w = 0; w < n_work; ++w) {
            if (!scores) continue;
            int r = n_sel > 0 ? sel_rows[w / Hq] : (int)(w / Hq);
            int hq = (int)(w % Hq);
            int b = row_seq[r];
            int i = r - q_indptr[b];
            int n = kv_len_before[b] + i + 1;
            size_t qo = ((size_t)r * (size_t)Hq + (size_t)hq) * (size_t)d;
            attend_row(Hkv, d, P, page_indices + page_indptr[b], kv_pool, q + qo, hq / G, n, scale,
                       scores, out + qo, lse + (size_t)r * (size_t)Hq + (size_t)hq);
        }
        free(scores);
    }
    free(row_seq);
    return fail ? -2 : 0;
}
