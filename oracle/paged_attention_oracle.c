/*
 * CPU oracle for one continuous-batching serving iteration over a paged KV
 * cache: KV append followed by grouped-query attention over mixed
 * chunked-prefill and decode sequences.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the correctness reference the CUDA
 * path is compared with and the timed CPU baseline.  Nothing in the product
 * path may call it, and it shares no code with the CUDA sources.
 *
 * The paper models this operator only through its cost (App. B, Eq.
 * "serve-latency": a decode step k attends a context of k tokens including
 * the new one; prefill is the longer-query operation; Eq. "roofline" gives its
 * time) and names paged KV memory and chunked prefill as the data-plane
 * techniques of the served systems (App. H).  It does not print the operator,
 * so the oracle is the textbook definition of scaled-dot-product attention
 * written out, evaluated in fp64 on exactly widened bf16 inputs:
 *
 *   append:    position p = ctx_len - q_len + t of sequence s lives in
 *              page  = block_table[s][p div 16], slot = p mod 16;
 *              K[page][kv_head][slot][:] <- k_new[row][kv_head][:]  (bit copy)
 *   page copy: page src_ids[i] (all kv heads, K and V) -> page dst_ids[i], all
 *              pairs at once (KV-cache migration between plans, Sec. 5.1 Phase 2)
 *   attention: query row (s,t), q head h, kv head g = h div (Hq/Hkv):
 *              x_j = scale * <q, k_j>  for j = 0..p   (causal bound j <= p)
 *              m = max_j x_j,  l = sum_j exp(x_j - m)
 *              out = sum_j exp(x_j - m) v_j / l,   lse = m + ln l
 *
 * No tiling, no online softmax, no splitting: one (s,t,h) at a time, three
 * passes over j.  OpenMP only distributes independent (sequence, head) pairs.
 *
 * Pins (tests/test_oracle_pins.py): dense brute force on contiguous tensors,
 * softmax rows summing to 1, single-token context returning V, identical
 * keys returning the mean of V, q = 0 giving lse = ln(p+1), page-permutation
 * invariance, split/merge identity, chunking identity, append replay; for the
 * page copy: attention unchanged after moving every page to another pool and
 * remapping the block tables, numpy's simultaneous gather/scatter, refusals.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_PAGE 16

/* exact widening: bf16 is the upper half of an IEEE-754 binary32 */
static double bf16_to_f64(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* element offset of (page, kv_head, slot, 0) in a [num_pages][Hkv][16][d] plane */
static size_t pool_off(int64_t page, int kv_head, int slot, int Hkv, int d)
{
    return (((size_t)page * Hkv + kv_head) * ORACLE_PAGE + slot) * (size_t)d;
}

/*
 * KV append.  Returns 0, or -1 if a needed block-table entry is outside
 * [0, num_pages) or a length is inconsistent (nothing is written for that row).
 */
int oracle_kv_append(uint16_t *K, uint16_t *V, int num_pages, int Hkv, int d,
                     int B, const int32_t *q_lens, const int32_t *ctx_lens,
                     const int32_t *block_tables, int table_stride,
                     const uint16_t *k_new, const uint16_t *v_new)
{
    int rc = 0;
    size_t row = 0;
    for (int s = 0; s < B; ++s) {
        for (int t = 0; t < q_lens[s]; ++t, ++row) {
            int p = ctx_lens[s] - q_lens[s] + t;
            if (p < 0 || p / ORACLE_PAGE >= table_stride) { rc = -1; continue; }
            int32_t page = block_tables[(size_t)s * table_stride + p / ORACLE_PAGE];
            int slot = p % ORACLE_PAGE;
            if (page < 0 || page >= num_pages) { rc = -1; continue; }
            for (int g = 0; g < Hkv; ++g) {
                size_t dst = pool_off(page, g, slot, Hkv, d);
                size_t src = (row * Hkv + g) * (size_t)d;
                memcpy(K + dst, k_new + src, (size_t)d * sizeof(uint16_t));
                memcpy(V + dst, v_new + src, (size_t)d * sizeof(uint16_t));
            }
        }
    }
    return rc;
}

/*
 * KV page copy (Sec. 5.1, execution model, Phase 2 "Reconfiguration": the transition between two
 * plans migrates KV caches; a page is the unit that moves).  For i = 0..n-1 the
 * whole page src_ids[i] of the source planes -- every kv head, every slot, both
 * K and V -- is copied bit for bit to page dst_ids[i] of the destination
 * planes.  All sources are read before any destination is written (the copies
 * are simultaneous: a page may be both a source and another pair's
 * destination), so the result does not depend on the order of the pairs.
 * Returns 0, or -1 (nothing written) if an id is out of range or a destination
 * appears twice.  The planes may be the same (copy inside one pool).
 */
int oracle_copy_pages(uint16_t *K_dst, uint16_t *V_dst, int num_pages_dst,
                      const uint16_t *K_src, const uint16_t *V_src, int num_pages_src,
                      int Hkv, int d, int n, const int32_t *dst_ids, const int32_t *src_ids)
{
    const size_t page_elems = (size_t)Hkv * ORACLE_PAGE * (size_t)d;
    for (int i = 0; i < n; ++i) {
        if (dst_ids[i] < 0 || dst_ids[i] >= num_pages_dst) return -1;
        if (src_ids[i] < 0 || src_ids[i] >= num_pages_src) return -1;
        for (int j = 0; j < i; ++j)
            if (dst_ids[j] == dst_ids[i]) return -1;
    }
    if (n <= 0) return 0;
    uint16_t *tmp = (uint16_t *)malloc(2 * (size_t)n * page_elems * sizeof(uint16_t));
    if (!tmp) return -1;
    for (int i = 0; i < n; ++i) {
        memcpy(tmp + (2 * (size_t)i) * page_elems, K_src + (size_t)src_ids[i] * page_elems, page_elems * sizeof(uint16_t));
        memcpy(tmp + (2 * (size_t)i + 1) * page_elems, V_src + (size_t)src_ids[i] * page_elems, page_elems * sizeof(uint16_t));
    }
    for (int i = 0; i < n; ++i) {
        memcpy(K_dst + (size_t)dst_ids[i] * page_elems, tmp + (2 * (size_t)i) * page_elems, page_elems * sizeof(uint16_t));
        memcpy(V_dst + (size_t)dst_ids[i] * page_elems, tmp + (2 * (size_t)i + 1) * page_elems, page_elems * sizeof(uint16_t));
    }
    free(tmp);
    return 0;
}

/*
 * Attention of one query vector over keys 0..p of one sequence.
 * qv: d bf16 values; bt: that sequence's block-table row; x: scratch of p+1 doubles.
 * Optionally returns the softmax weights in x (normalised), for the row-sum pin.
 */
static void attend_one(const uint16_t *K, const uint16_t *V, int Hkv, int d,
                       const int32_t *bt, int p, const uint16_t *qv, int g,
                       double scale, double *x, double *out, double *lse)
{
    double m = -INFINITY;
    for (int j = 0; j <= p; ++j) {
        const uint16_t *kj = K + pool_off(bt[j / ORACLE_PAGE], g, j % ORACLE_PAGE, Hkv, d);
        double dot = 0.0;
        for (int c = 0; c < d; ++c) dot += bf16_to_f64(qv[c]) * bf16_to_f64(kj[c]);
        x[j] = scale * dot;
        if (x[j] > m) m = x[j];
    }
    double l = 0.0;
    for (int j = 0; j <= p; ++j) { x[j] = exp(x[j] - m); l += x[j]; }
    for (int c = 0; c < d; ++c) out[c] = 0.0;
    for (int j = 0; j <= p; ++j) {
        const uint16_t *vj = V + pool_off(bt[j / ORACLE_PAGE], g, j % ORACLE_PAGE, Hkv, d);
        for (int c = 0; c < d; ++c) out[c] += x[j] * bf16_to_f64(vj[c]);
    }
    for (int c = 0; c < d; ++c) out[c] /= l;
    for (int j = 0; j <= p; ++j) x[j] /= l;
    *lse = m + log(l);
}

/*
 * Attention for every new token of the batch.
 * q: [N_new][Hq][d] bf16; out: [N_new][Hq][d] fp64; lse: [N_new][Hq] fp64.
 * scale <= 0 selects 1/sqrt(d).  Pool planes must already contain the
 * iteration's appended tokens.
 */
void oracle_attention(const uint16_t *K, const uint16_t *V, int Hkv, int d, int Hq,
                      int B, const int32_t *q_lens, const int32_t *ctx_lens,
                      const int32_t *block_tables, int table_stride,
                      const uint16_t *q, double scale, double *out, double *lse)
{
    if (scale <= 0.0) scale = 1.0 / sqrt((double)d);
    int G = Hq / Hkv;
    int64_t *row0 = (int64_t *)malloc(sizeof(int64_t) * (size_t)(B + 1));
    row0[0] = 0;
    int max_ctx = 1;
    for (int s = 0; s < B; ++s) {
        row0[s + 1] = row0[s] + q_lens[s];
        if (ctx_lens[s] > max_ctx) max_ctx = ctx_lens[s];
    }
#pragma omp parallel
    {
        double *x = (double *)malloc(sizeof(double) * (size_t)max_ctx);
#pragma omp for collapse(2) schedule(dynamic, 1)
        for (int s = 0; s < B; ++s) {
            for (int h = 0; h < Hq; ++h) {
                const int32_t *bt = block_tables + (size_t)s * table_stride;
                for (int t = 0; t < q_lens[s]; ++t) {
                    int64_t row = row0[s] + t;
                    int p = ctx_lens[s] - q_lens[s] + t;
                    size_t o = ((size_t)row * Hq + h);
                    attend_one(K, V, Hkv, d, bt, p, q + o * d, h / G, scale, x,
                               out + o * d, lse + o);
                }
            }
        }
        free(x);
    }
    free(row0);
}

/*
 * Attention for selected outputs only: sample i is (sequence seq[i], new-token
 * index tok[i], q head head[i]); out: [n][d], lse: [n].  Used where the whole
 * batch is too large to evaluate on the CPU.
 */
void oracle_attention_samples(const uint16_t *K, const uint16_t *V, int Hkv, int d, int Hq,
                              int B, const int32_t *q_lens, const int32_t *ctx_lens,
                              const int32_t *block_tables, int table_stride,
                              const uint16_t *q, double scale,
                              int n, const int32_t *seq, const int32_t *tok, const int32_t *head,
                              double *out, double *lse)
{
    if (scale <= 0.0) scale = 1.0 / sqrt((double)d);
    int G = Hq / Hkv;
    int64_t *row0 = (int64_t *)malloc(sizeof(int64_t) * (size_t)(B + 1));
    row0[0] = 0;
    int max_ctx = 1;
    for (int s = 0; s < B; ++s) {
        row0[s + 1] = row0[s] + q_lens[s];
        if (ctx_lens[s] > max_ctx) max_ctx = ctx_lens[s];
    }
#pragma omp parallel
    {
        double *x = (double *)malloc(sizeof(double) * (size_t)max_ctx);
#pragma omp for schedule(dynamic, 1)
        for (int i = 0; i < n; ++i) {
            int s = seq[i], t = tok[i], h = head[i];
            int p = ctx_lens[s] - q_lens[s] + t;
            size_t o = ((size_t)(row0[s] + t) * Hq + h);
            attend_one(K, V, Hkv, d, block_tables + (size_t)s * table_stride, p,
                       q + o * d, h / G, scale, x, out + (size_t)i * d, lse + i);
        }
        free(x);
    }
    free(row0);
}

/*
 * Softmax weights of one output (normalised, length p+1) -- for the
 * "rows sum to 1" pin.  Returns p+1.
 */
int oracle_softmax_row(const uint16_t *K, const uint16_t *V, int Hkv, int d, int Hq,
                       const int32_t *bt_row, int p, const uint16_t *qv, int head,
                       double scale, double *weights)
{
    if (scale <= 0.0) scale = 1.0 / sqrt((double)d);
    double *out = (double *)malloc(sizeof(double) * (size_t)d);
    double lse;
    attend_one(K, V, Hkv, d, bt_row, p, qv, head / (Hq / Hkv), scale, weights, out, &lse);
    free(out);
    return p + 1;
}

/*
 * Merge of split partial results over disjoint key ranges of the same query:
 *   lse = m* + ln sum_k exp(lse_k - m*),  o = sum_k exp(lse_k - lse) o_k,
 * with m* = max_k lse_k.  o_parts: [n_parts][d] (each normalised), lse_parts: [n_parts].
 */
void oracle_merge_partials(int n_parts, int d, const double *o_parts, const double *lse_parts,
                           double *o, double *lse)
{
    double mstar = -INFINITY;
    for (int k = 0; k < n_parts; ++k) if (lse_parts[k] > mstar) mstar = lse_parts[k];
    double sum = 0.0;
    for (int k = 0; k < n_parts; ++k) sum += exp(lse_parts[k] - mstar);
    *lse = mstar + log(sum);
    for (int c = 0; c < d; ++c) o[c] = 0.0;
    for (int k = 0; k < n_parts; ++k) {
        double w = exp(lse_parts[k] - *lse);
        for (int c = 0; c < d; ++c) o[c] += w * o_parts[(size_t)k * d + c];
    }
}

/*
 * Attention of one query over the key range [j0, j1) only (a split): the same
 * definition restricted to that range.  Used by the split/merge identity pin.
 */
void oracle_attention_range(const uint16_t *K, const uint16_t *V, int Hkv, int d, int Hq,
                            const int32_t *bt_row, int j0, int j1, const uint16_t *qv, int head,
                            double scale, double *out, double *lse)
{
    if (scale <= 0.0) scale = 1.0 / sqrt((double)d);
    int g = head / (Hq / Hkv);
    double m = -INFINITY;
    double *x = (double *)malloc(sizeof(double) * (size_t)(j1 - j0 > 0 ? j1 - j0 : 1));
    for (int j = j0; j < j1; ++j) {
        const uint16_t *kj = K + pool_off(bt_row[j / ORACLE_PAGE], g, j % ORACLE_PAGE, Hkv, d);
        double dot = 0.0;
        for (int c = 0; c < d; ++c) dot += bf16_to_f64(qv[c]) * bf16_to_f64(kj[c]);
        x[j - j0] = scale * dot;
        if (x[j - j0] > m) m = x[j - j0];
    }
    double l = 0.0;
    for (int j = j0; j < j1; ++j) { x[j - j0] = exp(x[j - j0] - m); l += x[j - j0]; }
    for (int c = 0; c < d; ++c) out[c] = 0.0;
    for (int j = j0; j < j1; ++j) {
        const uint16_t *vj = V + pool_off(bt_row[j / ORACLE_PAGE], g, j % ORACLE_PAGE, Hkv, d);
        for (int c = 0; c < d; ++c) out[c] += x[j - j0] * bf16_to_f64(vj[c]);
    }
    for (int c = 0; c < d; ++c) out[c] /= l;
    *lse = m + log(l);
    free(x);
}
