/*
 * CPU oracle for decode-phase sparse MLA attention.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain definition that the CUDA path is checked against.
 * It is never linked into, imported by, or called from the product library; only the
 * test-suite, the smoke check and the benchmark's cpu-baseline leg may use it.  It shares
 * no code, header, table or constant with the CUDA sources.
 *
 * What it computes (paper, "OmniAttn: Problem Formulation", Eq. 1, left-hand side):
 *     softmax(Q K_M^T * scale) V_M
 * i.e. exact attention restricted to the selected index set M, here for one decode query
 * per (request, head).  The paper's Eq. 2 (sink + recent) is one way to build M; this
 * oracle accepts any index list.  The MLA reading (one latent row per token, K = all
 * d_qk columns, V = the first d_v columns, every head of a request sharing M) and the
 * paged cache are the task's shapes; the paper's "Layer-wise Compression" paragraph only
 * says the scheme is MLA-compatible and that all heads of a layer share one pattern.
 *
 * Everything is two-pass fp64: scores, then max, then exp/sum, then the weighted sum.
 * No tiling, no online recurrence, no fusion.  bf16 inputs are widened exactly.
 * The working type of oracle_attend_rows is the typedef `real` (double unless the file is
 * compiled with -DORACLE_REAL=float): the fp64 build is the oracle every test compares with;
 * the float build of the same source exists only to be timed as the "plain fp32 CPU" figure
 * of the benchmark and is never used as a reference.
 *
 * Parity status of each exported function (pins live in tests/test_oracle_pins.py):
 *   oracle_resolve_rows      pinned (hand-written tables, histogram/spike constructions)
 *   oracle_attend_rows       pinned (library dense attention, brute force, closed forms)
 *   oracle_sparse_mla_decode pinned (composition of the two above + relabel invariance)
 *   oracle_splitkv_combine   pinned (any partition merges to the unsplit result)
 * The paper's quality claim (sparse ~ dense on a trained model) is NOT pinned: parity
 * unpinned for that claim; it needs trained weights and evaluation suites.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#ifndef ORACLE_REAL
#define ORACLE_REAL double
#endif
typedef ORACLE_REAL real;

/* bf16 bit pattern -> double, exact (bf16 is the top half of an IEEE-754 binary32). */
static double bf16_to_double(uint16_t bits)
{
    uint32_t w = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/*
 * Index resolution: logical token position -> physical row of the paged pool.
 *   row = page_table[b][t / page_size] * page_size + t % page_size
 * rows[b][j] is written for j < sel_len[b]; entries beyond are set to -1.
 * Returns 0, or a 1-based count of contract violations (negative / out-of-range token
 * position, page id outside the pool, sel_len outside [0,max_sel]); violating entries
 * resolve to -1 and the caller must treat that as a failed precondition.
 */
int oracle_resolve_rows(int batch, int page_size, int64_t num_pages, int max_pages_per_req,
                        int max_sel, const int32_t *page_table, const int32_t *sel_idx,
                        const int32_t *sel_len, int64_t *rows)
{
    int bad = 0;
    for (int b = 0; b < batch; ++b) {
        int n = sel_len[b];
        if (n < 0 || n > max_sel) {
            ++bad;
            n = 0;
        }
        for (int j = 0; j < max_sel; ++j) {
            int64_t r = -1;
            if (j < n) {
                int32_t t = sel_idx[(size_t)b * max_sel + j];
                if (t < 0 || t / page_size >= max_pages_per_req) {
                    ++bad;
                } else {
                    int32_t page = page_table[(size_t)b * max_pages_per_req + t / page_size];
                    if (page < 0 || (int64_t)page >= num_pages)
                        ++bad;
                    else
                        r = (int64_t)page * page_size + t % page_size;
                }
            }
            rows[(size_t)b * max_sel + j] = r;
        }
    }
    return bad;
}

/*
 * Attention over already-gathered rows.
 *   q      bf16 bits [batch, heads, d_qk]
 *   krows  bf16 bits [batch, max_sel, d_qk]   (row j of request b = the latent row of its
 *                                              j-th selected token; V = first d_v columns)
 *   n[b]   number of valid rows of request b
 *   out    fp64 [batch, heads, d_v],  lse fp64 [batch, heads] (natural log of scaled scores)
 *   wsum   optional fp64 [batch, heads]: sum of the softmax weights (should be 1)
 * n[b] == 0 gives out = 0 and lse = -inf.
 */
void oracle_attend_rows(int batch, int heads, int d_qk, int d_v, int max_sel, double scale,
                        const uint16_t *q, const uint16_t *krows, const int32_t *n,
                        double *out, double *lse, double *wsum)
{
    const long total = (long)batch * heads;
#pragma omp parallel
    {
        real *x = (real *)malloc(sizeof(real) * (size_t)(max_sel > 0 ? max_sel : 1));
        real *qd = (real *)malloc(sizeof(real) * (size_t)d_qk);
        real *oa = (real *)malloc(sizeof(real) * (size_t)(d_v > 0 ? d_v : 1));
#pragma omp for schedule(dynamic, 1)
        for (long bh = 0; bh < total; ++bh) {
            const int b = (int)(bh / heads);
            const int nb = n[b];
            double *o = out + (size_t)bh * d_v;
            for (int d = 0; d < d_v; ++d)
                oa[d] = (real)0.0;
            if (nb <= 0) {
                for (int d = 0; d < d_v; ++d)
                    o[d] = 0.0;
                lse[bh] = -INFINITY;
                if (wsum)
                    wsum[bh] = 0.0;
                continue;
            }
            for (int c = 0; c < d_qk; ++c)
                qd[c] = (real)bf16_to_double(q[(size_t)bh * d_qk + c]);
            const uint16_t *kb = krows + (size_t)b * max_sel * d_qk;
            /* pass 1: scaled scores x_j = scale * <q, k_j> */
            for (int j = 0; j < nb; ++j) {
                const uint16_t *k = kb + (size_t)j * d_qk;
                real acc = (real)0.0;
                for (int c = 0; c < d_qk; ++c)
                    acc += qd[c] * (real)bf16_to_double(k[c]);
                x[j] = (real)scale * acc;
            }
            /* pass 2: max, partition function */
            real m = x[0];
            for (int j = 1; j < nb; ++j)
                if (x[j] > m)
                    m = x[j];
            real z = (real)0.0;
            for (int j = 0; j < nb; ++j)
                z += (real)exp((double)(x[j] - m));
            lse[bh] = (double)(m + (real)log((double)z));
            /* pass 3: weighted sum of the value part of each row */
            real ws = (real)0.0;
            for (int j = 0; j < nb; ++j) {
                const real w = (real)exp((double)(x[j] - m)) / z;
                ws += w;
                const uint16_t *v = kb + (size_t)j * d_qk;
                for (int d = 0; d < d_v; ++d)
                    oa[d] += w * (real)bf16_to_double(v[d]);
            }
            for (int d = 0; d < d_v; ++d)
                o[d] = (double)oa[d];
            if (wsum)
                wsum[bh] = (double)ws;
        }
        free(x);
        free(qd);
        free(oa);
    }
}

/*
 * Full path on a host-resident pool: resolve, gather, attend.
 *   kv_cache bf16 bits [num_pages, page_size, d_qk]
 * rows_out (optional) receives the resolved physical rows [batch, max_sel].
 * Returns the violation count of oracle_resolve_rows (nothing is computed if non-zero).
 */
int oracle_sparse_mla_decode(int batch, int heads, int d_qk, int d_v, int page_size,
                             int64_t num_pages, int max_pages_per_req, int max_sel,
                             double scale, const uint16_t *q, const uint16_t *kv_cache,
                             const int32_t *page_table, const int32_t *sel_idx,
                             const int32_t *sel_len, double *out, double *lse,
                             int64_t *rows_out)
{
    const size_t nrows = (size_t)batch * (size_t)(max_sel > 0 ? max_sel : 1);
    int64_t *rows = (int64_t *)malloc(sizeof(int64_t) * nrows);
    int bad = oracle_resolve_rows(batch, page_size, num_pages, max_pages_per_req, max_sel,
                                  page_table, sel_idx, sel_len, rows);
    if (rows_out)
        memcpy(rows_out, rows, sizeof(int64_t) * (size_t)batch * max_sel);
    if (bad) {
        free(rows);
        return bad;
    }
    uint16_t *krows = (uint16_t *)calloc(nrows * (size_t)d_qk, sizeof(uint16_t));
    for (int b = 0; b < batch; ++b)
        for (int j = 0; j < sel_len[b]; ++j)
            memcpy(krows + ((size_t)b * max_sel + j) * d_qk,
                   kv_cache + (size_t)rows[(size_t)b * max_sel + j] * d_qk,
                   sizeof(uint16_t) * (size_t)d_qk);
    oracle_attend_rows(batch, heads, d_qk, d_v, max_sel, scale, q, krows, sel_len, out, lse,
                       NULL);
    free(krows);
    free(rows);
    return 0;
}

/*
 * Merge of split-KV partial results (each partial normalised by its own partition
 * function, carrying its own log-sum-exp):
 *   lse = m* + ln sum_s exp(lse_s - m*),  out = sum_s exp(lse_s - lse) * out_s
 * part_out fp64 [batch, max_splits, heads, d_v], part_lse fp64 [batch, max_splits, heads],
 * num_splits[b] in [0, max_splits].  A partial with lse = -inf has weight 0; if every
 * partial is empty the result is out = 0, lse = -inf.
 */
void oracle_splitkv_combine(int batch, int heads, int d_v, int max_splits,
                            const double *part_out, const double *part_lse,
                            const int32_t *num_splits, double *out, double *lse)
{
    for (int b = 0; b < batch; ++b)
        for (int h = 0; h < heads; ++h) {
            const int ns = num_splits[b];
            double m = -INFINITY;
            for (int s = 0; s < ns; ++s) {
                double l = part_lse[((size_t)b * max_splits + s) * heads + h];
                if (l > m)
                    m = l;
            }
            double *o = out + ((size_t)b * heads + h) * d_v;
            for (int d = 0; d < d_v; ++d)
                o[d] = 0.0;
            if (m == -INFINITY) {
                lse[(size_t)b * heads + h] = -INFINITY;
                continue;
            }
            double z = 0.0;
            for (int s = 0; s < ns; ++s)
                z += exp(part_lse[((size_t)b * max_splits + s) * heads + h] - m);
            const double L = m + log(z);
            lse[(size_t)b * heads + h] = L;
            for (int s = 0; s < ns; ++s) {
                const double l = part_lse[((size_t)b * max_splits + s) * heads + h];
                if (l == -INFINITY)
                    continue;
                const double w = exp(l - L);
                const double *po = part_out + (((size_t)b * max_splits + s) * heads + h) * d_v;
                for (int d = 0; d < d_v; ++d)
                    o[d] += w * po[d];
            }
        }
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
