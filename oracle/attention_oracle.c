/*
 * Reference oracle for scaled dot-product attention (TEST INFRASTRUCTURE ONLY).
 *
 * This file is a plain, slow, fp64 CPU statement of what the fused attention
 * forward pass computes.  It exists so that tests, the smoke check and the
 * benchmark's cpu_baseline leg can compare the CUDA path against something
 * written directly from the definition.  Nothing on the product path may
 * include, link, import or execute it, and it shares no code with the CUDA
 * kernels.
 *
 * What it follows
 *   - Eq. 1 of the paper: Attention(Q,K,V) = softmax(Q K^T / sqrt(d_k)) V for one
 *     head, with Q in R^{lq x dk}, K in R^{lk x dk}, V in R^{lk x dv}; the
 *     computation is replicated over H heads (Section 2.1).
 *   - Causal mode (the "causal masking" operator of Section 1 and the mask
 *     step of Algorithm 1): key j takes part in query row i only when
 *     j <= i + (Sk - Sq).  For Sq == Sk, the only case the paper runs, this
 *     is "a token sees itself and everything before it".
 *   - Grouped-query attention (Section 4.4): query head hq reads kv head
 *     hq / (Hq / Hkv).
 *   - lse = m + ln(l), the natural-log sum of exponentials of the scaled
 *     scores.  The paper's kernel returns (G', u, s) (Algorithm 1) and divides
 *     at the end; lse is the same information in one number per row.
 *
 * FlashAttention reaches this result exactly up to rounding order, so the
 * oracle is the definition itself: three plain passes per query row (scores
 * and their maximum; exponentials and their sum; weighted sum of V rows).  No
 * tiling, no online recurrence, no exp2, no reordering.
 *
 * Parity pins (tests run without a GPU): a hand-derived 2x2 example with
 * closed-form values, rows of P summing to one, constant V, a single key,
 * Q = 0 closed form, masked entries contributing nothing, shift invariance,
 * key permutation invariance, the split/merge identity, GQA == repeated MHA,
 * the sharp-softmax limit, and brute force against a structurally different
 * numpy implementation on tiny shapes.
 *
 * Layouts (row-major, contiguous): Q [B,Hq,Sq,dqk], K [B,Hkv,Sk,dqk],
 * V [B,Hkv,Sk,dv], O [B,Hq,Sq,dv] (fp64), lse [B,Hq,Sq] (fp64).
 * Rows without any visible key give O = 0 and lse = -inf.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ELEM_F64 = 0, ELEM_BF16 = 1 };

/* bf16 is the upper half of an IEEE binary32: widening is exact. */
static inline double bf16_bits_to_double(uint16_t h) {
    uint32_t w = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

static inline void widen_row(const void *base, size_t off, int n, int kind, double *dst) {
    if (kind == ELEM_F64) {
        const double *p = (const double *)base + off;
        for (int t = 0; t < n; ++t) dst[t] = p[t];
    } else {
        const uint16_t *p = (const uint16_t *)base + off;
        for (int t = 0; t < n; ++t) dst[t] = bf16_bits_to_double(p[t]);
    }
}

/*
 * One query row (b, hq, i).  `scores` is scratch of length Sk, `krow`/`vrow`
 * scratch of length max(dqk, dv), `qrow` of length dqk.  If `p_out` is not
 * NULL it receives the normalised probabilities P[i, 0..Sk) (zeros where
 * masked).
 */
static void attention_row(const void *Q, const void *K, const void *V, int kind,
                          int Hq, int Hkv, int Sq, int Sk, int dqk, int dv,
                          int causal, double scale, int b, int hq, int i,
                          double *o_row, double *lse_out, double *p_out,
                          double *scores, double *qrow, double *kvrow) {
    const int group = Hq / Hkv;
    const int kvh = hq / group;
    /* number of visible keys: all of them, or j <= i + (Sk - Sq) */
    long nvis = Sk;
    if (causal) {
        nvis = (long)i + (long)Sk - (long)Sq + 1;
        if (nvis > Sk) nvis = Sk;
        if (nvis < 0) nvis = 0;
    }
    for (int c = 0; c < dv; ++c) o_row[c] = 0.0;
    if (p_out) for (int j = 0; j < Sk; ++j) p_out[j] = 0.0;
    if (nvis == 0) {
        *lse_out = -INFINITY;
        return;
    }
    const size_t q_off = (((size_t)b * Hq + hq) * Sq + i) * (size_t)dqk;
    const size_t k_base = ((size_t)b * Hkv + kvh) * (size_t)Sk * dqk;
    const size_t v_base = ((size_t)b * Hkv + kvh) * (size_t)Sk * dv;
    widen_row(Q, q_off, dqk, kind, qrow);

    /* pass 1: scaled scores and their maximum */
    double m = -INFINITY;
    for (long j = 0; j < nvis; ++j) {
        widen_row(K, k_base + (size_t)j * dqk, dqk, kind, kvrow);
        double acc = 0.0;
        for (int t = 0; t < dqk; ++t) acc += qrow[t] * kvrow[t];
        const double s = scale * acc;
        scores[j] = s;
        if (s > m) m = s;
    }
    /* pass 2: exponentials relative to the maximum, and their sum */
    double l = 0.0;
    for (long j = 0; j < nvis; ++j) {
        const double e = exp(scores[j] - m);
        scores[j] = e;
        l += e;
    }
    /* pass 3: weighted sum of the value rows, then one division by l */
    for (long j = 0; j < nvis; ++j) {
        widen_row(V, v_base + (size_t)j * dv, dv, kind, kvrow);
        const double w = scores[j];
        for (int c = 0; c < dv; ++c) o_row[c] += w * kvrow[c];
    }
    const double inv_l = 1.0 / l;
    for (int c = 0; c < dv; ++c) o_row[c] *= inv_l;
    *lse_out = m + log(l);
    if (p_out) for (long j = 0; j < nvis; ++j) p_out[j] = scores[j] * inv_l;
}

/*
 * Attention for a list of query rows.
 *   rows    : NULL -> every (b, hq, i) in order, O is [B,Hq,Sq,dv], lse [B,Hq,Sq].
 *             else `n_rows` triples (b, hq, i) as int64; O is [n_rows, dv], lse [n_rows].
 *   kind    : 0 = inputs are fp64, 1 = inputs are bf16 bit patterns (uint16).
 *   threads : <= 0 -> OpenMP default.
 * Returns 0, or a negative number for an invalid argument / failed allocation.
 */
int oracle_attention(const void *Q, const void *K, const void *V, int kind,
                     int B, int Hq, int Hkv, int Sq, int Sk, int dqk, int dv,
                     int causal, double scale,
                     const int64_t *rows, int64_t n_rows,
                     double *O, double *lse, int threads) {
    if (!Q || !K || !V || !O || !lse) return -1;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || dqk <= 0 || dv <= 0) return -2;
    if (Hq % Hkv != 0) return -3;
    if (kind != ELEM_F64 && kind != ELEM_BF16) return -4;
    const int64_t total = rows ? n_rows : (int64_t)B * Hq * Sq;
    if (rows) {
        for (int64_t r = 0; r < n_rows; ++r) {
            const int64_t b = rows[3 * r], h = rows[3 * r + 1], i = rows[3 * r + 2];
            if (b < 0 || b >= B || h < 0 || h >= Hq || i < 0 || i >= Sq) return -5;
        }
    }
    const int dmax = dqk > dv ? dqk : dv;
    int failed = 0;
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#else
    (void)threads;
#endif
#pragma omp parallel
    {
        double *scores = (double *)malloc(sizeof(double) * (size_t)Sk);
        double *qrow = (double *)malloc(sizeof(double) * (size_t)dqk);
        double *kvrow = (double *)malloc(sizeof(double) * (size_t)dmax);
        if (!scores || !qrow || !kvrow) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(dynamic, 16)
            for (int64_t r = 0; r < total; ++r) {
                int b, hq, i;
                if (rows) {
                    b = (int)rows[3 * r]; hq = (int)rows[3 * r + 1]; i = (int)rows[3 * r + 2];
                } else {
                    i = (int)(r % Sq);
                    hq = (int)((r / Sq) % Hq);
                    b = (int)(r / ((int64_t)Sq * Hq));
                }
                attention_row(Q, K, V, kind, Hq, Hkv, Sq, Sk, dqk, dv, causal, scale,
                              b, hq, i, O + (size_t)r * dv, lse + r, NULL,
                              scores, qrow, kvrow);
            }
        }
        free(scores); free(qrow); free(kvrow);
    }
    return failed ? -6 : 0;
}

/* Debug entry: probabilities P[i, 0..Sk) of one row, plus its O row and lse. */
int oracle_attention_prow(const void *Q, const void *K, const void *V, int kind,
                          int B, int Hq, int Hkv, int Sq, int Sk, int dqk, int dv,
                          int causal, double scale, int b, int hq, int i,
                          double *P_row, double *O_row, double *lse) {
    if (!Q || !K || !V || !P_row || !O_row || !lse) return -1;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || dqk <= 0 || dv <= 0) return -2;
    if (Hq % Hkv != 0) return -3;
    if (kind != ELEM_F64 && kind != ELEM_BF16) return -4;
    if (b < 0 || b >= B || hq < 0 || hq >= Hq || i < 0 || i >= Sq) return -5;
    const int dmax = dqk > dv ? dqk : dv;
    double *scores = (double *)malloc(sizeof(double) * (size_t)Sk);
    double *qrow = (double *)malloc(sizeof(double) * (size_t)dqk);
    double *kvrow = (double *)malloc(sizeof(double) * (size_t)dmax);
    int rc = 0;
    if (!scores || !qrow || !kvrow) rc = -6;
    else attention_row(Q, K, V, kind, Hq, Hkv, Sq, Sk, dqk, dv, causal, scale,
                       b, hq, i, O_row, lse, P_row, scores, qrow, kvrow);
    free(scores); free(qrow); free(kvrow);
    return rc;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
