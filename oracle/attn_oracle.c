/*
 * attn_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A slow, plain, double-precision CPU statement of scaled-dot-product attention,
 *
 *     O = softmax(Q K^T * scale [+ causal mask]) V          (paper, Section 2.2,
 *                                                            "Attention computation")
 *
 * plus the per-row log-sum-exp of the scaled, visible scores.  The paper's tiled
 * "running maximum / running sum" formulation is only a faster route to this same
 * value, so this file writes out the definition itself: all scores of one query
 * row, their maximum, the exponentials, the sum, the weighted average of V rows.
 * Nothing is blocked, fused, reordered or approximated.
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call this.
 * It shares no code, header, table or constant with the CUDA library.
 *
 * Conventions (the paper fixes none of them; they are the library's documented ones):
 *   - Q [B, Sq, Hq, D], K and V [B, Sk, Hkv, D], D innermost, BF16 bit patterns
 *     (uint16: the upper half of the IEEE-754 binary32 pattern).
 *   - query head hq reads key/value head hq / (Hq / Hkv)  (grouped-query attention,
 *     Section 4.3: consecutive query heads share one KV head).
 *   - causal != 0: key j is visible to query i iff j <= i + (Sk - Sq)
 *     (lower-triangular for Sq == Sk, Section 4.1 "causal masking").
 *   - LSE is the natural log of the sum of exp(scale * q.k_j) over visible keys.
 *   - A row with no visible key gives O = 0 and LSE = -inf.
 *
 * Parity pins for every function here live in tests/test_oracle_pins.py.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_double(uint16_t bits)
{
    uint32_t w = (uint32_t)bits << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/* number of visible keys of query row i (they are always keys 0 .. n-1) */
static int64_t visible_keys(int64_t i, int64_t Sq, int64_t Sk, int causal)
{
    if (!causal) return Sk;
    int64_t n = i + (Sk - Sq) + 1;
    if (n < 0) n = 0;
    if (n > Sk) n = Sk;
    return n;
}

/*
 * One query row.  `s` is caller-provided scratch of Sk doubles; on return s[j]
 * holds the normalised weight p_j for visible j and 0 for masked j.
 * o_row: D doubles.  Returns the row's LSE.
 */
static double one_row(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                      int64_t Hq, int64_t Hkv, int64_t Sq, int64_t Sk, int64_t D,
                      int causal, double scale,
                      int64_t b, int64_t hq, int64_t i,
                      double *s, double *o_row)
{
    const int64_t g = Hq / Hkv;
    const int64_t hkv = hq / g;
    const int64_t nvis = visible_keys(i, Sq, Sk, causal);
    const uint16_t *qrow = q + ((b * Sq + i) * Hq + hq) * D;

    for (int64_t d = 0; d < D; ++d) o_row[d] = 0.0;
    for (int64_t j = 0; j < Sk; ++j) s[j] = 0.0;
    if (nvis == 0) return -INFINITY;

    /* scores s_j = scale * <q_i, k_j> */
    double m = -INFINITY;
    for (int64_t j = 0; j < nvis; ++j) {
        const uint16_t *krow = k + ((b * Sk + j) * Hkv + hkv) * D;
        double acc = 0.0;
        for (int64_t d = 0; d < D; ++d)
            acc += bf16_to_double(qrow[d]) * bf16_to_double(krow[d]);
        s[j] = scale * acc;
        if (s[j] > m) m = s[j];
    }
    /* softmax over the visible keys */
    double l = 0.0;
    for (int64_t j = 0; j < nvis; ++j) {
        s[j] = exp(s[j] - m);
        l += s[j];
    }
    for (int64_t j = 0; j < nvis; ++j) s[j] /= l;
    /* O_i = sum_j p_j v_j */
    for (int64_t j = 0; j < nvis; ++j) {
        const uint16_t *vrow = v + ((b * Sk + j) * Hkv + hkv) * D;
        for (int64_t d = 0; d < D; ++d)
            o_row[d] += s[j] * bf16_to_double(vrow[d]);
    }
    return m + log(l);
}

static int check_shape(int64_t B, int64_t Hq, int64_t Hkv, int64_t Sq, int64_t Sk, int64_t D)
{
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || D <= 0) return 1;
    if (Hq % Hkv != 0) return 1;
    return 0;
}

/*
 * Selected rows.  rows = n_rows triples (b, hq, i).  o: [n_rows, D] doubles,
 * lse: [n_rows] doubles.  Returns 0, or 1 on a bad shape / index, 2 on allocation
 * failure.
 */
int attn_oracle_rows(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                     int64_t B, int64_t Hq, int64_t Hkv, int64_t Sq, int64_t Sk, int64_t D,
                     int causal, float scale,
                     const int32_t *rows, int64_t n_rows,
                     double *o, double *lse, int n_threads)
{
    if (check_shape(B, Hq, Hkv, Sq, Sk, D) || n_rows < 0) return 1;
    for (int64_t r = 0; r < n_rows; ++r) {
        if (rows[3 * r] < 0 || rows[3 * r] >= B || rows[3 * r + 1] < 0 || rows[3 * r + 1] >= Hq ||
            rows[3 * r + 2] < 0 || rows[3 * r + 2] >= Sq)
            return 1;
    }
    if (n_threads < 1) n_threads = 1;
    int failed = 0;
#pragma omp parallel num_threads(n_threads)
    {
        double *s = (double *)malloc((size_t)Sk * sizeof(double));
        if (!s) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 4)
        for (int64_t r = 0; r < n_rows; ++r) {
            if (!s) continue;
            lse[r] = one_row(q, k, v, Hq, Hkv, Sq, Sk, D, causal, (double)scale,
                             rows[3 * r], rows[3 * r + 1], rows[3 * r + 2], s, o + r * D);
        }
        free(s);
    }
    return failed ? 2 : 0;
}

/*
 * Every row.  o: [B, Sq, Hq, D] doubles (same index order as Q), lse: [B, Hq, Sq].
 */
int attn_oracle_full(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                     int64_t B, int64_t Hq, int64_t Hkv, int64_t Sq, int64_t Sk, int64_t D,
                     int causal, float scale,
                     double *o, double *lse, int n_threads)
{
    if (check_shape(B, Hq, Hkv, Sq, Sk, D)) return 1;
    if (n_threads < 1) n_threads = 1;
    int failed = 0;
    const int64_t total = B * Hq * Sq;
#pragma omp parallel num_threads(n_threads)
    {
        double *s = (double *)malloc((size_t)Sk * sizeof(double));
        if (!s) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 16)
        for (int64_t r = 0; r < total; ++r) {
            if (!s) continue;
            const int64_t i = r % Sq;
            const int64_t hq = (r / Sq) % Hq;
            const int64_t b = r / (Sq * Hq);
            lse[(b * Hq + hq) * Sq + i] =
                one_row(q, k, v, Hq, Hkv, Sq, Sk, D, causal, (double)scale, b, hq, i, s,
                        o + ((b * Sq + i) * Hq + hq) * D);
        }
        free(s);
    }
    return failed ? 2 : 0;
}

/*
 * The normalised softmax weights p_j (Sk doubles, 0 where masked) of one row:
 * lets a test check that they are a probability vector.
 */
int attn_oracle_weights(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                        int64_t B, int64_t Hq, int64_t Hkv, int64_t Sq, int64_t Sk, int64_t D,
                        int causal, float scale,
                        int64_t b, int64_t hq, int64_t i, double *p)
{
    if (check_shape(B, Hq, Hkv, Sq, Sk, D)) return 1;
    if (b < 0 || b >= B || hq < 0 || hq >= Hq || i < 0 || i >= Sq) return 1;
    double *o_row = (double *)malloc((size_t)D * sizeof(double));
    if (!o_row) return 2;
    one_row(q, k, v, Hq, Hkv, Sq, Sk, D, causal, (double)scale, b, hq, i, p, o_row);
    free(o_row);
    return 0;
}

/*
 * Merge of two partial attention results over disjoint key sets (the identity behind
 * splitting the key sequence, a direct consequence of the softmax definition in Section 2.2):
 * with LSE = log(exp(LSE1) + exp(LSE2)) and w_i = exp(LSE_i - LSE),  O = w1 O1 + w2 O2.
 * o1, o2: BF16 bit patterns [rows, D]; lse1, lse2: fp32 [rows] (as the GPU library stores them);
 * o: double [rows, D]; lse: double [rows].  A part with LSE = -inf (no visible key) has weight 0;
 * if both parts are empty the row is O = 0, LSE = -inf.
 */
int attn_oracle_merge(const uint16_t *o1, const float *lse1, const uint16_t *o2, const float *lse2,
                      int64_t rows, int64_t D, double *o, double *lse)
{
    if (rows <= 0 || D <= 0) return 1;
    for (int64_t r = 0; r < rows; ++r) {
        const double a = (double)lse1[r], b = (double)lse2[r];
        const double m = a > b ? a : b;
        if (m == -INFINITY) {
            lse[r] = -INFINITY;
            for (int64_t d = 0; d < D; ++d) o[r * D + d] = 0.0;
            continue;
        }
        const double tot = m + log(exp(a - m) + exp(b - m));
        const double w1 = exp(a - tot), w2 = exp(b - tot);
        lse[r] = tot;
        for (int64_t d = 0; d < D; ++d)
            o[r * D + d] = w1 * bf16_to_double(o1[r * D + d]) + w2 * bf16_to_double(o2[r * D + d]);
    }
    return 0;
}

/*
 * Merge of n partial attention results over pairwise disjoint key sets: the same identity
 * applied to n parts at once.  LSE = log(sum_i exp(LSE_i)),  O = sum_i exp(LSE_i - LSE) O_i.
 * o_parts: BF16 bit patterns [n, rows, D]; lse_parts: fp32 [n, rows]; o: double [rows, D];
 * lse: double [rows].  Parts with LSE = -inf have weight 0; if every part is empty the row is
 * O = 0, LSE = -inf.
 */
int attn_oracle_merge_n(const uint16_t *o_parts, const float *lse_parts, int64_t n, int64_t rows, int64_t D,
                        double *o, double *lse)
{
    if (n <= 0 || rows <= 0 || D <= 0) return 1;
    for (int64_t r = 0; r < rows; ++r) {
        double m = -INFINITY;
        for (int64_t i = 0; i < n; ++i) {
            const double a = (double)lse_parts[i * rows + r];
            if (a > m) m = a;
        }
        for (int64_t d = 0; d < D; ++d) o[r * D + d] = 0.0;
        if (m == -INFINITY) {
            lse[r] = -INFINITY;
            continue;
        }
        double sum = 0.0;
        for (int64_t i = 0; i < n; ++i) sum += exp((double)lse_parts[i * rows + r] - m);
        const double tot = m + log(sum);
        lse[r] = tot;
        for (int64_t i = 0; i < n; ++i) {
            const double w = exp((double)lse_parts[i * rows + r] - tot);
            if (w == 0.0) continue;
            for (int64_t d = 0; d < D; ++d)
                o[r * D + d] += w * bf16_to_double(o_parts[(i * rows + r) * D + d]);
        }
    }
    return 0;
}
