/*
 * CPU oracle for SlimAttention over an INT8 KV cache.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain, double-precision statement of what the GPU
 * library computes.  It exists so that tests can compare the CUDA kernels
 * against it and so that a CPU baseline can be timed beside them.  It shares
 * no code with the CUDA path and nothing in the product may call it.
 *
 * What it follows:
 *   - Quantiser: the INT8 KV cache of Section 2.2, one scale per (token,
 *     kv head), K and V separately.  The paper gives no formula; the
 *     format used is symmetric codes in [-127, 127], scale = absmax / 127 kept
 *     in fp32, round half to even, evaluated on the exact ratio 127*x/absmax.
 *   - Attention: SlimAttention (Section 2.1) computes, for a block of query
 *     rows, the whole score row against all keys, then one softmax over that
 *     row, then the product with V.  No correction terms exist, so the result
 *     is the textbook softmax attention; the oracle is that definition written
 *     row by row, which is also the order Section 2.1 describes.
 *   - Split/merge: the decode kernel splits the key range and merges the
 *     pieces with the log-sum-exp identity; slim_oracle_partial and
 *     slim_oracle_merge state that identity so a test can show it reproduces
 *     the unsplit row.
 *   - Eq. (1): bytes of KV cache touched per generated token.
 *
 * Layout used here (the oracle's own; contiguous, no pages):
 *   x bf16 rows:      [n_rows][D]            uint16 bit patterns
 *   codes:            [L][Hkv][D]            int8
 *   scales:           [L][Hkv]               float
 *   q:                [nq][Hq][D]            uint16 bf16 bit patterns
 *   out:              [n_sel][Hq][D]         double
 *
 * All pins are in tests/test_oracle_*.py: exact rational arithmetic for the
 * quantiser, dense numpy softmax attention on tiny shapes, closed forms
 * (two-key softmax = logistic, equal keys -> mean of V), invariants and a
 * hand-worked three-token example.  No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_double(uint16_t h)
{
    uint32_t w = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/* Quantise n_rows rows of D bf16 values (Section 2.2; one scale per row, a row
 * being one (token, kv-head) of K or of V).
 *   amax  = max_d |x_d|
 *   scale = fl32(amax / 127)
 *   code  = clamp(round_half_even(127 * x_d / amax), -127, 127)
 *   amax == 0 -> scale 0 and all codes 0.
 * 127*x_d is exact in double; the quotient is never within double rounding of
 * a half-integer unless it is exactly one (bf16 significands have 8 bits), so
 * rint() in the default rounding mode gives the exact round-half-even. */
void slim_oracle_quantize(const uint16_t *x, int64_t n_rows, int32_t D,
                          int8_t *codes, float *scales)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < n_rows; ++r) {
        const uint16_t *row = x + r * D;
        double amax = 0.0;
        for (int d = 0; d < D; ++d) {
            double a = fabs(bf16_to_double(row[d]));
            if (a > amax) amax = a;
        }
        if (amax == 0.0) {
            scales[r] = 0.0f;
            for (int d = 0; d < D; ++d) codes[r * D + d] = 0;
            continue;
        }
        scales[r] = (float)(amax / 127.0);
        for (int d = 0; d < D; ++d) {
            double c = rint(127.0 * bf16_to_double(row[d]) / amax);
            if (c > 127.0) c = 127.0;
            if (c < -127.0) c = -127.0;
            codes[r * D + d] = (int8_t)c;
        }
    }
}

/* Dequantised element: (double)code * (double)scale. */
static inline double deq(const int8_t *codes, const float *scales,
                         int64_t tok, int32_t head, int32_t Hkv, int32_t D, int32_t d)
{
    return (double)codes[(tok * Hkv + head) * D + d] * (double)scales[tok * Hkv + head];
}

/* Scores of one query row against keys [j0, j1): s_j = sm_scale * q . k^_j. */
static void score_row(const uint16_t *qrow, const int8_t *kc, const float *ks,
                      int64_t j0, int64_t j1, int32_t g, int32_t Hkv, int32_t D,
                      double sm_scale, double *s)
{
    for (int64_t j = j0; j < j1; ++j) {
        double acc = 0.0;
        for (int d = 0; d < D; ++d)
            acc += bf16_to_double(qrow[d]) * deq(kc, ks, j, g, Hkv, D, d);
        s[j - j0] = sm_scale * acc;
    }
}

/* SlimAttention for one sequence (Section 2.1): for each selected query row
 * and each query head, the full score row over the visible keys, one softmax,
 * then the product with V.
 *   query t (0-based among the nq rows) sees keys j <= kv_len - nq + t
 *   (so j <= t when nq == kv_len; decode is nq == 1 and sees every key).
 *   query head h reads kv head h / (Hq / Hkv).
 * sel lists the query indices to compute (NULL = all nq rows, n_sel ignored).
 * out[n_sel][Hq][D] in double. */
void slim_oracle_attention(const uint16_t *q, const int8_t *kc, const float *ks,
                           const int8_t *vc, const float *vs,
                           int32_t nq, int32_t kv_len, int32_t Hq, int32_t Hkv, int32_t D,
                           double sm_scale, const int32_t *sel, int32_t n_sel, double *out)
{
    const int32_t G = Hq / Hkv;
    const int32_t n_rows = sel ? n_sel : nq;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)(kv_len > 0 ? kv_len : 1));
#pragma omp for collapse(2) schedule(dynamic, 1)
        for (int32_t r = 0; r < n_rows; ++r) {
            for (int32_t h = 0; h < Hq; ++h) {
                const int32_t t = sel ? sel[r] : r;
                const int32_t g = h / G;
                const int64_t n_vis = (int64_t)kv_len - nq + t + 1;
                double *o = out + ((int64_t)r * Hq + h) * D;
                for (int d = 0; d < D; ++d) o[d] = 0.0;
                if (n_vis <= 0) continue;
                const uint16_t *qrow = q + ((int64_t)t * Hq + h) * D;
                score_row(qrow, kc, ks, 0, n_vis, g, Hkv, D, sm_scale, s);
                double m = s[0];
                for (int64_t j = 1; j < n_vis; ++j) if (s[j] > m) m = s[j];
                double sum = 0.0;
                for (int64_t j = 0; j < n_vis; ++j) { s[j] = exp(s[j] - m); sum += s[j]; }
                for (int64_t j = 0; j < n_vis; ++j) {
                    const double p = s[j] / sum;
                    for (int d = 0; d < D; ++d) o[d] += p * deq(vc, vs, j, g, Hkv, D, d);
                }
            }
        }
        free(s);
    }
}

/* One piece of a split decode row: keys [j0, j1) of kv head g for query row
 * qrow[D].  Returns m = max_j s_j, l = sum_j exp(s_j - m) and the
 * unnormalised O_d = sum_j exp(s_j - m) * v^_{j,d}.  j1 > j0 required. */
void slim_oracle_partial(const uint16_t *qrow, const int8_t *kc, const float *ks,
                         const int8_t *vc, const float *vs,
                         int32_t j0, int32_t j1, int32_t g, int32_t Hkv, int32_t D,
                         double sm_scale, double *m_out, double *l_out, double *O)
{
    double *s = (double *)malloc(sizeof(double) * (size_t)(j1 - j0));
    score_row(qrow, kc, ks, j0, j1, g, Hkv, D, sm_scale, s);
    double m = s[0];
    for (int32_t j = 1; j < j1 - j0; ++j) if (s[j] > m) m = s[j];
    double l = 0.0;
    for (int d = 0; d < D; ++d) O[d] = 0.0;
    for (int32_t j = 0; j < j1 - j0; ++j) {
        const double e = exp(s[j] - m);
        l += e;
        for (int d = 0; d < D; ++d) O[d] += e * deq(vc, vs, j0 + j, g, Hkv, D, d);
    }
    *m_out = m;
    *l_out = l;
    free(s);
}

/* Merge of n pieces: M = max m_c; l = sum l_c e^{m_c - M};
 * o = sum O_c e^{m_c - M} / l. */
void slim_oracle_merge(const double *m, const double *l, const double *O,
                       int32_t n, int32_t D, double *o)
{
    double M = m[0];
    for (int32_t c = 1; c < n; ++c) if (m[c] > M) M = m[c];
    double L = 0.0;
    for (int d = 0; d < D; ++d) o[d] = 0.0;
    for (int32_t c = 0; c < n; ++c) {
        const double w = exp(m[c] - M);
        L += l[c] * w;
        for (int d = 0; d < D; ++d) o[d] += O[(int64_t)c * D + d] * w;
    }
    for (int d = 0; d < D; ++d) o[d] /= L;
}

/* Eq. (1): bytes of KV cache read to generate one token,
 * 2 * b * (L_i + L_o) * l * n_head * s_head * s_d. */
double slim_oracle_kv_bytes(double b, double L_in, double L_out, double layers,
                            double n_head, double s_head, double s_d)
{
    return 2.0 * b * (L_in + L_out) * layers * n_head * s_head * s_d;
}
