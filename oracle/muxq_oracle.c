/*
 * MUXQ oracle -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow CPU statement of what the MUXQ quantized linear layer computes, written from
 * the paper's equations (Eq. 1-7 and the outlier criterion of Section III-C).  It exists so
 * that the CUDA library can be checked against something that can be verified by eye.  It
 * shares no code, header, table or helper with the CUDA path, and the product never calls
 * it: only the tests, the smoke check and the benchmark's "cpu_baseline" leg may.
 *
 * Build: gcc -O2 -fopenmp -ffp-contract=off -fPIC -shared (no -ffast-math).  Every fp32
 * operation below is a single IEEE round-to-nearest-even operation; no fused multiply-add.
 *
 * Pins (see tests/test_oracle_*.py): hand-worked example, brute force in int64/fp64 on tiny
 * inputs, Eq. 6 exact reconstruction, error bound s/2, the r = 0 reduction to textbook abs-max
 * quantization, integer identity against the "x4 on outlier columns" form, fake-quant
 * cross-check, metamorphic relations.
 * Parity unpinned: which scale the authors' code gives Aux (shared with Body, or its own) --
 * nothing printed in the paper discriminates.  Both readings are implemented (aux_own flag).
 *
 * Notation (paper): X [M,K] fp16 activations, W [K,N] fp16 weights, O = outlier channel
 * (column) set of X, r = |O|, e = exp factor, c = 2^e - 1, q = 2^(bits-1) - 1.
 * fp16 values travel as raw uint16_t bit patterns.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_ERR_ARG 1
#define ORACLE_ERR_NONFINITE 2
#define ORACLE_ERR_CAPACITY 5

/* ---- IEEE binary16 <-> binary32, written from the format definition ------------------- */

/* binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits.  Widening is exact. */
float oracle_f16_to_f32(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int ex = (h >> 10) & 0x1f;
    int fr = h & 0x3ff;
    float v;
    if (ex == 0) {
        v = ldexpf((float)fr, -24); /* zero / subnormal: fr * 2^-24 */
    } else if (ex == 31) {
        v = fr ? NAN : INFINITY;
    } else {
        v = ldexpf((float)(fr | 0x400), ex - 25); /* (1024+fr) * 2^(ex-15-10) */
    }
    return sign ? -v : v;
}

/* binary32 -> binary16 with round-to-nearest-even (Eq. 3 writes the output as FP16). */
uint16_t oracle_f32_to_f16(float f)
{
    uint16_t sign = signbit(f) ? 0x8000u : 0;
    float a = fabsf(f);
    if (isnan(a)) return (uint16_t)(sign | 0x7e00u);
    if (a >= 65520.0f) return (uint16_t)(sign | 0x7c00u); /* rounds to infinity */
    if (a < ldexpf(1.0f, -14)) {
        /* subnormal target: spacing 2^-24.  a * 2^24 is exact (power-of-two scaling). */
        float t = nearbyintf(ldexpf(a, 24));
        return (uint16_t)(sign | (uint16_t)t); /* t == 1024 lands on the smallest normal */
    }
    int ex;
    float m = frexpf(a, &ex);            /* a = m * 2^ex, m in [0.5, 1) */
    float t = nearbyintf(ldexpf(m, 11)); /* 11 significant bits; ties to even; in [1024, 2048] */
    if (t == 2048.0f) { t = 1024.0f; ex += 1; }
    int be = ex - 1 + 15;                /* biased exponent of 1.xxx * 2^(ex-1) */
    return (uint16_t)(sign | (uint16_t)(be << 10) | ((uint16_t)t & 0x3ff));
}

static int qmax_of_bits(int bits) { return (1 << (bits - 1)) - 1; } /* Eq. 1: 2^7 - 1 for 8 bits */

/* Eq. 1 / Eq. 2 rounding: true division, round half to even, symmetric clamp to [-q, q]. */
static int8_t quantize_one(float v, float s, int q)
{
    float t = nearbyintf(v / s);
    if (t > (float)q) t = (float)q;
    if (t < (float)-q) t = (float)-q;
    return (int8_t)t;
}

/* abs-max scale of Eq. 1 / Eq. 2; an all-zero unit gets scale 1. */
static float scale_of(float amax, int q) { return amax > 0.0f ? amax / (float)q : 1.0f; }

/* ---- Step 1: per-channel abs-max (Section III-C criterion looks at channel magnitudes) -- */
int oracle_colmax(const uint16_t *x, int M, int K, int ldx, float *colmax)
{
    if (!x || !colmax || M <= 0 || K <= 0 || ldx < K) return ORACLE_ERR_ARG;
    for (int k = 0; k < K; ++k) colmax[k] = 0.0f;
    for (int m = 0; m < M; ++m)
        for (int k = 0; k < K; ++k) {
            float v = oracle_f16_to_f32(x[(size_t)m * ldx + k]);
            if (!isfinite(v)) return ORACLE_ERR_NONFINITE;
            float a = fabsf(v);
            if (a > colmax[k]) colmax[k] = a;
        }
    return ORACLE_OK;
}

/* ---- Step 2: O = channels holding at least one element of magnitude > tau (strict) ------ */
/* Writes all detected indices (ascending) up to cap; *r is the true count.                  */
int oracle_detect(const float *colmax, int K, float tau, int32_t *O, int cap, int32_t *r)
{
    int n = 0;
    for (int k = 0; k < K; ++k)
        if (colmax[k] > tau) {
            if (n < cap) O[n] = k;
            ++n;
        }
    *r = n;
    return n > cap ? ORACLE_ERR_CAPACITY : ORACLE_OK;
}

/* ---- Steps 3-4: Body and Aux in the real domain (Eq. 4, Eq. 5) -------------------------- */
/* body[m,k] = x[m,k] * 2^-e for k in O, else x[m,k];  aux[m,j] = body[m,O_j].  Exact in fp32. */
int oracle_decompose(const uint16_t *x, int M, int K, int ldx, const int32_t *O, int r, int e,
                     float *body /*[M,K]*/, float *aux /*[M,r] or NULL*/)
{
    unsigned char *is_out = (unsigned char *)calloc((size_t)K, 1);
    if (!is_out) return ORACLE_ERR_ARG;
    for (int j = 0; j < r; ++j) is_out[O[j]] = 1;
    for (int m = 0; m < M; ++m)
        for (int k = 0; k < K; ++k) {
            float v = oracle_f16_to_f32(x[(size_t)m * ldx + k]);
            body[(size_t)m * K + k] = is_out[k] ? ldexpf(v, -e) : v;
        }
    if (aux)
        for (int m = 0; m < M; ++m)
            for (int j = 0; j < r; ++j) aux[(size_t)m * r + j] = body[(size_t)m * K + O[j]];
    free(is_out);
    return ORACLE_OK;
}

/* ---- Steps 5-6: abs-max scales and INT codes of Body and Aux (Eq. 1) -------------------- */
/* per_token = 0: one scale for the tensor (s_x[0], s_a[0]); 1: one per row (s_x[m], s_a[m]). */
/* aux_own = 0: Aux is quantized with Body's scale (so aux_q == body_q[:,O]); 1: own abs-max. */
int oracle_quantize_act(const float *body, const float *aux, int M, int K, int r, int bits,
                        int per_token, int aux_own, float *s_x, float *s_a, int8_t *body_q,
                        int8_t *aux_q)
{
    int q = qmax_of_bits(bits);
    if (!per_token) {
        float bm = 0.0f, am = 0.0f;
        for (size_t i = 0; i < (size_t)M * K; ++i)
            if (fabsf(body[i]) > bm) bm = fabsf(body[i]);
        for (size_t i = 0; i < (size_t)M * r; ++i)
            if (fabsf(aux[i]) > am) am = fabsf(aux[i]);
        s_x[0] = scale_of(bm, q);
        s_a[0] = aux_own ? scale_of(am, q) : s_x[0];
    } else {
        for (int m = 0; m < M; ++m) {
            float bm = 0.0f, am = 0.0f;
            for (int k = 0; k < K; ++k)
                if (fabsf(body[(size_t)m * K + k]) > bm) bm = fabsf(body[(size_t)m * K + k]);
            for (int j = 0; j < r; ++j)
                if (fabsf(aux[(size_t)m * r + j]) > am) am = fabsf(aux[(size_t)m * r + j]);
            s_x[m] = scale_of(bm, q);
            s_a[m] = aux_own ? scale_of(am, q) : s_x[m];
        }
    }
    for (int m = 0; m < M; ++m) {
        float sx = per_token ? s_x[m] : s_x[0];
        float sa = per_token ? s_a[m] : s_a[0];
        for (int k = 0; k < K; ++k)
            body_q[(size_t)m * K + k] = quantize_one(body[(size_t)m * K + k], sx, q);
        for (int j = 0; j < r; ++j)
            aux_q[(size_t)m * r + j] = quantize_one(aux[(size_t)m * r + j], sa, q);
    }
    return ORACLE_OK;
}

/* ---- Step 7: weight quantization (Eq. 2), per tensor or per output channel n ------------ */
/* w is [K,N] row-major fp16 (ldw >= N); w_q is [K,N] row-major; s_w is [1] or [N].           */
int oracle_quantize_weight(const uint16_t *w, int K, int N, int ldw, int bits, int per_channel,
                           int8_t *w_q, float *s_w)
{
    if (!w || !w_q || !s_w || K <= 0 || N <= 0 || ldw < N) return ORACLE_ERR_ARG;
    int q = qmax_of_bits(bits);
    int ns = per_channel ? N : 1;
    float *amax = (float *)calloc((size_t)ns, sizeof(float));
    if (!amax) return ORACLE_ERR_ARG;
    for (int k = 0; k < K; ++k)
        for (int n = 0; n < N; ++n) {
            float v = oracle_f16_to_f32(w[(size_t)k * ldw + n]);
            if (!isfinite(v)) { free(amax); return ORACLE_ERR_NONFINITE; }
            float a = fabsf(v);
            int u = per_channel ? n : 0;
            if (a > amax[u]) amax[u] = a;
        }
    for (int u = 0; u < ns; ++u) s_w[u] = scale_of(amax[u], q);
    for (int k = 0; k < K; ++k)
        for (int n = 0; n < N; ++n)
            w_q[(size_t)k * N + n] =
                quantize_one(oracle_f16_to_f32(w[(size_t)k * ldw + n]), s_w[per_channel ? n : 0], q);
    free(amax);
    return ORACLE_OK;
}

/* ---- Step 8: the two integer products of Eq. 7 ------------------------------------------ */
/* acc_b = Body_q . W_q ; acc_a = Aux_q . W_q[O,:] ; int32.  rows (may be NULL) selects which */
/* rows of Body_q / Aux_q are multiplied; outputs are [n_rows, N].                            */
int oracle_products(const int8_t *body_q, const int8_t *aux_q, const int8_t *w_q, int M, int K,
                    int N, const int32_t *O, int r, const int32_t *rows, int n_rows,
                    int32_t *acc_b, int32_t *acc_a)
{
    if (!rows) n_rows = M;
#pragma omp parallel for schedule(static)
    for (int i = 0; i < n_rows; ++i) {
        int m = rows ? rows[i] : i;
        int32_t *pb = acc_b + (size_t)i * N;
        int32_t *pa = acc_a + (size_t)i * N;
        for (int n = 0; n < N; ++n) { pb[n] = 0; pa[n] = 0; }
        for (int k = 0; k < K; ++k) {
            int32_t a = body_q[(size_t)m * K + k];
            const int8_t *wr = w_q + (size_t)k * N;
            for (int n = 0; n < N; ++n) pb[n] += a * (int32_t)wr[n];
        }
        for (int j = 0; j < r; ++j) {
            int32_t a = aux_q[(size_t)m * r + j];
            const int8_t *wr = w_q + (size_t)O[j] * N;
            for (int n = 0; n < N; ++n) pa[n] += a * (int32_t)wr[n];
        }
    }
    return ORACLE_OK;
}

/* ---- Steps 9-10: weighted sum (Eq. 7) and dequantization (Eq. 3) ------------------------ */
/* shared scale: acc = acc_b + c*acc_a (int32), y = (s_x*s_w)*float(acc).                     */
/* own scale:    y = (s_x*s_w)*float(acc_b) + float(c)*((s_a*s_w)*float(acc_a)), acc = 0.     */
int oracle_combine_dequant(const int32_t *acc_b, const int32_t *acc_a, int M, int N, int e,
                           const int32_t *rows, int n_rows, const float *s_x, const float *s_a,
                           int per_token, const float *s_w, int per_channel, int aux_own,
                           int32_t *acc, float *y32, uint16_t *y16)
{
    int c = (1 << e) - 1;
    if (!rows) n_rows = M;
    for (int i = 0; i < n_rows; ++i) {
        int m = rows ? rows[i] : i;
        float sx = per_token ? s_x[m] : s_x[0];
        float sa = per_token ? s_a[m] : s_a[0];
        for (int n = 0; n < N; ++n) {
            size_t o = (size_t)i * N + n;
            float sw = per_channel ? s_w[n] : s_w[0];
            float y;
            if (!aux_own) {
                acc[o] = acc_b[o] + c * acc_a[o];
                float sxw = sx * sw;
                y = sxw * (float)acc[o];
            } else {
                acc[o] = 0;
                float t1 = sx * sw;
                t1 = t1 * (float)acc_b[o];
                float t2 = sa * sw;
                t2 = t2 * (float)acc_a[o];
                t2 = (float)c * t2;
                y = t1 + t2;
            }
            y32[o] = y;
            y16[o] = oracle_f32_to_f16(y);
        }
    }
    return ORACLE_OK;
}

/* ---- Whole activation side + products for one layer call, steps 1-6 and 8-10 in order --- */
/* Weights come in already quantized (step 7 is done once per weight).  Any output pointer    */
/* may be NULL except y32/y16.  Returns ORACLE_ERR_CAPACITY when r > cap (r_out is still set). */
int oracle_linear(const uint16_t *x, int M, int K, int ldx, const int8_t *w_q /*[K,N]*/,
                  const float *s_w, int N, float tau, int e, int act_bits, int per_vector,
                  int aux_own, int cap, const int32_t *rows, int n_rows,
                  /* outputs */
                  float *colmax, int32_t *O, int32_t *r_out, float *s_x, float *s_a,
                  int8_t *body_q /*[M,K]*/, int8_t *aux_q /*[M,cap]*/, int32_t *acc_b,
                  int32_t *acc_a, int32_t *acc, float *y32, uint16_t *y16)
{
    if (!x || !w_q || !s_w || !y32 || !y16 || M <= 0 || K <= 0 || N <= 0 || ldx < K || cap < 0)
        return ORACLE_ERR_ARG;
    if (!rows) n_rows = M;
    int rc = ORACLE_OK;
    int ns = per_vector ? M : 1;
    float *colmax_l = (float *)malloc((size_t)K * sizeof(float));
    int32_t *O_l = (int32_t *)malloc((size_t)(cap > 0 ? cap : 1) * sizeof(int32_t));
    float *body = (float *)malloc((size_t)M * K * sizeof(float));
    float *aux = NULL;
    float *sx_l = (float *)malloc((size_t)ns * sizeof(float));
    float *sa_l = (float *)malloc((size_t)ns * sizeof(float));
    int8_t *bq_l = (int8_t *)malloc((size_t)M * K);
    int8_t *aq_l = NULL;
    int32_t *ab_l = (int32_t *)malloc((size_t)n_rows * N * sizeof(int32_t));
    int32_t *aa_l = (int32_t *)malloc((size_t)n_rows * N * sizeof(int32_t));
    int32_t *ac_l = (int32_t *)malloc((size_t)n_rows * N * sizeof(int32_t));
    int32_t r = 0;

    rc = oracle_colmax(x, M, K, ldx, colmax_l);                       /* step 1 */
    if (rc) goto done;
    rc = oracle_detect(colmax_l, K, tau, O_l, cap, &r);               /* step 2 */
    if (r_out) *r_out = r;
    if (colmax) memcpy(colmax, colmax_l, (size_t)K * sizeof(float));
    if (O) memcpy(O, O_l, (size_t)(r < cap ? r : cap) * sizeof(int32_t));
    if (rc) goto done;
    aux = (float *)malloc((size_t)M * (r > 0 ? r : 1) * sizeof(float));
    aq_l = (int8_t *)malloc((size_t)M * (r > 0 ? r : 1));
    oracle_decompose(x, M, K, ldx, O_l, r, e, body, aux);             /* steps 3-4 */
    oracle_quantize_act(body, aux, M, K, r, act_bits, per_vector, aux_own, sx_l, sa_l, bq_l,
                        aq_l);                                        /* steps 5-6 */
    oracle_products(bq_l, aq_l, w_q, M, K, N, O_l, r, rows, n_rows, ab_l, aa_l); /* step 8 */
    oracle_combine_dequant(ab_l, aa_l, M, N, e, rows, n_rows, sx_l, sa_l, per_vector, s_w,
                           per_vector, aux_own, ac_l, y32, y16);      /* steps 9-10 */
    if (s_x) memcpy(s_x, sx_l, (size_t)ns * sizeof(float));
    if (s_a) memcpy(s_a, sa_l, (size_t)ns * sizeof(float));
    if (body_q) memcpy(body_q, bq_l, (size_t)M * K);
    if (aux_q)
        for (int m = 0; m < M; ++m)
            for (int j = 0; j < cap; ++j) aux_q[(size_t)m * cap + j] = j < r ? aq_l[(size_t)m * r + j] : 0;
    if (acc_b) memcpy(acc_b, ab_l, (size_t)n_rows * N * sizeof(int32_t));
    if (acc_a) memcpy(acc_a, aa_l, (size_t)n_rows * N * sizeof(int32_t));
    if (acc) memcpy(acc, ac_l, (size_t)n_rows * N * sizeof(int32_t));
done:
    free(colmax_l); free(O_l); free(body); free(aux); free(sx_l); free(sa_l);
    free(bq_l); free(aq_l); free(ab_l); free(aa_l); free(ac_l);
    return rc;
}

/* Threads the row loop of oracle_products uses (reported by the benchmark's CPU leg). */
int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
