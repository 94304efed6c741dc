/*
 * CPU oracle for attention weights and row-wise Softmax.
 *
 * TEST INFRASTRUCTURE, not product code: only the test-suite, the smoke check
 * and the benchmark's CPU-baseline leg may build, link or call this file.  It
 * shares no code, header, table or helper with the CUDA path.
 *
 * What it computes (every step in IEEE double precision, no blocking, no
 * online rescaling, no exp2 tricks - the definition written out):
 *
 *   scores      s_ij = sum_c Q_ic * K_jc                 (Section IV, Attention(Q,K,V))
 *   scaling     z_ij = scale * s_ij                      (Section IV, the 1/sqrt(d_k) factor)
 *   row max     m_i  = max_j z_ij                        (Eq. 1)
 *   weights     P_ij = exp(z_ij - m_i) / sum_k exp(z_ik - m_i)
 *                                                        (Eq. 1; equal to the Softmax
 *                                                         definition of Section VI)
 *
 * The order of steps inside a row is the one Section VI-A gives for the CPU
 * program, in its "caching" form: find the maximum, subtract it, exponentiate
 * and sum while keeping the exponentials, divide by the sum.
 *
 * Readings taken where the paper is silent:
 *   - the Softmax runs over the key index j (last axis);
 *   - inputs Q, K are bfloat16 bit patterns decoded exactly; precomputed scores
 *     S are float32 widened exactly;
 *   - `scale` is the float the caller hands over, widened to double (not a
 *     freshly computed 1/sqrt(d));
 *   - max subtraction is always applied;
 *   - the output is double and is never rounded to a narrower type here.
 *
 *   attention   O_ic = sum_j P_ij * V_jc                 (Section IV: Attention(Q,K,V) =
 *                                                         softmax(Q K^T / sqrt(d_k)) V)
 *
 * Parity pins (tests/test_oracle_pins.py): rows sum to 1 and lie in [0,1];
 * identical keys give exactly 1/N; permuting keys permutes columns; shift
 * invariance (Eq. 1); two-key logistic closed form; geometric-series closed
 * form; one-hot limit; 4x4 brute force of the un-shifted definition in long
 * double; float64 library softmax on the same decoded inputs.  For the product
 * with V: V of ones gives ones; unit-vector columns of V give column sums of P;
 * identical keys give the mean of V; a single key gives that key's V; linearity
 * in V; 4x4 brute force in long double; float64 library softmax times V.
 *
 * Rows are independent (Section VI), so threads split rows statically and
 * nothing else is parallelised.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ---- exact decoding of the narrow input types ------------------------------------- */

static double bf16_to_double(uint16_t bits)
{
    uint32_t w = ((uint32_t)bits) << 16; /* bfloat16 = upper half of a binary32 */
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/* ---- one row of Eq. 1 on already scaled scores z[0..n) ------------------------------ */

static void softmax_row_f64(const double *z, double *p, long n)
{
    double m = z[0];
    for (long j = 1; j < n; ++j)
        if (z[j] > m)
            m = z[j];
    double l = 0.0;
    for (long j = 0; j < n; ++j) {
        p[j] = exp(z[j] - m); /* kept ("cached") for the divide below */
        l += p[j];
    }
    for (long j = 0; j < n; ++j)
        p[j] = p[j] / l;
}

/* ---- static row partition over threads ---------------------------------------------- */

typedef void (*row_fn)(void *ctx, long row_index, double *scratch);

typedef struct {
    row_fn fn;
    void *ctx;
    long begin, end;
    long scratch_len;
    int failed;
} span_t;

static void *run_span(void *arg)
{
    span_t *s = (span_t *)arg;
    double *scratch = NULL;
    if (s->scratch_len > 0) {
        scratch = (double *)malloc(sizeof(double) * (size_t)s->scratch_len);
        if (!scratch) {
            s->failed = 1;
            return NULL;
        }
    }
    for (long r = s->begin; r < s->end; ++r)
        s->fn(s->ctx, r, scratch);
    free(scratch);
    return NULL;
}

static int for_each_row(row_fn fn, void *ctx, long nrows, long scratch_len, int nthreads)
{
    if (nthreads < 1)
        nthreads = 1;
    if ((long)nthreads > nrows)
        nthreads = nrows > 0 ? (int)nrows : 1;
    span_t *spans = (span_t *)calloc((size_t)nthreads, sizeof(span_t));
    pthread_t *tids = (pthread_t *)calloc((size_t)nthreads, sizeof(pthread_t));
    if (!spans || !tids) {
        free(spans);
        free(tids);
        return -1;
    }
    long q = nrows / nthreads, rem = nrows % nthreads, at = 0;
    for (int t = 0; t < nthreads; ++t) {
        long take = q + (t < rem ? 1 : 0);
        spans[t].fn = fn;
        spans[t].ctx = ctx;
        spans[t].begin = at;
        spans[t].end = at + take;
        spans[t].scratch_len = scratch_len;
        at += take;
    }
    int rc = 0;
    if (nthreads == 1) {
        run_span(&spans[0]);
    } else {
        for (int t = 0; t < nthreads; ++t)
            if (pthread_create(&tids[t], NULL, run_span, &spans[t]) != 0) {
                run_span(&spans[t]);
                tids[t] = 0;
            }
        for (int t = 0; t < nthreads; ++t)
            if (tids[t])
                pthread_join(tids[t], NULL);
    }
    for (int t = 0; t < nthreads; ++t)
        if (spans[t].failed)
            rc = -1;
    free(spans);
    free(tids);
    return rc;
}

/* ---- row Softmax of precomputed scores (Section VI definition, Eq. 1) --------------- */

typedef struct {
    const float *S;
    double *P;
    long cols;
    const long *row_ids; /* NULL = all rows in order */
} rows_ctx;

static void rows_one(void *vctx, long r, double *z)
{
    rows_ctx *c = (rows_ctx *)vctx;
    long src = c->row_ids ? c->row_ids[r] : r;
    const float *s = c->S + (size_t)src * (size_t)c->cols;
    for (long j = 0; j < c->cols; ++j)
        z[j] = (double)s[j];
    softmax_row_f64(z, c->P + (size_t)r * (size_t)c->cols, c->cols);
}

/* S: rows x cols float32, row-major.  P: rows x cols double, row-major. */
int oracle_softmax_rows(const float *S, double *P, long rows, long cols, int nthreads)
{
    if (!S || !P || rows < 1 || cols < 1)
        return -2;
    rows_ctx c = {S, P, cols, NULL};
    return for_each_row(rows_one, &c, rows, cols, nthreads);
}

/* Only the listed rows of S; P is n_ids x cols. */
int oracle_softmax_rows_subset(const float *S, double *P, long cols, const long *row_ids,
                               long n_ids, int nthreads)
{
    if (!S || !P || !row_ids || n_ids < 1 || cols < 1)
        return -2;
    rows_ctx c = {S, P, cols, row_ids};
    return for_each_row(rows_one, &c, n_ids, cols, nthreads);
}

/* ---- attention weights softmax(scale * Q K^T) (Section IV; Section VII states the
 *      same product for n x d_k inputs and an n x n output) --------------------------- */

typedef struct {
    const uint16_t *Q, *K; /* [B*H, N, d] bfloat16 bit patterns */
    double *P;
    long N, d;
    double scale;
    const long *row_ids; /* global row = bh * N + i; NULL = all rows in order */
} attn_ctx;

static void attn_one(void *vctx, long r, double *scratch)
{
    attn_ctx *c = (attn_ctx *)vctx;
    long g = c->row_ids ? c->row_ids[r] : r;
    long bh = g / c->N;
    const uint16_t *q = c->Q + (size_t)g * (size_t)c->d;
    const uint16_t *Kh = c->K + (size_t)bh * (size_t)c->N * (size_t)c->d;
    double *qd = scratch;        /* d decoded query values */
    double *z = scratch + c->d;  /* N scaled scores        */
    for (long t = 0; t < c->d; ++t)
        qd[t] = bf16_to_double(q[t]);
    for (long j = 0; j < c->N; ++j) {
        const uint16_t *k = Kh + (size_t)j * (size_t)c->d;
        double s = 0.0;
        for (long t = 0; t < c->d; ++t)
            s += qd[t] * bf16_to_double(k[t]);
        z[j] = c->scale * s;
    }
    softmax_row_f64(z, c->P + (size_t)r * (size_t)c->N, c->N);
}

/* Q, K: [B, H, N, d] bfloat16 bits.  P: [B, H, N, N] double. */
int oracle_attnw(const uint16_t *Q, const uint16_t *K, double *P, long B, long H, long N, long d,
                 float scale, int nthreads)
{
    if (!Q || !K || !P || B < 1 || H < 1 || N < 1 || d < 1)
        return -2;
    attn_ctx c = {Q, K, P, N, d, (double)scale, NULL};
    return for_each_row(attn_one, &c, B * H * N, N + d, nthreads);
}

/* Only the listed global rows (bh * N + i); P is n_ids x N. */
int oracle_attnw_rows(const uint16_t *Q, const uint16_t *K, double *P, long B, long H, long N,
                      long d, float scale, const long *row_ids, long n_ids, int nthreads)
{
    if (!Q || !K || !P || !row_ids || B < 1 || H < 1 || N < 1 || d < 1 || n_ids < 1)
        return -2;
    for (long r = 0; r < n_ids; ++r)
        if (row_ids[r] < 0 || row_ids[r] >= B * H * N)
            return -3;
    attn_ctx c = {Q, K, P, N, d, (double)scale, row_ids};
    return for_each_row(attn_one, &c, n_ids, N + d, nthreads);
}

/* ---- attention O = softmax(scale * Q K^T) V (Section IV) ------------------------------
 * One output row: the row of weights as above, then the weighted sum of the value vectors,
 * c ascending inside j ascending, all in double. */

typedef struct {
    attn_ctx a;        /* P is unused here */
    const uint16_t *V; /* [B*H, N, d] bfloat16 bit patterns */
    double *O;         /* one row of d doubles per listed row */
} attnv_ctx;

static void attnv_one(void *vctx, long r, double *scratch)
{
    attnv_ctx *c = (attnv_ctx *)vctx;
    long N = c->a.N, d = c->a.d;
    long g = c->a.row_ids ? c->a.row_ids[r] : r;
    long bh = g / N;
    const uint16_t *q = c->a.Q + (size_t)g * (size_t)d;
    const uint16_t *Kh = c->a.K + (size_t)bh * (size_t)N * (size_t)d;
    const uint16_t *Vh = c->V + (size_t)bh * (size_t)N * (size_t)d;
    double *qd = scratch;         /* d decoded query values */
    double *z = scratch + d;      /* N scaled scores        */
    double *p = scratch + d + N;  /* N weights              */
    double *o = c->O + (size_t)r * (size_t)d;
    for (long t = 0; t < d; ++t)
        qd[t] = bf16_to_double(q[t]);
    for (long j = 0; j < N; ++j) {
        const uint16_t *k = Kh + (size_t)j * (size_t)d;
        double s = 0.0;
        for (long t = 0; t < d; ++t)
            s += qd[t] * bf16_to_double(k[t]);
        z[j] = c->a.scale * s;
    }
    softmax_row_f64(z, p, N);
    for (long t = 0; t < d; ++t)
        o[t] = 0.0;
    for (long j = 0; j < N; ++j) {
        const uint16_t *v = Vh + (size_t)j * (size_t)d;
        for (long t = 0; t < d; ++t)
            o[t] += p[j] * bf16_to_double(v[t]);
    }
}

/* Q, K, V: [B, H, N, d] bfloat16 bits.  O: [B, H, N, d] double. */
int oracle_attn(const uint16_t *Q, const uint16_t *K, const uint16_t *V, double *O, long B, long H, long N,
                long d, float scale, int nthreads)
{
    if (!Q || !K || !V || !O || B < 1 || H < 1 || N < 1 || d < 1)
        return -2;
    attnv_ctx c = {{Q, K, NULL, N, d, (double)scale, NULL}, V, O};
    return for_each_row(attnv_one, &c, B * H * N, 2 * N + d, nthreads);
}

/* Only the listed global rows (bh * N + i); O is n_ids x d. */
int oracle_attn_rows(const uint16_t *Q, const uint16_t *K, const uint16_t *V, double *O, long B, long H,
                     long N, long d, float scale, const long *row_ids, long n_ids, int nthreads)
{
    if (!Q || !K || !V || !O || !row_ids || B < 1 || H < 1 || N < 1 || d < 1 || n_ids < 1)
        return -2;
    for (long r = 0; r < n_ids; ++r)
        if (row_ids[r] < 0 || row_ids[r] >= B * H * N)
            return -3;
    attnv_ctx c = {{Q, K, NULL, N, d, (double)scale, row_ids}, V, O};
    return for_each_row(attnv_one, &c, n_ids, 2 * N + d, nthreads);
}

/* Raw (unscaled) scores of the listed rows, for tests that look at one step alone. */
int oracle_scores_rows(const uint16_t *Q, const uint16_t *K, double *S, long B, long H, long N,
                       long d, const long *row_ids, long n_ids)
{
    if (!Q || !K || !S || !row_ids || B < 1 || H < 1 || N < 1 || d < 1 || n_ids < 1)
        return -2;
    for (long r = 0; r < n_ids; ++r) {
        long g = row_ids[r];
        if (g < 0 || g >= B * H * N)
            return -3;
        long bh = g / N;
        for (long j = 0; j < N; ++j) {
            double s = 0.0;
            for (long t = 0; t < d; ++t)
                s += bf16_to_double(Q[(size_t)g * (size_t)d + (size_t)t]) *
                     bf16_to_double(K[((size_t)bh * (size_t)N + (size_t)j) * (size_t)d + (size_t)t]);
            S[(size_t)r * (size_t)N + (size_t)j] = s;
        }
    }
    return 0;
}

/* ---- the linear transformation of the inputs into queries (or keys), Section IV: per head h,
 *      Q_h = X W_h, written out as Q[b,h,n,c] = sum_m X[b,n,m] * W[h,c,m], m ascending.
 *      X: [B, N, d_model] bfloat16 bits.  W: [H, d, d_model] bfloat16 bits (row c of head h holds column c of
 *      that head's parameter matrix).  Only the listed global rows (b*H + h)*N + n, or all rows when row_ids
 *      is NULL (then n_ids is ignored); out is rows x d. */
int oracle_project(const uint16_t *X, const uint16_t *W, double *out, long B, long N, long d_model, long H,
                   long d, const long *row_ids, long n_ids)
{
    if (!X || !W || !out || B < 1 || N < 1 || d_model < 1 || H < 1 || d < 1)
        return -2;
    long rows = row_ids ? n_ids : B * H * N;
    if (rows < 1)
        return -2;
    for (long r = 0; r < rows; ++r) {
        long g = row_ids ? row_ids[r] : r;
        if (g < 0 || g >= B * H * N)
            return -3;
        long n = g % N, h = (g / N) % H, b = g / (N * H);
        const uint16_t *x = X + ((size_t)b * (size_t)N + (size_t)n) * (size_t)d_model;
        for (long c = 0; c < d; ++c) {
            const uint16_t *w = W + ((size_t)h * (size_t)d + (size_t)c) * (size_t)d_model;
            double s = 0.0;
            for (long m = 0; m < d_model; ++m)
                s += bf16_to_double(x[m]) * bf16_to_double(w[m]);
            out[(size_t)r * (size_t)d + (size_t)c] = s;
        }
    }
    return 0;
}
