/*
 * fp64 CPU oracle for the fused operator chains (TEST INFRASTRUCTURE ONLY).
 *
 * This file is the yard-stick the CUDA path is compared against.  It is plain,
 * slow and written to be checked by eye; it shares no code, header, table or
 * constant with the CUDA library and must never be linked into or called from
 * the product path.  Only the tests, the smoke check and the bench's CPU
 * baseline leg use it.
 *
 * The paper (Section 5.3, "Task-wise Benchmark Analysis") describes the winning
 * pattern as fusing a heavy operator with the pointwise and reduction operators
 * that follow it, and replacing naive attention by a flash-attention kernel with
 * on-the-fly causal masking (Appendix C, "MinGPT", "HunyuanVideo").  It prints no
 * formula for those operators; each function below is therefore the textbook
 * definition of the named operator, written out directly.  Every chain has one
 * mathematically defined result, so the oracle is that definition in fp64 with
 * no blocking, fusion or re-ordering.
 *
 * All matrices are row-major doubles.  Rows are independent in every chain, so
 * "M" may be any gathered subset of rows.  OpenMP (if enabled at compile time)
 * only distributes independent rows over cores; it never splits a sum.
 *
 * Pins (see tests/test_oracle_pins.py): activations at tabulated points and the
 * identity f(y)-f(-y)=y; LayerNorm mean/variance closed forms and affine
 * invariance; softmax normalisation, shift invariance and the logistic closed
 * form; matmul against exact integer brute force, identity weights and a second
 * loop order; attention special cases (first row, constant V, zero Q, S=1,
 * key/value permutation) and the explicit masked dense form.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

enum { ACT_NONE = 0, ACT_GELU_ERF = 1, ACT_GELU_TANH = 2, ACT_SILU = 3 };
enum { RED_NONE = 0, RED_LAYERNORM = 1, RED_SOFTMAX = 2 };

/* GELU, exact form: y * Phi(y) with Phi the standard normal CDF. */
double oracle_gelu_erf(double y) { return 0.5 * y * (1.0 + erf(y / sqrt(2.0))); }

/* GELU, tanh form: 0.5 y (1 + tanh( sqrt(2/pi) (y + 0.044715 y^3) )). */
double oracle_gelu_tanh(double y)
{
    const double c = sqrt(2.0 / M_PI);
    return 0.5 * y * (1.0 + tanh(c * (y + 0.044715 * y * y * y)));
}

/* SiLU: y * sigmoid(y). */
double oracle_silu(double y) { return y / (1.0 + exp(-y)); }

double oracle_act(int act, double y)
{
    switch (act) {
    case ACT_GELU_ERF:  return oracle_gelu_erf(y);
    case ACT_GELU_TANH: return oracle_gelu_tanh(y);
    case ACT_SILU:      return oracle_silu(y);
    default:            return y;
    }
}

/* y[m,n] = sum_{k ascending} x[m,k] * w[k,n]  (+ b[n] if b != NULL).
 * w is [K,N] row-major.  The k loop is outermost per row only so that w is
 * walked along its contiguous dimension; each y[m,n] still receives its
 * products in ascending k. */
void oracle_linear(const double *x, const double *w, const double *b, double *y,
                   long M, long K, long N)
{
#pragma omp parallel for schedule(static)
    for (long m = 0; m < M; ++m) {
        double *yr = y + m * N;
        for (long n = 0; n < N; ++n) yr[n] = 0.0;
        for (long k = 0; k < K; ++k) {
            const double a = x[m * K + k];
            const double *wr = w + k * N;
            for (long n = 0; n < N; ++n) yr[n] += a * wr[n];
        }
        if (b) for (long n = 0; n < N; ++n) yr[n] += b[n];
    }
}

/* LayerNorm over the last dimension, in place: biased variance, two passes,
 * eps inside the square root; gamma/beta may be NULL (1 and 0). */
void oracle_layernorm_rows(double *v, long M, long N, const double *gamma,
                           const double *beta, double eps)
{
#pragma omp parallel for schedule(static)
    for (long m = 0; m < M; ++m) {
        double *r = v + m * N;
        double mean = 0.0, var = 0.0;
        for (long n = 0; n < N; ++n) mean += r[n];
        mean /= (double)N;
        for (long n = 0; n < N; ++n) var += (r[n] - mean) * (r[n] - mean);
        var /= (double)N;
        const double rstd = 1.0 / sqrt(var + eps);
        for (long n = 0; n < N; ++n) {
            double z = (r[n] - mean) * rstd;
            if (gamma) z *= gamma[n];
            if (beta) z += beta[n];
            r[n] = z;
        }
    }
}

/* softmax over the last dimension, in place, with the row maximum subtracted. */
void oracle_softmax_rows(double *v, long M, long N)
{
#pragma omp parallel for schedule(static)
    for (long m = 0; m < M; ++m) {
        double *r = v + m * N;
        double mx = r[0], sum = 0.0;
        for (long n = 1; n < N; ++n) if (r[n] > mx) mx = r[n];
        for (long n = 0; n < N; ++n) { r[n] = exp(r[n] - mx); sum += r[n]; }
        for (long n = 0; n < N; ++n) r[n] /= sum;
    }
}

/* Chain: out = reduce( scale * act(x @ w + bias) + residual ).
 * Order of the pointwise steps: bias, activation, scale, residual.
 * bias, residual, gamma, beta may be NULL. */
void oracle_linear_epilogue(const double *x, const double *w, const double *bias,
                            const double *residual, const double *gamma,
                            const double *beta, int act, double scale, int reduce,
                            double eps, double *out, long M, long K, long N)
{
    oracle_linear(x, w, bias, out, M, K, N);
    for (long i = 0; i < M * N; ++i) {
        double v = scale * oracle_act(act, out[i]);
        if (residual) v += residual[i];
        out[i] = v;
    }
    if (reduce == RED_LAYERNORM) oracle_layernorm_rows(out, M, N, gamma, beta, eps);
    else if (reduce == RED_SOFTMAX) oracle_softmax_rows(out, M, N);
}

/* Chain: pre-LN MLP block  out = x + act( LN(x) @ w1 + b1 ) @ w2 + b2.
 * x [M,D], w1 [D,F], w2 [F,D].  Nothing is rounded between the stages. */
int oracle_mlp_block(const double *x, const double *gamma, const double *beta,
                     double eps, const double *w1, const double *b1,
                     const double *w2, const double *b2, int act, double *out,
                     long M, long D, long F)
{
    double *z = (double *)malloc(sizeof(double) * (size_t)M * (size_t)D);
    double *h = (double *)malloc(sizeof(double) * (size_t)M * (size_t)F);
    if (!z || !h) { free(z); free(h); return 1; }
    memcpy(z, x, sizeof(double) * (size_t)M * (size_t)D);
    oracle_layernorm_rows(z, M, D, gamma, beta, eps);
    oracle_linear(z, w1, b1, h, M, D, F);
    for (long i = 0; i < M * F; ++i) h[i] = oracle_act(act, h[i]);
    oracle_linear(h, w2, b2, out, M, F, D);
    for (long i = 0; i < M * D; ++i) out[i] += x[i];
    free(z); free(h);
    return 0;
}

/* Attention for one head, for a chosen set of query rows.
 *   s[j]   = scale * sum_d q[d] * k[j,d]
 *   causal : only keys j <= i take part (i = the query's position)
 *   o[:]   = sum_j softmax_j(s)[j] * v[j,:]
 * q_rows [R,D] holds the queries, q_pos[R] their positions i; k, v are [S,D]. */
int oracle_attention_rows(const double *q_rows, const long *q_pos, long R,
                          const double *k, const double *v, long S, long D,
                          double scale, int causal, double *out)
{
    int fail = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (long r = 0; r < R; ++r) {
        const long i = q_pos[r];
        const long nkeys = causal ? i + 1 : S;
        double *s = (double *)malloc(sizeof(double) * (size_t)nkeys);
        if (!s) { fail = 1; continue; }
        for (long j = 0; j < nkeys; ++j) {
            double dot = 0.0;
            for (long d = 0; d < D; ++d) dot += q_rows[r * D + d] * k[j * D + d];
            s[j] = dot * scale;
        }
        oracle_softmax_rows(s, 1, nkeys);
        for (long d = 0; d < D; ++d) out[r * D + d] = 0.0;
        for (long j = 0; j < nkeys; ++j)
            for (long d = 0; d < D; ++d) out[r * D + d] += s[j] * v[j * D + d];
        free(s);
    }
    return fail;
}

/* Chain: pre-LN attention block with input and output projections, for one batch element.
 *   z   = LN(x)                       x [S,E]
 *   qkv = z @ w_qkv + b_qkv           [S,3E], columns q | k | v, each H heads of Dh (E = H*Dh)
 *   a[:, h*Dh:(h+1)*Dh] = attention(q_h, k_h, v_h)      per head
 *   out = x + a @ w_o + b_o
 * Nothing is rounded between the stages. */
int oracle_attention_block(const double *x, const double *gamma, const double *beta, double eps,
                           const double *w_qkv, const double *b_qkv, const double *w_o, const double *b_o,
                           double scale, int causal, double *out, long S, long E, long H)
{
    const long Dh = E / H;
    double *z = (double *)malloc(sizeof(double) * (size_t)S * (size_t)E);
    double *qkv = (double *)malloc(sizeof(double) * (size_t)S * (size_t)E * 3);
    double *a = (double *)malloc(sizeof(double) * (size_t)S * (size_t)E);
    double *qh = (double *)malloc(sizeof(double) * (size_t)S * (size_t)Dh * 4);
    long *pos = (long *)malloc(sizeof(long) * (size_t)S);
    int rc = 1;
    if (z && qkv && a && qh && pos) {
        double *kh = qh + S * Dh, *vh = kh + S * Dh, *oh = vh + S * Dh;
        memcpy(z, x, sizeof(double) * (size_t)S * (size_t)E);
        oracle_layernorm_rows(z, S, E, gamma, beta, eps);
        oracle_linear(z, w_qkv, b_qkv, qkv, S, E, 3 * E);
        for (long i = 0; i < S; ++i) pos[i] = i;
        rc = 0;
        for (long h = 0; h < H && !rc; ++h) {
            for (long i = 0; i < S; ++i)
                for (long d = 0; d < Dh; ++d) {
                    qh[i * Dh + d] = qkv[i * 3 * E + 0 * E + h * Dh + d];
                    kh[i * Dh + d] = qkv[i * 3 * E + 1 * E + h * Dh + d];
                    vh[i * Dh + d] = qkv[i * 3 * E + 2 * E + h * Dh + d];
                }
            rc = oracle_attention_rows(qh, pos, S, kh, vh, S, Dh, scale, causal, oh);
            for (long i = 0; i < S; ++i)
                for (long d = 0; d < Dh; ++d) a[i * E + h * Dh + d] = oh[i * Dh + d];
        }
        if (!rc) {
            oracle_linear(a, w_o, b_o, out, S, E, E);
            for (long i = 0; i < S * E; ++i) out[i] += x[i];
        }
    }
    free(z); free(qkv); free(a); free(qh); free(pos);
    return rc;
}
