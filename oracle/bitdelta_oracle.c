/*
 * BitDelta fused GEMM -- CPU oracle.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain definition that the CUDA library is checked
 * against.  Only the tests, the smoke check and the benchmark's CPU-baseline
 * leg may build or call it; the product path never does.  It shares no code,
 * header, table or helper with the CUDA sources.
 *
 * What it computes (the multi-tenant BitDelta product: a shared base weight
 * plus a per-tenant 1-bit delta scaled by a per-tenant scalar; the paper's
 * BitDelta paragraph in "Recently Published Kernels" fixes only the decode
 * s = 2*bit - 1, everything else is the task's formula):
 *
 *   Y[b,t,n] = sum_k x[b,t,k] * w[n,k]  +  alpha[b] * sum_k x[b,t,k] * s[b,n,k]
 *   s[b,n,k] = +1 if bit (k mod 32) of word bits[b,n,k div 32] is set, else -1
 *
 * x and w are bf16 bit patterns widened exactly to double, alpha is fp32
 * widened exactly to double, both sums run in double in plain k order and the
 * result is kept in double (never rounded to bf16).
 *
 * Parity pins: every function here is pinned by tests that do not reuse it
 * (hand-computed values, one-hot probes, numpy fp64 matmul on a dense S built
 * by independent Python code, brute-force Python loops, algebraic invariants;
 * for the extended product at the end of the file also numpy's float16 on
 * every finite pattern and closed forms of the sigmoid).
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* bf16 -> double: a bf16 is the upper 16 bits of an IEEE-754 binary32. */
static double bf16_to_double(uint16_t h)
{
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* sign of weight k in a packed row: bit = 1 means +1, bit = 0 means -1,
 * least-significant bit first along K. */
static double sign_at(const uint32_t *row_words, int k)
{
    uint32_t word = row_words[k / 32];
    uint32_t bit = (word >> (k % 32)) & 1u;
    return bit ? 1.0 : -1.0;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* pack: word[b,n,w] = sum_j [S[b,n,32w+j] > 0] << j.  K must be a multiple of 32. */
void oracle_pack(const int8_t *S, uint32_t *bits, int B, int N, int K)
{
    long long rows = (long long)B * N;
    int words = K / 32;
    for (long long r = 0; r < rows; ++r) {
        for (int w = 0; w < words; ++w) {
            uint32_t word = 0;
            for (int j = 0; j < 32; ++j) {
                if (S[r * K + 32 * w + j] > 0) word |= (1u << j);
            }
            bits[r * words + w] = word;
        }
    }
}

/* unpack: the inverse map to +1 / -1. */
void oracle_unpack(const uint32_t *bits, int8_t *S, int B, int N, int K)
{
    long long rows = (long long)B * N;
    int words = K / 32;
    for (long long r = 0; r < rows; ++r) {
        for (int k = 0; k < K; ++k) {
            S[r * K + k] = (int8_t)sign_at(bits + r * words, k);
        }
    }
}

/* Full result.  X [B,m,K] bf16 bits, W [N,K] bf16 bits, bits [B,N,K/32],
 * alpha [B] fp32, Y [B,m,N] double. */
void oracle_gemm(const uint16_t *X, const uint16_t *W, const uint32_t *bits,
                 const float *alpha, double *Y, int B, int m, int N, int K)
{
    int words = K / 32;
    double *xd = (double *)malloc(sizeof(double) * (size_t)B * m * K);
    double *wd = (double *)malloc(sizeof(double) * (size_t)N * K);
    for (size_t i = 0; i < (size_t)B * m * K; ++i) xd[i] = bf16_to_double(X[i]);
    for (size_t i = 0; i < (size_t)N * K; ++i) wd[i] = bf16_to_double(W[i]);

    long long rows = (long long)B * N;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)K);
#pragma omp for schedule(static)
        for (long long r = 0; r < rows; ++r) {
            int b = (int)(r / N);
            int n = (int)(r % N);
            const uint32_t *row_words = bits + (size_t)r * words;
            for (int k = 0; k < K; ++k) s[k] = sign_at(row_words, k);
            const double *wrow = wd + (size_t)n * K;
            double a = (double)alpha[b];
            for (int t = 0; t < m; ++t) {
                const double *xrow = xd + ((size_t)b * m + t) * K;
                double base = 0.0, delta = 0.0;
                for (int k = 0; k < K; ++k) {
                    base += xrow[k] * wrow[k];
                    delta += xrow[k] * s[k];
                }
                Y[((size_t)b * m + t) * N + n] = base + a * delta;
            }
        }
        free(s);
    }
    free(xd);
    free(wd);
}

/* The same definition evaluated only at `count` listed outputs
 * (idx holds count triples b,t,n); out[i] is Y[b,t,n].  Used where a full
 * result would take too long. */
void oracle_gemm_at(const uint16_t *X, const uint16_t *W, const uint32_t *bits,
                    const float *alpha, const int32_t *idx, int count, double *out,
                    int B, int m, int N, int K)
{
    int words = K / 32;
    (void)B;
#pragma omp parallel for schedule(static)
    for (int i = 0; i < count; ++i) {
        int b = idx[3 * i + 0], t = idx[3 * i + 1], n = idx[3 * i + 2];
        const uint16_t *xrow = X + ((size_t)b * m + t) * K;
        const uint16_t *wrow = W + (size_t)n * K;
        const uint32_t *row_words = bits + ((size_t)b * N + n) * words;
        double base = 0.0, delta = 0.0;
        for (int k = 0; k < K; ++k) {
            double x = bf16_to_double(xrow[k]);
            base += x * bf16_to_double(wrow[k]);
            delta += x * sign_at(row_words, k);
        }
        out[i] = base + (double)alpha[b] * delta;
    }
}

/*
 * compress: the step before the product -- derive a tenant's 1-bit delta from its fine-tuned weights
 * (the BitDelta method the paper cites in its BitDelta paragraph; the paper itself does not spell it
 * out, so this is the method's plain definition):
 *
 *   delta[b,n,k] = wf[b,n,k] - wb[n,k]                      (bf16 widened exactly to double)
 *   bit  (k mod 32) of bits[b,n,k div 32] = [delta > 0]     (so zero and negative deltas decode to -1)
 *   alpha[b] = (1 / (N K)) * sum_{n,k} |delta[b,n,k]|       (double, plain (n,k) order), rounded to fp32
 *
 * K must be a multiple of 32.
 */
void oracle_compress(const uint16_t *wf, const uint16_t *wb, uint32_t *bits, float *alpha, int B, int N, int K)
{
    int words = K / 32;
    for (int b = 0; b < B; ++b) {
        double sum_abs = 0.0;
        for (int n = 0; n < N; ++n) {
            for (int w = 0; w < words; ++w) {
                uint32_t word = 0;
                for (int j = 0; j < 32; ++j) {
                    int k = 32 * w + j;
                    double d = bf16_to_double(wf[((long long)b * N + n) * K + k]) - bf16_to_double(wb[(long long)n * K + k]);
                    if (d > 0.0) word |= (1u << j);
                    sum_abs += (d < 0.0) ? -d : d;
                }
                bits[((long long)b * N + n) * words + w] = word;
            }
        }
        alpha[b] = (float)(sum_abs / ((double)N * (double)K));
    }
}


/*
 * Extended product (an adjacent variant: the paper's own BitDelta kernel computes in FP16, and its suite
 * fuses activations into GEMM epilogues; neither is spelled out for this product, so this is the plain
 * definition):
 *
 *   Y[b,t,n] = act( sum_k x w  +  alpha[b] * sum_k x s  +  bias[n] )
 *
 * dtype 0: x, w, bias are bf16 bit patterns; dtype 1: IEEE-754 binary16 bit patterns.
 * bias may be NULL (no bias).  act 0: identity; act 1: SiLU, y * sigmoid(y) = y / (1 + exp(-y)).
 * act 2: SiLU gate of a gated MLP whose gate and up projections are interleaved along N: with
 *   z[b,t,n] = sum_k x w + alpha[b] sum_k x s + bias[n]   (N even),
 *   Y[b,t,i] = SiLU(z[b,t,2i]) * z[b,t,2i+1],   i < N/2     (row 2i: gate, row 2i+1: up),
 * so the result has N/2 features per token.
 * Everything is widened exactly to double; sums in double in plain k order; result kept in double.
 */
#include <math.h>

/* binary16 -> double by the format's definition: 1 sign, 5 exponent (bias 15), 10 fraction bits. */
static double half_to_double(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1F;
    int f = h & 0x3FF;
    double v;
    if (e == 0) v = ldexp((double)f, -24);                 /* zero and subnormals: f * 2^-24 */
    else if (e == 31) v = f ? NAN : INFINITY;
    else v = ldexp(1.0 + (double)f / 1024.0, e - 15);
    return sign ? -v : v;
}

void oracle_half_to_double(const uint16_t *h, double *out, long long count)
{
    for (long long i = 0; i < count; ++i) out[i] = half_to_double(h[i]);
}

static double widen16(uint16_t v, int dtype)
{
    return dtype == 1 ? half_to_double(v) : bf16_to_double(v);
}

static double silu(double y)
{
    return y / (1.0 + exp(-y));
}

static double finish(double y, double bias, int act)
{
    y += bias;
    if (act == 1) y = silu(y);
    return y;
}

/* z[b,t,n] before any activation */
static double preact(const uint16_t *X, const uint16_t *W, const uint32_t *bits, const float *alpha,
                     const uint16_t *bias, int b, int t, int n, int m, int N, int K, int dtype)
{
    int words = K / 32;
    const uint16_t *xrow = X + ((size_t)b * m + t) * K;
    const uint16_t *wrow = W + (size_t)n * K;
    const uint32_t *row_words = bits + ((size_t)b * N + n) * words;
    double base = 0.0, delta = 0.0;
    for (int k = 0; k < K; ++k) {
        double x = widen16(xrow[k], dtype);
        base += x * widen16(wrow[k], dtype);
        delta += x * sign_at(row_words, k);
    }
    return base + (double)alpha[b] * delta + (bias ? widen16(bias[n], dtype) : 0.0);
}

/* The extended definition at `count` listed outputs (idx holds count triples b,t,n), or, with idx == NULL,
 * at every output in (b,t,n) order (count is then ignored and out holds B*m*N values). */
void oracle_gemm_ex(const uint16_t *X, const uint16_t *W, const uint32_t *bits, const float *alpha,
                    const uint16_t *bias, const int32_t *idx, int count, double *out,
                    int B, int m, int N, int K, int dtype, int act)
{
    int words = K / 32;
    int No = (act == 2) ? N / 2 : N;   /* output features per token */
    long long total = idx ? (long long)count : (long long)B * m * No;
#pragma omp parallel for schedule(static)
    for (long long i = 0; i < total; ++i) {
        int b, t, n;
        if (idx) {
            b = idx[3 * i + 0]; t = idx[3 * i + 1]; n = idx[3 * i + 2];
        } else {
            n = (int)(i % No); t = (int)((i / No) % m); b = (int)(i / ((long long)No * m));
        }
        if (act == 2) {
            double gate = preact(X, W, bits, alpha, bias, b, t, 2 * n, m, N, K, dtype);
            double up = preact(X, W, bits, alpha, bias, b, t, 2 * n + 1, m, N, K, dtype);
            out[i] = silu(gate) * up;
            continue;
        }
        const uint16_t *xrow = X + ((size_t)b * m + t) * K;
        const uint16_t *wrow = W + (size_t)n * K;
        const uint32_t *row_words = bits + ((size_t)b * N + n) * words;
        double base = 0.0, delta = 0.0;
        for (int k = 0; k < K; ++k) {
            double x = widen16(xrow[k], dtype);
            base += x * widen16(wrow[k], dtype);
            delta += x * sign_at(row_words, k);
        }
        out[i] = finish(base + (double)alpha[b] * delta, bias ? widen16(bias[n], dtype) : 0.0, act);
    }
}
