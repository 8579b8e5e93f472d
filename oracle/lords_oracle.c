/*
 * lords_oracle.c -- CPU oracle for the LoRDS fused dequantize-and-multiply.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * path computes.  It shares no code, header, table or helper with the CUDA
 * library and must never be linked, imported or called by the product path.
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * What it computes (paper letters in brackets; here m = out-features, n =
 * in-features, M = tokens, r = rank):
 *
 *   S   = B * A                       Eq. 3  (S = BA, B: m x r, A: r x n)
 *   W^  = L[Q] (.) S                  Eq. 2 and Sec. 3.2/3.3: W^ = Q (.) (BA),
 *                                     Q_ij a level of the table L (Alg. 1, step 2.1)
 *   y   = x * W^T                     the linear layer; W is stored out x in (Table 7)
 *
 * All arithmetic is fp64, summed sequentially in index order.  Inputs are the
 * exact bytes the GPU path receives: bf16 bit patterns for x, B, A (widened
 * exactly), an fp32 level table, and the packed code bytes, which this file
 * decodes with its OWN reader of the written layout:
 *
 *   rows are packed independently, row i starts at byte i * n * bits / 8;
 *   bits = 4: byte b of a row holds code[2b] in its low nibble, code[2b+1] in its high nibble;
 *   bits = 3: every 32 consecutive codes form a 96-bit little-endian integer
 *             sum_j code[j] << (3 j), stored as 12 bytes, least significant first;
 *   bits = 2: byte b holds code[4b + q] in bits [2q, 2q+2).
 *
 * Pins (see tests/test_oracle_pins.py): block-wise equivalence against an
 * independent Eq. 2 block dequantiser, brute force on tiny inputs, rank-1
 * reduction to a library matmul, linearity in x, an exact-integer case with a
 * closed-form answer, pack known-answer bytes, and the rank rule of Table 7.
 * Not pinned: a forward output on real model weights -- the paper prints no
 * worked numeric example of the forward path ("parity unpinned" for that only).
 *
 * The backward of the layer with the codes frozen (multiplicative fine-tuning of B and A, Sec. 3.4;
 * the chain rule through W^ = L[Q] (.) (BA) as in Eq. 5's gradient with respect to S) is stated in
 * lords_oracle_backward: with g = dL/dy,
 *     dx = g W^,    dW^ = g^T x,    dS = dW^ (.) L[Q],    dB = dS A^T,    dA = B^T dS.
 * Pins: y is linear in every single entry of x, B and A, so replacing one entry by another bf16 value
 * changes the scalar sum(g (.) y) of two forward passes by exactly (difference) x (gradient entry);
 * the tests take such differences on sampled entries, and check <g, y> identities that follow from
 * linearity (sum(dx (.) x) = sum(dB (.) B) = sum(dA (.) A) = sum(g (.) y)).
 *
 * The gradients of quantisation-aware training with the straight-through estimator (Eq. 4-5) are in
 * lords_oracle_backward_qat.  Pins: dL/dW against a library matmul; a weight that its codes represent
 * exactly (W = L[Q] (.) S) has Q - W (/) S = 0, so dB = dA = 0; dL/dS differs from the fine-tuning
 * case above only by the term -dL/dW^ (.) (W (/) S), checked with the pinned fine-tuning gradients
 * and an array-wise quotient; linearity in g.
 *
 * The step before the path, the quantisation step of Alg. 1 (step 2.1), is stated here too
 * (lords_oracle_quantize): Q_ij = argmin over the levels v of (S_ij v - W_ij)^2 with S = BA, every
 * level tried in turn in fp64.  The paper does not say which level wins a tie: the lowest code does.
 * Pins: the codes of an exactly representable W^ are recovered; no other level has a smaller error
 * (an independent array-wise check); exact midpoints go to the lower code; negating S and W together
 * changes nothing; for S > 0 the code does not decrease as W grows.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_ERR_ARG (-1)
#define ORACLE_ERR_CODE_RANGE (-2)
#define ORACLE_ERR_NOMEM (-3)

static double bf16_to_f64(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static int group_ok(int64_t n, int bits)
{
    if (bits == 4) return n % 2 == 0;
    if (bits == 3) return n % 32 == 0;
    if (bits == 2) return n % 4 == 0;
    return 0;
}

/* Read code j of a packed row (bit offset j*bits in the row's little-endian bit stream). */
static unsigned read_code(const uint8_t *row, int64_t j, int bits)
{
    int64_t bit = j * bits;
    unsigned v = 0;
    for (int b = 0; b < bits; ++b) {
        int64_t p = bit + b;
        v |= (unsigned)((row[p >> 3] >> (p & 7)) & 1u) << b;
    }
    return v;
}

int64_t lords_oracle_packed_bytes(int64_t m, int64_t n, int bits)
{
    if (m < 0 || n < 0 || !group_ok(n, bits)) return ORACLE_ERR_ARG;
    return m * (n * bits / 8);
}

/* Layout writer, bit by bit from the written spec (used to build oracle inputs). */
int lords_oracle_pack_codes(const uint8_t *codes, int64_t m, int64_t n, int bits, uint8_t *packed)
{
    if (!codes || !packed || m < 0 || n < 0 || !group_ok(n, bits)) return ORACLE_ERR_ARG;
    int64_t row_bytes = n * bits / 8;
    memset(packed, 0, (size_t)(m * row_bytes));
    for (int64_t i = 0; i < m; ++i) {
        uint8_t *row = packed + i * row_bytes;
        for (int64_t j = 0; j < n; ++j) {
            unsigned c = codes[i * n + j];
            if (c >> bits) return ORACLE_ERR_CODE_RANGE;
            for (int b = 0; b < bits; ++b) {
                int64_t p = j * bits + b;
                row[p >> 3] |= (uint8_t)(((c >> b) & 1u) << (p & 7));
            }
        }
    }
    return ORACLE_OK;
}

int lords_oracle_unpack_codes(const uint8_t *packed, int64_t m, int64_t n, int bits, uint8_t *codes)
{
    if (!codes || !packed || m < 0 || n < 0 || !group_ok(n, bits)) return ORACLE_ERR_ARG;
    int64_t row_bytes = n * bits / 8;
    for (int64_t i = 0; i < m; ++i)
        for (int64_t j = 0; j < n; ++j)
            codes[i * n + j] = (uint8_t)read_code(packed + i * row_bytes, j, bits);
    return ORACLE_OK;
}

/* Row i of S = B A (Eq. 3), n doubles. */
static void scale_row(const uint16_t *B, const uint16_t *A, int64_t n, int64_t r, int64_t i, double *S_row)
{
    for (int64_t j = 0; j < n; ++j) {
        double s = 0.0;
        for (int64_t k = 0; k < r; ++k) s += bf16_to_f64(B[i * r + k]) * bf16_to_f64(A[k * n + j]);
        S_row[j] = s;
    }
}

/*
 * Rows of the dequantised weight W^ = L[Q] (.) (B A).  rows == NULL means rows 0..nrows-1.
 * W_out is nrows x n doubles.
 */
int lords_oracle_dequant_rows(const uint8_t *qpacked, const uint16_t *B, const uint16_t *A,
                              const float *codebook, int bits, int64_t m, int64_t n, int64_t r,
                              const int64_t *rows, int64_t nrows, double *W_out)
{
    if (!qpacked || !B || !A || !codebook || !W_out || m < 1 || n < 1 || r < 1 || !group_ok(n, bits))
        return ORACLE_ERR_ARG;
    int64_t row_bytes = n * bits / 8;
    for (int64_t q = 0; q < nrows; ++q) {
        int64_t i = rows ? rows[q] : q;
        if (i < 0 || i >= m) return ORACLE_ERR_ARG;
        double *W_row = W_out + q * n;
        scale_row(B, A, n, r, i, W_row);
        for (int64_t j = 0; j < n; ++j)
            W_row[j] = (double)codebook[read_code(qpacked + i * row_bytes, j, bits)] * W_row[j];
    }
    return ORACLE_OK;
}

/*
 * y[t][q] = sum_j x[t][j] * W^[rows[q]][j] for t < M, q < nrows, fp64.
 * rows == NULL means rows 0..nrows-1 (pass nrows = m for the full output).
 * y64 is M x nrows row-major.  Rows are independent and are spread over `threads`
 * OpenMP threads (<= 0: all available); the arithmetic of one output does not
 * depend on the thread count.  Returns the thread count used (> 0) or an error (< 0).
 */
int lords_oracle_forward(const uint16_t *x, const uint8_t *qpacked, const uint16_t *B, const uint16_t *A,
                         const float *codebook, int bits, int64_t M, int64_t m, int64_t n, int64_t r,
                         const int64_t *rows, int64_t nrows, double *y64, int threads)
{
    if (!x || !qpacked || !B || !A || !codebook || !y64 || M < 1 || m < 1 || n < 1 || r < 1 ||
        nrows < 0 || !group_ok(n, bits))
        return ORACLE_ERR_ARG;
    for (int64_t q = 0; q < nrows; ++q) {
        int64_t i = rows ? rows[q] : q;
        if (i < 0 || i >= m) return ORACLE_ERR_ARG;
    }
    int64_t row_bytes = n * bits / 8;
    int used = 1;
    int fail = 0;
#ifdef _OPENMP
    if (threads <= 0) threads = omp_get_max_threads();
    used = threads;
#else
    (void)threads;
#endif
    /* x widened once: M x n doubles */
    double *xd = (double *)malloc(sizeof(double) * (size_t)(M * n));
    if (!xd) return ORACLE_ERR_NOMEM;
    for (int64_t e = 0; e < M * n; ++e) xd[e] = bf16_to_f64(x[e]);

#pragma omp parallel num_threads(used)
    {
        double *W_row = (double *)malloc(sizeof(double) * (size_t)n);
        if (!W_row) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp for schedule(dynamic, 4)
        for (int64_t q = 0; q < nrows; ++q) {
            if (!W_row) continue;
            int64_t i = rows ? rows[q] : q;
            scale_row(B, A, n, r, i, W_row);                                   /* S_i = (BA)_i      */
            for (int64_t j = 0; j < n; ++j)                                    /* W^_ij = L[Q_ij] S_ij */
                W_row[j] = (double)codebook[read_code(qpacked + i * row_bytes, j, bits)] * W_row[j];
            for (int64_t t = 0; t < M; ++t) {                                  /* y_ti = sum_j x_tj W^_ij */
                double acc = 0.0;
                const double *xt = xd + t * n;
                for (int64_t j = 0; j < n; ++j) acc += xt[j] * W_row[j];
                y64[t * nrows + q] = acc;
            }
        }
        free(W_row);
    }
    free(xd);
    return fail ? ORACLE_ERR_NOMEM : used;
}

/*
 * Round fp64 values to bf16 with one round-to-nearest-even step (no intermediate
 * fp32 rounding) and return the bit patterns.  Values beyond the bf16 range become
 * infinities; NaN maps to a quiet NaN.
 */
void lords_oracle_round_bf16(const double *v, int64_t count, uint16_t *out)
{
    for (int64_t e = 0; e < count; ++e) {
        double d = v[e];
        uint16_t sign = (uint16_t)(signbit(d) ? 0x8000u : 0u);
        double a = fabs(d);
        if (isnan(d)) { out[e] = 0x7FC0u; continue; }
        if (a == 0.0) { out[e] = sign; continue; }
        int ex;
        (void)frexp(a, &ex);                 /* a = f * 2^ex, f in [0.5, 1) */
        int e2 = ex - 1;                     /* a = g * 2^e2, g in [1, 2)   */
        if (e2 < -126) e2 = -126;            /* subnormal range: fixed quantum 2^-133 */
        double quantum = ldexp(1.0, e2 - 7); /* 8-bit significand */
        double qv = nearbyint(a / quantum) * quantum; /* default rounding mode: nearest even */
        float f = (float)qv;                 /* exact: qv is a bf16 value or overflows to inf */
        if (qv > 3.3895313892515355e38) f = INFINITY;
        uint32_t u;
        memcpy(&u, &f, sizeof u);
        out[e] = (uint16_t)(sign | (uint16_t)(u >> 16));
    }
}

/* Equivalent-rank rule of Sec. 3.2 / App. A: r = floor(n m / (blk (n + m))). */
int64_t lords_oracle_equivalent_rank(int64_t rows, int64_t cols, int64_t blk)
{
    if (rows < 1 || cols < 1 || blk < 1) return ORACLE_ERR_ARG;
    return (rows * cols) / (blk * (rows + cols));
}

/*
 * Quantisation step (Alg. 1, step 2.1; Sec. 3.3 "nearest-neighbor search in the look-up table"):
 *   Q_ij = argmin_{c} (S_ij * L[c] - W_ij)^2,  S = B A (Eq. 3),  ties -> the lowest code.
 * W, B, A are bf16 bit patterns (W: m x n), widened exactly; all arithmetic fp64.
 *   codes_out  : m*n bytes, one code per byte
 *   runner_out : (may be NULL) the best code among the others (lowest code on ties)
 *   gap_out    : (may be NULL) |S L[runner] - W| - |S L[best] - W| >= 0: by how much the choice was clear
 *   mag_out    : (may be NULL) (sum_k |B_ik A_kj|) * max|L| + |W|: the magnitude the gap is to be compared with
 *                (a sum of r products rounds in proportion to the sum of their absolute values, which
 *                under cancellation is much larger than |S| itself)
 */
int lords_oracle_quantize(const uint16_t *W, const uint16_t *B, const uint16_t *A, const float *codebook, int bits,
                          int64_t m, int64_t n, int64_t r, uint8_t *codes_out, uint8_t *runner_out, double *gap_out,
                          double *mag_out)
{
    if (!W || !B || !A || !codebook || !codes_out || m < 0 || n < 0 || r < 1) return ORACLE_ERR_ARG;
    if (bits != 2 && bits != 3 && bits != 4) return ORACLE_ERR_ARG;
    const int levels = 1 << bits;
    double lmax = 0.0;
    for (int c = 0; c < levels; ++c)
        if (fabs((double)codebook[c]) > lmax) lmax = fabs((double)codebook[c]);
    int rc = ORACLE_OK;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < m; ++i) {
        double *S_row = (double *)malloc((size_t)(n > 0 ? n : 1) * sizeof(double));
        if (!S_row) {
#pragma omp critical
            rc = ORACLE_ERR_NOMEM;
            continue;
        }
        scale_row(B, A, n, r, i, S_row);
        for (int64_t j = 0; j < n; ++j) {
            const double w = bf16_to_f64(W[i * n + j]);
            int best = -1, runner = -1;
            double e_best = 0.0, e_runner = 0.0;
            for (int c = 0; c < levels; ++c) {
                const double d = S_row[j] * (double)codebook[c] - w;
                const double e = d * d;
                if (best < 0 || e < e_best) {
                    runner = best; e_runner = e_best;
                    best = c; e_best = e;
                } else if (runner < 0 || e < e_runner) {
                    runner = c; e_runner = e;
                }
            }
            codes_out[i * n + j] = (uint8_t)best;
            if (runner_out) runner_out[i * n + j] = (uint8_t)runner;
            if (gap_out) gap_out[i * n + j] = sqrt(e_runner) - sqrt(e_best);
            if (mag_out) {
                double sabs = 0.0;
                for (int64_t k = 0; k < r; ++k) sabs += fabs(bf16_to_f64(B[i * r + k]) * bf16_to_f64(A[k * n + j]));
                mag_out[i * n + j] = sabs * lmax + fabs(w);
            }
        }
        free(S_row);
    }
    return rc;
}

/*
 * Backward of y = x W^T, W^ = L[Q] (.) (B A), with the codes fixed (Sec. 3.4: only B and A are trained;
 * Eq. 5 gives the same chain rule through S = BA).  g = dL/dy is M x m (bf16 bit patterns, like x).
 *   dx = g W^                       M x n
 *   dW^ = g^T x                     m x n   (held row by row only)
 *   dS  = dW^ (.) L[Q]
 *   dB  = dS A^T                    m x r
 *   dA  = B^T dS                    r x n
 * Any of dx, dB, dA may be NULL.  fp64, sums in index order (dA: rows of W in order).
 */
int lords_oracle_backward(const uint16_t *g, const uint16_t *x, const uint8_t *qpacked, const uint16_t *B,
                          const uint16_t *A, const float *codebook, int bits, int64_t M, int64_t m, int64_t n,
                          int64_t r, double *dx, double *dB, double *dA)
{
    if (!g || !x || !qpacked || !B || !A || !codebook || M < 1 || m < 1 || n < 1 || r < 1 || !group_ok(n, bits))
        return ORACLE_ERR_ARG;
    int64_t row_bytes = n * bits / 8;
    double *S_row = (double *)malloc(sizeof(double) * (size_t)n);
    double *dS_row = (double *)malloc(sizeof(double) * (size_t)n);
    if (!S_row || !dS_row) {
        free(S_row); free(dS_row);
        return ORACLE_ERR_NOMEM;
    }
    if (dx) for (int64_t e = 0; e < M * n; ++e) dx[e] = 0.0;
    if (dA) for (int64_t e = 0; e < r * n; ++e) dA[e] = 0.0;
    for (int64_t i = 0; i < m; ++i) {
        const uint8_t *qrow = qpacked + i * row_bytes;
        scale_row(B, A, n, r, i, S_row);                                        /* S_i = (BA)_i */
        for (int64_t j = 0; j < n; ++j) {
            double level = (double)codebook[read_code(qrow, j, bits)];
            double dW = 0.0;                                                    /* dW^_ij = sum_t g_ti x_tj */
            for (int64_t t = 0; t < M; ++t) dW += bf16_to_f64(g[t * m + i]) * bf16_to_f64(x[t * n + j]);
            dS_row[j] = dW * level;                                             /* dS_ij = dW^_ij L[Q_ij] */
            if (dx) {
                double w = level * S_row[j];                                    /* W^_ij */
                for (int64_t t = 0; t < M; ++t) dx[t * n + j] += bf16_to_f64(g[t * m + i]) * w;
            }
        }
        if (dB)
            for (int64_t k = 0; k < r; ++k) {                                   /* dB_ik = sum_j dS_ij A_kj */
                double acc = 0.0;
                for (int64_t j = 0; j < n; ++j) acc += dS_row[j] * bf16_to_f64(A[k * n + j]);
                dB[i * r + k] = acc;
            }
        if (dA)
            for (int64_t k = 0; k < r; ++k) {                                   /* dA_kj += B_ik dS_ij */
                double b = bf16_to_f64(B[i * r + k]);
                for (int64_t j = 0; j < n; ++j) dA[k * n + j] += b * dS_row[j];
            }
    }
    free(S_row);
    free(dS_row);
    return ORACLE_OK;
}

/*
 * Backward of quantisation-aware training (Sec. 3.3, Eq. 4-5): the fake-quantised weight is
 * W^ = Round(W (/) S) (.) S with S = B A, and with the straight-through estimator
 *     dL/dW = dL/dW^                                  (Eq. 4)
 *     dL/dS = dL/dW^ (.) (Q - W (/) S)                (Eq. 5),   Q = Round(W (/) S) = the level L[code]
 * and then dB = dL/dS A^T, dA = B^T dL/dS as for any function of S = B A.  Here dL/dW^ = g^T x for
 * the layer y = x W^T, the codes are the given ones (the rounding has been done), and an element
 * whose S is exactly zero, where the quotient is undefined, gets dL/dS = 0.
 *   W   : bf16 [m][n], the latent full-precision weight
 *   dW  : m x n doubles (may be NULL), dB : m x r (may be NULL), dA : r x n (may be NULL)
 */
int lords_oracle_backward_qat(const uint16_t *g, const uint16_t *x, const uint16_t *W, const uint8_t *qpacked,
                              const uint16_t *B, const uint16_t *A, const float *codebook, int bits, int64_t M,
                              int64_t m, int64_t n, int64_t r, double *dW, double *dB, double *dA)
{
    if (!g || !x || !W || !qpacked || !B || !A || !codebook || M < 1 || m < 1 || n < 1 || r < 1 || !group_ok(n, bits))
        return ORACLE_ERR_ARG;
    int64_t row_bytes = n * bits / 8;
    double *S_row = (double *)malloc(sizeof(double) * (size_t)n);
    double *dS_row = (double *)malloc(sizeof(double) * (size_t)n);
    if (!S_row || !dS_row) {
        free(S_row); free(dS_row);
        return ORACLE_ERR_NOMEM;
    }
    if (dA) for (int64_t e = 0; e < r * n; ++e) dA[e] = 0.0;
    for (int64_t i = 0; i < m; ++i) {
        const uint8_t *qrow = qpacked + i * row_bytes;
        scale_row(B, A, n, r, i, S_row);
        for (int64_t j = 0; j < n; ++j) {
            double dWhat = 0.0;                                                 /* dL/dW^_ij = sum_t g_ti x_tj */
            for (int64_t t = 0; t < M; ++t) dWhat += bf16_to_f64(g[t * m + i]) * bf16_to_f64(x[t * n + j]);
            if (dW) dW[i * n + j] = dWhat;                                      /* Eq. 4 */
            double level = (double)codebook[read_code(qrow, j, bits)];
            dS_row[j] = S_row[j] != 0.0 ? dWhat * (level - bf16_to_f64(W[i * n + j]) / S_row[j]) : 0.0;   /* Eq. 5 */
        }
        if (dB)
            for (int64_t k = 0; k < r; ++k) {
                double acc = 0.0;
                for (int64_t j = 0; j < n; ++j) acc += dS_row[j] * bf16_to_f64(A[k * n + j]);
                dB[i * r + k] = acc;
            }
        if (dA)
            for (int64_t k = 0; k < r; ++k) {
                double b = bf16_to_f64(B[i * r + k]);
                for (int64_t j = 0; j < n; ++j) dA[k * n + j] += b * dS_row[j];
            }
    }
    free(S_row);
    free(dS_row);
    return ORACLE_OK;
}

