/*
 * CPU oracle for the MXInt (block floating point) linear layer of arXiv 2307.15517.
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, obviously-correct C.  It shares no code,
 * header, table or helper with the CUDA library and must never sit on the product
 * path: only the tests, the smoke check and the benchmark's CPU-baseline leg call it.
 *
 * What it follows (paper sections):
 *   - Sec. 2 "What are MX Formats?": MXInt == block floating point, one exponent shared
 *     by the block, which bounds the range of the block's values.
 *   - Sec. 4.1 "Software Design Parameters": the format is a tuple (B, e, m); average
 *     bits p = e/prod(B) + m + 1 (Eq. 1); e fixed to 8 bits.
 *   - Sec. 3.2 (software emulators): an MX operator == quantize inputs, run the plain
 *     floating-point operator on the dequantized values.
 *   - Sec. 3.2 (hardware operators, Fig. 3 right): the MXInt dot product multiplies and
 *     adds integer mantissas inside a block and applies the shared exponent once per block.
 *
 * The paper fixes neither the exponent derivation, the binary point nor the rounding.
 * The readings used here (w = total signed width, paper m = w - 1):
 *   E      = floor(log2(max|x| over the block)), stored as byte E+127 (the binary32
 *            exponent field of the block maximum); zero/subnormal maximum -> byte 0;
 *            Inf/NaN in the block -> byte 255, all mantissas 0.
 *   s      = 2^(E - (w-2))
 *   q      = clamp(round_half_even(x / s), -(2^(w-1)-1), +(2^(w-1)-1))
 *   x_hat  = q * s
 *   Y[i,j] = sum_b 2^(Ea[i,b] + Ew[j,b] - (wa-2) - (ww-2)) * sum_{k in b} qa[i,k] qw[j,k]
 *
 * Parity pins live in tests/test_oracle_pins.py (hand-worked blocks, exact rational brute
 * force, fp64 library matmul on representable inputs, invariants).  Unpinned by the paper
 * itself (pinned only by the readings above): rounding mode, binary-point position and the
 * symmetric clamp -- "parity unpinned" for those three choices.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define MXO_OK 0
#define MXO_BAD_ARG (-1)

static int mxo_args_ok(int64_t rows, int64_t K, int B, int w)
{
    if (rows < 0 || K < 0) return 0;
    if (B <= 0 || (K % B) != 0) return 0;
    if (w < 2 || w > 8) return 0;
    return 1;
}

/* Exponent byte of a non-negative float: its binary32 biased exponent field. */
static int mxo_exponent_byte(float amax)
{
    if (isnan(amax) || isinf(amax)) return 255;
    if (amax < 1.17549435082228750797e-38f) return 0; /* zero or subnormal */
    int ex;
    (void)frexpf(amax, &ex);          /* amax = f * 2^ex, f in [0.5, 1) */
    return (ex - 1) + 127;            /* floor(log2(amax)) + bias */
}

/*
 * Quantize x (rows x K, element (r,k) at x[r*stride_row + k*stride_k]) into int8 mantissas
 * q[r*K + k] and exponent bytes ebyte[r*(K/B) + k/B].  Blocks run along k.
 * nonfinite (nullable) receives the number of blocks that held an Inf or NaN.
 */
int mxo_quantize(const float *x, int64_t rows, int64_t K, int64_t stride_row, int64_t stride_k,
                 int B, int w, int8_t *q, uint8_t *ebyte, uint32_t *nonfinite)
{
    if (!mxo_args_ok(rows, K, B, w)) return MXO_BAD_ARG;
    const int64_t nb = K / B;
    const double qmax = (double)((1 << (w - 1)) - 1);
    uint32_t bad = 0;
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t b = 0; b < nb; ++b) {
            float amax = 0.0f;
            int any_nonfinite = 0;
            for (int k = 0; k < B; ++k) {
                float v = x[r * stride_row + (b * B + k) * stride_k];
                if (isnan(v) || isinf(v)) any_nonfinite = 1;
                float a = fabsf(v);
                if (a > amax) amax = a;
            }
            int8_t *qb = q + r * K + b * B;
            if (any_nonfinite) {
                ebyte[r * nb + b] = 255;
                for (int k = 0; k < B; ++k) qb[k] = 0;
                ++bad;
                continue;
            }
            const int eb = mxo_exponent_byte(amax);
            ebyte[r * nb + b] = (uint8_t)eb;
            const double s = ldexp(1.0, (eb - 127) - (w - 2));
            for (int k = 0; k < B; ++k) {
                double v = (double)x[r * stride_row + (b * B + k) * stride_k] / s; /* exact */
                double n = nearbyint(v);      /* default rounding mode: ties to even */
                if (n > qmax) n = qmax;
                if (n < -qmax) n = -qmax;
                qb[k] = (int8_t)n;
            }
        }
    }
    if (nonfinite) *nonfinite = bad;
    return MXO_OK;
}

/* x_hat = q * 2^(E-(w-2)); blocks with exponent byte 255 dequantize to NaN. */
int mxo_dequantize(const int8_t *q, const uint8_t *ebyte, int64_t rows, int64_t K, int B, int w,
                   double *xhat)
{
    if (!mxo_args_ok(rows, K, B, w)) return MXO_BAD_ARG;
    const int64_t nb = K / B;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k) {
            int eb = ebyte[r * nb + k / B];
            xhat[r * K + k] = (eb == 255) ? (double)NAN
                                          : ldexp((double)q[r * K + k], (eb - 127) - (w - 2));
        }
    return MXO_OK;
}

/*
 * Storage container: w <= 4 -> two two's-complement nibbles per byte, even k in the low
 * nibble; 5 <= w <= 8 -> one int8 per element.  out holds rows*K/2 or rows*K bytes.
 */
int mxo_pack(const int8_t *q, int64_t rows, int64_t K, int w, uint8_t *out)
{
    if (w < 2 || w > 8 || rows < 0 || K < 0 || (K & 1)) return MXO_BAD_ARG;
    const int64_t n = rows * K;
    if (w > 4) {
        memcpy(out, q, (size_t)n);
        return MXO_OK;
    }
    for (int64_t i = 0; i < n; i += 2) {
        uint8_t lo = (uint8_t)q[i] & 0xF, hi = (uint8_t)q[i + 1] & 0xF;
        out[i / 2] = (uint8_t)(lo | (hi << 4));
    }
    return MXO_OK;
}

int mxo_unpack(const uint8_t *in, int64_t rows, int64_t K, int w, int8_t *q)
{
    if (w < 2 || w > 8 || rows < 0 || K < 0 || (K & 1)) return MXO_BAD_ARG;
    const int64_t n = rows * K;
    if (w > 4) {
        memcpy(q, in, (size_t)n);
        return MXO_OK;
    }
    for (int64_t i = 0; i < n; i += 2) {
        int lo = in[i / 2] & 0xF, hi = in[i / 2] >> 4;
        q[i] = (int8_t)(lo >= 8 ? lo - 16 : lo);
        q[i + 1] = (int8_t)(hi >= 8 ? hi - 16 : hi);
    }
    return MXO_OK;
}

/* One output element: wide reference, sequential-fp32 variant and condition scale. */
static void mxo_dot(const int8_t *qa, const uint8_t *ea, int wa, const int8_t *qw,
                    const uint8_t *ew, int ww, int64_t K, int B, const float *bias_j,
                    float *y_ref, float *y_seq, double *S)
{
    const int64_t nb = K / B;
    long double wide = 0.0L;
    double sabs = 0.0;
    float seq = 0.0f;
    int poisoned = 0;
    for (int64_t b = 0; b < nb; ++b) {
        if (ea[b] == 255 || ew[b] == 255) { poisoned = 1; continue; }
        int64_t P = 0;
        for (int k = 0; k < B; ++k) P += (int64_t)qa[b * B + k] * (int64_t)qw[b * B + k];
        const int e = ((int)ea[b] - 127) + ((int)ew[b] - 127) - (wa - 2) - (ww - 2);
        const double t = ldexp((double)P, e); /* exact: |P| < 2^53 and e well inside double */
        wide += (long double)t;
        sabs += fabs(t);
        seq = seq + (float)t;                  /* fp32 add, ascending block order */
    }
    if (bias_j) {
        wide += (long double)*bias_j;
        sabs += fabs((double)*bias_j);
        seq = seq + *bias_j;
    }
    if (poisoned) {
        if (y_ref) *y_ref = NAN;
        if (y_seq) *y_seq = NAN;
        if (S) *S = (double)NAN;
        return;
    }
    if (y_ref) *y_ref = (float)wide;           /* one rounding to fp32 */
    if (y_seq) *y_seq = seq;
    if (S) *S = sabs;
}

/*
 * Y = A * W^T (+ bias).  qa [M,K], ea [M,K/B], qw [N,K], ew [N,K/B]; outputs [M,N]
 * (each nullable).  A and W must share the block size B.
 */
int mxo_gemm(const int8_t *qa, const uint8_t *ea, int wa, const int8_t *qw, const uint8_t *ew,
             int ww, int64_t M, int64_t N, int64_t K, int B, const float *bias, float *y_ref,
             float *y_seq, double *S)
{
    if (!mxo_args_ok(M, K, B, wa) || !mxo_args_ok(N, K, B, ww)) return MXO_BAD_ARG;
    const int64_t nb = K / B;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i)
        for (int64_t j = 0; j < N; ++j)
            mxo_dot(qa + i * K, ea + i * nb, wa, qw + j * K, ew + j * nb, ww, K, B,
                    bias ? bias + j : 0, y_ref ? y_ref + i * N + j : 0,
                    y_seq ? y_seq + i * N + j : 0, S ? S + i * N + j : 0);
    return MXO_OK;
}

/* The same, for n chosen output positions (si[t], sj[t]); outputs have n entries. */
int mxo_gemm_samples(const int8_t *qa, const uint8_t *ea, int wa, const int8_t *qw,
                     const uint8_t *ew, int ww, int64_t M, int64_t N, int64_t K, int B,
                     const float *bias, const int64_t *si, const int64_t *sj, int64_t n,
                     float *y_ref, float *y_seq, double *S)
{
    if (!mxo_args_ok(M, K, B, wa) || !mxo_args_ok(N, K, B, ww)) return MXO_BAD_ARG;
    const int64_t nb = K / B;
    for (int64_t t = 0; t < n; ++t)
        if (si[t] < 0 || si[t] >= M || sj[t] < 0 || sj[t] >= N) return MXO_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < n; ++t) {
        const int64_t i = si[t], j = sj[t];
        mxo_dot(qa + i * K, ea + i * nb, wa, qw + j * K, ew + j * nb, ww, K, B,
                bias ? bias + j : 0, y_ref ? y_ref + t : 0, y_seq ? y_seq + t : 0,
                S ? S + t : 0);
    }
    return MXO_OK;
}

/*
 * The operator with an MXInt result (Sec. 3.2, software emulators: the floating-point result of
 * an operation is quantized again to the output precision; Fig. 2: the LinearOp's result is
 * itself MXInt-typed).  The fp32 product y_ref (block terms summed exactly, rounded once, bias
 * included) is computed as in mxo_gemm, then each output row is quantized with mxo_quantize in
 * blocks of By along the output-feature axis N, which is the reduction axis of the next layer.
 * qy [M,N] int8, ey [M,N/By]; y_ref and S ([M,N], nullable) as in mxo_gemm.
 */
int mxo_gemm_requant(const int8_t *qa, const uint8_t *ea, int wa, const int8_t *qw,
                     const uint8_t *ew, int ww, int64_t M, int64_t N, int64_t K, int B,
                     const float *bias, int By, int wy, int8_t *qy, uint8_t *ey,
                     uint32_t *nonfinite, float *y_ref, double *S)
{
    if (!qy || !ey || !mxo_args_ok(M, N, By, wy)) return -1;
    float *y = y_ref ? y_ref : (float *)malloc((size_t)(M > 0 ? M : 1) * (size_t)(N > 0 ? N : 1) * sizeof(float));
    if (!y) return -2;
    int rc = mxo_gemm(qa, ea, wa, qw, ew, ww, M, N, K, B, bias, y, NULL, S);
    if (rc == 0) rc = mxo_quantize(y, M, N, N, 1, By, wy, qy, ey, nonfinite);
    if (!y_ref) free(y);
    return rc;
}

/*
 * Two-dimensional blocks (Sec. 4.1: a block has a shape; the paper's unified shape is (16, 2),
 * "block size 32", as in MXInt((16,2),8,7) of Fig. 2 and the worked 8.25-bit example after
 * Eq. 1).  Reading: B consecutive elements along the reduction axis k times BR adjacent rows
 * share one exponent, the exponent of the largest magnitude among the B*BR values.  rows must be
 * a multiple of BR.  q [rows,K] int8; ebyte [rows/BR, K/B].  Everything else as mxo_quantize.
 */
int mxo_quantize_2d(const float *x, int64_t rows, int64_t K, int64_t stride_row, int64_t stride_k,
                    int B, int BR, int w, int8_t *q, uint8_t *ebyte, uint32_t *nonfinite)
{
    if (!mxo_args_ok(rows, K, B, w) || BR < 1 || (rows % BR) != 0) return MXO_BAD_ARG;
    const int64_t nb = K / B;
    const double qmax = (double)((1 << (w - 1)) - 1);
    uint32_t bad = 0;
    for (int64_t r0 = 0; r0 < rows; r0 += BR) {
        for (int64_t b = 0; b < nb; ++b) {
            float amax = 0.0f;
            int any_nonfinite = 0;
            for (int dr = 0; dr < BR; ++dr)
                for (int k = 0; k < B; ++k) {
                    float v = x[(r0 + dr) * stride_row + (b * B + k) * stride_k];
                    if (isnan(v) || isinf(v)) any_nonfinite = 1;
                    float a = fabsf(v);
                    if (a > amax) amax = a;
                }
            const int eb = any_nonfinite ? 255 : mxo_exponent_byte(amax);
            ebyte[(r0 / BR) * nb + b] = (uint8_t)eb;
            if (any_nonfinite) ++bad;
            const double s = ldexp(1.0, (eb - 127) - (w - 2));
            for (int dr = 0; dr < BR; ++dr)
                for (int k = 0; k < B; ++k) {
                    double n = 0.0;
                    if (!any_nonfinite) {
                        n = nearbyint((double)x[(r0 + dr) * stride_row + (b * B + k) * stride_k] / s);
                        if (n > qmax) n = qmax;
                        if (n < -qmax) n = -qmax;
                    }
                    q[(r0 + dr) * K + b * B + k] = (int8_t)n;
                }
        }
    }
    if (nonfinite) *nonfinite = bad;
    return MXO_OK;
}

/* Exponent bytes of a tensor with (B, BR) blocks written out per row: out[r][b] = ebyte[r/BR][b]. */
int mxo_expand_exponent_rows(const uint8_t *ebyte, int64_t rows, int64_t nb, int BR, uint8_t *out)
{
    if (rows < 0 || nb < 0 || BR < 1 || (rows % BR) != 0) return MXO_BAD_ARG;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t b = 0; b < nb; ++b) out[r * nb + b] = ebyte[(r / BR) * nb + b];
    return MXO_OK;
}

/*
 * Cast between MXInt precisions (Sec. 3.2, "No mixed-arithmetic but mixed-precision quantization":
 * going from one mantissa width of the same format to another is an extension or a shortening of
 * the mantissas plus a shift of the exponent).  Reading: the cast is the quantizer applied to the
 * exactly decoded values -- shortening rounds to nearest even like every other rounding here, the
 * exponent is re-derived from the block's largest decoded magnitude, widening loses nothing.
 * Block sizes may differ between the two sides.
 */
int mxo_cast(const int8_t *q_in, const uint8_t *e_in, int64_t rows, int64_t K, int B_in, int w_in,
             int B_out, int w_out, int8_t *q_out, uint8_t *e_out, uint32_t *nonfinite)
{
    if (!mxo_args_ok(rows, K, B_in, w_in) || !mxo_args_ok(rows, K, B_out, w_out)) return MXO_BAD_ARG;
    const int64_t n = rows * K;
    double *xd = (double *)malloc((size_t)(n > 0 ? n : 1) * sizeof(double));
    float *xf = (float *)malloc((size_t)(n > 0 ? n : 1) * sizeof(float));
    if (!xd || !xf) { free(xd); free(xf); return -2; }
    int rc = mxo_dequantize(q_in, e_in, rows, K, B_in, w_in, xd);
    for (int64_t i = 0; i < n; ++i) xf[i] = (float)xd[i];      /* exact: <= 7 bits times a power of two */
    if (rc == 0) rc = mxo_quantize(xf, rows, K, K, 1, B_out, w_out, q_out, e_out, nonfinite);
    free(xd);
    free(xf);
    return rc;
}

/* Average bits per value, Eq. 1: p = e/prod(B) + m + 1 with m = w - 1. */
double mxo_format_bits(int block, int block_rows, int exp_bits, int w)
{
    return (double)exp_bits / ((double)block * (double)block_rows) + (double)(w - 1) + 1.0;
}

#ifdef _OPENMP
#include <omp.h>
int mxo_threads(void) { return omp_get_max_threads(); }
#else
int mxo_threads(void) { return 1; }
#endif
