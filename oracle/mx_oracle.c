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

/*
 * Dense storage (Eq. 1: a value costs its m mantissa bits plus the sign bit, nothing more): element k
 * of a row occupies bits [k*w, (k+1)*w) of the row's bit stream, two's complement, bit b of the stream
 * being bit (b % 8) of byte b / 8.  A row of K elements takes K*w/8 bytes (K % 8 == 0).
 */
int mxo_pack_dense(const int8_t *q, int64_t rows, int64_t K, int w, uint8_t *out)
{
    if (w < 2 || w > 8 || rows < 0 || K < 0 || (K % 8) != 0) return MXO_BAD_ARG;
    const int64_t row_bytes = K * w / 8;
    memset(out, 0, (size_t)(rows * row_bytes));
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k) {
            const unsigned field = (unsigned)q[r * K + k] & ((1u << w) - 1u);
            for (int b = 0; b < w; ++b)
                if ((field >> b) & 1u) {
                    const int64_t bit = k * w + b;
                    out[r * row_bytes + bit / 8] |= (uint8_t)(1u << (bit % 8));
                }
        }
    return MXO_OK;
}

int mxo_unpack_dense(const uint8_t *in, int64_t rows, int64_t K, int w, int8_t *q)
{
    if (w < 2 || w > 8 || rows < 0 || K < 0 || (K % 8) != 0) return MXO_BAD_ARG;
    const int64_t row_bytes = K * w / 8;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k) {
            int field = 0;
            for (int b = 0; b < w; ++b) {
                const int64_t bit = k * w + b;
                if ((in[r * row_bytes + bit / 8] >> (bit % 8)) & 1) field |= 1 << b;
            }
            if (field & (1 << (w - 1))) field -= 1 << w;      /* sign extension */
            q[r * K + k] = (int8_t)field;
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

/* ==================================================================================================
 * The two other MX formats of Sec. 2 "What are MX Formats?": Block Minifloat (BMF) and Block
 * Logarithm (BL).  The paper describes them in words only -- BMF "shares the exponent bias in a
 * block", BL "strips out the mantissa and shares the exponent bias, resulting in values that are
 * always powers of two" -- and compares them with MXInt in Table 1 and Fig. 5.  Readings taken here
 * (none is fixed by the paper: "parity unpinned" for all of them; pinned by the worked blocks and
 * invariants in tests/test_oracle_pins.py):
 *
 *   element  = sign bit, ebits-bit exponent field F (0 .. Fmax = 2^ebits - 1), mbits-bit mantissa T
 *              (BL: mbits = 0); one byte per element: code = sign << (ebits+mbits) | F << mbits | T
 *   block    = B consecutive elements along k share one byte: the shared bias, stored as beta + 127
 *              where 2^beta is the binade of the top exponent field (0: zero/subnormal block,
 *              255: the block holds Inf/NaN and decodes to NaN) -- "sharing the exponent bias":
 *              an element's exponent is F - (Fmax - beta)
 *   BMF value: F >= 1: (-1)^s * 2^(beta - (Fmax - F)) * (1 + T / 2^mbits)
 *              F == 0: (-1)^s * 2^(beta - (Fmax - 1)) * (T / 2^mbits)          (gradual underflow)
 *              beta = floor(log2(max |x|)); rounding to nearest, ties to even on the element's own
 *              grid, carries into the next binade, saturation at the largest code
 *   BL value : F >= 1: (-1)^s * 2^(beta - (Fmax - F)); F == 0: zero
 *              rounding in the log domain: |x| in [2^k, 2^(k+1)) goes to 2^(k+1) iff |x| >= sqrt(2) 2^k;
 *              beta = that rounded exponent of max |x|; below half a binade under the smallest
 *              power the value flushes to zero
 *   tiny     : a block whose maximum is below 2^-95 (shared byte < 32) is stored as a zero block
 *              (shared byte 0, which decodes to zeros whatever the codes): every decoded element of
 *              every other block then lies inside the range of bf16, so the formats decode to bf16
 *              exactly (at most 6 significant bits, exponent >= -133)
 *   limits   : BMF 1 + ebits + mbits <= 8, ebits <= 5;  BL ebits <= 5
 * ================================================================================================== */
#define MXO_KIND_BMF 1
#define MXO_KIND_BL 2

static int mxo_alt_args_ok(int kind, int64_t rows, int64_t K, int B, int ebits, int mbits)
{
    if (rows < 0 || K < 0 || B <= 0 || (K % B) != 0) return 0;
    if (kind == MXO_KIND_BMF) return ebits >= 1 && ebits <= 5 && mbits >= 1 && 1 + ebits + mbits <= 8;
    if (kind == MXO_KIND_BL) return ebits >= 1 && ebits <= 5 && mbits == 0;
    return 0;
}

/* round(log2(a)) for a finite a > 0: the exponent of the nearest power of two in the log domain. */
static int mxo_round_log2(double a)
{
    int ex;
    const double f = 2.0 * frexp(a, &ex);     /* a = f * 2^(ex-1), f in [1, 2) */
    /* f >= sqrt(2)  <=>  f*f >= 2; f has at most 24 significant bits, so f*f is exact in double */
    return (ex - 1) + (f * f >= 2.0 ? 1 : 0);
}

/* Magnitude code (F << mbits | T) of |x| = a on the BMF grid whose top field Fmax sits at 2^beta. */
static int mxo_bmf_code(double a, int beta, int ebits, int mbits)
{
    const int fmax = (1 << ebits) - 1;
    const int top = (fmax << mbits) | ((1 << mbits) - 1);
    if (a == 0.0) return 0;
    /* t = a in units of the subnormal step 2^(beta - (fmax - 1) - mbits): exact scaling */
    const double t = ldexp(a, -(beta - (fmax - 1) - mbits));
    double code;
    if (t < (double)(1 << mbits)) {
        code = nearbyint(t);                    /* F = 0 (a carry lands on F = 1, T = 0 by itself) */
    } else {
        int ex;
        (void)frexp(t, &ex);                    /* t in [2^(ex-1), 2^ex) */
        const int j = (ex - 1) - mbits;         /* binade above the subnormal range: F = j + 1 */
        const double sig = nearbyint(ldexp(t, -j));            /* in [2^mbits, 2^(mbits+1)] */
        code = (double)((j + 1) << mbits) + (sig - (double)(1 << mbits));  /* carry rolls into F */
    }
    if (code > (double)top) code = (double)top;
    return (int)code;
}

/*
 * x (rows x K, row stride ldx) -> one code byte per element, one shared byte per block of B along k.
 * kind 1: BMF(ebits, mbits), kind 2: BL(ebits).  nonfinite (nullable) counts blocks holding Inf/NaN.
 */
int mxo_alt_quantize(const float *x, int64_t rows, int64_t K, int64_t ldx, int kind, int B, int ebits,
                     int mbits, uint8_t *codes, uint8_t *shared, uint32_t *nonfinite)
{
    if (!mxo_alt_args_ok(kind, rows, K, B, ebits, mbits)) return MXO_BAD_ARG;
    const int64_t nb = K / B;
    const int fmax = (1 << ebits) - 1;
    uint32_t bad = 0;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t b = 0; b < nb; ++b) {
            const float *xb = x + r * ldx + b * B;
            uint8_t *cb = codes + r * K + b * B;
            float amax = 0.0f;
            int any_nonfinite = 0;
            for (int k = 0; k < B; ++k) {
                if (isnan(xb[k]) || isinf(xb[k])) any_nonfinite = 1;
                if (fabsf(xb[k]) > amax) amax = fabsf(xb[k]);
            }
            if (any_nonfinite) {
                shared[r * nb + b] = 255;
                memset(cb, 0, (size_t)B);
                ++bad;
                continue;
            }
            int sb = mxo_exponent_byte(amax);                  /* floor(log2 amax) + 127, 0 for zero/subnormal */
            if (kind == MXO_KIND_BL && sb > 0) {
                sb = mxo_round_log2((double)amax) + 127;
                if (sb > 254) sb = 254;
            }
            if (sb < 32) {                                     /* zero, subnormal or tiny block */
                shared[r * nb + b] = 0;
                memset(cb, 0, (size_t)B);
                continue;
            }
            shared[r * nb + b] = (uint8_t)sb;
            const int beta = sb - 127;
            for (int k = 0; k < B; ++k) {
                const double a = fabs((double)xb[k]);
                const int sign = signbit(xb[k]) ? 1 : 0;
                int mag;
                if (kind == MXO_KIND_BMF) {
                    mag = mxo_bmf_code(a, beta, ebits, mbits);
                } else if (a == 0.0) {
                    mag = 0;
                } else {
                    int f = mxo_round_log2(a) - beta + fmax;
                    mag = f > fmax ? fmax : (f < 1 ? 0 : f);
                }
                cb[k] = (uint8_t)((sign << (ebits + mbits)) | mag);
            }
        }
    if (nonfinite) *nonfinite = bad;
    return MXO_OK;
}

/* Decoded value of one code under a shared byte. */
static double mxo_alt_value(int kind, int code, int sb, int ebits, int mbits)
{
    if (sb == 255) return (double)NAN;
    if (sb == 0) return 0.0;
    const int fmax = (1 << ebits) - 1, beta = sb - 127;
    const int sign = (code >> (ebits + mbits)) & 1;
    const int f = (code >> mbits) & fmax, t = code & ((1 << mbits) - 1);
    double v;
    if (kind == MXO_KIND_BMF)
        v = f >= 1 ? ldexp(1.0 + ldexp((double)t, -mbits), beta - (fmax - f))
                   : ldexp(ldexp((double)t, -mbits), beta - (fmax - 1));
    else
        v = f >= 1 ? ldexp(1.0, beta - (fmax - f)) : 0.0;
    return sign ? -v : v;
}

int mxo_alt_dequantize(const uint8_t *codes, const uint8_t *shared, int64_t rows, int64_t K, int kind,
                       int B, int ebits, int mbits, double *xhat)
{
    if (!mxo_alt_args_ok(kind, rows, K, B, ebits, mbits)) return MXO_BAD_ARG;
    const int64_t nb = K / B;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k)
            xhat[r * K + k] = mxo_alt_value(kind, codes[r * K + k], shared[r * nb + k / B], ebits, mbits);
    return MXO_OK;
}

/*
 * Y = A W^T (+ bias) for operands in BMF or BL (Sec. 3.2, software emulator: the plain floating-point
 * operator on the dequantized values): every product of two decoded values is exact in double, the
 * products are summed in long double and rounded to fp32 once.  S = sum of |products| (+ |bias|).
 * An operand block with shared byte 255 makes the outputs it touches NaN.
 */
int mxo_alt_gemm(const uint8_t *ac, const uint8_t *as, int akind, int aeb, int amb, const uint8_t *wc,
                 const uint8_t *ws, int wkind, int web, int wmb, int64_t M, int64_t N, int64_t K, int B,
                 const float *bias, float *y_ref, double *S)
{
    if (!mxo_alt_args_ok(akind, M, K, B, aeb, amb) || !mxo_alt_args_ok(wkind, N, K, B, web, wmb))
        return MXO_BAD_ARG;
    const int64_t nb = K / B;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i)
        for (int64_t j = 0; j < N; ++j) {
            long double wide = 0.0L;
            double sabs = 0.0;
            int poisoned = 0;
            for (int64_t k = 0; k < K; ++k) {
                const int sa = as[i * nb + k / B], sw = ws[j * nb + k / B];
                if (sa == 255 || sw == 255) { poisoned = 1; continue; }
                const double t = mxo_alt_value(akind, ac[i * K + k], sa, aeb, amb) *
                                 mxo_alt_value(wkind, wc[j * K + k], sw, web, wmb);
                wide += (long double)t;
                sabs += fabs(t);
            }
            if (bias) {
                wide += (long double)bias[j];
                sabs += fabs((double)bias[j]);
            }
            y_ref[i * N + j] = poisoned ? NAN : (float)wide;
            if (S) S[i * N + j] = poisoned ? (double)NAN : sabs;
        }
    return MXO_OK;
}
