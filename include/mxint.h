/*
 * mxint.h -- C ABI of the MXInt linear-layer library for NVIDIA B200 (sm_100a).
 *
 * MXInt (arXiv 2307.15517, Sec. 2 "What are MX Formats?" and Sec. 4.1) is block floating
 * point: the values of a block share one 8-bit exponent and each keeps a short signed integer
 * mantissa.  A format is the tuple (B, e, m) of Sec. 4.1; this library fixes e = 8 and takes
 *   block      = number of consecutive elements along the reduction axis K sharing an exponent
 *   elem_bits  = w, the signed mantissa width INCLUDING its sign bit (the paper's m = w - 1)
 * so that the paper's "MXInt4" is elem_bits = 4 and its average size (Eq. 1) is
 * exp_bits/(block*block_rows) + elem_bits.
 *
 * Encoding of one block (E = exponent byte - 127):
 *   exponent byte = binary32 exponent field of the block's largest magnitude
 *                   (0 for an all-zero or subnormal block, 255 if the block holds Inf/NaN)
 *   mantissa q    = clamp(round_to_nearest_even(x * 2^-(E-(w-2))), -(2^(w-1)-1), 2^(w-1)-1)
 *   value         = q * 2^(E-(w-2));   a block with exponent byte 255 decodes to NaN
 * Containers: elem_bits <= 4 -> two two's-complement nibbles per byte, even k in the low
 * nibble, a row of K elements takes K/2 bytes; elem_bits 5..8 -> one int8 per element.
 * Exponent bytes: uint8 [rows, K/block], row-major.
 *
 * Conventions for every entry point:
 *   - All data pointers are DEVICE pointers owned by the caller.  The library neither
 *     allocates, frees nor keeps them.  Base pointers must be 16-byte aligned.
 *   - Every call works on the CURRENT CUDA device of the calling thread: all pointers must belong
 *     to it, `stream` must be one of its streams, and the library's per-device state (status
 *     word, tensor-map cache, the built-in scratch of mx_gemm_static) is that device's.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls are
 *     asynchronous on it and never synchronise the host, except mx_poll_status.
 *   - Arguments are validated on the host before anything is launched; a negative
 *     mx_status_t means nothing ran.  K must be a multiple of the block size.
 *   - There is no CPU fallback: on a machine without an sm_100 GPU the compute entry points
 *     return MX_ERR_ARCH / MX_ERR_CUDA.
 */
#ifndef MXINT_H_
#define MXINT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define MX_API __attribute__((visibility("default")))
#else
#define MX_API
#endif

typedef enum {
    MX_OK = 0,
    MX_ERR_NULL = -1,      /* a required pointer is NULL                                      */
    MX_ERR_SHAPE = -2,     /* K % block != 0, a negative size, a leading dimension too small  */
    MX_ERR_FORMAT = -3,    /* unsupported block / elem_bits / exp_bits / block_rows           */
    MX_ERR_ALIGN = -4,     /* a pointer or stride breaks the alignment rule                   */
    MX_ERR_WORKSPACE = -5, /* workspace NULL or smaller than mx_workspace_bytes()             */
    MX_ERR_CUDA = -6,      /* a CUDA runtime/driver call failed; see mx_last_cuda_error()     */
    MX_ERR_TIMEOUT = -7,   /* a bounded device-side wait expired (reported by mx_poll_status) */
    MX_ERR_ARCH = -8       /* the current device is not sm_100                                */
} mx_status_t;

typedef enum { MX_F32 = 0, MX_BF16 = 1 } mx_dtype_t;

/* Which kernel computes the block-scaled product. */
typedef enum {
    MX_ALGO_AUTO = 0,    /* M <= 16 and a streamable format (see mx_linear_grouped): MX_ALGO_STREAM;
                            everything else: MX_ALGO_TCGEN05                                       */
    MX_ALGO_SIMT = 1,    /* CUDA-core kernel: exact integer block sums, blocks added in ascending
                            order in fp32 (bit-reproducible; slow; mx_gemm needs no workspace)      */
    MX_ALGO_TCGEN05 = 2, /* tcgen05/TMEM tensor-core kernel on exactly decoded bf16 operands; a
                            separate pass decodes the packed weights into the workspace            */
    MX_ALGO_STREAM = 3,  /* weight-streaming kernel for M <= 16 (decode); see mx_linear_grouped for
                            its restrictions                                                       */
    MX_ALGO_TCGEN05_FUSED = 4, /* the same tensor-core kernel with the packed weights decoded inside
                            it by extra warps (no bf16 copy of W: workspace holds the activations
                            only; needs K % 32 == 0 and a 2-byte aligned w_exp, else it falls back to
                            the separate pass).  Saves memory, but the decode costs more issue slots
                            than the MMA leaves free, so it is slower than MX_ALGO_TCGEN05.          */
    MX_ALGO_TCGEN05_BLOCKWISE = 5, /* tensor-core kernel that gives every block its own accumulator: the tensor
                            pipe sums one block (exactly: all addends share one scale), the block terms
                            are added in fp32 registers with round-to-nearest in ascending block order --
                            the same bits as MX_ALGO_SIMT while every block term is a normal fp32 number.
                            Meets 1e-5 * S for any spread of the block exponents and any K; a fraction of
                            the throughput of MX_ALGO_TCGEN05 (a tensor-memory read per block).  fp32
                            result only.                                                                  */
    MX_ALGO_TCGEN05_MXF8 = 6 /* the hardware's block-scaled tensor-core path (tcgen05.mma.kind::mxf8f6f4 with one
                            E8M0 scale per 32 elements): the MXInt operator of Sec. 3.2 in silicon.  Exact for
                            the formats it can hold: block 32 and elem_bits <= 5 on BOTH operands (an element
                            q * 2^-(w-2) is an E4M3 number, the exponent byte is the E8M0 scale), K % 128 == 0,
                            container storage; anything else answers MX_ERR_FORMAT.  Twice the tensor peak of
                            the bf16 kernels; accumulation across blocks in fp32 as MX_ALGO_TCGEN05.  Workspace:
                            mx_workspace_bytes_ex with this algo.  mx_gemm_ex and mx_linear_ex only.            */
} mx_algo_t;

/* Accuracy of the product kernels against the exactly summed result (Sec. 3.2 leaves the accumulator
 * across blocks open; S[i,j] = sum_b |block term b|):
 *   MX_ALGO_SIMT, MX_ALGO_STREAM : exact block sums, one fp32 rounding per block, ascending blocks;
 *                                  bit-reproducible.
 *   MX_ALGO_TCGEN05(_FUSED), AUTO for M > 16, the _q / batched / static entry points : the tensor
 *                                  pipe aligns the 16 products of a step and the accumulator to the
 *                                  largest and truncates, so the guaranteed bound is
 *                                  ceil(K/16) * 17 * 2^-23 * S; it is approached only when block
 *                                  scales inside one row differ by many binades.  On operands whose
 *                                  block exponents spread over <= 2^6 per row (every LLM-shaped
 *                                  workload measured: N(0, sigma) weights, outlier-channel or
 *                                  Student-t activations, K up to 16384) the error stays below
 *                                  1e-5 * S, typically below 1e-6 * S.
 *   MX_ALGO_TCGEN05_BLOCKWISE    : exact block sums out of the tensor pipe, one fp32 rounding per block,
 *                                  ascending blocks: the result of MX_ALGO_SIMT, bit for bit, whatever
 *                                  the operands (block terms inside the fp32 normal range). */

/* The (B, e, m) tuple of Sec. 4.1. */
typedef struct {
    int32_t block;      /* 16 or 32 elements along K share one exponent                        */
    int32_t elem_bits;  /* w = 2..8, sign included (paper m = w - 1)                           */
    int32_t exp_bits;   /* 8 (the paper fixes the shared exponent to 8 bits)                   */
    int32_t block_rows; /* 1, or 2: two adjacent rows share their exponents, the paper's (16,2) */
    int32_t packing;    /* 0: container (below); 1: dense, elem_bits bits per element (Eq. 1)      */
} mx_format_t;

/* Dense storage (packing == 1): Eq. 1 charges a value m + 1 bits, so a row of K mantissas takes
 * K * elem_bits / 8 bytes: element k sits in bits [k*w, (k+1)*w) of the row's bit stream, two's
 * complement, stream bit b being bit b % 8 of byte b / 8 (for w = 4 and w = 8 this IS the container).
 * It is the form for tensors at rest -- weights: mx_pack_dense converts a quantized tensor into it,
 * mx_unpack_dense back, mx_mant_bytes gives its size, and mx_dequantize, mx_gemm(_ex) with the
 * tensor-core kernels, mx_gemm_q and the weight operand of mx_linear(_ex) / mx_linear_q read it
 * directly.  Everything else (the quantizer's output, casts, the CUDA-core, streaming, in-kernel
 * decode, batched, grouped and static entry points, activation and result formats) takes the
 * container only and answers MX_ERR_FORMAT to packing == 1. */

/* Two-row blocks (block_rows == 2; Sec. 4.1 and Fig. 2: the paper's unified block shape is
 * (16,2), "block size 32"): `block` consecutive elements along K times two adjacent rows (2r and
 * 2r+1) share one exponent, that of the largest magnitude among them.  The exponent array of a
 * [rows, K] tensor is then uint8 [rows/2, K/block] and rows must be even (MX_ERR_SHAPE).
 * Accepted by mx_quantize (stride_k == 1), mx_dequantize, mx_gemm / mx_linear and their _q forms
 * for either operand with MX_ALGO_AUTO, MX_ALGO_TCGEN05(_BLOCKWISE) and MX_ALGO_SIMT, as the result
 * format fy of the _q forms (rows of Y pair up: exponent array [M/2, N/fy.block]), by
 * mx_gemm_batched (items must start on even rows) and by MX_ALGO_STREAM / mx_linear_grouped for
 * either operand (an even number of tokens when the activations pair up; weights in this form are
 * read with plain loads instead of staged boxes); the in-kernel decode (MX_ALGO_TCGEN05_FUSED), the
 * fused attention and the static entry point take one-row blocks only (MX_ERR_FORMAT). */

/* ---- size helpers (host only, no CUDA call) ------------------------------------------- */

/* Bytes of the mantissa container / of the exponent array of a [rows, K] tensor; 0 on a bad
 * format or shape. */
MX_API size_t mx_mant_bytes(int64_t rows, int64_t K, mx_format_t f);
MX_API size_t mx_exp_bytes(int64_t rows, int64_t K, mx_format_t f);

/* Average bits per value, Eq. 1 of the paper: exp_bits/(block*block_rows) + (w-1) + 1.
 * MXInt((16,2),8,7) -> 8.25.  Returns 0 on a bad format. */
MX_API double mx_format_bits(mx_format_t f);

/* Scratch bytes mx_gemm / mx_linear need for these sizes with MX_ALGO_AUTO (the maximum over
 * the kernels AUTO may pick).  The workspace must be 256-byte aligned. */
MX_API size_t mx_workspace_bytes(int64_t M, int64_t N, int64_t K, mx_format_t fa, mx_format_t fw);

/* The same for an explicitly named kernel (0 for an unknown algo or a bad format). */
MX_API size_t mx_workspace_bytes_ex(int64_t M, int64_t N, int64_t K, mx_format_t fa, mx_format_t fw,
                                    mx_algo_t algo);

/* Container <-> dense storage of the mantissas of a [rows, K] tensor (the exponent array is the same
 * for both).  `f` names widths and block; its packing field is ignored.  Both arrays are device
 * memory, the container 16-byte aligned. */
MX_API mx_status_t mx_pack_dense(const void *mant, int64_t rows, int64_t K, mx_format_t f, void *dense_out,
                                 void *stream);
MX_API mx_status_t mx_unpack_dense(const void *dense, int64_t rows, int64_t K, mx_format_t f, void *mant_out,
                                   void *stream);

MX_API const char *mx_status_string(mx_status_t s);

/* Text of the last CUDA error this library saw on the calling thread ("" if none). */
MX_API const char *mx_last_cuda_error(void);

/* ---- quantizer (Sec. 3.2, software emulator: floating point -> MXInt) ------------------ */

/*
 * Quantize x, a [rows, K] tensor of `dt` whose element (r, k) sits at
 * x[r*stride_row + k*stride_k] (strides in elements), block by block along k.
 *   stride_k == 1 : rows are contiguous along K (fast path; stride_row % 8 == 0 required).
 *   stride_k != 1 : blocks run along a strided axis (e.g. V of attention quantized along the
 *                   token axis for the P*V product).
 * mant_out receives mx_mant_bytes(rows,K,f) bytes, exp_out mx_exp_bytes(rows,K,f) bytes, both
 * row-major and dense.  nonfinite_count (nullable, device uint32) is incremented once per
 * block that holds an Inf or NaN; such a block gets exponent byte 255 and zero mantissas.
 */
MX_API mx_status_t mx_quantize(const void *x, mx_dtype_t dt, int64_t rows, int64_t K,
                        int64_t stride_row, int64_t stride_k, mx_format_t f, void *mant_out,
                        uint8_t *exp_out, uint32_t *nonfinite_count, void *stream);

/* Inverse map (Sec. 3.2: the software emulator of a format converts between it and floating point in
 * both directions; here a test helper): out[r*ld_out + k] = q * 2^(E-(w-2)) as `dt` (exact in both
 * fp32 and bf16); NaN for blocks with exponent byte 255. */
MX_API mx_status_t mx_dequantize(const void *mant, const uint8_t *exps, int64_t rows, int64_t K,
                          mx_format_t f, void *out, mx_dtype_t dt, int64_t ld_out, void *stream);

/*
 * Cast an MXInt tensor to another MXInt format (Sec. 3.2, "No mixed-arithmetic but mixed-precision
 * quantization": another mantissa width of the same format costs an extension or shortening of
 * the mantissas and an exponent shift).  Defined as mx_quantize applied to the exactly decoded
 * values: shortening rounds to nearest even and re-derives the block exponent, widening is exact,
 * a cast to the same format is the identity.  Block sizes may differ; one-row blocks only.
 * Arrays as for mx_quantize (dense rows); nonfinite_count as there.
 */
MX_API mx_status_t mx_cast(const void *mant_in, const uint8_t *exp_in, mx_format_t f_in, int64_t rows,
                           int64_t K, mx_format_t f_out, void *mant_out, uint8_t *exp_out,
                           uint32_t *nonfinite_count, void *stream);

/* ---- block-scaled product (Sec. 3.2, MXInt dot-product operator, Fig. 3 right) --------- */

/*
 * Y[M,N] = A[M,K] * W[N,K]^T (+ bias[N]) where both operands are MXInt tensors blocked along K:
 *   Y[i,j] = sum_b 2^(Ea[i,b]+Ew[j,b]-(wa-2)-(ww-2)) * sum_{k in block b} qa[i,k]*qw[j,k]
 * accumulated in fp32.  fa.block must equal fw.block; elem_bits may differ (e.g. A8/W4).
 * y is fp32 with leading dimension ldy >= N (elements).  Any block with exponent byte 255
 * makes the outputs it touches NaN.  workspace: see mx_workspace_bytes (may be NULL for
 * MX_ALGO_SIMT / MX_ALGO_STREAM).
 */
MX_API mx_status_t mx_gemm(const void *a_mant, const uint8_t *a_exp, mx_format_t fa,
                    const void *w_mant, const uint8_t *w_exp, mx_format_t fw, int64_t M,
                    int64_t N, int64_t K, const float *bias, float *y, int64_t ldy,
                    void *workspace, size_t workspace_bytes, void *stream);

/* The same with the kernel named explicitly. */
MX_API mx_status_t mx_gemm_ex(const void *a_mant, const uint8_t *a_exp, mx_format_t fa,
                       const void *w_mant, const uint8_t *w_exp, mx_format_t fw, int64_t M,
                       int64_t N, int64_t K, const float *bias, float *y, int64_t ldy,
                       void *workspace, size_t workspace_bytes, mx_algo_t algo, void *stream);

/* ---- the MXInt linear layer (Fig. 2: LinearOp with MXInt activations and weights) ------ */

/*
 * Y[M,N] = Q_fa(X)[M,K] * W[N,K]^T (+ bias): quantizes the activations x ([M,K] of `dt`,
 * leading dimension ldx elements, ldx % 8 == 0) to format fa on the fly and multiplies them
 * with weights already stored in format fw.  Equivalent to mx_quantize followed by mx_gemm,
 * but the quantized activations go straight to the product kernel's operand layout.
 */
MX_API mx_status_t mx_linear(const void *x, mx_dtype_t dt, int64_t M, int64_t K, int64_t ldx,
                      mx_format_t fa, const void *w_mant, const uint8_t *w_exp, mx_format_t fw,
                      int64_t N, const float *bias, float *y, int64_t ldy, void *workspace,
                      size_t workspace_bytes, void *stream);

MX_API mx_status_t mx_linear_ex(const void *x, mx_dtype_t dt, int64_t M, int64_t K, int64_t ldx,
                         mx_format_t fa, const void *w_mant, const uint8_t *w_exp,
                         mx_format_t fw, int64_t N, const float *bias, float *y, int64_t ldy,
                         void *workspace, size_t workspace_bytes, mx_algo_t algo, void *stream);

/* ---- decode: a few tokens against many weight matrices (weights streamed once) ---------- */

/* One layer of a grouped call: the arguments of mx_linear. */
typedef struct {
    const void *x;          /* [M, K] activations of `dt`, leading dimension ldx (elements)     */
    mx_dtype_t dt;
    int64_t M, K, ldx;      /* M = number of tokens, 1..16                                      */
    mx_format_t fa;         /* activation format (block 32)                                     */
    const void *w_mant;     /* [N, K/2] packed weights (elem_bits <= 4, block 32)               */
    const uint8_t *w_exp;   /* [N, K/32], 4-byte aligned                                        */
    mx_format_t fw;
    int64_t N;
    const float *bias;      /* nullable, [N]                                                    */
    float *y;               /* [M, ldy]                                                         */
    int64_t ldy;
} mx_linear_args_t;

/*
 * Sec. 1 and Sec. 6 motivate MX formats by the memory footprint of the parameters: at a few tokens per
 * step a layer's time is the time to stream its packed weights once.  This call
 * runs n_layers independent MXInt linear layers with few tokens each (decode) in ONE kernel
 * launch: every distinct activation tensor is quantized to its format once (layers that name
 * the same x, shape and format share it), then a single persistent kernel streams all weight
 * matrices from HBM exactly once.  Per output the integer block sums are exact and the blocks are
 * added in fp32, in ascending order whenever there are enough weight rows to fill the GPU without
 * cutting K (always the case for tens of layers).  `layers` is HOST memory (read during the
 * call).  Restrictions: M <= 16, both formats block 32, weights elem_bits <= 4, K % 128 == 0,
 * M*K small enough to stage in shared memory (M = 16: K <= 18432); otherwise MX_ERR_SHAPE /
 * MX_ERR_FORMAT.  mx_linear(_ex) with MX_ALGO_STREAM is the one-layer form of this call.
 */
MX_API size_t mx_linear_grouped_workspace_bytes(const mx_linear_args_t *layers, int32_t n_layers);
MX_API mx_status_t mx_linear_grouped(const mx_linear_args_t *layers, int32_t n_layers,
                                     void *workspace, size_t workspace_bytes, void *stream);

/* ---- batched product and fp32 glue (the attention matmuls and the rest of a decoder block) --- */

/*
 * `batch` independent products Y_b[M,N] = A_b[M,K] * W_b[N,K]^T of MXInt operands that live inside
 * larger packed tensors: row r of A_b starts `r*lda + b*stride_a` ELEMENTS into the packed tensor
 * (mantissa byte offset = elements * container bits / 8, exponent offset = elements / block), same
 * for W with ldw / stride_w; Y_b = y + b*stride_y with leading dimension ldy.  The attention
 * matmuls of Fig. 1 (tensors "A" = Q K^T and "B" = P V) are this call: heads side by side in a
 * [tokens, heads*d] tensor give lda = heads*d, stride_a = d.  lda, ldw, stride_a, stride_w must be
 * multiples of the block size and of 8.  Tensor-core kernel, one launch for all items after one
 * decode launch per operand; workspace from mx_gemm_batched_workspace_bytes.
 */
MX_API size_t mx_gemm_batched_workspace_bytes(int64_t M, int64_t N, int64_t K, int64_t batch);
MX_API mx_status_t mx_gemm_batched(const void *a_mant, const uint8_t *a_exp, mx_format_t fa,
                                   int64_t lda, int64_t stride_a, const void *w_mant,
                                   const uint8_t *w_exp, mx_format_t fw, int64_t ldw, int64_t stride_w,
                                   int64_t M, int64_t N, int64_t K, int64_t batch, float *y,
                                   int64_t ldy, int64_t stride_y, void *workspace,
                                   size_t workspace_bytes, void *stream);

/* The paper keeps LayerNorm, softmax and the activation function in floating point around the MX
 * operators (Fig. 1(d)); these are plain fp32 row kernels.  cols <= 8192.
 *   mx_layernorm : y[r,:] = (x[r,:] - mean) / sqrt(var + eps) * gamma + beta  (gamma/beta nullable)
 *   mx_softmax   : in place, s[r,j] = softmax_j(scale * s[r,j]); with causal != 0 only columns
 *                  j <= (r % rows_per_batch) take part and the rest become 0
 *   mx_relu_add  : y[i] = (relu ? max(a[i], 0) : a[i]) + (b ? b[i] : 0); y may alias a or b */
MX_API mx_status_t mx_layernorm(const float *x, int64_t ldx, const float *gamma, const float *beta,
                                float eps, int64_t rows, int64_t cols, float *y, int64_t ldy,
                                void *stream);
MX_API mx_status_t mx_softmax(float *s, int64_t ld, int64_t rows, int64_t cols, float scale,
                              int causal, int64_t rows_per_batch, void *stream);
MX_API mx_status_t mx_relu_add(const float *a, const float *b, float *y, int64_t n, int relu,
                               void *stream);

/* mx_softmax followed by mx_quantize of its result, in one pass and without the fp32 probabilities
 * ever reaching memory (Fig. 1(d): the probabilities are an MXInt operand of the P V product):
 * p = Q_fp(softmax(scale * s)) with blocks of fp.block along the columns (the key/token axis, the
 * reduction axis of P V).  s: device fp32 [rows, ld] (read only, ld % 4 == 0); p_mant: device,
 * [rows, cols/2] bytes (fp.elem_bits <= 4) or [rows, cols] int8; p_exp: device uint8
 * [rows, cols/fp.block]; cols <= 8192, cols % fp.block == 0 (MX_ERR_SHAPE); one-row blocks only. */
MX_API mx_status_t mx_softmax_q(const float *s, int64_t ld, int64_t rows, int64_t cols, float scale,
                                int causal, int64_t rows_per_batch, mx_format_t fp, void *p_mant,
                                uint8_t *p_exp, void *stream);

/*
 * Fused attention of one transformer block (Fig. 1(d); the matmuls "A" = Q K^T and "B" = P V of Fig. 1(a)/(b)
 * are MXInt operators, softmax stays in floating point): per head h of `heads` heads of dimension head_dim,
 *   S_h = Q_h K_h^T                      Q, K: MXInt [seq, heads*head_dim], format fqk, blocks along the head dimension
 *   P_h = Q_fp(softmax(scale * S_h))     causal != 0: query i attends keys 0..i; P quantized to fp along the keys
 *   ctx[:, h*head_dim ..] = P_h V_h      V given TRANSPOSED: MXInt [heads*head_dim, seq], format fv, blocks along the tokens
 * i.e. mx_gemm_batched -> mx_softmax_q -> mx_gemm_batched in one kernel: the scores and the probabilities
 * (heads * seq * seq values each) never reach memory.  Same arithmetic as that sequence up to the fp32
 * rounding of the softmax row sums (two sweeps over the key tiles: maximum and sum first, then the
 * probabilities normalised with the final values, quantized and multiplied).
 *   ctx      : device fp32 [seq, ldc], ldc >= heads*head_dim, ldc % 4 == 0, 16-byte aligned
 *   p_mant_out, p_exp_out : nullable; when given, the quantized probabilities are also written there
 *              ([heads*seq, seq/2 or seq] and [heads*seq, seq/fp.block]; masked positions 0) -- for checks
 *   workspace: mx_attention_workspace_bytes(seq, heads, head_dim) (the three operands as bf16), 256-byte aligned
 * Restrictions: head_dim 128 or 64, seq % 32 == 0 (whole blocks along the keys; the last tile of 128 queries or keys
 * may be ragged), scale > 0, container storage, one-row blocks; otherwise MX_ERR_SHAPE / MX_ERR_FORMAT (use the
 * three separate calls then).
 */
MX_API size_t mx_attention_workspace_bytes(int64_t seq, int64_t heads, int64_t head_dim);
MX_API mx_status_t mx_attention(const void *q_mant, const uint8_t *q_exp, const void *k_mant, const uint8_t *k_exp,
                                mx_format_t fqk, const void *vt_mant, const uint8_t *vt_exp, mx_format_t fv,
                                int64_t seq, int64_t heads, int64_t head_dim, float scale, int causal, mx_format_t fp,
                                float *ctx, int64_t ldc, void *p_mant_out, uint8_t *p_exp_out, void *workspace,
                                size_t workspace_bytes, void *stream);

/*
 * The same with the three operands still in floating point (what mx_linear is to mx_gemm): q, k, v are
 * [seq, heads*head_dim] tensors of `dt` with leading dimensions ldq, ldk, ldv (elements, multiples of 8;
 * slices of one fused projection result are fine), 16-byte aligned.  q and k are quantized to fqk in blocks
 * along the head dimension, v to fv in blocks along the TOKENS (its slow axis; no transposed copy is needed
 * from the caller), each in one pass that writes the tensor-core operand directly -- the packed codes never
 * reach memory.  Equal to mx_quantize (x3) followed by mx_attention, bit for bit.  Workspace and
 * restrictions as for mx_attention.
 */
MX_API mx_status_t mx_attention_fp(const void *q, const void *k, const void *v, mx_dtype_t dt, int64_t ldq,
                                   int64_t ldk, int64_t ldv, mx_format_t fqk, mx_format_t fv, int64_t seq,
                                   int64_t heads, int64_t head_dim, float scale, int causal, mx_format_t fp,
                                   float *ctx, int64_t ldc, void *workspace, size_t workspace_bytes,
                                   void *stream);

/* ---- device status (the paper has no counterpart: it describes no runtime) ---------------- */

/*
 * Every device-side wait in this library (mbarrier polls of the tensor-core pipeline) gives up
 * after a bounded time, records the fact in a per-device status word and lets the kernel
 * return.  mx_poll_status synchronises `stream`, reads and clears that word and returns
 * MX_ERR_TIMEOUT if any wait expired since the last poll, MX_ERR_CUDA if the stream reported
 * an error, else MX_OK.  Outputs of a call that timed out are undefined.
 */
MX_API mx_status_t mx_poll_status(void *stream);

/*
 * Self-test of that mechanism: launches one warp that waits, with the same bounded wait the
 * product kernels use, on a barrier nobody arrives on.  The wait gives up after `limit_us`
 * microseconds (1 .. 100000, else MX_ERR_SHAPE), the kernel records the expiry and returns
 * normally; the next mx_poll_status on that stream then reports MX_ERR_TIMEOUT (and clears it).
 * Nothing faults or hangs; the device and the context stay usable.
 */
MX_API mx_status_t mx_selftest_wait_expiry(uint32_t limit_us, void *stream);

/* ---- the layer with an MXInt result ------------------------------------------------------------
 *
 * Sec. 3.2 (software emulators): an operator's floating-point result is quantized again to the
 * output precision; Fig. 2: the LinearOp's result is itself MXInt-typed, and Sec. 3.2 ("No
 * mixed-arithmetic but mixed-precision quantization") notes that going from one MXInt width to
 * another is cheap.  These two calls are mx_gemm / mx_linear with that last step done in the
 * product kernel's epilogue: instead of fp32 values they write Q_fy(A W^T + bias), quantized in
 * blocks of fy.block along N -- the reduction axis of the layer that consumes the result -- with
 * the same rule as mx_quantize (exponent of the block's largest magnitude, round to nearest even,
 * symmetric clamp; a block holding Inf/NaN gets exponent byte 255 and zero mantissas).
 *   y_mant : device, [M, N/2] bytes (fy.elem_bits <= 4) or [M, N] int8, dense rows, 16-byte aligned
 *   y_exp  : device, uint8 [M, N/fy.block]
 *   nonfinite_count : device, nullable; incremented once per non-finite block (not cleared here)
 * N % fy.block must be 0 (MX_ERR_SHAPE); fy.block may differ from fa.block.  Always the
 * tensor-core kernel; workspace as for MX_ALGO_TCGEN05.  The fp32 accumulation order is the
 * tensor pipe's, so a value within the product's tolerance of a rounding boundary may take either
 * neighbouring code.  Other arguments, ownership and errors as for mx_gemm / mx_linear.
 */
MX_API mx_status_t mx_gemm_q(const void *a_mant, const uint8_t *a_exp, mx_format_t fa,
                      const void *w_mant, const uint8_t *w_exp, mx_format_t fw, int64_t M,
                      int64_t N, int64_t K, const float *bias, mx_format_t fy, void *y_mant,
                      uint8_t *y_exp, uint32_t *nonfinite_count, void *workspace,
                      size_t workspace_bytes, void *stream);

MX_API mx_status_t mx_linear_q(const void *x, mx_dtype_t dt, int64_t M, int64_t K, int64_t ldx,
                        mx_format_t fa, const void *w_mant, const uint8_t *w_exp, mx_format_t fw,
                        int64_t N, const float *bias, mx_format_t fy, void *y_mant,
                        uint8_t *y_exp, uint32_t *nonfinite_count, void *workspace,
                        size_t workspace_bytes, void *stream);

/* ---- the product with a fused element-wise tail ------------------------------------------------
 *
 * Fig. 1(d): between the MX operators of a decoder block sit LayerNorm, a bias, the activation function and the
 * skip connection, all in floating point.  These two calls are mx_gemm / mx_linear (fp32 result y) or
 * mx_gemm_q / mx_linear_q (MXInt result fy, y_mant, y_exp) with that tail applied in the product kernel's
 * epilogue, on the fp32 accumulator, before the result is stored or quantized:
 *     out[i,j] = act(acc[i,j] + bias[j]) + residual[i*ldr + j],   act(t) = relu ? (t < 0 ? 0 : t) : t
 * so no separate pass over the fp32 tensor remains.  Exactly one of y and y_mant is non-null
 * (MX_ERR_NULL otherwise); fy is ignored for an fp32 result.  ep may be NULL (no tail).
 * residual is device fp32, 4-byte aligned (16-byte aligned with ldr % 4 == 0 takes vector loads),
 * ldr >= N (MX_ERR_SHAPE); it may alias y only element for element (y = residual in place is fine).
 * Always the tensor-core kernels; workspace as for MX_ALGO_TCGEN05.  Everything else as for the calls
 * named above.
 */
typedef struct {
    const float *bias;      /* device, [N], nullable                                   */
    int32_t relu;           /* != 0: clamp negatives to zero after the bias (NaN stays) */
    const float *residual;  /* device, [M, ldr] fp32, nullable: added last             */
    int64_t ldr;            /* elements between the rows of residual                   */
} mx_epilogue_t;

MX_API mx_status_t mx_gemm_fused(const void *a_mant, const uint8_t *a_exp, mx_format_t fa,
                          const void *w_mant, const uint8_t *w_exp, mx_format_t fw, int64_t M,
                          int64_t N, int64_t K, const mx_epilogue_t *ep, float *y, int64_t ldy,
                          mx_format_t fy, void *y_mant, uint8_t *y_exp, void *workspace,
                          size_t workspace_bytes, void *stream);

/* What happens to the rows of x before they are quantized (mx_linear_fused only; NULL = nothing).
 * layernorm != 0: every row is layer-normalised first, y = (x - mean) / sqrt(var + ln_eps) * ln_gamma + ln_beta
 * (ln_gamma / ln_beta device fp32 [K], nullable = 1 / 0), with the arithmetic of mx_layernorm, bit for bit, and
 * goes straight to the quantizer: the normalised fp32 tensor is never stored (Fig. 1(d): LayerNorm stays in
 * floating point in front of the MX linears).  Needs fp32 x, K % 32 == 0, K <= 8192, one-row container formats
 * (MX_ERR_FORMAT / MX_ERR_SHAPE otherwise). */
typedef struct {
    int32_t layernorm;
    const float *ln_gamma;
    const float *ln_beta;
    float ln_eps;
} mx_prologue_t;

MX_API mx_status_t mx_linear_fused(const void *x, mx_dtype_t dt, int64_t M, int64_t K, int64_t ldx,
                            mx_format_t fa, const mx_prologue_t *pro, const void *w_mant,
                            const uint8_t *w_exp, mx_format_t fw, int64_t N, const mx_epilogue_t *ep,
                            float *y, int64_t ldy, mx_format_t fy, void *y_mant, uint8_t *y_exp,
                            void *workspace, size_t workspace_bytes, void *stream);

/* ---- the other MX formats of the paper: Block Minifloat and Block Logarithm ---------------------
 *
 * Sec. 2 "What are MX Formats?" puts two more block formats beside MXInt and Table 1 / Fig. 5 compare
 * them: Block Minifloat (BMF) "shares the exponent bias in a block" -- every element is a small
 * floating-point number --, Block Logarithm (BL) "strips out the mantissa and shares the exponent
 * bias", so every value is a power of two.  The paper gives no bit-level definition; this library's
 * reading (stated in full because results depend on it):
 *   element : one byte, sign << (elem_exp_bits + elem_man_bits) | F << elem_man_bits | T
 *             (F = exponent field, 0 .. Fmax = 2^elem_exp_bits - 1; T = mantissa; BL: elem_man_bits = 0)
 *   shared  : one byte per `block` consecutive elements along K = 127 + beta, 2^beta being the binade
 *             of the top field Fmax; 0 = zero block (decodes to zeros whatever the codes),
 *             255 = the block holds Inf/NaN (codes 0, decodes to NaN)
 *   BMF     : F >= 1: (-1)^s 2^(beta-(Fmax-F)) (1 + T / 2^man);  F == 0: (-1)^s 2^(beta-(Fmax-1)) T / 2^man;
 *             beta = floor(log2 max|x|); round to nearest even on the element's own grid, carries into
 *             the next binade, saturation at the largest code
 *   BL      : F >= 1: (-1)^s 2^(beta-(Fmax-F));  F == 0: zero;  rounding in the log domain (a value
 *             goes to the next power of two iff its significand is >= sqrt(2)), beta = the rounded
 *             exponent of max|x|; more than half a binade below the smallest power flushes to zero
 *   a block whose maximum is below 2^-95 is stored as a zero block, so that every decoded element
 *   is exactly a bf16 number and the formats can feed the bf16 tensor-core product without loss
 *   limits  : block 16 or 32;  BMF 1 + exp + man <= 8, exp <= 5, man >= 1;  BL exp <= 5
 * Average bits per value: 8 / block + 1 + elem_exp_bits + elem_man_bits (the analogue of Eq. 1).
 */
typedef enum { MX_ELEM_BMF = 1, MX_ELEM_BL = 2 } mx_elem_kind_t;
typedef struct {
    int32_t kind;           /* mx_elem_kind_t                                                  */
    int32_t block;          /* 16 or 32 elements along K share one bias byte                   */
    int32_t elem_exp_bits;  /* exponent bits of an element                                     */
    int32_t elem_man_bits;  /* mantissa bits of an element (0 for MX_ELEM_BL)                  */
} mx_alt_format_t;

/* x ([rows, K] of `dt`, leading dimension ldx elements, ldx % 8 == 0, K % block == 0) -> codes (device,
 * uint8 [rows, K], 16-byte aligned) and shared bytes (device, uint8 [rows, K/block]).
 * nonfinite_count (device, nullable) is incremented once per block holding Inf/NaN. */
MX_API mx_status_t mx_alt_quantize(const void *x, mx_dtype_t dt, int64_t rows, int64_t K, int64_t ldx,
                                   mx_alt_format_t f, uint8_t *codes, uint8_t *shared,
                                   uint32_t *nonfinite_count, void *stream);

/* Inverse map: out[r*ld_out + k] = decoded value as `dt` (exact in fp32 and in bf16); ld_out % 8 == 0. */
MX_API mx_status_t mx_alt_dequantize(const uint8_t *codes, const uint8_t *shared, int64_t rows, int64_t K,
                                     mx_alt_format_t f, void *out, mx_dtype_t dt, int64_t ld_out,
                                     void *stream);

/* Y[M,N] = A[M,K] W[N,K]^T (+ bias) on operands in BMF or BL (kinds and bit splits may differ, the
 * block sizes must be equal): Sec. 3.2's emulated operator -- the floating-point product of the
 * decoded values -- on the tensor-core kernels of mx_gemm, fp32 accumulation.  Workspace:
 * mx_alt_gemm_workspace_bytes (both operands as bf16), 256-byte aligned.  Tolerance as for mx_gemm
 * with S = sum_k |a_k w_k|.  Other conventions as for mx_gemm. */
MX_API size_t mx_alt_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K);
MX_API mx_status_t mx_alt_gemm(const uint8_t *a_codes, const uint8_t *a_shared, mx_alt_format_t fa,
                               const uint8_t *w_codes, const uint8_t *w_shared, mx_alt_format_t fw,
                               int64_t M, int64_t N, int64_t K, const float *bias, float *y, int64_t ldy,
                               void *workspace, size_t workspace_bytes, void *stream);

/* ---- product for callers that cannot allocate (the paper has no counterpart) -----------------
 *
 * Some callers of this library have no way to obtain device memory at the point where they
 * need the product: a plugin running inside a host application that owns the allocator and
 * forbids cudaMalloc after start-up, a real-time loop with a no-allocation rule, or code that
 * runs while another component holds the device's memory pool.  mx_gemm and mx_linear need a
 * caller-provided workspace for the decoded bf16 operands; mx_gemm_static needs none.  It is
 * the tensor-core product of mx_gemm_ex(..., MX_ALGO_TCGEN05) with that workspace replaced by
 * a fixed array of MX_STATIC_SCRATCH_BYTES that is part of the library's device image (every
 * GPU that loads the library holds these bytes until the process exits).  The caller still
 * passes all inputs and the output; arguments, layouts and result are those of mx_gemm.
 *
 *  - Limit: 2*(M+N)*K bytes (each operand rounded up to 256) must fit in MX_STATIC_SCRATCH_BYTES,
 *    e.g. M = N = K = 2048.  Larger problems return MX_ERR_WORKSPACE without launching
 *    anything; mx_last_cuda_error() then holds the sizes.
 *  - The call creates no buffer, event or handle: no cudaMalloc/cudaFree, no allocating library
 *    routine.  The first call on a device looks up the array's device address and sets a kernel
 *    attribute; make that first call before any stream capture begins.
 *  - The array used is the CURRENT device's copy; the operands must live on that device.
 *  - All calls on a device share the one array.  It keeps the previous call's bytes; the call
 *    rewrites every byte it later reads, so nothing has to be cleared.  Two calls whose kernels
 *    can overlap on the GPU (different streams, or different host threads) race on it: issue
 *    them on one stream or order them with events. */
#define MX_STATIC_SCRATCH_BYTES (32u << 20)
MX_API mx_status_t mx_gemm_static(const void *a_mant, const uint8_t *a_exp, mx_format_t fa,
                                  const void *w_mant, const uint8_t *w_exp, mx_format_t fw,
                                  int64_t M, int64_t N, int64_t K, const float *bias, float *y,
                                  int64_t ldy, void *stream);

/* ---- launch profile (benchmark support; the paper has no counterpart) ---------------------
 *
 * Between mx_profile_begin and mx_profile_end the library brackets each of its kernel launches
 * with a pair of CUDA events on the launch stream.  mx_profile_end waits for them and returns,
 * per kernel kind, the summed device time in milliseconds and the number of launches (arrays of
 * MX_KERNEL_KINDS entries, host memory).  Kinds: 0 quantize (incl. casts and the transposing
 * quantizer), 1 dequantize, 2 tensor-core GEMM, 3 CUDA-core GEMM, 4 weight-streaming GEMM, 5 operand
 * preparation of mx_linear (activation quantize + weight decode in one launch), 6 fp32 glue
 * (LayerNorm, softmax with fp32 or MXInt result, ReLU/add).  Not thread-safe with respect to concurrent
 * compute calls on other host threads being attributed correctly; meant for one stream. */
#define MX_KERNEL_KINDS 8
MX_API mx_status_t mx_profile_begin(void);
MX_API mx_status_t mx_profile_end(double *ms_per_kind, int64_t *launches_per_kind);

#ifdef __cplusplus
}
#endif
#endif /* MXINT_H_ */
