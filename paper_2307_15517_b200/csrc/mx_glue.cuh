// fp32 glue of a transformer block around the MXInt products (the paper keeps LayerNorm, softmax and
// the activation function outside the MX data path; Fig. 1(d) shows the block).  Plain
// HBM-bound row kernels: one CTA per row, values held in registers between the passes.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "mx_quantize.cuh"

namespace mx {

constexpr int GLUE_THREADS = 256;
constexpr int GLUE_MAX_PER_THREAD = 32;          // rows of up to 8192 values stay in registers

__device__ __forceinline__ float block_sum(float v, float *scratch)
{
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    __syncthreads();                              // scratch may still be read from a previous call
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = 0.f;
#pragma unroll
    for (int i = 0; i < GLUE_THREADS / 32; ++i) t += scratch[i];
    return t;
}
__device__ __forceinline__ float block_max(float v, float *scratch)
{
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, d));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = scratch[0];
#pragma unroll
    for (int i = 1; i < GLUE_THREADS / 32; ++i) t = fmaxf(t, scratch[i]);
    return t;
}

// y[r, :] = (x[r, :] - mean) / sqrt(var + eps) * gamma + beta, two-pass variance.
template <int PER>
__global__ void __launch_bounds__(GLUE_THREADS)
layernorm_kernel(const float *__restrict__ x, int64_t ldx, const float *__restrict__ gamma,
                 const float *__restrict__ beta, float eps, int cols, float *__restrict__ y, int64_t ldy)
{
    __shared__ float scratch[GLUE_THREADS / 32];
    const float *xr = x + (int64_t)blockIdx.x * ldx;
    float v[PER];
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const int c = threadIdx.x + i * GLUE_THREADS;
        v[i] = c < cols ? xr[c] : 0.f;
        s += v[i];
    }
    const float mean = block_sum(s, scratch) / (float)cols;
    float q = 0.f;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const int c = threadIdx.x + i * GLUE_THREADS;
        const float d = c < cols ? v[i] - mean : 0.f;
        q += d * d;
    }
    const float rstd = 1.0f / sqrtf(block_sum(q, scratch) / (float)cols + eps);
    float *yr = y + (int64_t)blockIdx.x * ldy;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const int c = threadIdx.x + i * GLUE_THREADS;
        if (c < cols) yr[c] = (v[i] - mean) * rstd * (gamma ? gamma[c] : 1.f) + (beta ? beta[c] : 0.f);
    }
}

// The operand pass of a layer whose input is layer-normalised first (Fig. 1(d): LayerNorm in floating point in
// front of the MX linears): CTA r < M normalises row r exactly as layernorm_kernel does (same ownership of the
// elements, same order of every sum: the values are bit-identical to that kernel's), quantizes them to MXInt --
// element c of the row sits in thread c % 256, so a block of 16 or 32 columns is a group of neighbouring lanes and
// its maximum one round of shuffles -- and writes the exact bf16 operand; the fp32 normalised tensor never exists.
// After its row every CTA decodes its share of the packed weights (decode_bf16_body), so one launch prepares both
// operands of the product, as prep_operands_kernel does for a plain layer.
struct PrepLnJob {
    const float *x;           // [M, K] fp32, leading dimension ldx
    int64_t M, K, ldx;
    const float *gamma, *beta;   // nullable
    float eps;
    int wa, block;
    __nv_bfloat16 *a_hat;     // [M, K]
    const uint8_t *w_mant, *w_exp;
    int64_t N;
    int ww;
    __nv_bfloat16 *w_hat;     // [N, K]
    int w_row_shift;
};

template <int PER, bool NIBBLE>
__global__ void __launch_bounds__(GLUE_THREADS, 4)
prep_ln_operands_kernel(const PrepLnJob j)
{
    __shared__ float scratch[GLUE_THREADS / 32];
    ptx::dep_wait();
    ptx::dep_trigger();
    const int cols = (int)j.K;
    for (int64_t r = blockIdx.x; r < j.M; r += gridDim.x) {
        const float *xr = j.x + r * j.ldx;
        float v[PER];
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const int c = threadIdx.x + i * GLUE_THREADS;
            v[i] = c < cols ? xr[c] : 0.f;
            s += v[i];
        }
        const float mean = block_sum(s, scratch) / (float)cols;
        float q = 0.f;
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const int c = threadIdx.x + i * GLUE_THREADS;
            const float d = c < cols ? v[i] - mean : 0.f;
            q += d * d;
        }
        const float rstd = 1.0f / sqrtf(block_sum(q, scratch) / (float)cols + j.eps);
        __nv_bfloat16 *ar = j.a_hat + r * j.K;
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const int c = threadIdx.x + i * GLUE_THREADS;           // K % block == 0: a block is all inside or all outside
            const float y = c < cols ? (v[i] - mean) * rstd * (j.gamma ? j.gamma[c] : 1.f) + (j.beta ? j.beta[c] : 0.f) : 0.f;
            uint32_t amax = __float_as_uint(absmax_nan(0.f, y));
#pragma unroll
            for (int d = 1; d < 32; d <<= 1)
                if (d < j.block) amax = max(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, d));
            const float y8[8] = {y, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            float xh[8];
            encode8_full(y8, (int)(amax >> 23), j.wa, xh);          // the library's rounding; only xh[0] is used
            if (c < cols) ar[c] = __float2bfloat16_rn(xh[0]);
        }
    }
    PackedStrides ps;
    ps.mant_ld = NIBBLE ? j.K / 2 : j.K;
    ps.exp_ld = j.K / j.block;
    ps.mant_batch = ps.exp_batch = ps.out_batch = 0;
    ps.exp_row_shift = j.w_row_shift;
    const int warps = blockDim.x >> 5;
    decode_bf16_body<NIBBLE, 2>(j.w_mant, j.w_exp, j.N, j.K, j.block, j.ww, j.w_hat, j.K, ps,
                                (int64_t)blockIdx.x * warps + (threadIdx.x >> 5), (int64_t)gridDim.x * warps);
}

// In place: s[r, j] = softmax_j(scale * s[r, j]) over j < limit, 0 elsewhere; limit = cols, or
// (r % rows_per_batch) + 1 with the causal mask.
template <int PER>
__global__ void __launch_bounds__(GLUE_THREADS)
softmax_kernel(float *__restrict__ s, int64_t ld, int cols, float scale, int causal, int64_t rows_per_batch)
{
    __shared__ float scratch[GLUE_THREADS / 32];
    float *row = s + (int64_t)blockIdx.x * ld;
    const int limit = causal ? (int)((int64_t)blockIdx.x % rows_per_batch) + 1 : cols;
    float v[PER];
    float m = -INFINITY;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const int c = threadIdx.x + i * GLUE_THREADS;
        v[i] = (c < cols && c < limit) ? row[c] * scale : -INFINITY;
        m = fmaxf(m, v[i]);
    }
    m = block_max(m, scratch);
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        v[i] = v[i] == -INFINITY ? 0.f : expf(v[i] - m);
        sum += v[i];
    }
    const float inv = 1.0f / block_sum(sum, scratch);
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const int c = threadIdx.x + i * GLUE_THREADS;
        if (c < cols) row[c] = v[i] * inv;
    }
}

// The same softmax with an MXInt result (the probabilities are the quantized left operand of the
// P V product, Fig. 1(d)): p[r, :] = Q(softmax(scale * s[r, :])) with blocks of BLOCK along the
// columns, written as packed mantissas [rows, cols/2 or cols] and exponent bytes [rows, cols/BLOCK];
// no fp32 probabilities are written.  A thread holds 8 consecutive columns per chunk, so a block
// is 2 or 4 neighbouring lanes; rounding as in the quantizer.  cols % 8 == 0, cols % BLOCK == 0.
template <int PER8, int BLOCK>
__global__ void __launch_bounds__(GLUE_THREADS)
softmax_q_kernel(const float *__restrict__ s, int64_t ld, int cols, float scale, int causal, int64_t rows_per_batch,
                 int w, uint8_t *__restrict__ p_mant, uint8_t *__restrict__ p_exp)
{
    __shared__ float scratch[GLUE_THREADS / 32];
    constexpr int LANES = BLOCK / 8, LANE_SHIFT = BLOCK == 16 ? 1 : 2;
    const float *row = s + (int64_t)blockIdx.x * ld;
    const int limit = causal ? (int)((int64_t)blockIdx.x % rows_per_batch) + 1 : cols;
    const int chunks = cols >> 3;
    float v[PER8][8];
    float m = -INFINITY;
#pragma unroll
    for (int i = 0; i < PER8; ++i) {
        const int ch = threadIdx.x + i * GLUE_THREADS;
        if (ch < chunks) {
            const float4 a = *reinterpret_cast<const float4 *>(row + ch * 8);
            const float4 b = *reinterpret_cast<const float4 *>(row + ch * 8 + 4);
            const float t[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
            for (int j = 0; j < 8; ++j) v[i][j] = (ch * 8 + j < limit) ? t[j] * scale : -INFINITY;
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) v[i][j] = -INFINITY;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) m = fmaxf(m, v[i][j]);
    }
    m = block_max(m, scratch);
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < PER8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            v[i][j] = v[i][j] == -INFINITY ? 0.f : expf(v[i][j] - m);
            sum += v[i][j];
        }
    const float inv = 1.0f / block_sum(sum, scratch);
    const bool nibble = w <= 4;
    const int64_t mant_ld = nibble ? (cols >> 1) : cols, nb_row = cols / BLOCK;
#pragma unroll
    for (int i = 0; i < PER8; ++i) {
        const int ch = threadIdx.x + i * GLUE_THREADS;
        float am = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            v[i][j] *= inv;
            am = absmax_nan(am, v[i][j]);
        }
        uint32_t amax = __float_as_uint(am);
#pragma unroll
        for (int d = 1; d < LANES; d <<= 1) amax = max(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, d));
        if (ch < chunks) {
            const int ebyte = (int)(amax >> 23);
            const uint2 pk = encode8_packed(v[i], ebyte, w);
            if (nibble) *reinterpret_cast<uint32_t *>(p_mant + (int64_t)blockIdx.x * mant_ld + ch * 4) = pk.x;
            else *reinterpret_cast<uint2 *>(p_mant + (int64_t)blockIdx.x * mant_ld + ch * 8) = pk;
            if ((threadIdx.x & (LANES - 1)) == 0) p_exp[(int64_t)blockIdx.x * nb_row + (ch >> LANE_SHIFT)] = (uint8_t)ebyte;
        }
    }
}

// y = (relu ? max(a, 0) : a) + (b ? b : 0), elementwise over n values (y may alias a or b).
__global__ void __launch_bounds__(GLUE_THREADS)
relu_add_kernel(const float *a, const float *b, float *y, int64_t n, int relu)
{
    for (int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4; i < n;
         i += (int64_t)gridDim.x * blockDim.x * 4) {
        if (i + 4 <= n) {
            float4 va = *reinterpret_cast<const float4 *>(a + i);
            if (relu) {                                  // NaN stays NaN
                va.x = va.x < 0.f ? 0.f : va.x; va.y = va.y < 0.f ? 0.f : va.y;
                va.z = va.z < 0.f ? 0.f : va.z; va.w = va.w < 0.f ? 0.f : va.w;
            }
            if (b) {
                const float4 vb = *reinterpret_cast<const float4 *>(b + i);
                va.x += vb.x; va.y += vb.y; va.z += vb.z; va.w += vb.w;
            }
            *reinterpret_cast<float4 *>(y + i) = va;
        } else {
            for (int64_t j = i; j < n; ++j) {
                float t = a[j];
                if (relu) t = t < 0.f ? 0.f : t;
                y[j] = b ? t + b[j] : t;
            }
        }
    }
}

}  // namespace mx
