// fp32 glue of a transformer block around the MXInt products (the paper keeps LayerNorm, softmax and
// the activation function outside the MX data path; Fig. 1(d) shows the block).  Plain
// HBM-bound row kernels: one CTA per row, values held in registers between the passes.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

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
