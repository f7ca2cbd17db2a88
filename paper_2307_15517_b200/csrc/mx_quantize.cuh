// MXInt quantizer and its inverse (Sec. 3.2 software emulator; format of Sec. 2 / Sec. 4.1).
//
// HBM-bound streaming kernels.  One thread owns 8 consecutive elements of a row (32 B of fp32
// or 16 B of bf16, one or two 128-bit loads); the 2 (block 16) or 4 (block 32) lanes that
// cover one block exchange their largest magnitude with warp shuffles, so the shared exponent
// costs no shared memory and no second pass over the data.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mx {

// 2^(e) for e in [-127, 127], built from its bit pattern (2^-127 is a subnormal).
__device__ __forceinline__ float pow2_from_biased(int biased /* e + 127, 0..254 */)
{
    return __uint_as_float(biased == 0 ? 0x00400000u : ((uint32_t)biased << 23));
}

// Decode scale of a block: 2^(E-(w-2)) split into two exactly representable factors.
// value = (q * 2^-(w-2)) * 2^E
__device__ __forceinline__ float small_neg_pow2(int w) { return __uint_as_float((uint32_t)(127 - (w - 2)) << 23); }

__device__ __forceinline__ float decode_value(int q, int ebyte, int w)
{
    if (ebyte == 255) return __uint_as_float(0x7FC00000u);
    // |q| * 2^-(w-2) < 2, so neither product can overflow and both are exact
    return ((float)q * small_neg_pow2(w)) * pow2_from_biased(ebyte);
}

// Round one value to its mantissa: x * 2^-E * 2^(w-2), nearest-even, symmetric clamp.
__device__ __forceinline__ int encode_value(float x, float inv_pow2_E, float pow2_wm2, int qmax)
{
    int q = __float2int_rn(x * inv_pow2_E * pow2_wm2);
    return max(-qmax, min(qmax, q));
}

struct QuantOut {
    uint8_t *mant;        // packed mantissas (nullable)
    uint8_t *exps;        // exponent bytes (nullable together with mant)
    __nv_bfloat16 *xhat;  // decoded values as bf16, [rows, ld_xhat] (nullable)
    int64_t ld_xhat;
    uint32_t *nonfinite;  // nullable
};

template <typename InT> struct Load8;
template <> struct Load8<float> {
    static __device__ __forceinline__ void run(const float *p, float (&v)[8])
    {
        const float4 a = __ldg(reinterpret_cast<const float4 *>(p));
        const float4 b = __ldg(reinterpret_cast<const float4 *>(p) + 1);
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
        v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    }
};
template <> struct Load8<__nv_bfloat16> {
    static __device__ __forceinline__ void run(const __nv_bfloat16 *p, float (&v)[8])
    {
        const uint4 a = __ldg(reinterpret_cast<const uint4 *>(p));
        const uint32_t u[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(u[i] << 16);          // bf16 -> fp32 is a 16-bit shift
            v[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u);
        }
    }
};

// rows x K, rows contiguous along K with leading dimension ldx.  BLOCK in {16, 32}.
template <typename InT, int BLOCK>
__global__ void __launch_bounds__(256)
quantize_rows_kernel(const InT *__restrict__ x, int64_t rows, int64_t K, int64_t ldx, int w,
                     QuantOut out)
{
    constexpr int LANES = BLOCK / 8;                    // lanes sharing one block
    const int64_t chunks_per_row = K >> 3;
    const int64_t total = rows * chunks_per_row;
    const int qmax = (1 << (w - 1)) - 1;
    const float pow2_wm2 = (float)(1 << (w - 2));
    const bool nibble = w <= 4;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    // trip count is uniform over the warp so that the shuffles below see all 32 lanes
    const int64_t first = (int64_t)blockIdx.x * blockDim.x + (threadIdx.x & ~31);
    for (int64_t base = first; base < total; base += stride) {
        const int64_t c = base + (threadIdx.x & 31);
        const bool live = c < total;
        const int64_t row = live ? c / chunks_per_row : 0;
        const int64_t kc = live ? c - row * chunks_per_row : 0;
        float v[8];
        if (live) {
            Load8<InT>::run(x + row * ldx + kc * 8, v);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = 0.f;
        }
        uint32_t amax = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) amax = max(amax, __float_as_uint(v[i]) & 0x7FFFFFFFu);
#pragma unroll
        for (int d = 1; d < LANES; d <<= 1) amax = max(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, d));
        const int ebyte = (int)(amax >> 23);            // 255 <=> an Inf or NaN in the block
        const bool bad = ebyte == 255;
        const float inv_pow2_E = pow2_from_biased(254 - (bad ? 254 : ebyte));
        int q[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) q[i] = bad ? 0 : encode_value(v[i], inv_pow2_E, pow2_wm2, qmax);
        if (!live) continue;
        const bool leader = (threadIdx.x & (LANES - 1)) == 0;
        if (out.mant) {
            if (nibble) {
                uint32_t p = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) p |= ((uint32_t)q[i] & 0xFu) << (4 * i);
                *reinterpret_cast<uint32_t *>(out.mant + row * (K >> 1) + kc * 4) = p;
            } else {
                uint2 p;
                p.x = ((uint32_t)q[0] & 0xFF) | (((uint32_t)q[1] & 0xFF) << 8) |
                      (((uint32_t)q[2] & 0xFF) << 16) | ((uint32_t)q[3] << 24);
                p.y = ((uint32_t)q[4] & 0xFF) | (((uint32_t)q[5] & 0xFF) << 8) |
                      (((uint32_t)q[6] & 0xFF) << 16) | ((uint32_t)q[7] << 24);
                *reinterpret_cast<uint2 *>(out.mant + row * K + kc * 8) = p;
            }
            if (leader) out.exps[row * (K / BLOCK) + kc / LANES] = (uint8_t)ebyte;
        }
        if (out.xhat) {
            uint32_t h[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const __nv_bfloat16 lo = __float2bfloat16_rn(decode_value(q[2 * i], ebyte, w));
                const __nv_bfloat16 hi = __float2bfloat16_rn(decode_value(q[2 * i + 1], ebyte, w));
                h[i] = (uint32_t)__bfloat16_as_ushort(lo) | ((uint32_t)__bfloat16_as_ushort(hi) << 16);
            }
            *reinterpret_cast<uint4 *>(out.xhat + row * out.ld_xhat + kc * 8) =
                make_uint4(h[0], h[1], h[2], h[3]);
        }
        if (bad && leader && out.nonfinite) atomicAdd(out.nonfinite, 1u);
    }
}

// Generic-stride variant (blocks along a strided axis): one thread per block, plain loads.
// Element (r, k) at x[r*stride_row + k*stride_k].  Threads are laid out with r fastest so that
// stride_row == 1 (a transposed view) still reads coalesced.
template <typename InT>
__global__ void __launch_bounds__(256)
quantize_strided_kernel(const InT *__restrict__ x, int64_t rows, int64_t K, int64_t stride_row,
                        int64_t stride_k, int block, int w, QuantOut out)
{
    const int64_t nb = K / block;
    const int64_t total = rows * nb;
    const int qmax = (1 << (w - 1)) - 1;
    const float pow2_wm2 = (float)(1 << (w - 2));
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
         t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t b = t / rows, row = t - b * rows;
        const InT *p = x + row * stride_row + b * block * stride_k;
        uint32_t amax = 0;
        for (int k = 0; k < block; ++k)
            amax = max(amax, __float_as_uint((float)p[k * stride_k]) & 0x7FFFFFFFu);
        const int ebyte = (int)(amax >> 23);
        const bool bad = ebyte == 255;
        const float inv_pow2_E = pow2_from_biased(254 - (bad ? 254 : ebyte));
        out.exps[row * nb + b] = (uint8_t)ebyte;
        if (bad && out.nonfinite) atomicAdd(out.nonfinite, 1u);
        for (int k = 0; k < block; k += 2) {
            const int q0 = bad ? 0 : encode_value((float)p[k * stride_k], inv_pow2_E, pow2_wm2, qmax);
            const int q1 = bad ? 0 : encode_value((float)p[(k + 1) * stride_k], inv_pow2_E, pow2_wm2, qmax);
            if (w <= 4) {
                out.mant[row * (K >> 1) + ((b * block + k) >> 1)] = (uint8_t)((q0 & 0xF) | ((q1 & 0xF) << 4));
            } else {
                out.mant[row * K + b * block + k] = (uint8_t)q0;
                out.mant[row * K + b * block + k + 1] = (uint8_t)q1;
            }
        }
    }
}

// (mant, exps) -> decoded values, 8 elements per thread.
template <typename OutT>
__global__ void __launch_bounds__(256)
dequantize_kernel(const uint8_t *__restrict__ mant, const uint8_t *__restrict__ exps, int64_t rows,
                  int64_t K, int block, int w, OutT *__restrict__ out, int64_t ld_out)
{
    const int64_t chunks_per_row = K >> 3;
    const int64_t total = rows * chunks_per_row;
    for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < total;
         c += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = c / chunks_per_row, kc = c - row * chunks_per_row;
        const int ebyte = __ldg(exps + row * (K / block) + (kc * 8) / block);
        int q[8];
        if (w <= 4) {
            const uint32_t p = __ldg(reinterpret_cast<const uint32_t *>(mant + row * (K >> 1) + kc * 4));
#pragma unroll
            for (int i = 0; i < 8; ++i) q[i] = ((int)(p << (28 - 4 * i))) >> 28;
        } else {
            const uint2 p = __ldg(reinterpret_cast<const uint2 *>(mant + row * K + kc * 8));
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                q[i] = ((int)(p.x << (24 - 8 * i))) >> 24;
                q[4 + i] = ((int)(p.y << (24 - 8 * i))) >> 24;
            }
        }
        OutT *o = out + row * ld_out + kc * 8;
        if constexpr (sizeof(OutT) == 4) {
            float4 a, b;
            a.x = decode_value(q[0], ebyte, w); a.y = decode_value(q[1], ebyte, w);
            a.z = decode_value(q[2], ebyte, w); a.w = decode_value(q[3], ebyte, w);
            b.x = decode_value(q[4], ebyte, w); b.y = decode_value(q[5], ebyte, w);
            b.z = decode_value(q[6], ebyte, w); b.w = decode_value(q[7], ebyte, w);
            reinterpret_cast<float4 *>(o)[0] = a;
            reinterpret_cast<float4 *>(o)[1] = b;
        } else {
            uint32_t h[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const __nv_bfloat16 lo = __float2bfloat16_rn(decode_value(q[2 * i], ebyte, w));
                const __nv_bfloat16 hi = __float2bfloat16_rn(decode_value(q[2 * i + 1], ebyte, w));
                h[i] = (uint32_t)__bfloat16_as_ushort(lo) | ((uint32_t)__bfloat16_as_ushort(hi) << 16);
            }
            *reinterpret_cast<uint4 *>(o) = make_uint4(h[0], h[1], h[2], h[3]);
        }
    }
}

}  // namespace mx
