// CUDA-core MXInt product: the literal form of the MXInt dot-product operator (Sec. 3.2,
// Fig. 3 right) -- integer multiply-adds on the mantissas of one block, one shared-exponent
// shift per block, blocks added in ascending order in fp32.  Deterministic and bit-reproducible;
// used as the on-device cross-check of the tensor-core kernel and for tiny problems.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace mx {

// 8 consecutive mantissas of a row as two int8x4 words.
__device__ __forceinline__ void load8_as_s8x4(const uint8_t *__restrict__ mant, int64_t row,
                                              int64_t K, int64_t k8, bool nibble, uint32_t &lo,
                                              uint32_t &hi)
{
    if (nibble) {
        const uint32_t p = __ldg(reinterpret_cast<const uint32_t *>(mant + row * (K >> 1) + k8 * 4));
        uint32_t b[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) b[i] = (uint32_t)((((int)(p << (28 - 4 * i))) >> 28) & 0xFF);
        lo = b[0] | (b[1] << 8) | (b[2] << 16) | (b[3] << 24);
        hi = b[4] | (b[5] << 8) | (b[6] << 16) | (b[7] << 24);
    } else {
        const uint2 p = __ldg(reinterpret_cast<const uint2 *>(mant + row * K + k8 * 8));
        lo = p.x;
        hi = p.y;
    }
}

// One thread per output element; 16x16 outputs per CTA.
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const uint8_t *__restrict__ a_mant, const uint8_t *__restrict__ a_exp, int wa,
                 const uint8_t *__restrict__ w_mant, const uint8_t *__restrict__ w_exp, int ww,
                 int64_t M, int64_t N, int64_t K, int block, const float *__restrict__ bias,
                 float *__restrict__ y, int64_t ldy, int a_row_shift, int w_row_shift)
{
    const int64_t j = (int64_t)blockIdx.x * 16 + (threadIdx.x & 15);
    const int64_t i = (int64_t)blockIdx.y * 16 + (threadIdx.x >> 4);
    if (i >= M || j >= N) return;
    const int64_t nb = K / block;
    const bool a_nib = wa <= 4, w_nib = ww <= 4;
    const int shift0 = -254 - (wa - 2) - (ww - 2);
    float acc = 0.f;
    bool poisoned = false;
    for (int64_t b = 0; b < nb; ++b) {
        int P = 0;
        for (int c = 0; c < block / 8; ++c) {
            uint32_t al, ah, wl, wh;
            load8_as_s8x4(a_mant, i, K, b * (block / 8) + c, a_nib, al, ah);
            load8_as_s8x4(w_mant, j, K, b * (block / 8) + c, w_nib, wl, wh);
            P = __dp4a((int)al, (int)wl, P);
            P = __dp4a((int)ah, (int)wh, P);
        }
        const int ea = a_exp[(i >> a_row_shift) * nb + b], ew = w_exp[(j >> w_row_shift) * nb + b];   // shifts: two-row blocks
        poisoned |= (ea == 255) | (ew == 255);
        acc = acc + ldexpf((float)P, ea + ew + shift0);   // |P| < 2^24: exact before the add
    }
    if (bias) acc = acc + bias[j];
    y[i * ldy + j] = poisoned ? __uint_as_float(0x7FC00000u) : acc;
}

}  // namespace mx
