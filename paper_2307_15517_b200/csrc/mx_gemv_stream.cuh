// Decode-shaped MXInt product: a handful of tokens (T <= 16) against weight matrices that are
// streamed from HBM exactly once (Sec. 3.2 MXInt dot-product operator; the paper motivates MX
// formats by the memory footprint of the parameters, Sec. 1 / Sec. 6).
//
// HBM-bound, so the layout of the loads and the number of bytes in flight decide, not the math.
// The math is the literal operator: integer multiply-adds over one block of 32, one shared
// scale per block, blocks added in ascending order in fp32 -- bit-identical to the CUDA-core
// kernel when a row's blocks are not split over warps.
//
//  * weights  : packed 4-bit mantissas [N, K/2] + exponent bytes [N, K/32] (block 32), read with
//               coalesced 32-bit loads, four blocks (and their four exponent bytes) per step,
//               the next step's ten registers prefetched while the current one is consumed.
//  * tokens   : already quantized (int8 or nibble container); each CTA stages them once per
//               layer into shared memory in the operand order of the integer MMA below, with
//               their float block scales and the per-block sums needed to undo the +8 offset.
//  * per block: nibble ^ 8 = q + 8 is an unsigned byte after one AND/shift, so a 16-row x 32-k
//               tile of weights is the A operand of mma.sync.m16n8k32 (u8 x s8 -> s32) with no
//               sign extension; the accumulator starts at 0x4B400000 - 8 * sum(qa), so the result
//               register IS the float 1.5*2^23 + P (P = exact integer block sum), and two FMAs
//               per output apply the weight scale (removing the 1.5*2^23) and the token scale.
//
// A warp owns 16 weight rows.  With split > 1 the K range of a row tile is cut into `split`
// contiguous pieces handled by consecutive warps of one CTA and summed in piece order through
// shared memory (deterministic, but no longer the ascending single chain).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "mx_quantize.cuh"

namespace mx {

struct StreamLayer {
    const uint8_t *w_mant;   // [N, K/2] nibbles
    const uint8_t *w_exp;    // [N, K/32]
    const uint8_t *a_mant;   // [T, K] int8 or [T, K/2] nibbles (a_bits <= 4)
    const uint8_t *a_exp;    // [T, K/32]
    const float *bias;       // nullable
    float *y;                // [T, ldy]
    int64_t ldy;
    int N, K, T;
    int a_bits, w_bits;
    int tile_begin;          // index of this layer's first 16-row tile in the launch
    int n_tiles;             // ceil(N / 16)
};

struct StreamParams {
    const StreamLayer *layers;   // device memory
    int n_layers;
    int total_tiles;
    int split;                   // 1, 2, 4 or 8
    int max_nb;                  // largest K/32 over the layers (sizes the shared-memory arrays)
};

constexpr int STREAM_THREADS = 256;
constexpr int STREAM_MAGIC_INT = 0x4B400000;        // bit pattern of 1.5 * 2^23
constexpr float STREAM_MAGIC = 12582912.0f;

template <int NT> constexpr size_t stream_smem_bytes(int max_nb)
{
    // operand words + token scales + accumulator seeds + split-K exchange
    return (size_t)max_nb * NT * 8 * (4 * 8 + 4 + 4) + 8 * NT * 4 * 32 * 4;
}

__device__ __forceinline__ void mma_u8s8_m16n8k32(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                                  uint32_t a3, uint32_t b0, uint32_t b1, int c0, int c1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%10,%11,%12,%13};"
        : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(c0), "r"(c1), "r"(c0), "r"(c1));
}

// NT = number of 8-token column tiles (1: T <= 8, 2: T <= 16).
template <int NT>
__global__ void __launch_bounds__(STREAM_THREADS)
gemv_stream_kernel(const StreamParams p)
{
    extern __shared__ __align__(16) uint8_t smem[];
    constexpr int TP = NT * 8;                                   // padded token count
    uint2 *sB = reinterpret_cast<uint2 *>(smem);                 // [nb][TP][4]: (even-k word, odd-k word)
    float *sSa = reinterpret_cast<float *>(smem + (size_t)p.max_nb * TP * 32);   // [nb][TP]
    int *sC = reinterpret_cast<int *>(sSa + (size_t)p.max_nb * TP);              // [nb][TP]
    float *sRed = reinterpret_cast<float *>(sC + (size_t)p.max_nb * TP);         // [8][NT][4][32]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int S = p.split, TPR = 8 / S;                          // row tiles per round of the CTA

    const int per = (p.total_tiles + gridDim.x - 1) / gridDim.x;
    int tile_lo = blockIdx.x * per;
    const int tile_hi = min(tile_lo + per, p.total_tiles);
    int li = 0;
    while (li + 1 < p.n_layers && p.layers[li + 1].tile_begin <= tile_lo) ++li;

    while (tile_lo < tile_hi) {
        const StreamLayer L = p.layers[li];
        const int l_end = min(tile_hi, L.tile_begin + L.n_tiles);
        const int nb = L.K >> 5;

        // ---- stage this layer's tokens: operand words, block scales, accumulator seeds ----
        __syncthreads();                                         // previous layer fully consumed
        for (int i = threadIdx.x; i < nb * TP * 4; i += STREAM_THREADS) {
            const int tq = i & 3, tok = (i >> 2) % TP, b = (i >> 2) / TP;
            uint32_t lo = 0, hi = 0;                             // 8 mantissas, k = 32b + 8tq ..
            if (tok < L.T) {
                if (L.a_bits <= 4) {
                    const uint32_t pk = __ldg(reinterpret_cast<const uint32_t *>(
                        L.a_mant + (int64_t)tok * (L.K >> 1) + b * 16 + tq * 4));
                    uint32_t by[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) by[j] = (uint32_t)((((int)(pk << (28 - 4 * j))) >> 28) & 0xFF);
                    lo = by[0] | (by[1] << 8) | (by[2] << 16) | (by[3] << 24);
                    hi = by[4] | (by[5] << 8) | (by[6] << 16) | (by[7] << 24);
                } else {
                    const uint2 v = __ldg(reinterpret_cast<const uint2 *>(
                        L.a_mant + (int64_t)tok * L.K + b * 32 + tq * 8));
                    lo = v.x;
                    hi = v.y;
                }
            }
            // MMA slots 4t..4t+3 take the even k of this group of 8, slots 16+4t.. the odd k
            sB[i] = make_uint2(__byte_perm(lo, hi, 0x6420), __byte_perm(lo, hi, 0x7531));
            int sum = __dp4a((int)lo, 0x01010101, __dp4a((int)hi, 0x01010101, 0));
            sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 1);
            sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 2);         // the 4 groups of one block
            if (tq == 0) {
                const int eb = tok < L.T ? (int)__ldg(L.a_exp + (int64_t)tok * nb + b) : 0;
                sSa[b * TP + tok] = f32_scale(eb, L.a_bits);
                sC[b * TP + tok] = STREAM_MAGIC_INT - 8 * sum;
            }
        }
        __syncthreads();

        const int64_t w_ld = L.K >> 1;
        for (int base = tile_lo; base < l_end; base += TPR) {
            const int tile = base + warp / S, s = warp % S;
            const bool active = tile < l_end;
            float acc[NT][4];
#pragma unroll
            for (int n = 0; n < NT; ++n)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[n][j] = 0.f;
            const int r0 = (tile - L.tile_begin) * 16;
            if (active) {
                const int rowA = min(r0 + g, L.N - 1), rowB = min(r0 + g + 8, L.N - 1);
                const uint8_t *mA = L.w_mant + (int64_t)rowA * w_ld + t * 4;
                const uint8_t *mB = L.w_mant + (int64_t)rowB * w_ld + t * 4;
                const uint8_t *eA = L.w_exp + (int64_t)rowA * nb;
                const uint8_t *eB = L.w_exp + (int64_t)rowB * nb;
                const int b_lo = (nb / S) * s, b_hi = b_lo + nb / S;       // nb % (4*S) == 0
                uint32_t wa[4], wb[4], ea, eb;
                auto fetch = [&](int b, uint32_t (&xa)[4], uint32_t (&xb)[4], uint32_t &xea, uint32_t &xeb) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        xa[j] = __ldcs(reinterpret_cast<const uint32_t *>(mA + (b + j) * 16));
                        xb[j] = __ldcs(reinterpret_cast<const uint32_t *>(mB + (b + j) * 16));
                    }
                    xea = __ldcs(reinterpret_cast<const uint32_t *>(eA + b));
                    xeb = __ldcs(reinterpret_cast<const uint32_t *>(eB + b));
                };
                fetch(b_lo, wa, wb, ea, eb);
                for (int b = b_lo; b < b_hi; b += 4) {
                    uint32_t na[4], nbw[4], nea = 0, neb = 0;
                    if (b + 4 < b_hi) fetch(b + 4, na, nbw, nea, neb);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int ebA = (int)((ea >> (8 * j)) & 0xFF), ebB = (int)((eb >> (8 * j)) & 0xFF);
                        const float swA = f32_scale(ebA, L.w_bits), swB = f32_scale(ebB, L.w_bits);
                        // far up the exponent range 1.5*2^23 * scale is not finite: take two steps there
                        const bool top = (ebA > 225 && ebA != 255) || (ebB > 225 && ebB != 255);
                        const float mwA = -STREAM_MAGIC * swA, mwB = -STREAM_MAGIC * swB;
                        const uint32_t pa = wa[j] ^ 0x88888888u, pb = wb[j] ^ 0x88888888u;
                        const uint32_t a0 = pa & 0x0F0F0F0Fu, a2 = (pa >> 4) & 0x0F0F0F0Fu;
                        const uint32_t a1 = pb & 0x0F0F0F0Fu, a3 = (pb >> 4) & 0x0F0F0F0Fu;
                        const int blk = b + j;
#pragma unroll
                        for (int n = 0; n < NT; ++n) {
                            const uint2 bf = sB[(blk * TP + n * 8 + g) * 4 + t];
                            const int2 c = *reinterpret_cast<const int2 *>(&sC[blk * TP + n * 8 + 2 * t]);
                            const float2 sa = *reinterpret_cast<const float2 *>(&sSa[blk * TP + n * 8 + 2 * t]);
                            int d[4];
                            mma_u8s8_m16n8k32(d, a0, a1, a2, a3, bf.x, bf.y, c.x, c.y);
                            float p0, p1, p2, p3;                 // P * weight scale, exact
                            if (!top) {
                                p0 = fmaf(__int_as_float(d[0]), swA, mwA);
                                p1 = fmaf(__int_as_float(d[1]), swA, mwA);
                                p2 = fmaf(__int_as_float(d[2]), swB, mwB);
                                p3 = fmaf(__int_as_float(d[3]), swB, mwB);
                            } else {
                                p0 = (__int_as_float(d[0]) - STREAM_MAGIC) * swA;
                                p1 = (__int_as_float(d[1]) - STREAM_MAGIC) * swA;
                                p2 = (__int_as_float(d[2]) - STREAM_MAGIC) * swB;
                                p3 = (__int_as_float(d[3]) - STREAM_MAGIC) * swB;
                            }
                            acc[n][0] = fmaf(p0, sa.x, acc[n][0]);   // one rounding per block, ascending
                            acc[n][1] = fmaf(p1, sa.y, acc[n][1]);
                            acc[n][2] = fmaf(p2, sa.x, acc[n][2]);
                            acc[n][3] = fmaf(p3, sa.y, acc[n][3]);
                        }
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        wa[j] = na[j];
                        wb[j] = nbw[j];
                    }
                    ea = nea;
                    eb = neb;
                }
            }
            if (S > 1) {                                             // CTA-uniform branch
                __syncthreads();
#pragma unroll
                for (int n = 0; n < NT; ++n)
#pragma unroll
                    for (int j = 0; j < 4; ++j) sRed[((warp * NT + n) * 4 + j) * 32 + lane] = acc[n][j];
                __syncthreads();
                if (s == 0 && active) {
#pragma unroll
                    for (int n = 0; n < NT; ++n)
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            float v = acc[n][j];
                            for (int q = 1; q < S; ++q) v += sRed[(((warp + q) * NT + n) * 4 + j) * 32 + lane];
                            acc[n][j] = v;
                        }
                }
            }
            if (active && s == 0) {
#pragma unroll
                for (int n = 0; n < NT; ++n)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int row = r0 + g + (j >> 1) * 8, tok = n * 8 + 2 * t + (j & 1);
                        if (row < L.N && tok < L.T)
                            L.y[(int64_t)tok * L.ldy + row] = L.bias ? acc[n][j] + __ldg(L.bias + row) : acc[n][j];
                    }
            }
        }
        tile_lo = l_end;
        ++li;
    }
}

}  // namespace mx
