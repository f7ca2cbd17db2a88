// The two other MX formats the paper compares with MXInt (Sec. 2 "What are MX Formats?", Table 1,
// Fig. 5): Block Minifloat (BMF: every element a small floating-point number, the exponent bias shared
// by the block) and Block Logarithm (BL: sign and exponent only, every value a power of two, bias
// shared).  Quantizers and the exact decode to bf16 that feeds the same tensor-core product as MXInt.
//
// Encoding (the paper gives words only; these are the library's readings, stated in mxint.h):
//   element  = one byte: sign << (ebits+mbits) | F << mbits | T   (F: ebits-bit exponent field, T: mantissa)
//   shared   = one byte per block of B along k: 127 + beta, 2^beta = binade of the top field Fmax = 2^ebits - 1;
//              0 = zero block (decodes to zeros), 255 = the block holds Inf/NaN (decodes to NaN)
//   BMF      : F >= 1: +-2^(beta-(Fmax-F)) (1 + T/2^mbits);  F == 0: +-2^(beta-(Fmax-1)) T/2^mbits;
//              beta = floor(log2 max|x|), round to nearest even on the element's grid, saturating
//   BL       : F >= 1: +-2^(beta-(Fmax-F));  F == 0: zero;  rounding in the log domain (up iff the
//              significand is >= sqrt(2)), beta = rounded exponent of max|x|
//   a block whose maximum is below 2^-95 is stored as a zero block, so every decoded value is a bf16 number
//
// HBM-bound streaming kernels with the same work split as the MXInt quantizer: a warp item is one row
// times 256 elements, a lane owns 8 consecutive elements, the 2 or 4 lanes of a block exchange their
// maximum with shuffles.  All arithmetic is on the binary32 bit pattern: no rounding instruction is
// involved, so the codes are the definition's bit for bit.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mx_ptx.cuh"
#include "mx_quantize.cuh"

namespace mx {

enum AltKind { ALT_BMF = 1, ALT_BL = 2 };

struct AltFormat {
    int kind, block, ebits, mbits;
};

// 2^s for s in [-149, 127] from its bit pattern.
__device__ __forceinline__ float pow2_any(int s)
{
    return __uint_as_float(s >= -126 ? (uint32_t)(s + 127) << 23 : 1u << (s + 149));
}

// Magnitude code of one finite value with bit pattern `a` (sign cleared) in a block with shared byte sb >= 32.
__device__ __forceinline__ uint32_t alt_code(uint32_t a, int sb, const AltFormat &f)
{
    const int fmax = (1 << f.ebits) - 1;
    const int ex = (int)(a >> 23);
    const uint32_t man = a & 0x007FFFFFu;
    if (f.kind == ALT_BL) {
        if (ex == 0) return 0u;                                         // zero or binary32 subnormal
        const int F = ex + (man >= 0x003504F4u ? 1 : 0) - sb + fmax;    // significand >= sqrt(2): next power
        return (uint32_t)(F > fmax ? fmax : (F < 1 ? 0 : F));
    }
    const int F = ex - sb + fmax;                                       // exponent field if the value is normal in the format
    const uint32_t top = (uint32_t)(fmax << f.mbits) | ((1u << f.mbits) - 1u);
    uint32_t code;
    if (F >= 1 && ex > 0) {
        // keep mbits of the 23 mantissa bits, nearest even; a carry rolls into the exponent field
        const int sh = 23 - f.mbits;
        const uint32_t T = (man + (1u << (sh - 1)) - 1u + ((man >> sh) & 1u)) >> sh;
        code = ((uint32_t)F << f.mbits) + T;
    } else {
        // below the format's normal range: units of its subnormal step 2^(beta-(Fmax-1)-mbits), two exact scalings
        const float t = (__uint_as_float(a) * pow2_any(127 - sb)) * pow2_any(fmax - 1 + f.mbits);
        code = (uint32_t)__float2int_rn(t);                             // <= 2^mbits: lands on F = 1, T = 0 by itself
    }
    return code > top ? top : code;
}

// Decoded value of a code byte under shared byte sb (exact in fp32 and in bf16).
__device__ __forceinline__ float alt_value(uint32_t code, int sb, const AltFormat &f)
{
    if (sb == 255) return __uint_as_float(0x7FC00000u);
    if (sb == 0) return 0.f;
    const int fmax = (1 << f.ebits) - 1;
    const uint32_t mag = code & ((1u << (f.ebits + f.mbits)) - 1u);
    const int F = (int)(mag >> f.mbits);
    const uint32_t T = mag & ((1u << f.mbits) - 1u);
    const uint32_t sig = F ? (1u << f.mbits) + T : T;                    // BL: mbits = 0, sig = 1 or 0
    const float v = (float)sig * pow2_any(sb - 127 - fmax + (F > 1 ? F : 1) - f.mbits);
    return ((code >> (f.ebits + f.mbits)) & 1u) ? -v : v;
}

template <typename InT, int BLOCK>
__global__ void __launch_bounds__(256)
alt_quantize_kernel(const InT *__restrict__ x, int64_t rows, int64_t K, int64_t ldx, AltFormat f,
                    uint8_t *__restrict__ codes, uint8_t *__restrict__ shared, uint32_t *nonfinite)
{
    ptx::dep_wait();
    ptx::dep_trigger();
    constexpr int LANES = BLOCK / 8, LANE_SHIFT = BLOCK == 16 ? 1 : 2;
    const int lane = threadIdx.x & 31;
    const int64_t cpr = K >> 3, segs = (cpr + 31) >> 5, n_items = rows * segs;
    const int64_t n_warps = (int64_t)gridDim.x * (blockDim.x >> 5), nb_row = K / BLOCK;
    const bool leader = (lane & (LANES - 1)) == 0;
    for (int64_t it = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); it < n_items; it += n_warps) {
        const int64_t row = it / segs, kc = (it - row * segs) * 32 + lane;
        const bool live = kc < cpr;
        float v[8];
        if (live) {
            Load8<InT>::run(x + row * ldx + kc * 8, v);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = 0.f;
        }
        float am = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) am = absmax_nan(am, v[i]);
        uint32_t amax = __float_as_uint(am);
#pragma unroll
        for (int d = 1; d < LANES; d <<= 1) amax = max(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, d));
        if (!live) continue;
        int sb = (int)(amax >> 23);                                      // 255 <=> an Inf or NaN in the block
        const bool bad = sb == 255;
        if (!bad) {
            if (f.kind == ALT_BL && sb > 0) sb = min(sb + ((amax & 0x007FFFFFu) >= 0x003504F4u ? 1 : 0), 254);
            if (sb < 32) sb = 0;                                         // zero, subnormal or tiny block
        }
        uint32_t c[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t bits = __float_as_uint(v[i]);
            const uint32_t mag = (bad || sb == 0) ? 0u : alt_code(bits & 0x7FFFFFFFu, sb, f);
            c[i] = (bad || sb == 0) ? 0u : (((bits >> 31) << (f.ebits + f.mbits)) | mag);
        }
        *reinterpret_cast<uint2 *>(codes + row * K + kc * 8) =
            make_uint2(c[0] | (c[1] << 8) | (c[2] << 16) | (c[3] << 24), c[4] | (c[5] << 8) | (c[6] << 16) | (c[7] << 24));
        if (leader) {
            shared[row * nb_row + (kc >> LANE_SHIFT)] = (uint8_t)sb;
            if (bad && nonfinite) atomicAdd(nonfinite, 1u);
        }
    }
}

// codes + shared bytes -> decoded values (bf16: the MMA operand form; fp32: test helper), 8 per thread.
template <typename OutT>
__global__ void __launch_bounds__(256)
alt_decode_kernel(const uint8_t *__restrict__ codes, const uint8_t *__restrict__ shared, int64_t rows, int64_t K, AltFormat f,
                  OutT *__restrict__ out, int64_t ld_out)
{
    ptx::dep_wait();
    ptx::dep_trigger();
    const int64_t cpr = K >> 3, total = rows * cpr, nb_row = K / f.block;
    const int sh = f.block == 16 ? 1 : 2;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = t / cpr, kc = t - row * cpr;
        const uint2 p = __ldg(reinterpret_cast<const uint2 *>(codes + row * K + kc * 8));
        const int sb = __ldg(shared + row * nb_row + (kc >> sh));
        float v[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[i] = alt_value((p.x >> (8 * i)) & 0xFFu, sb, f);
            v[4 + i] = alt_value((p.y >> (8 * i)) & 0xFFu, sb, f);
        }
        OutT *o = out + row * ld_out + kc * 8;
        if constexpr (sizeof(OutT) == 4) {
            reinterpret_cast<float4 *>(o)[0] = make_float4(v[0], v[1], v[2], v[3]);
            reinterpret_cast<float4 *>(o)[1] = make_float4(v[4], v[5], v[6], v[7]);
        } else {
            uint32_t h[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) h[i] = as_u32(__floats2bfloat162_rn(v[2 * i], v[2 * i + 1]));
            *reinterpret_cast<uint4 *>(o) = make_uint4(h[0], h[1], h[2], h[3]);
        }
    }
}

}  // namespace mx
