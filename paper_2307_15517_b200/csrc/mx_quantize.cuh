// MXInt quantizer and its inverse (Sec. 3.2 software emulator; format of Sec. 2 / Sec. 4.1).
//
// HBM-bound streaming kernels.  One thread owns 8 consecutive elements of a row (32 B of fp32
// or 16 B of bf16, one or two 128-bit loads); the 2 (block 16) or 4 (block 32) lanes that
// cover one block exchange their largest magnitude with warp shuffles, so the shared exponent
// costs no shared memory and no second pass over the data.
#pragma once
#include "mx_ptx.cuh"
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

// ---- fast exact decode of packed mantissas to bf16 (the MMA operand form) -------------------
// bf16 bit pattern of the block scale 2^(E-(w-2)), both halves; e_field = Ebyte - (w-2) may be
// <= 0 (bf16 subnormal scale) and Ebyte 255 marks a non-finite block (NaN scale).
__device__ __forceinline__ uint32_t bf16x2_scale_bits(int ebyte, int w)
{
    const int e = ebyte - (w - 2);
    uint32_t b = e > 0 ? ((uint32_t)e << 7) : (1u << (6 + e));
    if (ebyte == 255) b = 0x7FC0u;
    return b | (b << 16);
}
__device__ __forceinline__ __nv_bfloat162 as_bf162(uint32_t u)
{
    return *reinterpret_cast<__nv_bfloat162 *>(&u);
}
__device__ __forceinline__ uint32_t as_u32(__nv_bfloat162 v)
{
    return *reinterpret_cast<uint32_t *>(&v);
}

// Slow but range-safe decode of 8 mantissas (used for blocks whose scale is within 2^8 of the
// top of the bf16 range, where the fused multiply-add below would overflow its constant).
__device__ __forceinline__ void decode8_safe(const int (&q)[8], int ebyte, int w, uint32_t (&out)[4])
{
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat16 lo = __float2bfloat16_rn(decode_value(q[2 * i], ebyte, w));
        const __nv_bfloat16 hi = __float2bfloat16_rn(decode_value(q[2 * i + 1], ebyte, w));
        out[i] = (uint32_t)__bfloat16_as_ushort(lo) | ((uint32_t)__bfloat16_as_ushort(hi) << 16);
    }
}

// 8 two's-complement nibbles (k ascending from bit 0) -> 8 bf16 values q * s, exact, for a
// power-of-two scale s (bf16x2, both halves) and c = -136 * s.
// nibble ^ 8 = q + 8 in [0,15]; 0x4300 | that is the bf16 number 128 + (q + 8); one bf16x2 fma
// gives (136 + q) * s - 136 * s = q * s with a single, exact rounding.
__device__ __forceinline__ void decode8_nibbles(uint32_t p, __nv_bfloat162 s, __nv_bfloat162 c,
                                                uint32_t (&out)[4])
{
    uint32_t v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t x = (((p >> (4 * i)) & 0x000F000Fu) ^ 0x00080008u) | 0x43004300u;   // (n_i, n_{i+4})
        v[i] = as_u32(__hfma2(as_bf162(x), s, c));
    }
    out[0] = __byte_perm(v[0], v[1], 0x5410);      // (k0, k1)
    out[1] = __byte_perm(v[2], v[3], 0x5410);      // (k2, k3)
    out[2] = __byte_perm(v[0], v[1], 0x7632);      // (k4, k5)
    out[3] = __byte_perm(v[2], v[3], 0x7632);      // (k6, k7)
}
// The fma constant -136*s must stay finite: scale field (Ebyte - (w-2)) at most 240.
__device__ __forceinline__ bool nibble_fast_ok(int ebyte, int w) { return ebyte == 255 || ebyte - (w - 2) <= 240; }

// 8 int8 mantissas (two words, k ascending) -> 8 bf16 values q * s, exact, for a power-of-two
// fp32 scale s and c = -(2^23 + 128) * s.  byte ^ 0x80 = q + 128; 0x4B000000 | that is the float
// 2^23 + (q + 128); one fp32 fma removes the offset and applies the scale.
__device__ __forceinline__ void decode8_bytes(uint32_t p0, uint32_t p1, float s, float c, uint32_t (&out)[4])
{
    const uint32_t t0 = p0 ^ 0x80808080u, t1 = p1 ^ 0x80808080u;
    float f[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[i] = fmaf(__uint_as_float(__byte_perm(t0, 0x4B000000u, 0x7540 | i)), s, c);
        f[4 + i] = fmaf(__uint_as_float(__byte_perm(t1, 0x4B000000u, 0x7540 | i)), s, c);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) out[i] = as_u32(__floats2bfloat162_rn(f[2 * i], f[2 * i + 1]));
}
__device__ __forceinline__ bool byte_fast_ok(int ebyte, int w) { return ebyte == 255 || ebyte - (w - 2) <= 225; }
__device__ __forceinline__ float f32_scale(int ebyte, int w)
{
    const int e = ebyte - (w - 2);
    return ebyte == 255 ? __uint_as_float(0x7FC00000u)
                        : __uint_as_float(e > 0 ? ((uint32_t)e << 23) : (1u << (22 + e)));
}

// Row and batch strides (bytes) of a packed source and (elements) of the decoded output.
struct PackedStrides {
    int64_t mant_ld, exp_ld;          // bytes between rows of the mantissa / exponent arrays
    int64_t mant_batch, exp_batch;    // bytes between batch items
    int64_t out_batch;                // elements between batch items of the output
    int exp_row_shift;                // 1: two adjacent rows share one row of exponent bytes (two-row blocks)
};

struct QuantOut {
    uint8_t *mant;        // packed mantissas (nullable)
    uint8_t *exps;        // exponent bytes (nullable together with mant)
    __nv_bfloat16 *xhat;  // decoded values as bf16, [rows, ld_xhat] (nullable)
    int64_t ld_xhat;
    uint32_t *nonfinite;  // nullable
    int xhat_perm;        // 1: inside every group of 8 consecutive k, xhat holds k in the order
                          // 0,4,1,5,2,6,3,7 (the operand order of the W_NIBBLE_PERM product kernel)
};

template <typename InT> struct Load8;
template <> struct Load8<float> {
    static __device__ __forceinline__ void run(const float *p, float (&v)[8])
    {
        const float4 a = __ldcs(reinterpret_cast<const float4 *>(p));      // read once: evict first
        const float4 b = __ldcs(reinterpret_cast<const float4 *>(p) + 1);
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
        v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    }
};
template <> struct Load8<__nv_bfloat16> {
    static __device__ __forceinline__ void run(const __nv_bfloat16 *p, float (&v)[8])
    {
        const uint4 a = __ldcs(reinterpret_cast<const uint4 *>(p));
        const uint32_t u[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(u[i] << 16);          // bf16 -> fp32 is a 16-bit shift
            v[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u);
        }
    }
};

// Largest magnitude so far, NaN-propagating (a NaN comes out as 0x7FFFFFFF, exponent field 255).
__device__ __forceinline__ float absmax_nan(float m, float x)
{
    float d;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(m), "f"(fabsf(x)));
    return d;
}

// Eight values of one block (exponent byte `ebyte`, width w) -> their packed mantissas: one word of
// two's-complement nibbles (w <= 4, returned in p.x) or two words of int8; xh receives the decoded
// values.  Same arithmetic as
// quantize_rows_body below (add-only rounding with the block-scaled magic constant, the
// multiply-based form for blocks near the top of the range or holding Inf/NaN).
__device__ __forceinline__ uint2 encode8_full(const float (&v)[8], int ebyte, int w, float (&xh)[8])
{
    const bool nibble = w <= 4;
    const int qmax = (1 << (w - 1)) - 1;
    const uint32_t off = nibble ? 8u : 128u;
    const bool bad = ebyte == 255;
    uint32_t f[8], corr;
    if (ebyte <= 229 + w) {
        const uint32_t mb = ((uint32_t)(ebyte + 25 - w) << 23) | 0x00400000u;
        const float M = __uint_as_float(mb);
        const float lo = __uint_as_float(mb - (uint32_t)qmax), hi = __uint_as_float(mb + (uint32_t)qmax);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float t = fminf(fmaxf(v[i] + M, lo), hi);
            f[i] = __float_as_uint(t);
            xh[i] = t - M;                                   // the decoded value q * s, exactly
        }
        corr = mb - off;
    } else {
        const float qmaxf = (float)qmax, pow2_wm2 = (float)(1 << (w - 2));
        const float inv_pow2_E = pow2_from_biased(254 - (bad ? 254 : ebyte));
        const float dec_small = small_neg_pow2(w), dec_big = pow2_from_biased(bad ? 127 : ebyte);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float s = (v[i] * inv_pow2_E) * pow2_wm2;
            const float t = fminf(fmaxf(s, -qmaxf), qmaxf) + 12582912.f;
            f[i] = bad ? off : __float_as_uint(t) - 0x4B400000u + off;
            xh[i] = bad ? __uint_as_float(0x7FC00000u) : ((t - 12582912.f) * dec_small) * dec_big;
        }
        corr = 0;
    }
    uint2 p = make_uint2(0, 0);
    if (nibble) {
#pragma unroll
        for (int i = 0; i < 8; ++i) p.x += f[i] << (4 * i);
        p.x = (p.x - corr * 0x11111111u) ^ 0x88888888u;
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            p.x += f[i] << (8 * i);
            p.y += f[4 + i] << (8 * i);
        }
        p.x = (p.x - corr * 0x01010101u) ^ 0x80808080u;
        p.y = (p.y - corr * 0x01010101u) ^ 0x80808080u;
    }
    return p;
}
__device__ __forceinline__ uint2 encode8_packed(const float (&v)[8], int ebyte, int w)
{
    float unused[8];
    return encode8_full(v, ebyte, w, unused);
}

// rows x K, rows contiguous along K with leading dimension ldx.  BLOCK in {16, 32}.
//
// Work item of a warp = (row, segment of 256 elements): lane l owns the 8 elements starting at
// k = segment*256 + 8*l, so a warp reads 1 KB of fp32 contiguously.  A warp walks its items with
// a fixed stride; (row, segment) advance by the stride's quotient and remainder, so the only
// divisions are at set-up.  UNROLL items per warp and iteration have all their loads issued
// before any arithmetic (UNROLL * 32 bytes in flight per thread).
//
// Rounding without a multiply or a conversion: the block scale is s = 2^es, es = E-127-(w-2).
// M = 1.5 * 2^(23+es) has ulp s, so the adder rounds x + M to a multiple of s (nearest, ties to
// even; M's significand is even, so ties fall on even q) and the low bits of the sum's pattern
// are those of M plus q.  Clamping the sum to [M - qmax*s, M + qmax*s] is the symmetric clamp of
// q, and (sum - M) is the decoded value q*s, exactly.  The patterns of a word's 8 (4) values are
// added up with shifts; one multiply-subtract removes M's pattern from every field and leaves
// q + OFF >= 1 there (OFF = 8 / 128), one XOR restores two's complement.
// M needs a biased exponent E + 25 - w <= 254: blocks above that (|x| >= 2^102) take the
// multiply-based path below, as do blocks holding an Inf or NaN.
template <typename InT, int BLOCK, int UNROLL>
__device__ __forceinline__ void quantize_rows_body(const InT *__restrict__ x, int64_t rows, int64_t K,
                                                   int64_t ldx, int w, const QuantOut &out,
                                                   int64_t warp_id, int64_t n_warps)
{
    constexpr int LANES = BLOCK / 8;                    // lanes sharing one block
    constexpr int LANE_SHIFT = BLOCK == 16 ? 1 : 2;
    const int lane = threadIdx.x & 31;
    const int cpr = (int)(K >> 3);                      // 8-element chunks per row
    const int segs = (cpr + 31) >> 5;                   // 256-element segments per row
    const bool nibble = w <= 4;
    const bool leader = (lane & (LANES - 1)) == 0;
    const int64_t nb_row = K >> (BLOCK == 16 ? 4 : 5);
    const int64_t mant_ld = nibble ? (K >> 1) : K;

    const int64_t step = n_warps * UNROLL;
    const int64_t step_row = step / segs;
    const int step_seg = (int)(step - step_row * segs);
    int64_t row[UNROLL];
    int seg[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
        const int64_t it = warp_id + u * n_warps;
        row[u] = it / segs;
        seg[u] = (int)(it - row[u] * segs);
    }

    while (row[0] < rows) {                             // warp-uniform: items ascend with u
        float v[UNROLL][8];
        int kc[UNROLL];
        bool live[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            kc[u] = seg[u] * 32 + lane;
            live[u] = row[u] < rows && kc[u] < cpr;
            if (live[u]) {
                Load8<InT>::run(x + row[u] * ldx + (int64_t)kc[u] * 8, v[u]);
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) v[u][i] = 0.f;
            }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            float am = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) am = absmax_nan(am, v[u][i]);
            uint32_t amax = __float_as_uint(am);
#pragma unroll
            for (int d = 1; d < LANES; d <<= 1) amax = max(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, d));
            if (live[u]) {
                const int ebyte = (int)(amax >> 23);        // 255 <=> an Inf or NaN in the block
                const bool bad = ebyte == 255;
                float xh[8];                                // decoded values (when asked for)
                const uint2 pk = encode8_full(v[u], ebyte, w, xh);      // the one rounding routine of this library
                if (out.mant) {
                    if (nibble) *reinterpret_cast<uint32_t *>(out.mant + row[u] * mant_ld + (int64_t)kc[u] * 4) = pk.x;
                    else *reinterpret_cast<uint2 *>(out.mant + row[u] * mant_ld + (int64_t)kc[u] * 8) = pk;
                    if (leader) out.exps[row[u] * nb_row + (kc[u] >> LANE_SHIFT)] = (uint8_t)ebyte;
                }
                if (out.xhat) {
                    // q * 2^(E-127-(w-2)) as bf16 (exact: <= 7 significant bits)
                    uint32_t h[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        h[i] = out.xhat_perm ? as_u32(__floats2bfloat162_rn(xh[i], xh[i + 4]))
                                             : as_u32(__floats2bfloat162_rn(xh[2 * i], xh[2 * i + 1]));
                    *reinterpret_cast<uint4 *>(out.xhat + row[u] * out.ld_xhat + (int64_t)kc[u] * 8) =
                        make_uint4(h[0], h[1], h[2], h[3]);
                }
                if (bad && leader && out.nonfinite) atomicAdd(out.nonfinite, 1u);
            }
            row[u] += step_row;
            seg[u] += step_seg;
            if (seg[u] >= segs) { seg[u] -= segs; ++row[u]; }
        }
    }
}

template <typename InT, int BLOCK, int UNROLL>
__global__ void __launch_bounds__(256)
quantize_rows_kernel(const InT *__restrict__ x, int64_t rows, int64_t K, int64_t ldx, int w,
                     QuantOut out)
{
    ptx::dep_wait();
    ptx::dep_trigger();
    quantize_rows_body<InT, BLOCK, UNROLL>(x, rows, K, ldx, w, out,
                                           (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5),
                                           (int64_t)gridDim.x * (blockDim.x >> 5));
}

// Two-row blocks (the paper's (16,2) block shape, Sec. 4.1 / Fig. 2): BLOCK elements along K times
// two adjacent rows share one exponent.  Work item of a warp = (pair of rows, segment of 256
// elements); a lane owns 8 elements of each row, so the block maximum is a maximum over 16
// registers and one or two shuffles.  Same rounding arithmetic as the one-row kernel; exponent
// bytes [rows/2, K/BLOCK].  rows must be even.
template <typename InT, int BLOCK>
__device__ __forceinline__ void quantize_rows2_body(const InT *__restrict__ x, int64_t rows, int64_t K, int64_t ldx,
                                                    int w, const QuantOut &out, int64_t warp_id, int64_t n_warps)
{
    constexpr int LANES = BLOCK / 8;
    constexpr int LANE_SHIFT = BLOCK == 16 ? 1 : 2;
    const int lane = threadIdx.x & 31;
    const int64_t cpr = K >> 3, segs = (cpr + 31) >> 5, n_items = (rows >> 1) * segs;
    const bool nibble = w <= 4, leader = (lane & (LANES - 1)) == 0;
    const int64_t nb_row = K / BLOCK, mant_ld = nibble ? (K >> 1) : K;
    for (int64_t it = warp_id; it < n_items; it += n_warps) {
        const int64_t pr = it / segs, kc = (it - pr * segs) * 32 + lane;
        const bool live = kc < cpr;
        float v[2][8];
        float am = 0.f;
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            if (live) {
                Load8<InT>::run(x + (2 * pr + r) * ldx + kc * 8, v[r]);
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) v[r][i] = 0.f;
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) am = absmax_nan(am, v[r][i]);
        }
        uint32_t amax = __float_as_uint(am);
#pragma unroll
        for (int d = 1; d < LANES; d <<= 1) amax = max(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, d));
        if (!live) continue;
        const int ebyte = (int)(amax >> 23);                // 255 <=> an Inf or NaN in the block
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int64_t row = 2 * pr + r;
            float xh[8];
            const uint2 pk = encode8_full(v[r], ebyte, w, xh);
            if (out.mant) {
                if (nibble) *reinterpret_cast<uint32_t *>(out.mant + row * mant_ld + kc * 4) = pk.x;
                else *reinterpret_cast<uint2 *>(out.mant + row * mant_ld + kc * 8) = pk;
            }
            if (out.xhat) {
                uint32_t h[4];
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    h[i] = out.xhat_perm ? as_u32(__floats2bfloat162_rn(xh[i], xh[i + 4]))
                                         : as_u32(__floats2bfloat162_rn(xh[2 * i], xh[2 * i + 1]));
                *reinterpret_cast<uint4 *>(out.xhat + row * out.ld_xhat + kc * 8) = make_uint4(h[0], h[1], h[2], h[3]);
            }
        }
        if (leader) {
            if (out.mant) out.exps[pr * nb_row + (kc >> LANE_SHIFT)] = (uint8_t)ebyte;
            if (ebyte == 255 && out.nonfinite) atomicAdd(out.nonfinite, 1u);
        }
    }
}

template <typename InT, int BLOCK>
__global__ void __launch_bounds__(256)
quantize_rows2_kernel(const InT *__restrict__ x, int64_t rows, int64_t K, int64_t ldx, int w, QuantOut out)
{
    ptx::dep_wait();
    ptx::dep_trigger();
    quantize_rows2_body<InT, BLOCK>(x, rows, K, ldx, w, out, (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5),
                                    (int64_t)gridDim.x * (blockDim.x >> 5));
}

// Cast between MXInt formats (Sec. 3.2: a different mantissa width of the same format): the
// quantizer on the exactly decoded values of an MXInt tensor, without the fp32 copy in between.
// Warp item = (row, segment of 256 elements), 8 elements per lane; one-row blocks on both sides.
template <int BLOCK_OUT>
__global__ void __launch_bounds__(256)
cast_rows_kernel(const uint8_t *__restrict__ mant_in, const uint8_t *__restrict__ exp_in, int block_in, int w_in,
                 int64_t rows, int64_t K, int w_out, QuantOut out)
{
    ptx::dep_wait();
    ptx::dep_trigger();
    constexpr int LANES = BLOCK_OUT / 8;
    constexpr int LANE_SHIFT = BLOCK_OUT == 16 ? 1 : 2;
    const int lane = threadIdx.x & 31;
    const int64_t cpr = K >> 3, segs = (cpr + 31) >> 5, n_items = rows * segs;
    const int64_t n_warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const bool nib_in = w_in <= 4, nib_out = w_out <= 4, leader = (lane & (LANES - 1)) == 0;
    const int in_shift = block_in == 16 ? 1 : 2;                    // 8-element chunks per input block, as a shift
    const int64_t nb_in = K / block_in, nb_out = K / BLOCK_OUT;
    const int64_t ld_in = nib_in ? (K >> 1) : K, ld_out = nib_out ? (K >> 1) : K;
    for (int64_t it = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); it < n_items; it += n_warps) {
        const int64_t row = it / segs, kc = (it - row * segs) * 32 + lane;
        const bool live = kc < cpr;
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = 0.f;
        if (live) {
            const int eb = __ldg(exp_in + row * nb_in + (kc >> in_shift));
            int q[8];
            if (nib_in) {
                const uint32_t p = __ldg(reinterpret_cast<const uint32_t *>(mant_in + row * ld_in + kc * 4));
#pragma unroll
                for (int i = 0; i < 8; ++i) q[i] = ((int)(p << (28 - 4 * i))) >> 28;
            } else {
                const uint2 p = __ldg(reinterpret_cast<const uint2 *>(mant_in + row * ld_in + kc * 8));
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    q[i] = ((int)(p.x << (24 - 8 * i))) >> 24;
                    q[4 + i] = ((int)(p.y << (24 - 8 * i))) >> 24;
                }
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = decode_value(q[i], eb, w_in);      // exact in fp32
        }
        float am = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) am = absmax_nan(am, v[i]);
        uint32_t amax = __float_as_uint(am);
#pragma unroll
        for (int d = 1; d < LANES; d <<= 1) amax = max(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, d));
        if (!live) continue;
        const int ebyte = (int)(amax >> 23);
        const uint2 pk = encode8_packed(v, ebyte, w_out);
        if (nib_out) *reinterpret_cast<uint32_t *>(out.mant + row * ld_out + kc * 4) = pk.x;
        else *reinterpret_cast<uint2 *>(out.mant + row * ld_out + kc * 8) = pk;
        if (leader) {
            out.exps[row * nb_out + (kc >> LANE_SHIFT)] = (uint8_t)ebyte;
            if (ebyte == 255 && out.nonfinite) atomicAdd(out.nonfinite, 1u);
        }
    }
}

// Several tensors in one launch (the distinct activation tensors of a grouped decode call):
// blockIdx.y selects the tensor, blockIdx.x strides over its rows.
struct QuantJob {
    const void *x;
    int64_t rows, K, ldx;
    int w, block, dt;        // dt: 0 = fp32, 1 = bf16
    QuantOut out;
};

template <typename InT, int DT>
__global__ void __launch_bounds__(256)
quantize_multi_kernel(const QuantJob *__restrict__ jobs)
{
    ptx::dep_wait();
    ptx::dep_trigger();
    const QuantJob j = jobs[blockIdx.y];
    if (j.dt != DT) return;
    const int64_t warp_id = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t n_warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    if (j.block == 16)
        quantize_rows_body<InT, 16, 2>(static_cast<const InT *>(j.x), j.rows, j.K, j.ldx, j.w, j.out, warp_id, n_warps);
    else
        quantize_rows_body<InT, 32, 2>(static_cast<const InT *>(j.x), j.rows, j.K, j.ldx, j.w, j.out, warp_id, n_warps);
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

// Blocks along the slow axis of a row-major tensor (stride_row == 1: x[r, k] = base[k * stride_k + r],
// e.g. V of attention quantized along the token axis).  A CTA owns 32 rows r and walks k in tiles of
// 256: every warp reads 128 contiguous bytes per k (coalesced), the tile is transposed through
// shared memory, then 8 lanes cover the 256 k of one row -- 32 consecutive k each, i.e. two blocks
// of 16 or one of 32 -- so that they write 128 (nibbles) or 256 contiguous bytes per row.
// Tile element (r, k) sits at r * 264 + k + k / 32: with this padding both the transposing store
// and the per-lane reads are (nearly) free of bank conflicts.
// CTA-wide body (256 threads, every thread must call it): CTA `cta` of `n_ctas` walks the 32 x 256 tiles.
template <typename InT>
__device__ __forceinline__ void quantize_transposed_body(float *tile, const InT *__restrict__ x, int64_t rows, int64_t K,
                                                         int64_t stride_k, int block, int w, const QuantOut &out,
                                                         int cta, int n_ctas)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool nibble = w <= 4;
    const int64_t nb_row = K / block, mant_ld = nibble ? (K >> 1) : K;
    const int64_t row_tiles = (rows + 31) >> 5, k_tiles = (K + 255) >> 8;
    for (int64_t tix = cta; tix < row_tiles * k_tiles; tix += n_ctas) {
        const int64_t r0 = (tix % row_tiles) * 32, k0 = (tix / row_tiles) * 256;
        __syncthreads();                                    // the previous tile has been consumed
#pragma unroll 4
        for (int kk = warp; kk < 256; kk += 8) {
            const int64_t k = k0 + kk;
            float v = 0.f;
            if (k < K && r0 + lane < rows) v = (float)x[k * stride_k + r0 + lane];
            tile[lane * 264 + kk + (kk >> 5)] = v;
        }
        __syncthreads();
        const int r = threadIdx.x >> 3, kg = threadIdx.x & 7;       // 32 k starting at k0 + 32 * kg of row r0 + r
        const int64_t row = r0 + r, kb = k0 + 32 * kg;
        if (row < rows && kb < K) {                                  // K % block == 0 and 32 % block == 0: whole blocks
            const float *src = tile + r * 264 + kg * 33;
            float v[4][8];
            uint32_t amax[2] = {0u, 0u};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                float am = 0.f;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    v[c][i] = src[c * 8 + i];
                    am = absmax_nan(am, v[c][i]);
                }
                amax[c >> 1] = max(amax[c >> 1], __float_as_uint(am));
            }
            if (block == 32) amax[0] = amax[1] = max(amax[0], amax[1]);
            uint2 pk[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                float xh[8];
                pk[c] = encode8_full(v[c], (int)(amax[c >> 1] >> 23), w, xh);
                if (out.xhat) {                                       // the decoded values, exact in bf16
                    uint4 h;
                    h.x = as_u32(__floats2bfloat162_rn(xh[0], xh[1]));
                    h.y = as_u32(__floats2bfloat162_rn(xh[2], xh[3]));
                    h.z = as_u32(__floats2bfloat162_rn(xh[4], xh[5]));
                    h.w = as_u32(__floats2bfloat162_rn(xh[6], xh[7]));
                    *reinterpret_cast<uint4 *>(out.xhat + row * out.ld_xhat + kb + 8 * c) = h;
                }
            }
            if (!out.mant) continue;                                  // operand form only
            if (nibble)
                *reinterpret_cast<uint4 *>(out.mant + row * mant_ld + (kb >> 1)) = make_uint4(pk[0].x, pk[1].x, pk[2].x, pk[3].x);
            else {
                uint4 *dst = reinterpret_cast<uint4 *>(out.mant + row * mant_ld + kb);
                dst[0] = make_uint4(pk[0].x, pk[0].y, pk[1].x, pk[1].y);
                dst[1] = make_uint4(pk[2].x, pk[2].y, pk[3].x, pk[3].y);
            }
            const int e0 = (int)(amax[0] >> 23), e1 = (int)(amax[1] >> 23);
            if (block == 32) {
                out.exps[row * nb_row + (kb >> 5)] = (uint8_t)e0;
                if (e0 == 255 && out.nonfinite) atomicAdd(out.nonfinite, 1u);
            } else {
                out.exps[row * nb_row + (kb >> 4)] = (uint8_t)e0;
                out.exps[row * nb_row + (kb >> 4) + 1] = (uint8_t)e1;
                if (out.nonfinite) {
                    if (e0 == 255) atomicAdd(out.nonfinite, 1u);
                    if (e1 == 255) atomicAdd(out.nonfinite, 1u);
                }
            }
        }
    }
}

template <typename InT>
__global__ void __launch_bounds__(256)
quantize_transposed_kernel(const InT *__restrict__ x, int64_t rows, int64_t K, int64_t stride_k, int block, int w,
                           QuantOut out)
{
    __shared__ float tile[32 * 264];
    quantize_transposed_body<InT>(tile, x, rows, K, stride_k, block, w, out, (int)blockIdx.x, (int)gridDim.x);
}

// The three operands of the fused attention in one launch (256 threads per CTA): every warp takes its share of the
// rows of q and of k (blocks along the head dimension, written in operand form), then every CTA its share of the
// tiles of v (blocks along the tokens, written transposed).
struct AttnOperandsJob {
    const void *q, *k, *v;
    int64_t seq, hid, ldq, ldk, ldv;
    int block_qk, w_qk, block_v, w_v;
    __nv_bfloat16 *q_hat, *k_hat;      // [seq, hid]
    __nv_bfloat16 *v_hat;              // [hid, seq]
};

template <typename InT>
__global__ void __launch_bounds__(256)
attention_operands_kernel(const AttnOperandsJob j)
{
    __shared__ float tile[32 * 264];
    ptx::dep_wait();
    ptx::dep_trigger();
    const int warps = blockDim.x >> 5;
    const int64_t wid = (int64_t)blockIdx.x * warps + (threadIdx.x >> 5), nw = (int64_t)gridDim.x * warps;
    const QuantOut oq{nullptr, nullptr, j.q_hat, j.hid, nullptr, 0}, ok{nullptr, nullptr, j.k_hat, j.hid, nullptr, 0};
    if (j.block_qk == 16) {
        quantize_rows_body<InT, 16, 2>(static_cast<const InT *>(j.q), j.seq, j.hid, j.ldq, j.w_qk, oq, wid, nw);
        quantize_rows_body<InT, 16, 2>(static_cast<const InT *>(j.k), j.seq, j.hid, j.ldk, j.w_qk, ok, wid, nw);
    } else {
        quantize_rows_body<InT, 32, 2>(static_cast<const InT *>(j.q), j.seq, j.hid, j.ldq, j.w_qk, oq, wid, nw);
        quantize_rows_body<InT, 32, 2>(static_cast<const InT *>(j.k), j.seq, j.hid, j.ldk, j.w_qk, ok, wid, nw);
    }
    const QuantOut ov{nullptr, nullptr, j.v_hat, j.seq, nullptr, 0};
    quantize_transposed_body<InT>(tile, static_cast<const InT *>(j.v), j.hid, j.seq, j.ldv, j.block_v, j.w_v, ov,
                                  (int)blockIdx.x, (int)gridDim.x);
}

// (mant, exps) -> decoded values, 8 elements per thread.
template <typename OutT>
__global__ void __launch_bounds__(256)
dequantize_kernel(const uint8_t *__restrict__ mant, const uint8_t *__restrict__ exps, int64_t rows,
                  int64_t K, int block, int w, OutT *__restrict__ out, int64_t ld_out, PackedStrides ps)
{
    mant += (int64_t)blockIdx.y * ps.mant_batch;
    exps += (int64_t)blockIdx.y * ps.exp_batch;
    out += (int64_t)blockIdx.y * ps.out_batch;
    const int64_t chunks_per_row = K >> 3;
    const int exp_shift = block == 16 ? 1 : 2;          // 8-element chunks per block, as a shift
    // chunks are walked with a fixed stride: (row, chunk) advance by its quotient and remainder
    const int64_t step = (int64_t)gridDim.x * blockDim.x;
    const int64_t step_row = step / chunks_per_row, step_kc = step - step_row * chunks_per_row;
    const int64_t first = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    int64_t row = first / chunks_per_row, kc = first - row * chunks_per_row;
    for (; row < rows; row += step_row, kc += step_kc) {
        if (kc >= chunks_per_row) {
            kc -= chunks_per_row;
            if (++row >= rows) break;
        }
        const int ebyte = __ldg(exps + (row >> ps.exp_row_shift) * ps.exp_ld + (kc >> exp_shift));
        int q[8];
        if (w <= 4) {
            const uint32_t p = __ldg(reinterpret_cast<const uint32_t *>(mant + row * ps.mant_ld + kc * 4));
#pragma unroll
            for (int i = 0; i < 8; ++i) q[i] = ((int)(p << (28 - 4 * i))) >> 28;
        } else {
            const uint2 p = __ldg(reinterpret_cast<const uint2 *>(mant + row * ps.mant_ld + kc * 8));
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


// 32 consecutive elements of a row (one 16-byte word of nibbles, or two of int8) and their exponent
// byte(s) `e` (block 16: low byte = first half, next byte = second half; block 32: one byte) ->
// 32 exact bf16 values, o[j] = elements 8j .. 8j + 7.
template <bool NIBBLE>
__device__ __forceinline__ void decode32(const uint4 (&m)[NIBBLE ? 1 : 2], uint32_t e, bool b16, int w, uint32_t (&o)[4][4])
{
    const int e0 = (int)(e & 0xFF), e1 = b16 ? (int)((e >> 8) & 0xFF) : e0;
    const uint32_t w8[8] = {m[0].x, m[0].y, m[0].z, m[0].w,
                            m[NIBBLE ? 0 : 1].x, m[NIBBLE ? 0 : 1].y, m[NIBBLE ? 0 : 1].z, m[NIBBLE ? 0 : 1].w};
    if (NIBBLE) {
        if (nibble_fast_ok(e0, w) && nibble_fast_ok(e1, w)) {
            const __nv_bfloat162 m136 = as_bf162(0xC308C308u);       // -136
            const __nv_bfloat162 s0 = as_bf162(bf16x2_scale_bits(e0, w));
            const __nv_bfloat162 s1 = as_bf162(bf16x2_scale_bits(e1, w));
            const __nv_bfloat162 c0 = __hmul2(s0, m136), c1 = __hmul2(s1, m136);
            decode8_nibbles(w8[0], s0, c0, o[0]);
            decode8_nibbles(w8[1], s0, c0, o[1]);
            decode8_nibbles(w8[2], s1, c1, o[2]);
            decode8_nibbles(w8[3], s1, c1, o[3]);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                int q[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) q[i] = ((int)(w8[j] << (28 - 4 * i))) >> 28;
                decode8_safe(q, j < 2 ? e0 : e1, w, o[j]);
            }
        }
    } else {
        if (byte_fast_ok(e0, w) && byte_fast_ok(e1, w)) {
            const float s0 = f32_scale(e0, w), s1 = f32_scale(e1, w);
            const float c0 = -8388736.0f * s0, c1 = -8388736.0f * s1;   // -(2^23+128)*s, exact
            decode8_bytes(w8[0], w8[1], s0, c0, o[0]);
            decode8_bytes(w8[2], w8[3], s0, c0, o[1]);
            decode8_bytes(w8[4], w8[5], s1, c1, o[2]);
            decode8_bytes(w8[6], w8[7], s1, c1, o[3]);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                int q[8];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    q[i] = ((int)(w8[2 * j] << (24 - 8 * i))) >> 24;
                    q[4 + i] = ((int)(w8[2 * j + 1] << (24 - 8 * i))) >> 24;
                }
                decode8_safe(q, j < 2 ? e0 : e1, w, o[j]);
            }
        }
    }
}

// (mant, exps) -> bf16 operand, 32 elements per thread: one 16-byte (nibbles) or two 16-byte
// (int8) loads, four 16-byte stores.  Work item of a warp = (row, segment of 1024 elements);
// UNROLL items per warp are loaded before any is decoded so that several loads are in flight.
// Requires K % 32 == 0 (rows of the packed tensor 16-byte aligned).  Element order and values
// are those of dequantize_kernel.
template <bool NIBBLE, int UNROLL>
__device__ __forceinline__ void decode_bf16_body(const uint8_t *__restrict__ mant, const uint8_t *__restrict__ exps,
                                                 int64_t rows, int64_t K, int block, int w,
                                                 __nv_bfloat16 *__restrict__ out, int64_t ld_out,
                                                 const PackedStrides &ps, int64_t warp_id, int64_t n_warps)
{
    const int lane = threadIdx.x & 31;
    const int ipr = (int)(K >> 5);                      // 32-element items per row
    const int segs = (ipr + 31) >> 5;
    const bool b16 = block == 16;
    const int exp_shift = b16 ? 4 : 5;
    const int64_t nb_row = ps.exp_ld;
    // items are walked with a fixed stride: (row, segment) advance by its quotient and remainder
    const int64_t step = n_warps * UNROLL;
    const int64_t step_row = step / segs;
    const int step_seg = (int)(step - step_row * segs);
    int64_t cur_row[UNROLL];
    int cur_seg[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
        const int64_t it = warp_id + u * n_warps;
        cur_row[u] = it / segs;
        cur_seg[u] = (int)(it - cur_row[u] * segs);
    }
    while (cur_row[0] < rows) {                         // warp-uniform: items ascend with u
        uint4 m[UNROLL][NIBBLE ? 1 : 2];
        uint32_t e[UNROLL];
        int64_t row[UNROLL], kc[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            kc[u] = cur_seg[u] * 32 + lane;
            row[u] = (cur_row[u] < rows && kc[u] < ipr) ? cur_row[u] : -1;
            cur_row[u] += step_row;
            cur_seg[u] += step_seg;
            if (cur_seg[u] >= segs) { cur_seg[u] -= segs; ++cur_row[u]; }
            if (row[u] >= 0) {
                if (NIBBLE) {
                    m[u][0] = __ldcs(reinterpret_cast<const uint4 *>(mant + row[u] * ps.mant_ld + kc[u] * 16));
                } else {
                    const uint4 *src = reinterpret_cast<const uint4 *>(mant + row[u] * ps.mant_ld + kc[u] * 32);
                    m[u][0] = __ldcs(src);
                    m[u][NIBBLE ? 0 : 1] = __ldcs(src + 1);
                }
                const uint8_t *ep = exps + (row[u] >> ps.exp_row_shift) * nb_row + ((kc[u] * 32) >> exp_shift);
                e[u] = b16 ? (uint32_t)ep[0] | ((uint32_t)ep[1] << 8) : (uint32_t)ep[0];
            }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            if (row[u] < 0) continue;
            uint32_t o[4][4];
            decode32<NIBBLE>(m[u], e[u], b16, w, o);
            uint4 *dst = reinterpret_cast<uint4 *>(out + row[u] * ld_out + kc[u] * 32);
#pragma unroll
            for (int j = 0; j < 4; ++j) dst[j] = make_uint4(o[j][0], o[j][1], o[j][2], o[j][3]);
        }
    }
}


template <bool NIBBLE, int UNROLL>
__global__ void __launch_bounds__(256)
decode_bf16_kernel(const uint8_t *__restrict__ mant, const uint8_t *__restrict__ exps, int64_t rows,
                   int64_t K, int block, int w, __nv_bfloat16 *__restrict__ out, int64_t ld_out,
                   PackedStrides ps)
{
    ptx::dep_wait();
    ptx::dep_trigger();
    // blockIdx.y = batch item; rows of the packed source may be wider than K (a column slice)
    decode_bf16_body<NIBBLE, UNROLL>(mant + (int64_t)blockIdx.y * ps.mant_batch,
                                     exps + (int64_t)blockIdx.y * ps.exp_batch, rows, K, block, w,
                                     out + (int64_t)blockIdx.y * ps.out_batch, ld_out, ps,
                                     (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5),
                                     (int64_t)gridDim.x * (blockDim.x >> 5));
}

// Both packed operands of a product -> their bf16 operand forms in one launch: every warp takes its share of the
// rows of A, then of W (the product that follows needs both; two launches would each pay their own ramp and tail).
struct DecodePairJob {
    const uint8_t *a_mant, *a_exp, *w_mant, *w_exp;
    int64_t M, N, K;
    int block, wa, ww, a_row_shift, w_row_shift;
    __nv_bfloat16 *a_hat, *w_hat;
};

template <bool NIB_A, bool NIB_W>
__global__ void __launch_bounds__(256)
decode_pair_kernel(const DecodePairJob j)
{
    ptx::dep_wait();
    ptx::dep_trigger();
    const int warps = blockDim.x >> 5;
    const int64_t wid = (int64_t)blockIdx.x * warps + (threadIdx.x >> 5), nw = (int64_t)gridDim.x * warps;
    PackedStrides ps;
    ps.exp_ld = j.K / j.block;
    ps.mant_batch = ps.exp_batch = ps.out_batch = 0;
    ps.mant_ld = NIB_A ? j.K / 2 : j.K;
    ps.exp_row_shift = j.a_row_shift;
    decode_bf16_body<NIB_A, 2>(j.a_mant, j.a_exp, j.M, j.K, j.block, j.wa, j.a_hat, j.K, ps, wid, nw);
    ps.mant_ld = NIB_W ? j.K / 2 : j.K;
    ps.exp_row_shift = j.w_row_shift;
    decode_bf16_body<NIB_W, 2>(j.w_mant, j.w_exp, j.N, j.K, j.block, j.ww, j.w_hat, j.K, ps, wid, nw);
}

// ---- dense storage: w bits per element (Eq. 1 counts m + 1 bits per value) ---------------------
// Element k of a row sits in bits [k*w, (k+1)*w) of the row's bit stream (two's complement; stream
// bit b = bit b % 8 of byte b / 8); a row takes K*w/8 bytes.  Eight consecutive elements are exactly w
// bytes, which is a thread's unit in the three kernels below (byte loads and stores: w = 3, 5, 6 leave
// no wider alignment).

// The 8*w bits of eight elements starting at byte address p.
__device__ __forceinline__ uint64_t dense_load8(const uint8_t *p, int w)
{
    uint64_t v = 0;
    for (int i = 0; i < w; ++i) v |= (uint64_t)__ldg(p + i) << (8 * i);
    return v;
}
__device__ __forceinline__ int dense_field(uint64_t v, int i, int w)
{
    const int f = (int)((v >> (i * w)) & ((1u << w) - 1u));
    return (f << (32 - w)) >> (32 - w);                         // sign extension
}

// container (nibbles for w <= 4, int8 above) -> dense
__global__ void __launch_bounds__(256)
dense_pack_kernel(const uint8_t *__restrict__ mant, int64_t rows, int64_t K, int w, uint8_t *__restrict__ dense)
{
    ptx::dep_wait();
    ptx::dep_trigger();
    const int64_t cpr = K >> 3, total = rows * cpr;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = t / cpr, kc = t - row * cpr;
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
        uint64_t v = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) v |= (uint64_t)((uint32_t)q[i] & ((1u << w) - 1u)) << (i * w);
        uint8_t *dst = dense + row * (K * w / 8) + kc * w;
        for (int i = 0; i < w; ++i) dst[i] = (uint8_t)(v >> (8 * i));
    }
}

// dense -> container
__global__ void __launch_bounds__(256)
dense_unpack_kernel(const uint8_t *__restrict__ dense, int64_t rows, int64_t K, int w, uint8_t *__restrict__ mant)
{
    ptx::dep_wait();
    ptx::dep_trigger();
    const int64_t cpr = K >> 3, total = rows * cpr;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = t / cpr, kc = t - row * cpr;
        const uint64_t v = dense_load8(dense + row * (K * w / 8) + kc * w, w);
        if (w <= 4) {
            uint32_t p = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) p |= ((uint32_t)dense_field(v, i, w) & 0xFu) << (4 * i);
            *reinterpret_cast<uint32_t *>(mant + row * (K >> 1) + kc * 4) = p;
        } else {
            uint2 p = make_uint2(0, 0);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                p.x |= ((uint32_t)dense_field(v, i, w) & 0xFFu) << (8 * i);
                p.y |= ((uint32_t)dense_field(v, 4 + i, w) & 0xFFu) << (8 * i);
            }
            *reinterpret_cast<uint2 *>(mant + row * K + kc * 8) = p;
        }
    }
}

// dense mantissas + exponent bytes -> decoded values (fp32, or bf16: the MMA operand form), 8 per thread
template <typename OutT>
__global__ void __launch_bounds__(256)
dequantize_dense_kernel(const uint8_t *__restrict__ dense, const uint8_t *__restrict__ exps, int64_t rows, int64_t K,
                        int block, int w, int exp_row_shift, OutT *__restrict__ out, int64_t ld_out)
{
    ptx::dep_wait();
    ptx::dep_trigger();
    const int64_t cpr = K >> 3, total = rows * cpr, nb_row = K / block;
    const int exp_shift = block == 16 ? 1 : 2;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = t / cpr, kc = t - row * cpr;
        const uint64_t v = dense_load8(dense + row * (K * w / 8) + kc * w, w);
        const int ebyte = __ldg(exps + (row >> exp_row_shift) * nb_row + (kc >> exp_shift));
        float f[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) f[i] = decode_value(dense_field(v, i, w), ebyte, w);
        OutT *o = out + row * ld_out + kc * 8;
        if constexpr (sizeof(OutT) == 4) {
            reinterpret_cast<float4 *>(o)[0] = make_float4(f[0], f[1], f[2], f[3]);
            reinterpret_cast<float4 *>(o)[1] = make_float4(f[4], f[5], f[6], f[7]);
        } else {
            uint32_t h[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) h[i] = as_u32(__floats2bfloat162_rn(f[2 * i], f[2 * i + 1]));
            *reinterpret_cast<uint4 *>(o) = make_uint4(h[0], h[1], h[2], h[3]);
        }
    }
}

// Both operands of the tensor-core product in one launch: the activations are quantized straight to
// their exact bf16 operand form and the packed weights decoded to theirs.  Two HBM-bound passes share
// one launch instead of queueing behind each other.
struct PrepJob {
    const void *x;            // activations [M, K] of InT, leading dimension ldx
    int64_t M, K, ldx;
    int wa, block;
    __nv_bfloat16 *a_hat;     // [M, K]
    const uint8_t *w_mant, *w_exp;
    int64_t N;
    int ww;
    __nv_bfloat16 *w_hat;     // [N, K]
    int w_row_shift;          // 1: the weights have two-row blocks
    int a_rows2;              // 1: the activations get two-row blocks
};

template <typename InT, bool NIBBLE>
__global__ void __launch_bounds__(256)
prep_operands_kernel(const PrepJob j)
{
    ptx::dep_wait();
    ptx::dep_trigger();
    const int warps = blockDim.x >> 5;
    // every warp takes its share of BOTH sides (its quantize items, then its decode items): the two sides cost
    // differently per byte, and with CTAs dedicated to one side each the cheaper side's SM slots sat idle while
    // the other finished (SMs active 63 % of the kernel's duration)
    const int64_t wid = (int64_t)blockIdx.x * warps + (threadIdx.x >> 5), nw = (int64_t)gridDim.x * warps;
    {
        QuantOut out{nullptr, nullptr, j.a_hat, j.K, nullptr};
        if (j.a_rows2) {
            if (j.block == 16) quantize_rows2_body<InT, 16>(static_cast<const InT *>(j.x), j.M, j.K, j.ldx, j.wa, out, wid, nw);
            else quantize_rows2_body<InT, 32>(static_cast<const InT *>(j.x), j.M, j.K, j.ldx, j.wa, out, wid, nw);
        } else if (j.block == 16) quantize_rows_body<InT, 16, 2>(static_cast<const InT *>(j.x), j.M, j.K, j.ldx, j.wa, out, wid, nw);
        else quantize_rows_body<InT, 32, 2>(static_cast<const InT *>(j.x), j.M, j.K, j.ldx, j.wa, out, wid, nw);
    }
    {
        PackedStrides ps;
        ps.mant_ld = NIBBLE ? j.K / 2 : j.K;
        ps.exp_ld = j.K / j.block;
        ps.mant_batch = ps.exp_batch = ps.out_batch = 0;
        ps.exp_row_shift = j.w_row_shift;
        decode_bf16_body<NIBBLE, 2>(j.w_mant, j.w_exp, j.N, j.K, j.block, j.ww, j.w_hat, j.K, ps, wid, nw);
    }
}

}  // namespace mx
