// Decode-shaped MXInt product: a handful of tokens (T <= 16) against weight matrices that are
// streamed from HBM exactly once (Sec. 3.2 MXInt dot-product operator; the paper motivates MX
// formats by the memory footprint of the parameters, Sec. 1 / Sec. 6).
//
// HBM-bound, so the layout of the loads and the number of bytes in flight decide, not the math.
// The math is the literal operator: integer multiply-adds over one block of 32, one shared
// scale per block, blocks added in ascending order in fp32 -- bit-identical to the CUDA-core
// kernel when a row's blocks are not split over warps.
//
//  * weights  : packed 4-bit mantissas [N, K/2] + exponent bytes [N, K/32] (block 32).  TMA
//               variant: every warp owns a two-stage ring of shared-memory stages, each filled by
//               three tiled TMA loads (16 rows x 256 mantissa bytes as two 128-byte swizzled boxes,
//               16 rows x 16 exponent bytes).  Register variant: coalesced 32-bit loads, four blocks
//               and their four exponent bytes per step, two register sets alternating.
//  * tokens   : already quantized (int8 or nibble container); each CTA stages them once per
//               layer into shared memory in the operand order of the integer MMA below, together
//               with their float block scales.
//  * per block: a two's-complement nibble moved into the HIGH half of a byte is the signed byte
//               16*q, so one shift/AND pair turns a packed word into the A operand of
//               mma.sync.m16n8k32 (s8 x s8 -> s32) with no sign extension; the accumulator starts
//               at 0x4B400000, so the result register IS the float 1.5*2^23 + 16*P (P = exact
//               integer block sum, |16 P| < 2^22), and two packed FMAs per output pair apply the
//               weight scale (removing the 1.5*2^23) and the token scale (which carries the 1/16).
//
// A warp owns 16 weight rows.  With split > 1 the K range of a row tile is cut into `split`
// contiguous pieces handled by consecutive warps of one CTA and summed in piece order through
// shared memory (deterministic, but no longer the ascending single chain).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

#include "mx_ptx.cuh"
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
    // two-row blocks (the paper's (16,2) shape): rows 2i and 2i+1 share row i of the exponent array.  Weights in
    // this form take the register variant of the kernel (the staged exponent boxes assume one row per weight row).
    int w_rows2, a_rows2;    // 0 or 1: shift applied to the row index of w_exp / a_exp
};

struct StreamParams {
    const StreamLayer *layers;   // device memory
    int n_layers;
    int total_tiles;
    int split;                   // 1, 2, 4 or 8
    int max_nb;                  // largest K/32 over the layers (sizes the shared-memory arrays)
    uint32_t *status;            // device status word (bit 0: a bounded wait expired)
    const CUtensorMap *tmaps;    // BULK: two maps per layer (device memory): [2l] over the packed
                                 // mantissas [N, K/2] bytes, box 128 x 16 rows, 128-byte swizzle;
                                 // [2l+1] over the exponent bytes [N, K/32], box 16 x 16 rows
};

// Geometry of the two variants.
//   register variant (BULK = false): 8 warps, each lane prefetches four blocks' words with 32-bit
//     loads; works for any K % 128 == 0.
//   TMA variant (BULK = true): 16 warps; every warp owns a ring of STAGES shared-memory stages.
//     A stage is 16 rows x 16 blocks: two tiled TMA loads of 16 rows x 128 mantissa bytes each
//     (issued back to back so that DRAM sees 256 contiguous bytes per row -- 128-byte pieces
//     alone reach only ~70 % of the HBM rate; 128-byte swizzle so that the 8 rows one fragment
//     load touches fall into different banks) plus one load of 16 rows x 16 exponent bytes.
//     Global data never passes through the load/store data pipe.  Needs K % 512 == 0 and
//     16-byte aligned exponent arrays.
template <int NT, bool BULK> struct StreamCfg {
    static constexpr int WARPS = BULK ? 16 : 8;
    static constexpr int THREADS = WARPS * 32;
    static constexpr int STAGES = 2;
    static constexpr int CH = BULK ? 16 : 4;                       // blocks of 32 per step and row
    static constexpr int MANT_BYTES = 16 * CH * 16;                // 4096: two boxes of 16 rows x 128 bytes
    static constexpr int STAGE_BYTES = MANT_BYTES + 16 * CH;       // + 16 rows x 16 exponent bytes
    static constexpr uint32_t STAGE_TX = STAGE_BYTES;
    static constexpr int TP = NT * 8;                              // padded token count
    static constexpr size_t tokens_bytes(int max_nb) { return (size_t)max_nb * TP * (32 + 4); }
    static constexpr size_t red_bytes() { return (size_t)WARPS * NT * 4 * 32 * 4; }
    static constexpr size_t smem_bytes(int max_nb)
    {
        // the split-K exchange buffer aliases the weight stages in the TMA variant
        return tokens_bytes(max_nb) +
               (BULK ? 1024 /* stage alignment */ + (size_t)WARPS * STAGES * STAGE_BYTES +
                           (size_t)WARPS * STAGES * 8 + 16
                     : red_bytes());
    }
};
constexpr uint64_t STREAM_WAIT_LIMIT_NS = 400ull * 1000 * 1000;
constexpr int STREAM_MAGIC_INT = 0x4B400000;        // bit pattern of 1.5 * 2^23
constexpr float STREAM_MAGIC = 12582912.0f;

// 1-D bulk copy global -> shared (no tensor map, no multicast); 16-byte aligned, size % 16 == 0.
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst_smem, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :
                 : "r"(dst_smem), "l"((uint64_t)src), "r"(bytes), "r"(bar)
                 : "memory");
}

__device__ __forceinline__ void mma_s8s8_m16n8k32(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                                  uint32_t a3, uint32_t b0, uint32_t b1, const int (&c)[4])
{
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%10,%11,%12,%13};"
        : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(c[0]), "r"(c[1]), "r"(c[2]), "r"(c[3]));
}

// Pairs of fp32 values in one 64-bit register and the sm_100 packed-pair arithmetic on them
// (each half rounds exactly like the scalar instruction).
typedef uint64_t f32x2_t;
__device__ __forceinline__ f32x2_t pack2(float lo, float hi)
{
    f32x2_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ f32x2_t pack2u(uint32_t lo, uint32_t hi)
{
    f32x2_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2_t v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2_t ffma2(f32x2_t a, f32x2_t b, f32x2_t c)
{
    f32x2_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ f32x2_t fmul2(f32x2_t a, f32x2_t b)
{
    f32x2_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// NT = number of 8-token column tiles (1: T <= 8, 2: T <= 16).
template <int NT, bool BULK>
__global__ void __launch_bounds__(StreamCfg<NT, BULK>::THREADS, 1)
gemv_stream_kernel(const StreamParams p)
{
    using Cfg = StreamCfg<NT, BULK>;
    constexpr int TP = Cfg::TP, WARPS = Cfg::WARPS, STAGES = Cfg::STAGES, CH = Cfg::CH;
    extern __shared__ __align__(16) uint8_t smem[];
    uint2 *sB = reinterpret_cast<uint2 *>(smem);                 // [nb][TP][4]: (even-k word, odd-k word)
    // [nb][TP] token block scales; they also carry the weights' binary point 2^-(ww-2) and the 1/16
    // of the shifted nibbles, so the weight scale below is the plain 2^(Ew-127)
    float *sCS = reinterpret_cast<float *>(smem + (size_t)p.max_nb * TP * 32);
    // BULK: [WARPS][STAGES][4096] swizzled mantissa stages (1024-byte aligned), then
    // [WARPS][STAGES][256] exponent stages; the split-K exchange buffer [WARPS][NT][4][32] reuses them
    uint8_t *sStage = reinterpret_cast<uint8_t *>(sCS + (size_t)p.max_nb * TP);
    if (BULK) sStage += (1024u - (ptx::smem_u32(sStage) & 1023u)) & 1023u;
    uint8_t *sExpStage = sStage + WARPS * STAGES * Cfg::MANT_BYTES;
    float *sRed = reinterpret_cast<float *>(sStage);
    uint8_t *sBar = sStage + (BULK ? WARPS * STAGES * Cfg::STAGE_BYTES : 0);     // [WARPS][STAGES] mbarriers
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(sBar + WARPS * STAGES * 8);
    uint32_t phase_bits = 0;                  // parity per stage barrier of this warp
    bool timed_out = false;
    if (BULK) {
        if (threadIdx.x == 0) {
            for (int i = 0; i < WARPS * STAGES; ++i) ptx::mbar_init(ptx::smem_u32(sBar) + 8 * i, 1);
            *abort_flag = 0;
            ptx::fence_mbar_init();
        }
        __syncthreads();
    }

    ptx::dep_wait();                          // the quantized tokens come from the previous launch
    if (threadIdx.x == 0) ptx::dep_trigger();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int S = p.split, TPR = WARPS / S;                      // row tiles per round of the CTA
    int swz[8];                               // this lane's byte offset of 16-byte chunk c in a swizzled box
#pragma unroll
    for (int c = 0; c < 8; ++c) swz[c] = g * 128 + ((c ^ g) << 4) + t * 4;

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
        for (int i = threadIdx.x; i < nb * TP * 4; i += Cfg::THREADS) {
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
            if (tq == 0) {
                const int eb = tok < L.T ? (int)__ldg(L.a_exp + (int64_t)(tok >> L.a_rows2) * nb + b) : 0;
                // 2^(Ea-127-(wa-2)) * 2^-(ww-2) * 2^-4, every factor an exact power of two
                sCS[b * TP + tok] = f32_scale(eb, L.a_bits) * small_neg_pow2(L.w_bits) * 0.0625f;
            }
        }
        __syncthreads();

        const int64_t w_ld = L.K >> 1;
        for (int base = tile_lo; base < l_end; base += TPR) {
            const int tile = base + warp / S, s = warp % S;
            const bool active = tile < l_end;
            f32x2_t accA[NT], accB[NT];        // rows g / g + 8, tokens (2t, 2t + 1) of each column tile
#pragma unroll
            for (int n = 0; n < NT; ++n) accA[n] = accB[n] = pack2(0.f, 0.f);
            const int r0 = (tile - L.tile_begin) * 16;
            if (active) {
                const int rowA = min(r0 + g, L.N - 1), rowB = min(r0 + g + 8, L.N - 1);
                const uint8_t *mA = L.w_mant + (int64_t)rowA * w_ld + t * 4;
                const uint8_t *mB = L.w_mant + (int64_t)rowB * w_ld + t * 4;
                const uint8_t *eA = L.w_exp + (int64_t)(rowA >> L.w_rows2) * nb;
                const uint8_t *eB = L.w_exp + (int64_t)(rowB >> L.w_rows2) * nb;
                const int b_lo = (nb / S) * s, b_hi = b_lo + nb / S;       // nb % (4*S) == 0
                struct Regs { uint32_t a[4], b[4], ea, eb; };
                // any exponent byte >= 226: 1.5*2^23 * 2^(E-127) is not finite, take two steps there
                auto near_top = [](uint32_t v) {
                    return ((v & 0x80808080u) & ((v & 0x7F7F7F7Fu) + 0x1E1E1E1Eu)) != 0u;
                };
                auto compute_g = [&](int b, const Regs &r, auto top_c) {
                    constexpr bool TOP = decltype(top_c)::value;
                    const f32x2_t neg_magic = pack2(-STREAM_MAGIC, -STREAM_MAGIC);
                    const int seed[4] = {STREAM_MAGIC_INT, STREAM_MAGIC_INT, STREAM_MAGIC_INT, STREAM_MAGIC_INT};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        // weight scale 2^(E-127): exponent byte moved into the float's exponent field
                        // (byte 0 -> the subnormal 2^-127, byte 255 -> Inf, which turns the block into NaN)
                        const uint32_t fa = j == 3 ? (r.ea >> 1) : (r.ea << (23 - 8 * j));
                        const uint32_t fb = j == 3 ? (r.eb >> 1) : (r.eb << (23 - 8 * j));
                        const uint32_t ba = max(fa & 0x7F800000u, 0x00400000u), bb = max(fb & 0x7F800000u, 0x00400000u);
                        const f32x2_t swA = pack2u(ba, ba), swB = pack2u(bb, bb);
                        const f32x2_t mwA = fmul2(swA, neg_magic), mwB = fmul2(swB, neg_magic);
                        // even-k nibbles shifted up, odd-k nibbles already in the high halves: bytes 16*q
                        const uint32_t a0 = (r.a[j] << 4) & 0xF0F0F0F0u, a2 = r.a[j] & 0xF0F0F0F0u;
                        const uint32_t a1 = (r.b[j] << 4) & 0xF0F0F0F0u, a3 = r.b[j] & 0xF0F0F0F0u;
                        const int blk = b + j;
#pragma unroll
                        for (int n = 0; n < NT; ++n) {
                            const uint2 bf = sB[(blk * TP + n * 8 + g) * 4 + t];
                            const f32x2_t sa = *reinterpret_cast<const f32x2_t *>(sCS + blk * TP + n * 8 + 2 * t);
                            int d[4];
                            mma_s8s8_m16n8k32(d, a0, a1, a2, a3, bf.x, bf.y, seed);
                            f32x2_t pA, pB;                       // P * weight scale (rows g, g + 8), exact
                            if (!TOP) {
                                pA = ffma2(pack2u((uint32_t)d[0], (uint32_t)d[1]), swA, mwA);
                                pB = ffma2(pack2u((uint32_t)d[2], (uint32_t)d[3]), swB, mwB);
                            } else {
                                // 1.5*2^23 * scale is not finite up here: subtract first; + 0 * scale keeps
                                // finite results and turns an Inf scale into NaN
                                const float wa_ = __uint_as_float(ba), wb_ = __uint_as_float(bb);
                                pA = pack2(fmaf(0.f, wa_, (__int_as_float(d[0]) - STREAM_MAGIC) * wa_),
                                           fmaf(0.f, wa_, (__int_as_float(d[1]) - STREAM_MAGIC) * wa_));
                                pB = pack2(fmaf(0.f, wb_, (__int_as_float(d[2]) - STREAM_MAGIC) * wb_),
                                           fmaf(0.f, wb_, (__int_as_float(d[3]) - STREAM_MAGIC) * wb_));
                            }
                            accA[n] = ffma2(pA, sa, accA[n]);     // one rounding per block, ascending blocks
                            accB[n] = ffma2(pB, sa, accB[n]);
                        }
                    }
                };
                // The two-step form is needed only when an exponent byte is >= 226.  The decision is taken
                // for the whole warp: the MMA inside is warp-collective and must never run divergent.
                auto compute = [&](int b, const Regs &r) {
                    if (__any_sync(0xFFFFFFFFu, near_top(r.ea | r.eb))) compute_g(b, r, std::true_type{});
                    else compute_g(b, r, std::false_type{});
                };
                if (!BULK) {
                    auto fetch = [&](int b, Regs &r) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            r.a[j] = __ldcs(reinterpret_cast<const uint32_t *>(mA + (b + j) * 16));
                            r.b[j] = __ldcs(reinterpret_cast<const uint32_t *>(mB + (b + j) * 16));
                        }
                        r.ea = __ldcs(reinterpret_cast<const uint32_t *>(eA + b));
                        r.eb = __ldcs(reinterpret_cast<const uint32_t *>(eB + b));
                    };
                    // two register sets alternate, so the prefetched words are never copied
                    Regs ra, rb;
                    fetch(b_lo, ra);
                    for (int b = b_lo; b < b_hi; b += 8) {
                        const bool second = b + 4 < b_hi;
                        if (second) fetch(b + 4, rb);
                        compute(b, ra);
                        if (b + 8 < b_hi) fetch(b + 8, ra);
                        if (second) compute(b + 4, rb);
                    }
                } else {
                    // one lane fills a stage with three tiled TMA loads: mantissa columns [x, x+128) and
                    // [x+128, x+256) of the 16 rows, and their 16 exponent bytes
                    uint8_t *my_stage = sStage + warp * STAGES * Cfg::MANT_BYTES;
                    uint8_t *my_exps = sExpStage + warp * STAGES * (16 * CH);
                    const uint32_t my_bar = ptx::smem_u32(sBar) + 8 * warp * STAGES;
                    const CUtensorMap *tm_m = p.tmaps + 2 * li, *tm_e = tm_m + 1;
                    const int nblk = b_hi - b_lo;                       // multiple of 16
                    auto issue = [&](int step, int st) {              // step: CH-block chunk index from b_lo
                        // after an expired wait (this warp's or, through the flag, another's) nothing new
                        // is put in flight: the CTA is about to return
                        if (lane == 0 && !timed_out && *abort_flag == 0) {
                            const uint32_t bar = my_bar + 8 * st;
                            const uint32_t dst = ptx::smem_u32(my_stage + st * Cfg::MANT_BYTES);
                            const int b = b_lo + step * CH;
                            ptx::mbar_arrive_expect_tx(bar, Cfg::STAGE_TX);
                            ptx::tma_load_2d(dst, tm_m, b * 16, r0, bar);                 // rows >= N read as zero
                            ptx::tma_load_2d(dst + 2048, tm_m, b * 16 + 128, r0, bar);
                            ptx::tma_load_2d(ptx::smem_u32(my_exps + st * (16 * CH)), tm_e, b, r0, bar);
                        }
                    };
                    const int nsteps = nblk / CH;
                    ptx::fence_proxy_async_smem();                      // earlier generic reads/writes of the stages
                    __syncwarp();
                    for (int i = 0; i < STAGES && i < nsteps; ++i) issue(i, i);
                    int st = 0;
                    for (int step = 0; step < nsteps && !timed_out; ++step) {
                        const bool ok = ptx::mbar_wait_bounded(my_bar + 8 * st, (phase_bits >> st) & 1u, abort_flag,
                                                               STREAM_WAIT_LIMIT_NS);
                        if (!__all_sync(0xFFFFFFFFu, ok)) {
                            timed_out = true;
                            *abort_flag = 1;                          // the other warps stop issuing as well
                            break;
                        }
                        phase_bits ^= 1u << st;
                        const uint8_t *sm = my_stage + st * Cfg::MANT_BYTES;
                        const uint8_t *se = my_exps + st * (16 * CH);
#pragma unroll
                        for (int q = 0; q < CH / 4; ++q) {
                            Regs r;
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                // box (c >> 3); inside it the 16-byte chunk c & 7 of row r sits at
                                // chunk (c & 7) ^ (r & 7); rows g and g + 8 share r & 7
                                const int c = q * 4 + j;
                                const int off = (c >> 3) * 2048 + swz[c & 7];
                                r.a[j] = *reinterpret_cast<const uint32_t *>(sm + off);
                                r.b[j] = *reinterpret_cast<const uint32_t *>(sm + off + 8 * 128);
                            }
                            r.ea = *reinterpret_cast<const uint32_t *>(se + g * 16 + q * 4);
                            r.eb = *reinterpret_cast<const uint32_t *>(se + (g + 8) * 16 + q * 4);
                            compute(b_lo + step * CH + q * 4, r);
                        }
                        __syncwarp();                                 // every lane is done reading the stage
                        if (step + STAGES < nsteps) {
                            ptx::fence_proxy_async_smem();
                            issue(step + STAGES, st);
                        }
                        if (++st == STAGES) st = 0;
                    }
                }
            }
            float acc[NT][4];
#pragma unroll
            for (int n = 0; n < NT; ++n) {
                unpack2(accA[n], acc[n][0], acc[n][1]);
                unpack2(accB[n], acc[n][2], acc[n][3]);
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
                __syncthreads();          // the exchange buffer shares memory with the weight stages
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
        if (BULK && __syncthreads_or(timed_out ? 1 : 0)) break;     // a bounded wait expired: give up
    }
    if (BULK && timed_out) {
        *abort_flag = 1;
        atomicOr(p.status, 1u);
        // copies already in flight get time to land before the CTA's shared memory is released
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 100000ull) __nanosleep(1000);
    }
    if (BULK) __syncthreads();                // no warp leaves while another may still be waiting out its copies
}

}  // namespace mx
