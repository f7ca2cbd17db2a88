// Fused MX attention for head dimensions 128 and 64 (Fig. 1(d): the block's two attention matmuls --
// tensors "A" = Q K^T and "B" = P V of Fig. 1(a)/(b) -- are MXInt operators, softmax stays in floating
// point): scores, causal mask, softmax, quantization of the probabilities and the context product in ONE
// kernel, so neither the fp32 scores (heads x seq x seq) nor the probabilities ever reach HBM.
//
// What is computed is exactly the unfused sequence of this library -- S = Q K^T on exactly decoded
// operands (blocks along the head dimension), p = expf(scale * s - m) / l over the unmasked keys of a
// row, P quantized to MXInt in blocks of 16 or 32 along the keys with the quantizer's rounding, O = P V
// with V quantized along the tokens -- up to the fp32 rounding of the row sum: m and l come from a first
// sweep over the key tiles (running maximum, running sum rescaled when the maximum moves), the second
// sweep recomputes each score tile, normalises with the FINAL m and l and quantizes, so a probability
// sees the same block exponent as in the unfused path.  Fully masked key tiles are skipped in both sweeps.
//
// One work item = (head, 128 queries); items are ordered long rows first and dealt to the persistent CTAs
// in alternating direction (round k: CTA b takes item k*G + b, then k*G + G-1-b, ...), which evens out the
// causal rows' unequal lengths.
//   warp 0      : TMA producer: Q tile once per item, K tiles (both sweeps), V^T tiles (second sweep)
//   warp 1      : tensor-memory allocation, MMA issue: S_j = Q K_j^T (8 steps of K = 16) into one of two
//                 score accumulators; O += P_j V_j (8 steps) into the context accumulator
//   warps 2..   : ROW_WARPS row warps: warp w reads TMEM lanes 32 * (w % 4) .. + 31 (its hardware window), i.e.
//                 32 query rows, and a slice of 128 / (ROW_WARPS / 4) key columns of every tile (the warps of a
//                 row combine their maxima and sums once, between the sweeps, through shared memory).
//                 Sweep 1: statistics; sweep 2: scores -> probabilities -> MXInt codes -> exact bf16 -> the
//                 swizzled P operand tile in shared memory; at the end the context tile out of tensor
//                 memory into global memory.  exp is ex2.approx on arguments pre-scaled by log2(e); the division
//                 by the row sum is a subtraction of its log2 inside that argument
// Every 128 x 128 bf16 tile is stored as two halves of 128 rows x 128 bytes (64 columns) with the
// 128-byte swizzle.  All waits are bounded.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mx_gemm_tc.cuh"
#include "mx_ptx.cuh"
#include "mx_quantize.cuh"

namespace mx {

// D_ = head dimension, 128 or 64.  Q and K tiles are [128 rows, D_] (D_/64 halves of 128 rows x 128 bytes), the V^T
// tile is [D_ rows, 128 keys] (two halves of D_ rows x 128 bytes), the P tile always [128, 128].
template <int D_> struct AttnCfgT {
    static constexpr int D = D_, BQ = 128, BKEY = 128;
    static constexpr uint32_t TILE_BYTES = 128 * D_ * 2;             // Q, K and V^T tiles: 32 KB or 16 KB
    static constexpr uint32_t HALF_BYTES = 128 * 128;                // 128 rows x 128 bytes: a half of Q, K or P
    static constexpr uint32_t V_HALF_BYTES = D_ * 128;               // D_ rows x 128 bytes: a half of V^T
    static constexpr uint32_t P_BYTES = 128 * 128 * 2;
    static constexpr int KST = 2, VST = 2;                           // K and V^T stage rings
    static constexpr int ROW_WARPS = 16;                             // 4 per TMEM lane quarter: 32 key columns each
    static constexpr int COLS_PER_WARP = 128 / (ROW_WARPS / 4);
    static constexpr int THREADS = 64 + 32 * ROW_WARPS;
    static constexpr uint32_t STATS_BYTES = 2 * (ROW_WARPS / 4) * 128 * 8;   // (maximum, sum) per row and column slice, two items deep
    static constexpr uint32_t SMEM_BYTES = (1 + KST + VST) * TILE_BYTES + P_BYTES + 512 + STATS_BYTES + 1024;    // Q, K ring, V ring, P
    static constexpr uint32_t TMEM_COLS = 512;                       // S0, S1 (128 columns each), O (D_ columns) at 0, 128, 256
};
using AttnCfg = AttnCfgT<128>;

struct AttnParams {
    float *ctx;               // [seq, ldc] fp32; head h writes columns h*D .. h*D+D-1
    int64_t ldc;
    int seq, heads;
    float scale;
    int causal;
    int p_bits, p_block;      // MXInt format of the probabilities (blocks along the keys)
    uint8_t *p_mant;          // nullable: the quantized probabilities [heads*seq, seq/2 or seq] (checks only)
    uint8_t *p_exp;           // nullable: [heads*seq, seq/p_block]
    uint32_t *status;
};

// D[tmem] (+)= A[smem tile] * B[smem tile]^T over K = 64 * HALVES (halves of four steps of 16); a_half / b_half
// are the byte distances between the halves of the two tiles.
template <int HALVES>
__device__ __forceinline__ void attn_mma(uint32_t d_tmem, uint32_t a_tile, uint32_t a_half, uint32_t b_tile, uint32_t b_half,
                                         uint32_t idesc, bool accumulate)
{
#pragma unroll
    for (int hh = 0; hh < HALVES; ++hh)
#pragma unroll
        for (int j = 0; j < 4; ++j)
            ptx::mma_bf16_ss(d_tmem, ptx::smem_desc_k_sw128(a_tile + hh * a_half, j * 32),
                             ptx::smem_desc_k_sw128(b_tile + hh * b_half, j * 32), idesc,
                             (accumulate || hh || j) ? 1u : 0u);
}

// Item of CTA b in round k of G CTAs: the direction alternates between rounds.
__device__ __forceinline__ int attn_item(uint32_t k, int b, int G) { return (int)k * G + ((k & 1u) ? G - 1 - b : b); }

// tmap_q, tmap_k: bf16 [seq, heads*D], box 64 x 128.  tmap_v: bf16 [heads*D, seq] (V transposed), box 64 x D.
__device__ __forceinline__ float exp2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float log2_approx(float x)
{
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int D_>
__global__ void __launch_bounds__(AttnCfgT<D_>::THREADS, 1)
attention_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                 const __grid_constant__ CUtensorMap tmap_v, const AttnParams p)
{
    using Cfg = AttnCfgT<D_>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    const uint32_t q_tile = smem_base;
    const uint32_t k_tiles = q_tile + Cfg::TILE_BYTES;
    const uint32_t v_tiles = k_tiles + Cfg::KST * Cfg::TILE_BYTES;
    const uint32_t p_tile = v_tiles + Cfg::VST * Cfg::TILE_BYTES;
    const uint32_t bar_base = p_tile + Cfg::P_BYTES;
    // barriers: 0 q_full, 1 q_empty, 2..3 k_full, 4..5 k_empty, 6..7 v_full, 8..9 v_empty, 10..11 s_full,
    //           12..13 s_empty, 14 p_full, 15 p_empty, 16 o_full, 17 o_empty, 18 row statistics written
    auto bar = [&](int i) { return bar_base + 8u * i; };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem_gen + (bar_base - smem_base) + 8 * 19);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    float2 *stats = reinterpret_cast<float2 *>(smem_gen + (bar_base - smem_base) + 512);    // [slice][row]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int i = 0; i < 19; ++i) {
            const bool by_rows = i == 12 || i == 13 || i == 14 || i == 17 || i == 18;      // arrived on by every row warp
            ptx::mbar_init(bar(i), by_rows ? Cfg::ROW_WARPS : 1);
        }
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_q);
        ptx::prefetch_tensormap(&tmap_k);
        ptx::prefetch_tensormap(&tmap_v);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(tmem_slot), Cfg::TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    ptx::dep_wait();
    if (threadIdx.x == 0) ptx::dep_trigger();

    const int q_tiles_n = (p.seq + Cfg::BQ - 1) / Cfg::BQ;      // the last tile may be ragged: loads beyond seq read zeros
    const int items = q_tiles_n * p.heads;
    bool timed_out = false;
    auto wait = [&](int i, uint32_t parity) { return ptx::mbar_wait_bounded(bar(i), parity, abort_flag, TC_WAIT_LIMIT_NS); };

    if (warp == 0) {
        if (lane == 0) {
            uint32_t n_item = 0, n_k = 0, n_v = 0;                    // uses so far of the Q tile and the two rings
            for (int w = attn_item(0, blockIdx.x, gridDim.x); w < items && !timed_out; ++n_item, w = attn_item(n_item, blockIdx.x, gridDim.x)) {
                const int qt = q_tiles_n - 1 - w / p.heads, h = w % p.heads;
                const int T = p.causal ? qt + 1 : q_tiles_n;
                if (!wait(1, (n_item & 1u) ^ 1u)) { timed_out = true; break; }
                ptx::mbar_arrive_expect_tx(bar(0), Cfg::TILE_BYTES);
                ptx::tma_load_2d(q_tile, &tmap_q, h * Cfg::D, qt * Cfg::BQ, bar(0));
                if (Cfg::D == 128) ptx::tma_load_2d(q_tile + Cfg::HALF_BYTES, &tmap_q, h * Cfg::D + 64, qt * Cfg::BQ, bar(0));
                for (int sweep = 0; sweep < 2 && !timed_out; ++sweep)
                    for (int j = 0; j < T; ++j) {
                        const uint32_t ks = n_k % Cfg::KST;
                        if (!wait(4 + ks, ((n_k / Cfg::KST) & 1u) ^ 1u)) { timed_out = true; break; }
                        ptx::mbar_arrive_expect_tx(bar(2 + ks), Cfg::TILE_BYTES);
                        const uint32_t kt = k_tiles + ks * Cfg::TILE_BYTES;
                        ptx::tma_load_2d(kt, &tmap_k, h * Cfg::D, j * Cfg::BKEY, bar(2 + ks));
                        if (Cfg::D == 128) ptx::tma_load_2d(kt + Cfg::HALF_BYTES, &tmap_k, h * Cfg::D + 64, j * Cfg::BKEY, bar(2 + ks));
                        ++n_k;
                        if (sweep == 1) {
                            const uint32_t vs = n_v % Cfg::VST;
                            if (!wait(8 + vs, ((n_v / Cfg::VST) & 1u) ^ 1u)) { timed_out = true; break; }
                            ptx::mbar_arrive_expect_tx(bar(6 + vs), Cfg::TILE_BYTES);
                            const uint32_t vt = v_tiles + vs * Cfg::TILE_BYTES;
                            ptx::tma_load_2d(vt, &tmap_v, j * Cfg::BKEY, h * Cfg::D, bar(6 + vs));
                            ptx::tma_load_2d(vt + Cfg::V_HALF_BYTES, &tmap_v, j * Cfg::BKEY + 64, h * Cfg::D, bar(6 + vs));
                            ++n_v;
                        }
                    }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::idesc_bf16_f32(128, 128), idesc_o = ptx::idesc_bf16_f32(128, Cfg::D);
            const uint32_t s_tmem[2] = {tmem_base, tmem_base + 128u}, o_tmem = tmem_base + 256u;
            uint32_t n_item = 0, n_k = 0, n_v = 0, n_s = 0, n_p = 0;
            // S_j = Q K_j^T into score accumulator n_s % 2
            auto issue_scores = [&]() -> bool {
                const uint32_t ks = n_k % Cfg::KST, si = n_s & 1u;
                if (!wait(2 + ks, (n_k / Cfg::KST) & 1u) || !wait(12 + si, ((n_s >> 1) & 1u) ^ 1u)) return false;
                ptx::tc_fence_after_sync();
                attn_mma<Cfg::D / 64>(s_tmem[si], q_tile, Cfg::HALF_BYTES, k_tiles + ks * Cfg::TILE_BYTES, Cfg::HALF_BYTES, idesc, false);
                ptx::mma_commit(bar(4 + ks));               // K stage free
                ptx::mma_commit(bar(10 + si));              // scores complete
                ++n_k;
                ++n_s;
                return true;
            };
            for (int w = attn_item(0, blockIdx.x, gridDim.x); w < items && !timed_out; ++n_item, w = attn_item(n_item, blockIdx.x, gridDim.x)) {
                const int qt = q_tiles_n - 1 - w / p.heads;
                const int T = p.causal ? qt + 1 : q_tiles_n;
                if (!wait(0, n_item & 1u)) { timed_out = true; break; }
                for (int j = 0; j < T && !timed_out; ++j)                       // sweep 1: statistics
                    if (!issue_scores()) timed_out = true;
                if (timed_out) break;
                if (!wait(17, (n_item & 1u) ^ 1u)) { timed_out = true; break; }  // previous item's context has been read
                if (!issue_scores()) { timed_out = true; break; }                // sweep 2: S_0
                for (int j = 0; j < T; ++j) {
                    if (j + 1 < T) {
                        if (!issue_scores()) { timed_out = true; break; }       // S_{j+1} runs under the softmax of S_j
                    } else {
                        ptx::mma_commit(bar(1));                                // every product that reads Q has been issued
                    }
                    const uint32_t vs = n_v % Cfg::VST;
                    if (!wait(14, n_p & 1u) || !wait(6 + vs, (n_v / Cfg::VST) & 1u)) { timed_out = true; break; }
                    ptx::tc_fence_after_sync();
                    attn_mma<2>(o_tmem, p_tile, Cfg::HALF_BYTES, v_tiles + vs * Cfg::TILE_BYTES, Cfg::V_HALF_BYTES, idesc_o, j > 0);
                    ptx::mma_commit(bar(8 + vs));            // V stage free
                    ptx::mma_commit(bar(15));                // P tile free
                    ++n_v;
                    ++n_p;
                }
                if (timed_out) break;
                ptx::mma_commit(bar(16));                    // context complete
            }
        }
        __syncwarp();
    } else {
        const int quad = warp & 3;
        const int slice = (warp - 2) >> 2;                   // which COLS_PER_WARP key columns of every tile
        constexpr int CHUNKS = Cfg::COLS_PER_WARP / 32;
        const int r = quad * 32 + lane;                      // this thread's query row inside the tile
        const uint32_t lane_tmem = tmem_base + ((uint32_t)(quad * 32) << 16);
        const uint32_t p_row = p_tile + (uint32_t)((r >> 3) * 1024 + (r & 7) * 128);
        const bool nibble = p.p_bits <= 4;
        const float scale2 = p.scale * 1.4426950408889634f;  // scores in units of log2: exp(x) = 2^(x log2 e)
        uint32_t n_item = 0, n_s = 0, n_p = 0;
        for (int w = attn_item(0, blockIdx.x, gridDim.x); w < items && !timed_out; ++n_item, w = attn_item(n_item, blockIdx.x, gridDim.x)) {
            const int qt = q_tiles_n - 1 - w / p.heads, h = w % p.heads;
            const int T = p.causal ? qt + 1 : q_tiles_n;
            const int qrow = qt * Cfg::BQ + r;
            float m = -INFINITY, l = 0.f;
            for (int sweep = 0; sweep < 2 && !timed_out; ++sweep) {
                if (sweep == 1) {
                    // combine the statistics of the row's column slices: one exchange per item.  The buffer
                    // alternates between items, so a warp that runs ahead never overwrites values still being read
                    float2 *st_buf = stats + (n_item & 1u) * (Cfg::ROW_WARPS / 4) * 128;
                    st_buf[slice * 128 + r] = make_float2(m, l);
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(bar(18));
                    if (!__all_sync(0xFFFFFFFFu, wait(18, n_item & 1u))) { timed_out = true; break; }
                    float mm = -INFINITY;
#pragma unroll
                    for (int q = 0; q < Cfg::ROW_WARPS / 4; ++q) mm = fmaxf(mm, st_buf[q * 128 + r].x);
                    float ll = 0.f;
#pragma unroll
                    for (int q = 0; q < Cfg::ROW_WARPS / 4; ++q) {
                        const float2 st = st_buf[q * 128 + r];
                        ll += st.x == -INFINITY ? 0.f : st.y * exp2_approx(st.x - mm);
                    }
                    m = mm;
                    l = ll;
                }
                // sweep 2 normalises inside the exponent: e / l = 2^(x - (m + log2 l))
                const float m_norm = sweep ? m + log2_approx(l) : 0.f;
                for (int j = 0; j < T; ++j) {
                    const uint32_t si = n_s & 1u;
                    if (!__all_sync(0xFFFFFFFFu, wait(10 + si, (n_s >> 1) & 1u))) { timed_out = true; break; }
                    ptx::tc_fence_after_sync();
                    // keys 0..limit of this tile take part: the causal bound and the end of the sequence
                    const int limit = min(p.causal ? qrow - j * Cfg::BKEY : Cfg::BKEY, p.seq - 1 - j * Cfg::BKEY);
#pragma unroll 1
                    for (int cc = 0; cc < CHUNKS; ++cc) {
                        const int c = slice * CHUNKS + cc;
                        uint32_t raw[32];
                        ptx::tmem_ld_32x32(lane_tmem + si * 128u + (uint32_t)(c * 32), raw);
                        ptx::tmem_ld_wait();
                        // raw scores; masked keys (only the diagonal tile of a causal row has any) become -inf
                        float v[32];
                        if (c * 32 + 31 <= limit) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(raw[i]);
                        } else {
#pragma unroll
                            for (int i = 0; i < 32; ++i) v[i] = (c * 32 + i <= limit) ? __uint_as_float(raw[i]) : -INFINITY;
                        }
                        // exp(scale * s - max) = 2^(s * scale2 - m) with m kept in log2 units: one FMA and one ex2
                        if (sweep == 0) {
                            float cm = -INFINITY;
#pragma unroll
                            for (int i = 0; i < 32; ++i) cm = fmaxf(cm, v[i]);
                            cm *= scale2;                               // scale2 > 0: the maximum commutes with the scaling
                            if (cm > m) {                               // the running sum follows the maximum
                                l *= exp2_approx(m - cm);
                                m = cm;
                            }
                            if (m != -INFINITY) {
                                float s = 0.f;
#pragma unroll
                                for (int i = 0; i < 32; ++i) s += exp2_approx(fmaf(v[i], scale2, -m));      // 2^-inf = 0 for masked keys
                                l += s;
                            }
                        } else {
                            uint32_t amax[2] = {0u, 0u};
#pragma unroll
                            for (int i = 0; i < 32; ++i) {
                                v[i] = exp2_approx(fmaf(v[i], scale2, -m_norm));
                                amax[i >> 4] = max(amax[i >> 4], __float_as_uint(v[i]));     // v >= 0: bits order like values
                            }
                            if (p.p_block == 32) amax[0] = amax[1] = max(amax[0], amax[1]);
                            // the previous P tile must have been consumed before the first store of this one
                            if (cc == 0 && !__all_sync(0xFFFFFFFFu, wait(15, (n_p & 1u) ^ 1u))) { timed_out = true; break; }
                            const int64_t prow = (int64_t)h * p.seq + qrow;
                            const int key0 = j * Cfg::BKEY + c * 32;
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                const int ebyte = (int)(amax[u >> 1] >> 23);
                                float v8[8], xh[8];
#pragma unroll
                                for (int i = 0; i < 8; ++i) v8[i] = v[8 * u + i];
                                const uint2 pk = encode8_full(v8, ebyte, p.p_bits, xh);
                                uint32_t hw[4];
#pragma unroll
                                for (int i = 0; i < 4; ++i) hw[i] = as_u32(__floats2bfloat162_rn(xh[2 * i], xh[2 * i + 1]));
                                const uint32_t dst = p_row + (uint32_t)(c >> 1) * Cfg::HALF_BYTES +
                                                     (uint32_t)((((c & 1) * 4 + u) ^ (r & 7)) << 4);
                                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(hw[0]), "r"(hw[1]),
                                             "r"(hw[2]), "r"(hw[3])
                                             : "memory");
                                if (p.p_mant && qrow < p.seq && key0 + 8 * u < p.seq) {
                                    if (nibble) *reinterpret_cast<uint32_t *>(p.p_mant + prow * (p.seq >> 1) + ((key0 + 8 * u) >> 1)) = pk.x;
                                    else *reinterpret_cast<uint2 *>(p.p_mant + prow * p.seq + key0 + 8 * u) = pk;
                                    if (p.p_block == 16 ? (u & 1) == 0 : u == 0)
                                        p.p_exp[prow * (p.seq / p.p_block) + (key0 + 8 * u) / p.p_block] = (uint8_t)ebyte;
                                }
                            }
                        }
                    }
                    if (timed_out) break;
                    ptx::tc_fence_before_sync();
                    if (sweep == 1) ptx::fence_proxy_async_smem();      // the P tile's stores -> visible to the MMA
                    __syncwarp();
                    if (lane == 0) {
                        ptx::mbar_arrive(bar(12 + si));                  // score accumulator free
                        if (sweep == 1) ptx::mbar_arrive(bar(14));       // this warp's piece of P is in place
                    }
                    ++n_s;
                    if (sweep == 1) ++n_p;
                }
            }
            if (timed_out) break;
            // ---- context tile: tensor memory -> global ----
            const bool ok = wait(16, n_item & 1u);
            if (!__all_sync(0xFFFFFFFFu, ok)) { timed_out = true; break; }
            ptx::tc_fence_after_sync();
            float *orow = p.ctx + (int64_t)qrow * p.ldc + h * Cfg::D;
#pragma unroll 1
            for (int cc = 0; cc < CHUNKS; ++cc) {
                const int c = slice * CHUNKS + cc;
                if (c * 32 >= Cfg::D) break;                 // head dimension 64: the first two column slices write it
                uint32_t raw[32];
                ptx::tmem_ld_32x32(lane_tmem + 256u + (uint32_t)(c * 32), raw);
                ptx::tmem_ld_wait();
                if (qrow >= p.seq) continue;                 // rows of a ragged last query tile
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    reinterpret_cast<float4 *>(orow + c * 32)[i] =
                        make_float4(__uint_as_float(raw[4 * i]), __uint_as_float(raw[4 * i + 1]), __uint_as_float(raw[4 * i + 2]),
                                    __uint_as_float(raw[4 * i + 3]));
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar(17));
        }
    }

    if (timed_out) {
        *abort_flag = 1;
        atomicOr(p.status, STATUS_TIMEOUT_BIT);
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 100000ull) __nanosleep(1000);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
    }
}

}  // namespace mx
