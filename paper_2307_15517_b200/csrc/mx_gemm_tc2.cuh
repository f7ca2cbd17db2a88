// Tensor-core MXInt product on CTA pairs (Sec. 3.2 MXInt dot-product operator; same arithmetic
// and operands as mx_gemm_tc.cuh: exactly decoded bf16 tiles, fp32 accumulation in tensor memory).
//
// Two CTAs on neighbouring SMs (a cluster of two) share one 256 x 256 output tile: each holds 128
// rows of A and 128 of the 256 rows of W per K step, one thread of the leader CTA issues
// tcgen05.mma.cta_group::2, and each CTA's tensor memory receives the 128 x 256 half of the tile
// that belongs to its rows.  Against the one-CTA 128 x 256 tile this cuts the bytes that pass
// through each SM's shared memory per flop by a third (32 KB instead of 48 KB per K step), which
// is what bounds that kernel, and leaves room for six stages instead of four.
//
//   warp 0      : TMA producer (one lane, in both CTAs; bytes are counted on the leader's barrier)
//   warp 1      : tensor-memory allocation (both CTAs), MMA issue (leader only)
//   warps 2..5  : epilogue of the CTA's own 128 rows (fp32, or MXInt as in the one-CTA kernel)
// Barriers: full[s] lives in the leader (one arrival + the bytes of both CTAs), empty[s] and
// tfull[a] in both (the MMA thread's commits are multicast to the pair), tempty[a] in the leader
// (eight arrivals: the four epilogue warps of both CTAs).  No TMA load is multicast.  Every wait
// is bounded; both CTAs always reach the closing cluster barrier.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mx_gemm_tc.cuh"
#include "mx_ptx.cuh"

namespace mx {

// ---- operand preparation inside the product kernel (PREP > 0) ---------------------------------------
// mx_linear has to turn fp32/bf16 activations into their quantized, exactly decoded bf16 operand and
// packed weights into theirs before the tensor cores can use them.  Both passes are HBM-bound while
// the product is tensor-bound, so with PREP extra warps per CTA they run INSIDE the product kernel,
// ahead of the tiles that need them, instead of in a launch of their own in front of it:
//   * work unit  = 256 consecutive k (one "K group" = four K steps) of 32 activation rows (quantize:
//                  block maximum, shared exponent, rounding, exact bf16) or of 128 weight rows (decode);
//                  32 warp items each, spread over the CTA's PREP warps
//   * order      = K group by K group for all activation panels and for the weight panels of the first
//                  wave of tiles, then the remaining weight panels in the order the tiles reach them;
//                  unit i belongs to CTA i % gridDim.x, so all CTAs advance through the list together
//   * hand-over  = one counter per (128-row panel, K group) in the workspace, zero at launch: every
//                  prep warp adds 1 after a release fence when its share of a unit is written; the TMA
//                  producer of a tile polls (acquire, bounded) the two counters of the K group it is
//                  about to load, then orders its TMA loads behind them with a proxy fence
// Prep warps never wait on anything, every CTA of the grid is resident (one per SM), so the consumers'
// waits always end; they are bounded like every other wait of the library.
struct FusedPrep {
    const void *x;              // activations [M, K], fp32 or bf16, leading dimension ldx
    int64_t ldx;
    int x_bf16;                 // 1: x is bf16
    int wa, ww;                 // mantissa widths of activations / weights
    int block;                  // 16 or 32, both operands
    __nv_bfloat16 *a_hat;       // [M, K] exact bf16 operand (written here)
    const uint8_t *w_mant;      // packed weights [N, K/2] (ww <= 4) or [N, K]
    const uint8_t *w_exp;       // [N, K/block]
    __nv_bfloat16 *w_hat;       // [N, K] (written here)
    uint32_t *flags;            // [(PA + PW) * G] progress counters, all zero at launch
    int PA, PW;                 // 128-row panels of A / W covered by the tile grid
    int G;                      // K groups = K / 256
    int W0;                     // weight panels the first wave of tiles needs
};
constexpr int PREP_KG = 256;    // elements per K group

__device__ __forceinline__ bool flag_wait_bounded(const uint32_t *flag, uint32_t target, volatile uint32_t *abort_flag,
                                                  uint64_t limit_ns)
{
    uint64_t t0 = 0;
    for (uint32_t it = 1;; ++it) {
        uint32_t v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
        if (v >= target) return true;
        if ((it & 0x7F) == 0) {
            if (*abort_flag) return false;
            const uint64_t now = ptx::globaltimer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns) return false;
        }
    }
}

// One decode unit: rows [r0, r0 + 128) x k [k0, k0 + 256) of the packed weights -> bf16.  A lane item
// is 32 elements (one or two 16-byte loads, four 16-byte stores); 8 lanes cover the 256 k of a row,
// so a warp item is 4 rows and the unit has 32 warp items.
template <bool NIBBLE>
__device__ __forceinline__ void decode_unit(const FusedPrep &fp, int N, int K, int r0, int k0, int pw, int n_pw, int lane)
{
    const bool b16 = fp.block == 16;
    const int64_t mant_ld = NIBBLE ? (K >> 1) : K, nb_row = K / fp.block;
    const int sub = lane >> 3, kc = lane & 7;                   // row within the warp item, 32-element chunk
#pragma unroll 2
    for (int wi = pw; wi < 32; wi += n_pw) {
        const int row = r0 + wi * 4 + sub;
        if (row < N) {
            const int k = k0 + kc * 32;
            uint4 m[NIBBLE ? 1 : 2];
            const uint4 *src = reinterpret_cast<const uint4 *>(fp.w_mant + (int64_t)row * mant_ld + (NIBBLE ? (k >> 1) : k));
            m[0] = __ldcs(src);
            if (!NIBBLE) m[NIBBLE ? 0 : 1] = __ldcs(src + 1);
            const uint8_t *ep = fp.w_exp + (int64_t)row * nb_row + k / fp.block;
            const uint32_t e = b16 ? (uint32_t)__ldg(ep) | ((uint32_t)__ldg(ep + 1) << 8) : (uint32_t)__ldg(ep);
            uint32_t o[4][4];
            decode32<NIBBLE>(m, e, b16, fp.ww, o);
            uint4 *dst = reinterpret_cast<uint4 *>(fp.w_hat + (int64_t)row * K + k);
#pragma unroll
            for (int j = 0; j < 4; ++j) dst[j] = make_uint4(o[j][0], o[j][1], o[j][2], o[j][3]);
        }
    }
}

// One quantize unit: rows [r0, r0 + rows) x k [k0, k0 + 256) of the activations -> exact bf16.
template <typename InT>
__device__ __forceinline__ void quantize_unit(const FusedPrep &fp, int K, int r0, int rows, int k0, int pw, int n_pw)
{
    QuantOut out{nullptr, nullptr, fp.a_hat + (int64_t)r0 * K + k0, K, nullptr, 0};
    const InT *x = static_cast<const InT *>(fp.x) + (int64_t)r0 * fp.ldx + k0;
    if (fp.block == 16) quantize_rows_body<InT, 16, 2>(x, rows, PREP_KG, fp.ldx, fp.wa, out, pw, n_pw);
    else quantize_rows_body<InT, 32, 2>(x, rows, PREP_KG, fp.ldx, fp.wa, out, pw, n_pw);
}

struct Tc2Cfg {
    static constexpr int BN = 256;                        // pair tile: 256 x 256
    static constexpr int STAGES = 6;
    static constexpr uint32_t A_BYTES = TC_BM * TC_BK * 2;          // this CTA's 128 rows of A
    static constexpr uint32_t W_BYTES = (BN / 2) * TC_BK * 2;       // this CTA's 128 rows of W
    static constexpr uint32_t STAGE_BYTES = A_BYTES + W_BYTES;
    static constexpr uint32_t BAR_BYTES = 256;
    static constexpr uint32_t EPI_BYTES = 4 * 2 * 4096;
    static constexpr uint32_t SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + BAR_BYTES + 1024;
    static constexpr uint32_t TMEM_COLS = 512;            // two accumulators of 256 columns
};

template <int PREP>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(TC_THREADS + 32 * PREP, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
                const __grid_constant__ CUtensorMap tmap_y, const TcParams p, const FusedPrep fp)
{
    using Cfg = Tc2Cfg;
    constexpr int STAGES = Cfg::STAGES, BN = Cfg::BN;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));

    const uint32_t epi_base = smem_base + STAGES * Cfg::STAGE_BYTES;
    const uint32_t bar_base = epi_base + Cfg::EPI_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem_gen + STAGES * Cfg::STAGE_BYTES + Cfg::EPI_BYTES + 8 * (2 * STAGES + 4));
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();         // 0: leader
    const bool leader = rank == 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(full_bar(s), 1);
            ptx::mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(tfull_bar(a), 1);
            ptx::mbar_init(tempty_bar(a), 8);              // four epilogue warps of each CTA
        }
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_a);
        ptx::prefetch_tensormap(&tmap_w);
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(ptx::smem_u32(tmem_slot), Cfg::TMEM_COLS);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();                                  // the peer's barriers exist before anyone signals them
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    ptx::dep_wait();
    if (threadIdx.x == 0) ptx::dep_trigger();

    const int num_tiles = p.tiles_m * p.tiles_n;          // pair tiles
    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    const int kblocks = (p.K + TC_BK - 1) / TC_BK;
    bool timed_out = false;

    if (warp == 0) {
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            for (int t = pair; t < num_tiles && !timed_out; t += npairs) {
                const int m0 = (t % p.tiles_m) * 256 + (int)rank * 128;
                const int n0 = (t / p.tiles_m) * BN + (int)rank * (BN / 2);
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (PREP > 0 && (kb & 3) == 0) {
                        // this CTA's 128 rows of A and of W in K group kb / 4: written by prep warps somewhere
                        // in the grid; their release/our acquire orders the data, the proxy fence orders the
                        // TMA loads (async proxy) behind it
                        const uint32_t *fa_ = fp.flags + (m0 >> 7) * fp.G + (kb >> 2);
                        const uint32_t *fw_ = fp.flags + (fp.PA + (n0 >> 7)) * fp.G + (kb >> 2);
                        if (!flag_wait_bounded(fa_, 4u * PREP, abort_flag, TC_WAIT_LIMIT_NS) ||
                            !flag_wait_bounded(fw_, (uint32_t)PREP, abort_flag, TC_WAIT_LIMIT_NS)) {
                            timed_out = true;
                            break;
                        }
                        asm volatile("fence.proxy.async.global;" ::: "memory");
                    }
                    if (!ptx::mbar_wait_bounded_cluster(empty_bar(s), ph ^ 1u, abort_flag, TC_WAIT_LIMIT_NS)) {
                        timed_out = true;
                        break;
                    }
                    if (leader) ptx::mbar_arrive_expect_tx(full_bar(s), 2 * Cfg::STAGE_BYTES);
                    const uint32_t leader_full = ptx::map_to_cta(full_bar(s), 0);
                    const uint32_t sa = smem_base + s * Cfg::STAGE_BYTES;
                    ptx::tma_load_2d_pair(sa, &tmap_a, kb * TC_BK, m0, leader_full);
                    ptx::tma_load_2d_pair(sa + Cfg::A_BYTES, &tmap_w, kb * TC_BK, n0, leader_full);
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0 && leader) {
            constexpr uint32_t idesc = ptx::idesc_bf16_f32(256, BN);
            int s = 0;
            uint32_t ph = 0;
            int it = 0;
            for (int t = pair; t < num_tiles && !timed_out; t += npairs, ++it) {
                const int acc = it & 1;
                const uint32_t acc_ph = (uint32_t)(it >> 1) & 1u;
                if (!ptx::mbar_wait_bounded_cluster(tempty_bar(acc), acc_ph ^ 1u, abort_flag, TC_WAIT_LIMIT_NS)) {
                    timed_out = true;
                    break;
                }
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!ptx::mbar_wait_bounded_cluster(full_bar(s), ph, abort_flag, TC_WAIT_LIMIT_NS)) {
                        timed_out = true;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    const uint32_t sa = smem_base + s * Cfg::STAGE_BYTES;
                    const uint32_t sw = sa + Cfg::A_BYTES;
#pragma unroll
                    for (int j = 0; j < TC_BK / 16; ++j) {
                        ptx::mma_bf16_ss_pair(d_tmem, ptx::smem_desc_k_sw128(sa, j * 32),
                                              ptx::smem_desc_k_sw128(sw, j * 32), idesc, (kb | j) != 0 ? 1u : 0u);
                    }
                    ptx::mma_commit_pair(empty_bar(s), 3);          // both CTAs may refill the stage
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (timed_out) break;
                ptx::mma_commit_pair(tfull_bar(acc), 3);            // both halves of the accumulator are complete
            }
        }
        __syncwarp();
    } else if (PREP > 0 && warp >= TC_THREADS / 32) {
        // ---- operand preparation (see FusedPrep): never waits ----
        const int pw = warp - TC_THREADS / 32;
        const int c1 = fp.PA * 4 + fp.W0;                    // units per K group in the first part of the list
        const int n1 = fp.G * c1;
        const int total = n1 + (fp.PW - fp.W0) * fp.G;
        for (int i = blockIdx.x; i < total; i += gridDim.x) {
            int g, panel, sub = 0;
            bool is_a = false;
            if (i < n1) {
                g = i / c1;
                const int u = i - g * c1;
                if (u < fp.PA * 4) { is_a = true; panel = u >> 2; sub = u & 3; }
                else panel = u - fp.PA * 4;
            } else {
                const int j = i - n1;
                panel = fp.W0 + j / fp.G;
                g = j - (j / fp.G) * fp.G;
            }
            const int k0 = g * PREP_KG;
            if (is_a) {
                const int r0 = panel * 128 + sub * 32;
                const int rows = min(32, p.M - r0);
                if (rows > 0) {
                    if (fp.x_bf16) quantize_unit<__nv_bfloat16>(fp, p.K, r0, rows, k0, pw, PREP);
                    else quantize_unit<float>(fp, p.K, r0, rows, k0, pw, PREP);
                }
            } else {
                if (fp.ww <= 4) decode_unit<true>(fp, p.N, p.K, panel * 128, k0, pw, PREP, lane);
                else decode_unit<false>(fp, p.N, p.K, panel * 128, k0, pw, PREP, lane);
            }
            __syncwarp();
            if (lane == 0) {
                __threadfence();                                // release: the warp's stores before the count
                atomicAdd(fp.flags + (is_a ? panel : fp.PA + panel) * fp.G + g, 1u);
            }
        }
    } else {
        const int quad = warp & 3;
        int it = 0;
        uint32_t epi_buf = 0;
        for (int t = pair; t < num_tiles && !timed_out; t += npairs, ++it) {
            const int acc = it & 1;
            const uint32_t acc_ph = (uint32_t)(it >> 1) & 1u;
            const int m0 = (t % p.tiles_m) * 256 + (int)rank * 128, n0 = (t / p.tiles_m) * BN;
            const bool ok = ptx::mbar_wait_bounded_cluster(tfull_bar(acc), acc_ph, abort_flag, TC_WAIT_LIMIT_NS);
            if (!__all_sync(0xFFFFFFFFu, ok)) {
                timed_out = true;
                break;
            }
            ptx::tc_fence_after_sync();
            const int row = m0 + quad * 32 + lane;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t r[32];
                ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * BN + c0), r);
                ptx::tmem_ld_wait();
                const int n = n0 + c0;
                if (p.yq_mant) {
                    store_mxint_chunk(p, row, n, r);
                    continue;
                }
                store_f32_chunk(p, &tmap_y, r, row, m0 + quad * 32, n, 0, epi_base + (uint32_t)(warp - 2) * 8192u, epi_buf, lane);
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(ptx::map_to_cta(tempty_bar(acc), 0));
        }
        if (p.tma_store && lane == 0) ptx::bulk_wait_group<0>();
    }

    if (timed_out) {
        *abort_flag = 1;
        atomicOr(p.status, STATUS_TIMEOUT_BIT);
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 100000ull) __nanosleep(1000);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();          // the peer no longer reads this CTA's shared memory or signals its barriers
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem_base, Cfg::TMEM_COLS);
    }
}

}  // namespace mx
