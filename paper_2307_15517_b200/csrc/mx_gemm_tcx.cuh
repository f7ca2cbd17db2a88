// Tensor-core MXInt product with two-level accumulation (Sec. 3.2 MXInt dot-product operator: the
// paper fixes the integer block sums and the one shared scale per block, not the width of the
// accumulator across blocks).
//
// The tensor pipe adds the 16 products of an MMA step and the running accumulator after aligning
// all 17 addends to the largest and cutting the rest off (no rounding).  With block scales that
// differ by many binades inside one row, a large running sum therefore eats the low bits of every
// later small block, once per step, for the whole reduction.  Here the pipe only ever sums ONE
// K step of 64 elements (four MMA steps, the first overwriting the accumulator): a chunk's loss is
// at most 3 * 16 cut-offs of one ulp of the chunk's own largest term, i.e. < 48 * 2^-23 * S_chunk,
// and the chunks are then added by the CUDA cores in fp32 registers with round-to-nearest, in
// ascending K order.  Summed over a row: |dY| < 48 * 2^-23 * S (= 5.7e-6 * S) from the pipe plus the
// ordinary rounding of K/64 fp32 additions, whatever the exponent spread and whatever K.
//
// Kernel: persistent, one CTA per SM, 128 x 128 tile, K step 64, four TMA stages, FOUR chunk
// accumulators of 128 columns in tensor memory (all 512 columns) so the MMA thread runs up to four
// chunks ahead of the drain.
//   warp 0      : TMA producer (one lane)
//   warp 1      : tensor-memory allocation, MMA issue (one lane)
//   warps 2..9  : drain: warp w reads TMEM lanes 32 * (w % 4) .. + 31 (the hardware's lane window of a
//                 warp), columns 64 * ((w - 2) / 4) .. + 63, of every chunk and adds them to 64 fp32
//                 registers per lane; after the tile's last chunk it writes its 32 x 64 piece of Y
// Costs against the single-accumulator kernels: the 128 x 128 tile moves twice the shared-memory
// bytes per flop of the 256-wide tiles, and every K step pays a TMEM read and 64 additions per lane.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mx_gemm_tc.cuh"
#include "mx_ptx.cuh"

namespace mx {

struct TcxCfg {
    static constexpr int BN = 128;
    static constexpr int STAGES = 4;
    static constexpr int ACCS = 4;                                   // chunk accumulators in tensor memory
    static constexpr int DRAIN_WARPS = 8;
    static constexpr int THREADS = 64 + 32 * DRAIN_WARPS;            // 320
    static constexpr uint32_t A_BYTES = TC_BM * TC_BK * 2;
    static constexpr uint32_t W_BYTES = BN * TC_BK * 2;
    static constexpr uint32_t STAGE_BYTES = A_BYTES + W_BYTES;       // 32 KB
    static constexpr uint32_t EPI_BYTES = DRAIN_WARPS * 2 * 4096;    // two 32x32 fp32 store buffers per drain warp
    static constexpr uint32_t BAR_BYTES = 256;
    static constexpr uint32_t SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + BAR_BYTES + 1024;
    static constexpr uint32_t TMEM_COLS = ACCS * BN;                 // 512
};

__global__ void __launch_bounds__(TcxCfg::THREADS, 1)
gemm_tcx_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
                const __grid_constant__ CUtensorMap tmap_y, const TcParams p)
{
    using Cfg = TcxCfg;
    constexpr int STAGES = Cfg::STAGES, BN = Cfg::BN, ACCS = Cfg::ACCS;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));

    const uint32_t epi_base = smem_base + STAGES * Cfg::STAGE_BYTES;
    const uint32_t bar_base = epi_base + Cfg::EPI_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + ACCS + a); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem_gen + STAGES * Cfg::STAGE_BYTES + Cfg::EPI_BYTES +
                                                       8 * (2 * STAGES + 2 * ACCS));
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(full_bar(s), 1);
            ptx::mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < ACCS; ++a) {
            ptx::mbar_init(tfull_bar(a), 1);
            ptx::mbar_init(tempty_bar(a), Cfg::DRAIN_WARPS);
        }
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_a);
        ptx::prefetch_tensormap(&tmap_w);
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

    const int num_tiles = p.tiles_m * p.tiles_n;
    const int kblocks = (p.K + TC_BK - 1) / TC_BK;           // one chunk per K step
    bool timed_out = false;

    if (warp == 0) {
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            for (int t = blockIdx.x; t < num_tiles && !timed_out; t += gridDim.x) {
                const int m0 = (t % p.tiles_m) * TC_BM, n0 = (t / p.tiles_m) * BN;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!ptx::mbar_wait_bounded(empty_bar(s), ph ^ 1u, abort_flag, TC_WAIT_LIMIT_NS)) {
                        timed_out = true;
                        break;
                    }
                    ptx::mbar_arrive_expect_tx(full_bar(s), Cfg::STAGE_BYTES);
                    const uint32_t sa = smem_base + s * Cfg::STAGE_BYTES;
                    ptx::tma_load_2d(sa, &tmap_a, kb * TC_BK, m0, full_bar(s));
                    ptx::tma_load_2d(sa + Cfg::A_BYTES, &tmap_w, kb * TC_BK, n0, full_bar(s));
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::idesc_bf16_f32(TC_BM, BN);
            int s = 0, a = 0;
            uint32_t ph = 0, aph = 0;
            for (int t = blockIdx.x; t < num_tiles && !timed_out; t += gridDim.x) {
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!ptx::mbar_wait_bounded(tempty_bar(a), aph ^ 1u, abort_flag, TC_WAIT_LIMIT_NS) ||
                        !ptx::mbar_wait_bounded(full_bar(s), ph, abort_flag, TC_WAIT_LIMIT_NS)) {
                        timed_out = true;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    const uint32_t d_tmem = tmem_base + (uint32_t)(a * BN);
                    const uint32_t sa = smem_base + s * Cfg::STAGE_BYTES;
                    const uint32_t sw = sa + Cfg::A_BYTES;
#pragma unroll
                    for (int j = 0; j < TC_BK / 16; ++j)       // the chunk starts from zero: j == 0 overwrites
                        ptx::mma_bf16_ss(d_tmem, ptx::smem_desc_k_sw128(sa, j * 32), ptx::smem_desc_k_sw128(sw, j * 32),
                                         idesc, j != 0 ? 1u : 0u);
                    ptx::mma_commit(empty_bar(s));             // stage free once these MMAs retire
                    ptx::mma_commit(tfull_bar(a));             // ... and the chunk's sum is complete
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                    if (++a == ACCS) { a = 0; aph ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else {
        const int quad = warp & 3;                             // TMEM lanes this warp may read
        const int half = (warp - 2) >> 2;                      // which 64 of the 128 columns
        int a = 0;
        uint32_t aph = 0, epi_buf = 0;
        for (int t = blockIdx.x; t < num_tiles && !timed_out; t += gridDim.x) {
            const int m0 = (t % p.tiles_m) * TC_BM, n0 = (t / p.tiles_m) * BN;
            float acc[64];
#pragma unroll
            for (int v = 0; v < 64; ++v) acc[v] = 0.f;
            for (int kb = 0; kb < kblocks; ++kb) {
                const bool ok = ptx::mbar_wait_bounded(tfull_bar(a), aph, abort_flag, TC_WAIT_LIMIT_NS);
                if (!__all_sync(0xFFFFFFFFu, ok)) {
                    timed_out = true;
                    break;
                }
                ptx::tc_fence_after_sync();
                const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(a * BN + half * 64);
                uint32_t r0[32], r1[32];
                ptx::tmem_ld_32x32(taddr, r0);
                ptx::tmem_ld_32x32(taddr + 32, r1);
                ptx::tmem_ld_wait();
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(tempty_bar(a));    // the values are in registers: the accumulator is free
#pragma unroll
                for (int v = 0; v < 32; ++v) {
                    acc[v] += __uint_as_float(r0[v]);              // ascending chunks, round to nearest
                    acc[32 + v] += __uint_as_float(r1[v]);
                }
                if (++a == ACCS) { a = 0; aph ^= 1u; }
            }
            if (timed_out) break;
            const int row = m0 + quad * 32 + lane;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t r[32];
#pragma unroll
                for (int v = 0; v < 32; ++v) r[v] = __float_as_uint(acc[32 * c + v]);
                store_f32_chunk(p, &tmap_y, r, row, m0 + quad * 32, n0 + half * 64 + 32 * c, 0,
                                epi_base + (uint32_t)(warp - 2) * 8192u, epi_buf, lane);
            }
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
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
    }
}

}  // namespace mx
