// Tensor-core MXInt product that follows the operator of Sec. 3.2 to the letter: exact integer sums
// inside each block, one shared scale per block, and the blocks added in fp32 in ascending order.
//
// The tensor pipe adds the 16 products of an MMA step and the running accumulator after aligning all
// addends to the largest and cutting the rest off (no rounding).  With block scales that differ by
// many binades inside one row, a large running sum therefore eats the low bits of every later small
// block.  Here the pipe only ever sums ONE block (one MMA step for blocks of 16, two for blocks of
// 32, the first overwriting the accumulator): all its addends are integers (< 2^14) times the same
// power of two and their sum stays below 2^19 times it, so nothing is cut off and the block term
// q-sum * 2^(Ea+Ew-(wa-2)-(ww-2)) arrives in tensor memory exactly.  The CUDA cores then add the block
// terms in fp32 registers with round-to-nearest, in ascending block order: bit for bit the
// sequential fp32 accumulation of the definition (as long as no block term leaves the fp32 normal
// range), and within (K/B) roundings of the exactly summed result whatever the exponent spread.
//
// Kernel: persistent, one CTA per SM, 128 x 128 tile, K step 64 per TMA stage, four stages, FOUR
// block accumulators of 128 columns in tensor memory (all 512 columns) so the MMA thread runs up
// to four blocks ahead of the drain.
//   warp 0      : TMA producer (one lane)
//   warp 1      : tensor-memory allocation, MMA issue (one lane)
//   warps 2..9  : drain: warp w reads TMEM lanes 32 * (w % 4) .. + 31 (the hardware's lane window of a
//                 warp), columns 64 * ((w - 2) / 4) .. + 63, of every block term and adds them to 64
//                 fp32 registers per lane (packed pairs); after the tile's last block it writes its
//                 32 x 64 piece of Y
// Costs against the single-accumulator kernels: the 128 x 128 tile moves twice the shared-memory
// bytes per flop of the 256-wide tiles, and every block pays a TMEM read and 64 additions per lane.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mx_gemm_tc.cuh"
#include "mx_ptx.cuh"

namespace mx {

// (lo, hi) pair of fp32 sums += (a, b); each half rounds to nearest like a scalar add.
__device__ __forceinline__ uint64_t add2_rn(uint64_t acc, uint32_t a, uint32_t b)
{
    uint64_t d;
    asm("{\n\t.reg .b64 t;\n\tmov.b64 t, {%2, %3};\n\tadd.rn.f32x2 %0, %1, t;\n\t}" : "=l"(d) : "l"(acc), "r"(a), "r"(b));
    return d;
}

struct TcxCfg {
    static constexpr int BN = 128;
    static constexpr int STAGES = 4;
    static constexpr int ACCS = 4;                                   // block accumulators in tensor memory
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
    const int kblocks = (p.K + TC_BK - 1) / TC_BK;           // TMA stages per tile
    const int steps_blk = p.block / 16;                      // MMA steps per block: 1 or 2
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
                for (int kb = 0; kb < kblocks && !timed_out; ++kb) {
                    if (!ptx::mbar_wait_bounded(full_bar(s), ph, abort_flag, TC_WAIT_LIMIT_NS)) {
                        timed_out = true;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    const uint32_t sa = smem_base + s * Cfg::STAGE_BYTES;
                    const uint32_t sw = sa + Cfg::A_BYTES;
                    const int steps = min(TC_BK, p.K - kb * TC_BK) / 16;      // K % block == 0: whole blocks
                    for (int j = 0; j < steps; ++j) {
                        const bool first = (j % steps_blk) == 0, last = ((j + 1) % steps_blk) == 0;
                        if (first) {
                            if (!ptx::mbar_wait_bounded(tempty_bar(a), aph ^ 1u, abort_flag, TC_WAIT_LIMIT_NS)) {
                                timed_out = true;
                                break;
                            }
                            ptx::tc_fence_after_sync();
                        }
                        ptx::mma_bf16_ss(tmem_base + (uint32_t)(a * BN), ptx::smem_desc_k_sw128(sa, j * 32),
                                         ptx::smem_desc_k_sw128(sw, j * 32), idesc, first ? 0u : 1u);   // a block starts from zero
                        if (last) {
                            ptx::mma_commit(tfull_bar(a));             // the block's sum is complete
                            if (++a == ACCS) { a = 0; aph ^= 1u; }
                        }
                    }
                    ptx::mma_commit(empty_bar(s));                 // stage free once these MMAs retire
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
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
            uint64_t acc[32];                                   // 64 fp32 sums as packed pairs
#pragma unroll
            for (int v = 0; v < 32; ++v) acc[v] = 0ull;
            const int nblocks = p.K / p.block;
            for (int b = 0; b < nblocks; ++b) {
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
                for (int v = 0; v < 16; ++v) {                     // ascending blocks, one rounding per block and output
                    acc[v] = add2_rn(acc[v], r0[2 * v], r0[2 * v + 1]);
                    acc[16 + v] = add2_rn(acc[16 + v], r1[2 * v], r1[2 * v + 1]);
                }
                if (++a == ACCS) { a = 0; aph ^= 1u; }
            }
            if (timed_out) break;
            const int row = m0 + quad * 32 + lane;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t r[32];
#pragma unroll
                for (int v = 0; v < 16; ++v) {
                    r[2 * v] = (uint32_t)acc[16 * c + v];
                    r[2 * v + 1] = (uint32_t)(acc[16 * c + v] >> 32);
                }
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
