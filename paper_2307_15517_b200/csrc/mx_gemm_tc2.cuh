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
//   warps 2..9  : epilogue of the CTA's own 128 rows (fp32, or MXInt as in the one-CTA kernel): warp w reads
//                 TMEM lanes 32 * (w % 4) .. + 31 and 128 of the 256 columns -- two warps per scheduler, so one
//                 warp's TMEM and memory latencies hide under the other's arithmetic, and the last tile's
//                 epilogue, which nothing overlaps, takes half as long
// Barriers: full[s] lives in the leader (one arrival + the bytes of both CTAs), empty[s] and
// tfull[a] in both (the MMA thread's commits are multicast to the pair), tempty[a] in the leader
// (sixteen arrivals: the eight epilogue warps of both CTAs).  No TMA load is multicast.  Every wait
// is bounded; both CTAs always reach the closing cluster barrier.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mx_gemm_tc.cuh"
#include "mx_ptx.cuh"

namespace mx {

struct Tc2Cfg {
    static constexpr int BN = 256;                        // pair tile: 256 x 256
    static constexpr int STAGES = 6;
    static constexpr uint32_t A_BYTES = TC_BM * TC_BK * 2;          // this CTA's 128 rows of A
    static constexpr uint32_t W_BYTES = (BN / 2) * TC_BK * 2;       // this CTA's 128 rows of W
    static constexpr uint32_t STAGE_BYTES = A_BYTES + W_BYTES;
    static constexpr uint32_t BAR_BYTES = 256;
    static constexpr int EPI_WARPS = 8;                   // two per TMEM lane quarter: 128 of the tile's 256 columns each
    static constexpr int THREADS = 64 + 32 * EPI_WARPS;
    static constexpr uint32_t EPI_BYTES = EPI_WARPS * 4096;         // one 32x32 fp32 store buffer per epilogue warp
    static constexpr uint32_t SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + BAR_BYTES + 1024;
    static constexpr uint32_t TMEM_COLS = 512;            // two accumulators of 256 columns
};

template <bool TAIL = false>
// At most 128 registers per thread (the block size would allow 204; the plain instantiation needs 110, the one with
// the fused tail 124): this launch follows an operand pass that fills the register file with its own CTAs, and as a
// programmatic dependent it becomes resident -- barriers, tensor memory, descriptor prefetch -- as soon as enough of
// those have left.  The smaller the footprint the earlier that is (step of four layers 0.2366 -> 0.2331 ms).
__global__ void __cluster_dims__(2, 1, 1) __maxnreg__(128)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
                const __grid_constant__ CUtensorMap tmap_y, const TcParams p)
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
            ptx::mbar_init(tempty_bar(a), 2 * Cfg::EPI_WARPS);      // the epilogue warps of both CTAs
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
    } else {
        const int quad = warp & 3;                           // TMEM lane quarter (the hardware's window for this warp)
        const int col0 = ((warp - 2) >> 2) * (BN / (Cfg::EPI_WARPS / 4));   // this warp's columns of the tile
        constexpr int COLS = BN / (Cfg::EPI_WARPS / 4);
        int it = 0;
        uint32_t epi_buf = 0;
        constexpr bool tail = TAIL;
        for (int t = pair; t < num_tiles && !timed_out; t += npairs, ++it) {
            const int acc = it & 1;
            const uint32_t acc_ph = (uint32_t)(it >> 1) & 1u;
            const int m0 = (t % p.tiles_m) * 256 + (int)rank * 128, n0 = (t / p.tiles_m) * BN;
            const int row = m0 + quad * 32 + lane;
            TailRegs ahead;
            if (tail) tail_fetch(p, row, n0 + col0, ahead);    // the first chunk's residual: in flight under the MMAs
            const bool ok = ptx::mbar_wait_bounded_cluster(tfull_bar(acc), acc_ph, abort_flag, TC_WAIT_LIMIT_NS);
            if (!__all_sync(0xFFFFFFFFu, ok)) {
                timed_out = true;
                break;
            }
            ptx::tc_fence_after_sync();
#pragma unroll 1
            for (int c0 = col0; c0 < col0 + COLS; c0 += 32) {
                if (!tail && p.frag_store) {
                    store_f32_frag(p, tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * BN + c0), m0 + quad * 32,
                                   n0 + c0, 0, lane);
                    continue;
                }
                uint32_t r[32];
                ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * BN + c0), r);
                TailRegs cur;
                if (tail) {
                    cur = ahead;                                                        // fetched a chunk ago: has arrived
                    if (c0 + 32 < col0 + COLS) tail_fetch(p, row, n0 + c0 + 32, ahead);  // in flight under this chunk
                }
                ptx::tmem_ld_wait();
                const int n = n0 + c0;
                if (tail) tail_apply(p, cur, n, r);
                if (p.yq_mant) {
                    store_mxint_chunk(p, row, n, r);
                    continue;
                }
                store_f32_chunk<1>(p, &tmap_y, r, row, m0 + quad * 32, n, 0, epi_base + (uint32_t)(warp - 2) * 4096u, epi_buf, lane);
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
