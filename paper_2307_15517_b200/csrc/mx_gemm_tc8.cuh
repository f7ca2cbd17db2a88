// MXInt product on the hardware's block-scaled tensor-core path (Sec. 3.2: the MXInt dot-product
// operator applies the shared exponent once per block -- tcgen05.mma.kind::mxf8f6f4.block_scale is
// that operator in silicon: 8-bit elements, one E8M0 power-of-two scale per 32 elements along K).
//
// Which MXInt tensors it represents exactly: blocks of 32 along K and mantissas of at most 5 bits on
// both operands.  An element q * 2^(E-(w-2)) is split as
//   element = q * 2^-(w-2)   as E4M3 (|q| <= 15 has at most 4 significant bits, 2^-(w-2) >= 2^-3: exact)
//   scale   = 2^E            as E8M0 = the MXInt exponent byte itself (byte 255 is E8M0's NaN: a block
//                            that held Inf/NaN poisons its outputs, as everywhere else)
// so nothing is rounded before the multiply; products are exact, the 32 products of a block are summed
// and scaled by 2^(Ea+Ew) by the tensor pipe, blocks accumulate in fp32 in tensor memory.
//
// Operand preparation (`pack_e4m3_kernel`): packed MXInt -> one E4M3 byte per element, rows of K bytes
// (fetched by TMA with the 128-byte swizzle, 128 elements per row of a stage), and the exponent bytes
// re-laid as the tensor pipe wants its scale factors: chunks of 512 bytes = 128 rows x 4 consecutive
// blocks, byte (row % 32) * 16 + (row / 32) * 4 + (block % 4), chunk index (block / 4) * row_chunks +
// row / 128.  A stage's chunk is copied shared -> tensor memory by `tcgen05.cp.32x128b.warpx4` (32 rows
// of 16 bytes, replicated to the four lane quarters: row m of the tile finds its four scale bytes in
// lane m % 32 of its quarter, column m / 32); the MMA of K sub-step j selects byte j with the
// scale-factor id fields of its instruction descriptor.
//
// Kernel: the one-CTA structure of gemm_tc_kernel -- persistent, 128 x 128 tile, two accumulators of 128
// columns, TMA producer warp, MMA warp, four epilogue warps, bounded waits -- with a K step of 128
// elements (four MMAs of K = 32), five stages of 33 KB (two operand tiles of 16 KB, two scale chunks).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mx_gemm_tc.cuh"
#include "mx_gemv_stream.cuh"
#include "mx_ptx.cuh"

namespace mx {

struct Tc8Cfg {
    static constexpr int BN = 128;
    static constexpr int BK = 128;                                   // elements (bytes) per stage row
    static constexpr int STAGES = 5;
    static constexpr uint32_t A_BYTES = TC_BM * BK;                  // 16 KB
    static constexpr uint32_t W_BYTES = BN * BK;                     // 16 KB
    static constexpr uint32_t SF_BYTES = 512;                        // one chunk: 128 rows x 4 blocks
    static constexpr uint32_t STAGE_BYTES = A_BYTES + W_BYTES + 2 * SF_BYTES;      // 33 KB
    static constexpr uint32_t STAGE_STRIDE = 34 * 1024;              // keeps every operand tile 1024-byte aligned
    static constexpr uint32_t EPI_BYTES = 4 * 2 * 4096;
    static constexpr uint32_t BAR_BYTES = 256;
    static constexpr uint32_t SMEM_BYTES = STAGES * STAGE_STRIDE + EPI_BYTES + BAR_BYTES + 1024;
    static constexpr uint32_t TMEM_COLS = 512;                       // 2 x 128 accumulator columns + scale columns
    static constexpr uint32_t SF_COL0 = 256;                         // first scale-factor column; 8 per stage
};

// E4M3 byte of q * 2^-sh, |q| <= 15, 0 <= sh <= 3 (exact: at most 4 significant bits, exponent >= -3).
__device__ __forceinline__ uint32_t e4m3_of_small_int(int q, int sh)
{
    const uint32_t n = (uint32_t)(q < 0 ? -q : q);
    if (n == 0) return 0u;
    const int p = 31 - __clz(n);                                     // n = 2^p * (1 + f), p in 0..3
    const uint32_t man = (n << (3 - p)) & 7u;
    return ((q < 0) ? 0x80u : 0u) | ((uint32_t)(p - sh + 7) << 3) | man;
}

// Packed MXInt (container) -> E4M3 elements [rows, K] and scale bytes in the chunk layout above.
// One thread = 8 consecutive elements.  exp_row_shift = 1: two-row blocks (rows 2i, 2i+1 share exponents).
__global__ void __launch_bounds__(256)
pack_e4m3_kernel(const uint8_t *__restrict__ mant, const uint8_t *__restrict__ exps, int64_t rows, int64_t K, int w,
                 int exp_row_shift, uint8_t *__restrict__ elems, uint8_t *__restrict__ sf, int64_t row_chunks)
{
    ptx::dep_wait();
    ptx::dep_trigger();
    const int64_t cpr = K >> 3, total = rows * cpr, nb_row = K >> 5;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = t / cpr, kc = t - row * cpr;
        const int ebyte = __ldg(exps + (row >> exp_row_shift) * nb_row + (kc >> 2));
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
        uint32_t b[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) b[i] = ebyte == 255 ? 0x7Fu : e4m3_of_small_int(q[i], w - 2);   // 0x7F: E4M3 NaN
        *reinterpret_cast<uint2 *>(elems + row * K + kc * 8) =
            make_uint2(b[0] | (b[1] << 8) | (b[2] << 16) | (b[3] << 24), b[4] | (b[5] << 8) | (b[6] << 16) | (b[7] << 24));
        if ((kc & 3) == 0) {
            const int64_t blk = kc >> 2, chunk = (blk >> 2) * row_chunks + (row >> 7);
            const int r = (int)(row & 127);
            sf[chunk * 512 + (r & 31) * 16 + (r >> 5) * 4 + (blk & 3)] = (uint8_t)ebyte;
        }
    }
}

// Instruction descriptor, kind::mxf8f6f4.block_scale: E4M3 x E4M3 -> fp32, both K-major, E8M0 scales;
// `sf_id` selects which of the four scale bytes of a tensor-memory cell this K sub-step uses.
__device__ __forceinline__ uint32_t idesc_mxf8_e4m3(int m, int n, uint32_t sf_id)
{
    return (sf_id << 4)                   // B scale-factor id
           | (0u << 7) | (0u << 10)       // A, B format: E4M3
           | ((uint32_t)(n >> 3) << 17) | (1u << 23)   // N, scale format E8M0
           | ((uint32_t)(m >> 4) << 24) | (sf_id << 29);   // M, A scale-factor id
}

// Shared-memory descriptor of a scale chunk: 32 rows of 16 bytes, no swizzle (groups of 8 rows 128 bytes apart).
__device__ __forceinline__ uint64_t smem_desc_sf_chunk(uint32_t addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(128u >> 4) << 32;         // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                   // descriptor version for tcgen05
    return d;                                 // layout type 0: no swizzle
}

__device__ __forceinline__ void tmem_cp_32x128b_warpx4(uint32_t taddr, uint64_t sdesc)
{
    asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}

__device__ __forceinline__ void mma_mxf8_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
        :
        : "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
        : "memory");
}

// tmap_a / tmap_w: E4M3 bytes [rows, K], box 128 x 128, 128-byte swizzle.  sfa / sfw: scale chunks.
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc8_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
                const __grid_constant__ CUtensorMap tmap_y, const TcParams p, const uint8_t *__restrict__ sfa,
                const uint8_t *__restrict__ sfw, int chunks_a, int chunks_w)
{
    using Cfg = Tc8Cfg;
    constexpr int STAGES = Cfg::STAGES, BN = Cfg::BN;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));

    const uint32_t epi_base = smem_base + STAGES * Cfg::STAGE_STRIDE;
    const uint32_t bar_base = epi_base + Cfg::EPI_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem_gen + STAGES * Cfg::STAGE_STRIDE + Cfg::EPI_BYTES + 8 * (2 * STAGES + 4));
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(full_bar(s), 1);
            ptx::mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(tfull_bar(a), 1);
            ptx::mbar_init(tempty_bar(a), 4);
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
    const int kblocks = p.K / Cfg::BK;                       // K % 128 == 0
    bool timed_out = false;

    if (warp == 0) {
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            for (int t = blockIdx.x; t < num_tiles && !timed_out; t += gridDim.x) {
                const int tm = t % p.tiles_m, tn = t / p.tiles_m;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!ptx::mbar_wait_bounded(empty_bar(s), ph ^ 1u, abort_flag, TC_WAIT_LIMIT_NS)) {
                        timed_out = true;
                        break;
                    }
                    ptx::mbar_arrive_expect_tx(full_bar(s), Cfg::STAGE_BYTES);
                    const uint32_t sa = smem_base + s * Cfg::STAGE_STRIDE;
                    ptx::tma_load_2d(sa, &tmap_a, kb * Cfg::BK, tm * TC_BM, full_bar(s));
                    ptx::tma_load_2d(sa + Cfg::A_BYTES, &tmap_w, kb * Cfg::BK, tn * BN, full_bar(s));
                    bulk_copy_g2s(sa + Cfg::A_BYTES + Cfg::W_BYTES, sfa + ((int64_t)kb * chunks_a + tm) * 512, 512, full_bar(s));
                    bulk_copy_g2s(sa + Cfg::A_BYTES + Cfg::W_BYTES + 512, sfw + ((int64_t)kb * chunks_w + tn) * 512, 512, full_bar(s));
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            int it = 0;
            for (int t = blockIdx.x; t < num_tiles && !timed_out; t += gridDim.x, ++it) {
                const int acc = it & 1;
                const uint32_t acc_ph = (uint32_t)(it >> 1) & 1u;
                if (!ptx::mbar_wait_bounded(tempty_bar(acc), acc_ph ^ 1u, abort_flag, TC_WAIT_LIMIT_NS)) {
                    timed_out = true;
                    break;
                }
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!ptx::mbar_wait_bounded(full_bar(s), ph, abort_flag, TC_WAIT_LIMIT_NS)) {
                        timed_out = true;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    const uint32_t sa = smem_base + s * Cfg::STAGE_STRIDE;
                    const uint32_t sw = sa + Cfg::A_BYTES, ssf = sw + Cfg::W_BYTES;
                    // this stage's scale bytes: shared -> tensor memory, executed in order ahead of the MMAs below
                    const uint32_t tsfa = tmem_base + Cfg::SF_COL0 + (uint32_t)(s * 8), tsfb = tsfa + 4;
                    tmem_cp_32x128b_warpx4(tsfa, smem_desc_sf_chunk(ssf));
                    tmem_cp_32x128b_warpx4(tsfb, smem_desc_sf_chunk(ssf + 512));
#pragma unroll
                    for (int j = 0; j < Cfg::BK / 32; ++j) {
                        mma_mxf8_ss(d_tmem, ptx::smem_desc_k_sw128(sa, j * 32), ptx::smem_desc_k_sw128(sw, j * 32),
                                    idesc_mxf8_e4m3(TC_BM, BN, (uint32_t)j), tsfa, tsfb, (kb | j) != 0 ? 1u : 0u);
                    }
                    ptx::mma_commit(empty_bar(s));
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (timed_out) break;
                ptx::mma_commit(tfull_bar(acc));
            }
        }
        __syncwarp();
    } else {
        const int quad = warp & 3;
        int it = 0;
        uint32_t epi_buf = 0;
        for (int t = blockIdx.x; t < num_tiles && !timed_out; t += gridDim.x, ++it) {
            const int acc = it & 1;
            const uint32_t acc_ph = (uint32_t)(it >> 1) & 1u;
            const int m0 = (t % p.tiles_m) * TC_BM, n0 = (t / p.tiles_m) * BN;
            const bool ok = ptx::mbar_wait_bounded(tfull_bar(acc), acc_ph, abort_flag, TC_WAIT_LIMIT_NS);
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
                store_f32_chunk(p, &tmap_y, r, row, m0 + quad * 32, n0 + c0, 0, epi_base + (uint32_t)(warp - 2) * 8192u, epi_buf, lane);
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(tempty_bar(acc));
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
