// Tensor-core MXInt product for prefill shapes (Sec. 3.2 MXInt dot-product operator, computed
// on tcgen05/TMEM).
//
// Why bf16 MMA and not int8 MMA: a decoded MXInt element q*2^(E-(w-2)) with |q| <= 127 has at
// most 7 significant bits and an 8-bit exponent, so it IS a bf16 number -- the conversion is
// exact, the product of two such numbers (<= 14 significant bits) is exact in fp32, and the
// shared exponents ride along inside the operands.  Only the fp32 accumulation rounds, which
// the paper's operator does as well.  An int8 MMA would need the accumulator pulled out of
// tensor memory and rescaled by 2^(Ea+Ew) once per block of 16/32 along K, i.e. a full
// TMEM -> register -> FMA pass per 128x256x32 step, several times longer than the MMA itself.
//
// Kernel: persistent, one CTA per SM, 128 x BN output tile, K step 64 (one 128-byte swizzled
// row of bf16), STAGES-deep TMA pipeline, two accumulators in tensor memory (2*BN <= 512
// columns) so that the epilogue of tile t overlaps the MMAs of tile t+1.
//   warp 0      : TMA producer (one lane)
//   warp 1      : tensor-memory allocation, MMA issue (one lane)
//   warps 2..   : epilogue, TMEM -> registers -> (+bias) -> global fp32 (eight warps in the plain kernel, two per
//                 TMEM lane quarter with half of the tile's columns each; four in the in-kernel-decode variants)
// Every mbarrier wait is bounded in time; on expiry the kernel raises a CTA-wide abort flag,
// records MX_ERR_TIMEOUT in the status word, frees its tensor memory and returns.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <cuda_bf16.h>

#include "mx_ptx.cuh"
#include "mx_quantize.cuh"

namespace mx {

// How the weight operand reaches shared memory.
//   W_BF16   : already decoded to bf16 in global memory, fetched by TMA (192 threads)
//   W_NIBBLE : packed 4-bit mantissas + exponent bytes, decoded in the kernel by 8 extra warps
//   W_INT8   : int8 mantissas + exponent bytes, decoded in the kernel by 8 extra warps
//   W_NIBBLE_PERM : as W_NIBBLE for K % 64 == 0, with the cheapest possible decode: inside every
//              group of 8 consecutive k the operand tile holds k in the order 0,4,1,5,2,6,3,7 (the
//              order in which a shift and a mask pull pairs of nibbles out of a packed word), and
//              the activation operand must have been written in the same order.  A dot product
//              does not care in which order its terms are visited.
enum WMode { W_BF16 = 0, W_NIBBLE = 1, W_INT8 = 2, W_NIBBLE_PERM = 3 };

constexpr int TC_BM = 128;
constexpr int TC_BK = 64;                                  // bf16 elements per 128-byte row
constexpr int TC_THREADS = 192;                            // producer, MMA, 4 epilogue warps
// plain kernel: eight epilogue warps (two per TMEM lane quarter, half of the tile's columns each: the epilogue of a
// CTA's last tile, which no MMA overlaps, takes half as long); fused modes: four, then 2 * BN weight-decode threads
// (one per tile row and half K step)
constexpr int tc_epi_warps(int wmode) { return wmode == 0 ? 8 : 4; }
constexpr int tc_threads(int bn, int wmode) { return wmode == 0 ? 64 + 32 * tc_epi_warps(0) : TC_THREADS + 2 * bn; }
// registers per thread: 128 at most, and what one block of that many threads can have
constexpr int tc_max_regs(int bn, int wmode)
{
    return 65536 / tc_threads(bn, wmode) >= 128 ? 128 : (65536 / tc_threads(bn, wmode)) / 16 * 16;
}
constexpr uint64_t TC_WAIT_LIMIT_NS = 400ull * 1000 * 1000; // 0.4 s per wait

constexpr uint32_t STATUS_TIMEOUT_BIT = 1u;

template <int BN> struct TcCfg {
    static constexpr int STAGES = (BN == 256) ? 4 : 6;
    static constexpr uint32_t A_BYTES = TC_BM * TC_BK * 2;
    static constexpr uint32_t W_BYTES = BN * TC_BK * 2;
    static constexpr uint32_t STAGE_BYTES = A_BYTES + W_BYTES;
    static constexpr uint32_t BAR_BYTES = 256;
    static constexpr uint32_t EPI_BYTES = 4 * 2 * 4096;    // per epilogue warp two 32x32 fp32 store buffers
    static constexpr uint32_t SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + BAR_BYTES + 1024; // + align slack
    static constexpr uint32_t TMEM_COLS = 2 * BN;          // 256 or 512: powers of two
};

struct TcParams {
    float *y;
    const float *bias;
    int64_t ldy;
    int M, N, K;
    int tiles_m, tiles_n;
    int tma_store;   // 1: the epilogue writes Y with tiled TMA stores (needs ldy % 4 == 0 and N % 4 == 0: the store
                     // clips at the tensor's extent in units of 16 bytes)
    int frag_store;  // 1 (fp32 result, no tail, ldy even, y 8-byte aligned): the epilogue reads the accumulator in the
                     // fragment shape and stores from registers, 32-byte sectors at a time, without shared memory
    // batch > 1 (W_BF16 kernels, fp32 result, no bias): `batch` independent products of the same
    // shape in one launch; the three tensor maps are rank 3 (z = item) and item b writes to
    // y + b * y_batch.  Tiles are numbered item-major.
    int batch;
    int64_t y_batch;
    uint32_t *status;
    // fused modes only: the packed weight operand
    const uint8_t *w_mant;
    const uint8_t *w_exp;
    int w_bits;    // signed mantissa width of W
    int block;     // 16 or 32
    // MXInt result (W_BF16 kernels only): when yq_mant is set the epilogue quantizes each row of the
    // tile in blocks of yq_block along N -- the reduction axis of the layer that consumes it -- and
    // writes mantissas [M, N/2] (yq_bits <= 4) or [M, N] and exponent bytes [M, N/yq_block]
    // instead of fp32 values (Sec. 3.2: the result is quantized to the output precision).
    uint8_t *yq_mant;
    uint8_t *yq_exp;
    uint32_t *yq_nonfinite;   // nullable: number of blocks that held Inf/NaN
    int yq_bits, yq_block;
    int yq_rows2;             // 1: rows 2i and 2i+1 share the exponent bytes (two-row blocks); exponents [M/2, N/yq_block]
    // Fused element-wise tail (one-CTA and CTA-pair kernels, batch == 1): when relu != 0 or residual is set the
    // epilogue forms  act(acc + ex_bias[n]) + residual[row, n]  (act = max(., 0) if relu) before the fp32 or MXInt
    // store; the host then passes the bias here and leaves `bias` null (Fig. 1(d): activation and skip
    // connection stay in floating point around the MX operators).
    const float *ex_bias;
    int relu;
    const float *residual;
    int64_t ldr;
};

// The residual values of a lane's 32 consecutive outputs (columns n .. n + 31) of row `row`.  Fetched one
// chunk ahead of their use: the loads cross the L2 while the previous chunk is processed (issued right before
// use they cost the epilogue warp a memory latency per chunk: 164 -> 225 us on 2048 x 16384 x 4096).
struct TailRegs { float4 res[8]; };

__device__ __forceinline__ void tail_fetch(const TcParams &p, int row, int n, TailRegs &t)
{
    if (!p.residual) return;
    const bool live = row < p.M && n < p.N;
    const float *res = p.residual + (int64_t)row * p.ldr + n;
    const bool vec = live && n + 32 <= p.N && ((p.ldr & 3) == 0) && ((reinterpret_cast<uintptr_t>(p.residual) & 15) == 0);
#pragma unroll
    for (int v = 0; v < 8; ++v) {
        if (vec) {
            t.res[v] = __ldg(reinterpret_cast<const float4 *>(res) + v);
        } else {
            const int c = n + 4 * v;
            t.res[v].x = live && c + 0 < p.N ? __ldg(res + 4 * v + 0) : 0.f;
            t.res[v].y = live && c + 1 < p.N ? __ldg(res + 4 * v + 1) : 0.f;
            t.res[v].z = live && c + 2 < p.N ? __ldg(res + 4 * v + 2) : 0.f;
            t.res[v].w = live && c + 3 < p.N ? __ldg(res + 4 * v + 3) : 0.f;
        }
    }
}

// act(acc + bias) + residual on those 32 outputs, in place.
__device__ __forceinline__ void tail_apply(const TcParams &p, const TailRegs &t, int n, uint32_t (&r)[32])
{
    const bool bvec = p.ex_bias && n + 32 <= p.N;          // the bias pointer is 16-byte aligned (checked on the host)
#pragma unroll
    for (int v = 0; v < 8; ++v) {
        float o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) o[i] = __uint_as_float(r[4 * v + i]);
        if (bvec) {
            const float4 bq = __ldg(reinterpret_cast<const float4 *>(p.ex_bias + n) + v);
            o[0] += bq.x; o[1] += bq.y; o[2] += bq.z; o[3] += bq.w;
        } else if (p.ex_bias) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (n + 4 * v + i < p.N) o[i] += __ldg(p.ex_bias + n + 4 * v + i);
        }
        if (p.relu) {
#pragma unroll
            for (int i = 0; i < 4; ++i) o[i] = o[i] < 0.f ? 0.f : o[i];       // NaN stays NaN
        }
        if (p.residual) {
            o[0] += t.res[v].x; o[1] += t.res[v].y; o[2] += t.res[v].z; o[3] += t.res[v].w;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) r[4 * v + i] = __float_as_uint(o[i]);
    }
}

// MXInt-result epilogue of one lane: r holds 32 consecutive fp32 outputs (columns n .. n + 31) of
// row `row`, i.e. one block of 32 or two blocks of 16 along N; no exchange between lanes is needed.
// Adds the bias, derives the exponent byte(s), rounds like the quantizer and stores 16 or 32
// mantissa bytes and one or two exponent bytes.
__device__ __forceinline__ void store_mxint_chunk(const TcParams &p, int row, int n, uint32_t (&r)[32])
{
    // every lane of the warp runs the shuffle below; lanes outside the matrix contribute zeros
    const bool live = row < p.M && n < p.N;
    const int64_t nb_row = p.N / p.yq_block;
    uint32_t amax[2] = {0u, 0u};
#pragma unroll
    for (int v = 0; v < 32; ++v) {
        float x = __uint_as_float(r[v]);
        if (p.bias && live && n + v < p.N) x += __ldg(p.bias + n + v);
        r[v] = __float_as_uint(x);
        if (live && n + v < p.N) amax[v >> 4] = max(amax[v >> 4], r[v] & 0x7FFFFFFFu);
    }
    if (p.yq_block == 32) amax[0] = amax[1] = max(amax[0], amax[1]);
    if (p.yq_rows2) {
        // rows 2i and 2i+1 are neighbouring lanes (the warp's first row is a multiple of 32; M is even)
        amax[0] = max(amax[0], __shfl_xor_sync(0xFFFFFFFFu, amax[0], 1));
        amax[1] = max(amax[1], __shfl_xor_sync(0xFFFFFFFFu, amax[1], 1));
    }
    if (!live) return;
    const bool writes_exp = !p.yq_rows2 || (row & 1) == 0;
    const int64_t erow = p.yq_rows2 ? (row >> 1) : row;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        if (n + 16 * h >= p.N) break;            // N % yq_block == 0: a half is all in or all out
        const int ebyte = (int)(amax[h] >> 23);   // 255 <=> an Inf or NaN in the block
        if ((p.yq_block == 16 || h == 0) && writes_exp) {
            p.yq_exp[erow * nb_row + (n + 16 * h) / p.yq_block] = (uint8_t)ebyte;
            if (ebyte == 255 && p.yq_nonfinite) atomicAdd(p.yq_nonfinite, 1u);
        }
        uint2 pk[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            float v8[8];
#pragma unroll
            for (int v = 0; v < 8; ++v) v8[v] = __uint_as_float(r[16 * h + 8 * u + v]);
            pk[u] = encode8_packed(v8, ebyte, p.yq_bits);
        }
        if (p.yq_bits <= 4)
            *reinterpret_cast<uint2 *>(p.yq_mant + (int64_t)row * (p.N >> 1) + ((n + 16 * h) >> 1)) =
                make_uint2(pk[0].x, pk[1].x);
        else
            *reinterpret_cast<uint4 *>(p.yq_mant + (int64_t)row * p.N + n + 16 * h) =
                make_uint4(pk[0].x, pk[0].y, pk[1].x, pk[1].y);
    }
}

// fp32 epilogue without shared memory: the 32 rows x 32 columns of a warp's chunk are read from tensor memory in
// the fragment shape (two loads of 16 lanes) and stored from registers; four neighbouring lanes write one 32-byte
// sector.  The staging of the tiled store costs the pair kernel shared-memory bandwidth, which is what bounds its
// main loop (see the header of mx_gemm_tc2.cuh).  taddr = the warp's lane quarter and the chunk's first column.
__device__ __forceinline__ void store_f32_frag(const TcParams &p, uint32_t taddr, int rows0, int n, int tb, int lane)
{
    uint32_t r[2][16];
    ptx::tmem_ld_16x256b_x4(taddr, r[0]);
    ptx::tmem_ld_16x256b_x4(taddr + (16u << 16), r[1]);
    ptx::tmem_ld_wait();
    if (n >= p.N || rows0 >= p.M) return;                  // warp-uniform
    float *y = p.y + (int64_t)tb * p.y_batch;
    const int cq = 2 * (lane & 3);
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            const int c = n + 8 * g + cq;
            float2 b = make_float2(0.f, 0.f);
            if (p.bias) {
                if (c + 1 < p.N) b = __ldg(reinterpret_cast<const float2 *>(p.bias + c));
                else if (c < p.N) b.x = __ldg(p.bias + c);
            }
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int row = rows0 + 16 * h + 8 * u + (lane >> 2);
                if (row >= p.M || c >= p.N) continue;
                const float2 v = make_float2(__uint_as_float(r[h][4 * g + 2 * u]) + b.x, __uint_as_float(r[h][4 * g + 2 * u + 1]) + b.y);
                float *dst = y + (int64_t)row * p.ldy + c;
                if (c + 1 < p.N) *reinterpret_cast<float2 *>(dst) = v;
                else *dst = v.x;
            }
        }
}

// fp32 epilogue of one lane: r holds 32 consecutive outputs (columns n .. n + 31) of row `row`; the
// warp's 32 rows start at `rows0`.  Adds the bias and writes the 32 x 32 block either through one of
// the warp's two 4 KB shared-memory buffers (`warp_bufs`, 128-byte swizzled box layout) and a tiled
// TMA store -- whole 128-byte lines reach L2, rows >= M and columns >= N are clipped by the store --
// or, when ldy % 4 != 0 or N % 4 != 0, with plain stores.  `epi_buf` counts the warp's TMA blocks (buffer parity).
// Shared by the one-CTA, the CTA-pair and the block-wise kernel.
// NBUF = 1: the warp has one 4 KB buffer and waits for its previous store to have been read.
template <int NBUF = 2>
__device__ __forceinline__ void store_f32_chunk(const TcParams &p, const CUtensorMap *tmap_y, uint32_t (&r)[32], int row,
                                                int rows0, int n, int tb, uint32_t warp_bufs, uint32_t &epi_buf, int lane)
{
    if (p.tma_store) {
        if (n < p.N && rows0 < p.M) {                      // warp-uniform
            const uint32_t buf = warp_bufs + (NBUF == 2 ? (epi_buf & 1u) * 4096u : 0u);
            if (lane == 0) ptx::bulk_wait_group_read<NBUF - 1>();   // the buffer used NBUF blocks ago is free
            __syncwarp();
#pragma unroll
            for (int v = 0; v < 8; ++v) {
                float4 o;
                o.x = __uint_as_float(r[4 * v + 0]);
                o.y = __uint_as_float(r[4 * v + 1]);
                o.z = __uint_as_float(r[4 * v + 2]);
                o.w = __uint_as_float(r[4 * v + 3]);
                if (p.bias) {
                    const int c = n + 4 * v;
                    if (c + 4 <= p.N) {
                        const float4 b = __ldg(reinterpret_cast<const float4 *>(p.bias + c));
                        o.x += b.x; o.y += b.y; o.z += b.z; o.w += b.w;
                    } else {
                        if (c + 0 < p.N) o.x += __ldg(p.bias + c + 0);
                        if (c + 1 < p.N) o.y += __ldg(p.bias + c + 1);
                        if (c + 2 < p.N) o.z += __ldg(p.bias + c + 2);
                    }
                }
                const uint32_t dst = buf + (uint32_t)lane * 128u + (uint32_t)((v ^ (lane & 7)) << 4);
                asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(o.x), "f"(o.y),
                             "f"(o.z), "f"(o.w)
                             : "memory");
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                if (p.batch > 1) ptx::tma_store_3d(tmap_y, n, rows0, tb, buf);
                else ptx::tma_store_2d(tmap_y, n, rows0, buf);
                ptx::bulk_commit_group();
            }
            ++epi_buf;
        }
    } else if (row < p.M && n < p.N) {
        float *yrow = p.y + (int64_t)tb * p.y_batch + (int64_t)row * p.ldy;
        const bool vec_ok = ((p.ldy & 3) == 0) && ((reinterpret_cast<uintptr_t>(p.y) & 15) == 0) && ((p.y_batch & 3) == 0);
        if (vec_ok && n + 32 <= p.N) {
#pragma unroll
            for (int v = 0; v < 8; ++v) {
                float4 o;
                o.x = __uint_as_float(r[4 * v + 0]);
                o.y = __uint_as_float(r[4 * v + 1]);
                o.z = __uint_as_float(r[4 * v + 2]);
                o.w = __uint_as_float(r[4 * v + 3]);
                if (p.bias) {
                    const float4 b = __ldg(reinterpret_cast<const float4 *>(p.bias + n) + v);
                    o.x += b.x; o.y += b.y; o.z += b.z; o.w += b.w;
                }
                reinterpret_cast<float4 *>(yrow + n)[v] = o;
            }
        } else {
#pragma unroll
            for (int v = 0; v < 32; ++v)
                if (n + v < p.N)
                    yrow[n + v] = p.bias ? __uint_as_float(r[v]) + __ldg(p.bias + n + v) : __uint_as_float(r[v]);
        }
    }
}

// Raw bytes of one (row, half K-step) item: 32 mantissas and their exponent bytes.
template <int WMODE> struct RawItem {
    uint4 m[WMODE == W_INT8 ? 2 : 1];
    uint32_t e;          // block 16: two exponent bytes (low = first block); block 32: one
};                       // an item outside the matrix is all zero bytes and decodes to +0

// TAIL: the instantiation whose epilogue applies the fused element-wise tail (it holds a chunk of residual values
// in registers; kept out of the plain kernel, which then fits the register cap without spills).
template <int BN, int WMODE, bool TAIL = false>
// (register cap: see the CTA-pair kernel; the block has tc_threads(BN, WMODE) threads)
__global__ void __maxnreg__(tc_max_regs(BN, WMODE))
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
               const __grid_constant__ CUtensorMap tmap_y, const TcParams p)
{
    using Cfg = TcCfg<BN>;
    constexpr bool FUSED = WMODE != W_BF16;
    constexpr int STAGES = Cfg::STAGES;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));

    const uint32_t epi_base = smem_base + STAGES * Cfg::STAGE_BYTES;        // 1024-byte aligned
    const uint32_t bar_base = epi_base + Cfg::EPI_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem_gen + STAGES * Cfg::STAGE_BYTES + Cfg::EPI_BYTES + 8 * (2 * STAGES + 4));
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            // full: the TMA lane's expect_tx arrival (+ one arrival per decode warp in the fused modes)
            // (the lean decode publishes a K step with one of its four groups only)
            ptx::mbar_init(full_bar(s), WMODE == W_NIBBLE_PERM ? 1 + BN / 64 : FUSED ? 1 + (2 * BN) / 32 : 1);
            ptx::mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(tfull_bar(a), 1);
            ptx::mbar_init(tempty_bar(a), tc_epi_warps(WMODE));          // one arrival per epilogue warp
        }
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_a);
        if (!FUSED) ptx::prefetch_tensormap(&tmap_w);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(tmem_slot), Cfg::TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // Everything above is private to this CTA; from here on global memory is read and written.
    ptx::dep_wait();
    if (threadIdx.x == 0) ptx::dep_trigger();

    const int tiles_item = p.tiles_m * p.tiles_n;
    const int num_tiles = tiles_item * p.batch;
    const int kblocks = (p.K + TC_BK - 1) / TC_BK;
    bool timed_out = false;

    if (warp == 0) {
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            for (int t = blockIdx.x; t < num_tiles && !timed_out; t += gridDim.x) {
                const int tb = t / tiles_item, tt = t - tb * tiles_item;
                const int m0 = (tt % p.tiles_m) * TC_BM, n0 = (tt / p.tiles_m) * BN;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!ptx::mbar_wait_bounded(empty_bar(s), ph ^ 1u, abort_flag, TC_WAIT_LIMIT_NS)) {
                        timed_out = true;
                        break;
                    }
                    ptx::mbar_arrive_expect_tx(full_bar(s), FUSED ? Cfg::A_BYTES : Cfg::STAGE_BYTES);
                    const uint32_t sa = smem_base + s * Cfg::STAGE_BYTES;
                    if (!FUSED && p.batch > 1) {
                        ptx::tma_load_3d(sa, &tmap_a, kb * TC_BK, m0, tb, full_bar(s));
                        ptx::tma_load_3d(sa + Cfg::A_BYTES, &tmap_w, kb * TC_BK, n0, tb, full_bar(s));
                    } else {
                        ptx::tma_load_2d(sa, &tmap_a, kb * TC_BK, m0, full_bar(s));
                        if (!FUSED) ptx::tma_load_2d(sa + Cfg::A_BYTES, &tmap_w, kb * TC_BK, n0, full_bar(s));
                    }
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::idesc_bf16_f32(TC_BM, BN);
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
                    const uint32_t sa = smem_base + s * Cfg::STAGE_BYTES;
                    const uint32_t sw = sa + Cfg::A_BYTES;
#pragma unroll
                    for (int j = 0; j < TC_BK / 16; ++j) {
                        ptx::mma_bf16_ss(d_tmem, ptx::smem_desc_k_sw128(sa, j * 32),
                                         ptx::smem_desc_k_sw128(sw, j * 32), idesc,
                                         (kb | j) != 0 ? 1u : 0u);
                    }
                    ptx::mma_commit(empty_bar(s));          // stage free once these MMAs retire
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (timed_out) break;
                ptx::mma_commit(tfull_bar(acc));            // accumulator complete
            }
        }
        __syncwarp();
    } else if (WMODE == W_NIBBLE_PERM && warp >= TC_THREADS / 32) {
        // ---- lean weight decode (see W_NIBBLE_PERM) ----
        // The 2 * BN decode threads form four groups; group g fills the operand tile of K steps
        // g, g + 4, g + 8, ...  A thread fetches the raw bytes of its next step right after it has
        // published the current one, so no global load of its own is in flight when it reaches the
        // proxy fence that precedes the publication (such a fence waits for them: with loads in
        // flight every K step pays a full L2 round trip), and the fetch has three K steps to land.
        // An item = 16 packed bytes (32 of the 64 k of a K step) of one tile row; a thread owns
        // four items per step, 32 rows apart (BN = 128) or 64 (BN = 256).  Rows past N read row
        // N - 1: their products land in columns that the epilogue never stores.
        constexpr int GSIZE = BN / 2;                      // threads per group
        constexpr int ITEMS = 4;
        const int dt = threadIdx.x - TC_THREADS;
        const int grp = dt / GSIZE, dl = dt % GSIZE;
        const int h = dl & 1, trow0 = dl >> 1;             // item q: tile row trow0 + q * GSIZE / 2
        const int my_tiles = blockIdx.x < num_tiles ? (num_tiles - 1 - blockIdx.x) / gridDim.x + 1 : 0;
        const int total = my_tiles * kblocks;
        const bool b16 = p.block == 16;
        const int64_t mant_ld = p.K >> 1, nb_row = p.K / p.block;
        const uint32_t row_off = (uint32_t)((trow0 >> 3) * 1024 + (trow0 & 7) * 128) + Cfg::A_BYTES;
        uint32_t chunk_off[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) chunk_off[j] = row_off + (uint32_t)(((h * 4 + j) ^ (trow0 & 7)) << 4);
        const int wsub = p.w_bits - 2;

        struct Raw { uint4 m; uint32_t e; };
        Raw raw[ITEMS];
        auto load = [&](int i) {
            if (i >= total) return;
            const int ti = i / kblocks, kb = i - ti * kblocks;
            const int n0 = ((blockIdx.x + ti * (int)gridDim.x) / p.tiles_m) * BN;
#pragma unroll
            for (int q = 0; q < ITEMS; ++q) {
                const int n = min(n0 + trow0 + q * (GSIZE / 2), p.N - 1);
                raw[q].m = __ldg(reinterpret_cast<const uint4 *>(p.w_mant + (int64_t)n * mant_ld + h * 16 + (int64_t)kb * 32));
                const uint8_t *ep = p.w_exp + (int64_t)n * nb_row;
                raw[q].e = b16 ? (uint32_t)__ldg(reinterpret_cast<const uint16_t *>(ep + h * 2 + kb * 4))
                               : (uint32_t)__ldg(ep + h + kb * 2);
            }
        };
        auto decode_store = [&](uint32_t stage, const Raw &r) {
            const int e0 = (int)(r.e & 0xFF), e1 = b16 ? (int)(r.e >> 8) : e0;
            const int f0 = e0 - wsub, f1 = e1 - wsub;
            const uint32_t w4[4] = {r.m.x, r.m.y, r.m.z, r.m.w};
            if ((unsigned)(f0 - 1) < 240u && (unsigned)(f1 - 1) < 240u) {
                // scale 2^(E-(w-2)) as bf16 in both halves; c = -136 * scale
                const uint32_t sb[2] = {(uint32_t)(f0 << 7) * 0x00010001u, (uint32_t)(f1 << 7) * 0x00010001u};
                const __nv_bfloat162 m136 = as_bf162(0xC308C308u);
                const __nv_bfloat162 cb[2] = {__hmul2(as_bf162(sb[0]), m136), __hmul2(as_bf162(sb[1]), m136)};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    // (w >> 4i) & 0x000F000F = nibbles i and i+4; ^ 0x43084308 turns each into the bf16
                    // number 128 + (q + 8); one fma gives (136 + q) * s - 136 * s = q * s exactly
                    uint32_t v[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t x = ((w4[j] >> (4 * i)) & 0x000F000Fu) ^ 0x43084308u;
                        v[i] = as_u32(__hfma2(as_bf162(x), as_bf162(sb[j >> 1]), cb[j >> 1]));
                    }
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stage + chunk_off[j]), "r"(v[0]),
                                 "r"(v[1]), "r"(v[2]), "r"(v[3])
                                 : "memory");
                }
            } else {                                        // zero / subnormal / top-of-range / non-finite scale
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    int q[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) q[i] = ((int)(w4[j] << (28 - 4 * i))) >> 28;
                    uint32_t o[4];
                    decode8_safe(q, j < 2 ? e0 : e1, p.w_bits, o);      // (k0,k1) (k2,k3) (k4,k5) (k6,k7)
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stage + chunk_off[j]),
                                 "r"(__byte_perm(o[0], o[2], 0x5410)), "r"(__byte_perm(o[0], o[2], 0x7632)),
                                 "r"(__byte_perm(o[1], o[3], 0x5410)), "r"(__byte_perm(o[1], o[3], 0x7632))
                                 : "memory");
                }
            }
        };
        load(grp);
        for (int i = grp; i < total; i += 4) {
            const int s = i % STAGES;
            const uint32_t ph = (uint32_t)(i / STAGES) & 1u;
            bool ok = true;
            if (lane == 0) ok = ptx::mbar_wait_bounded(empty_bar(s), ph ^ 1u, abort_flag, TC_WAIT_LIMIT_NS);
            if (!__shfl_sync(0xFFFFFFFFu, ok, 0)) {
                timed_out = true;
                break;
            }
            const uint32_t stage = smem_base + s * Cfg::STAGE_BYTES;
#pragma unroll
            for (int q = 0; q < ITEMS; ++q) decode_store(stage + (uint32_t)(q * GSIZE * 64), raw[q]);
            ptx::fence_proxy_async_smem();          // generic-proxy stores -> visible to the MMA
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(full_bar(s));
            load(i + 4);
        }
    } else if (FUSED && WMODE != W_NIBBLE_PERM && warp >= TC_THREADS / 32) {
        // ---- weight decode: packed mantissas + exponent bytes -> swizzled bf16 operand tile ----
        // Thread d owns half h = d & 1 (32 of the 64 k of a K step) of tile row d >> 1.  Raw
        // bytes are fetched three K steps ahead.
        constexpr int ITEMS = 1;
        const int d = threadIdx.x - TC_THREADS;
        const int h = d & 1;
        const int my_tiles = blockIdx.x < num_tiles ? (num_tiles - 1 - blockIdx.x) / gridDim.x + 1 : 0;
        const int total = my_tiles * kblocks;
        const int64_t mant_ld = WMODE == W_NIBBLE ? (p.K >> 1) : p.K;      // bytes per row
        const int nb_row = p.K / p.block;
        const bool b16 = p.block == 16;
        const int exp_shift = b16 ? 4 : 5;

        // load cursor: walks (tile, K step) in the order the steps are consumed
        int l_tile = blockIdx.x, l_kb = 0, l_i = 0;
        const uint8_t *l_mant = nullptr, *l_exp = nullptr;
        bool l_row_ok = false;
        auto load = [&](RawItem<WMODE> (&r)[ITEMS]) {
            r[0].e = 0;
#pragma unroll
            for (int j = 0; j < (WMODE == W_INT8 ? 2 : 1); ++j) r[0].m[j] = make_uint4(0, 0, 0, 0);
            if (l_i >= total) return;
            if (l_kb == 0) {                                   // new tile: this thread's weight row
                const int n = (l_tile / p.tiles_m) * BN + (d >> 1);
                l_row_ok = n < p.N;
                l_mant = p.w_mant + (int64_t)n * mant_ld;
                l_exp = p.w_exp + (int64_t)n * nb_row;
            }
            const int k0 = l_kb * TC_BK + h * 32;
            if (l_row_ok && k0 < p.K) {
                if (WMODE == W_NIBBLE) {
                    r[0].m[0] = __ldg(reinterpret_cast<const uint4 *>(l_mant + (k0 >> 1)));
                } else {
                    const uint4 *src = reinterpret_cast<const uint4 *>(l_mant + k0);
                    r[0].m[0] = __ldg(src);
                    r[0].m[WMODE == W_INT8 ? 1 : 0] = __ldg(src + 1);
                }
                const uint8_t *ep = l_exp + (k0 >> exp_shift);
                r[0].e = b16 ? (uint32_t)__ldg(reinterpret_cast<const uint16_t *>(ep)) : (uint32_t)__ldg(ep);
            }
            ++l_i;
            if (++l_kb == kblocks) { l_kb = 0; l_tile += gridDim.x; }
        };
        auto decode_store = [&](int s, const RawItem<WMODE> (&r)[ITEMS]) {
            uint8_t *sw = smem_gen + s * Cfg::STAGE_BYTES + Cfg::A_BYTES;
#pragma unroll
            for (int it = 0; it < ITEMS; ++it) {
                const int row = d >> 1;
                uint8_t *rowp = sw + (row >> 3) * 1024 + (row & 7) * 128;
                const int e0 = (int)(r[it].e & 0xFF), e1 = b16 ? (int)((r[it].e >> 8) & 0xFF) : e0;
                uint32_t o[4][4];
                const uint32_t w8[8] = {r[it].m[0].x, r[it].m[0].y, r[it].m[0].z, r[it].m[0].w,
                                        r[it].m[WMODE == W_INT8 ? 1 : 0].x, r[it].m[WMODE == W_INT8 ? 1 : 0].y,
                                        r[it].m[WMODE == W_INT8 ? 1 : 0].z, r[it].m[WMODE == W_INT8 ? 1 : 0].w};
                if (WMODE == W_NIBBLE) {
                    if (nibble_fast_ok(e0, p.w_bits) && nibble_fast_ok(e1, p.w_bits)) {
                        const __nv_bfloat162 m136 = as_bf162(0xC308C308u);       // -136
                        const __nv_bfloat162 s0 = as_bf162(bf16x2_scale_bits(e0, p.w_bits));
                        const __nv_bfloat162 s1 = as_bf162(bf16x2_scale_bits(e1, p.w_bits));
                        const __nv_bfloat162 c0 = __hmul2(s0, m136), c1 = __hmul2(s1, m136);
                        decode8_nibbles(w8[0], s0, c0, o[0]);
                        decode8_nibbles(w8[1], s0, c0, o[1]);
                        decode8_nibbles(w8[2], s1, c1, o[2]);
                        decode8_nibbles(w8[3], s1, c1, o[3]);
                    } else {                                    // scale near the top of the range
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            int q[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) q[i] = ((int)(w8[j] << (28 - 4 * i))) >> 28;
                            decode8_safe(q, j < 2 ? e0 : e1, p.w_bits, o[j]);
                        }
                    }
                } else {
                    if (byte_fast_ok(e0, p.w_bits) && byte_fast_ok(e1, p.w_bits)) {
                        const float s0 = f32_scale(e0, p.w_bits), s1 = f32_scale(e1, p.w_bits);
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
                            decode8_safe(q, j < 2 ? e0 : e1, p.w_bits, o[j]);
                        }
                    }
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int chunk = (h * 4 + j) ^ (row & 7);          // 128-byte swizzle
                    *reinterpret_cast<uint4 *>(rowp + chunk * 16) = make_uint4(o[j][0], o[j][1], o[j][2], o[j][3]);
                }
            }
        };

        // Three raw-byte buffers rotate without register moves: buffer b is decoded at steps
        // b, b+3, b+6, ... and refilled for step +3 right after, so each global load has almost
        // three K steps to land.
        int s = 0;
        uint32_t ph = 0;
        auto step = [&](int i, RawItem<WMODE> (&buf)[ITEMS]) -> bool {
            if (i >= total) return true;
            bool ok = true;
            if (lane == 0) ok = ptx::mbar_wait_bounded(empty_bar(s), ph ^ 1u, abort_flag, TC_WAIT_LIMIT_NS);
            if (!__shfl_sync(0xFFFFFFFFu, ok, 0)) return false;       // also orders the warp's stores
            decode_store(s, buf);
            ptx::fence_proxy_async_smem();          // generic-proxy stores -> visible to the MMA
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(full_bar(s));
            if (++s == STAGES) { s = 0; ph ^= 1u; }
            load(buf);
            return true;
        };
        RawItem<WMODE> b0[ITEMS], b1[ITEMS], b2[ITEMS];
        load(b0);
        load(b1);
        load(b2);
        for (int i = 0; i < total; i += 3) {
            if (!step(i, b0) || !step(i + 1, b1) || !step(i + 2, b2)) {
                timed_out = true;
                break;
            }
        }
    } else {
        const int quad = warp & 3;                          // TMEM lanes this warp may read
        constexpr int EPI_WARPS = tc_epi_warps(WMODE), COLS = BN / (EPI_WARPS / 4);
        const int col0 = ((warp - 2) >> 2) * COLS;          // this warp's columns of the tile
        int it = 0;
        uint32_t epi_buf = 0;                               // counts the warp's TMA store blocks (buffer parity)
        constexpr bool tail = TAIL && !FUSED;
        for (int t = blockIdx.x; t < num_tiles && !timed_out; t += gridDim.x, ++it) {
            const int acc = it & 1;
            const uint32_t acc_ph = (uint32_t)(it >> 1) & 1u;
            const int tb = t / tiles_item, tt = t - tb * tiles_item;
            const int m0 = (tt % p.tiles_m) * TC_BM, n0 = (tt / p.tiles_m) * BN;
            const int row = m0 + quad * 32 + lane;
            TailRegs ahead;
            if (tail) tail_fetch(p, row, n0 + col0, ahead);    // the first chunk's residual: in flight under the MMAs
            // every lane waits (acquire), then the warp agrees on the outcome so that the
            // warp-collective TMEM loads below are never executed by a partial warp
            const bool ok = ptx::mbar_wait_bounded(tfull_bar(acc), acc_ph, abort_flag, TC_WAIT_LIMIT_NS);
            if (!__all_sync(0xFFFFFFFFu, ok)) {
                timed_out = true;
                break;
            }
            ptx::tc_fence_after_sync();
#pragma unroll 1
            for (int c0 = col0; c0 < col0 + COLS; c0 += 32) {
                if (!FUSED && !tail && p.frag_store) {
                    store_f32_frag(p, tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * BN + c0), m0 + quad * 32,
                                   n0 + c0, tb, lane);
                    continue;
                }
                uint32_t r[32];
                ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * BN + c0), r);
                TailRegs cur;
                if (tail) {
                    cur = ahead;                                               // fetched a chunk ago: has arrived
                    if (c0 + 32 < col0 + COLS) tail_fetch(p, row, n0 + c0 + 32, ahead);  // in flight under this chunk
                }
                ptx::tmem_ld_wait();
                const int n = n0 + c0;
                if (tail) tail_apply(p, cur, n, r);
                if (!FUSED && p.yq_mant) {
                    store_mxint_chunk(p, row, n, r);
                    continue;
                }
                // eight warps share the 32 KB of store buffers: one 4 KB buffer each instead of two
                if (EPI_WARPS == 8)
                    store_f32_chunk<1>(p, &tmap_y, r, row, m0 + quad * 32, n, tb, epi_base + (uint32_t)(warp - 2) * 4096u, epi_buf, lane);
                else
                    store_f32_chunk<2>(p, &tmap_y, r, row, m0 + quad * 32, n, tb, epi_base + (uint32_t)(warp - 2) * 8192u, epi_buf, lane);
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(tempty_bar(acc));
        }
        if (p.tma_store && lane == 0) ptx::bulk_wait_group<0>();    // all of this warp's stores have landed
    }

    if (timed_out) {
        *abort_flag = 1;
        atomicOr(p.status, STATUS_TIMEOUT_BIT);
        // give copies that may still be in flight time to land before shared memory is released
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
