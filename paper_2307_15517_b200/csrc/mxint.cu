// C ABI of the MXInt linear-layer library: argument validation and kernel launches.
// Everything here is host code; the arithmetic lives in the kernels of the included headers.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <map>
#include <mutex>
#include <tuple>
#include <vector>

#include "../../include/mxint.h"
#include "mx_alt.cuh"
#include "mx_attention.cuh"
#include "mx_gemm_simt.cuh"
#include "mx_gemm_tc.cuh"
#include "mx_gemm_tc2.cuh"
#include "mx_gemm_tc8.cuh"
#include "mx_gemm_tcx.cuh"
#include "mx_gemv_stream.cuh"
#include "mx_glue.cuh"
#include "mx_quantize.cuh"

namespace {

constexpr int MAX_DEVICES = 64;
constexpr int SM_COUNT_FALLBACK = 148;

__device__ uint32_t g_status_word;      // per device: bit 0 = a bounded wait expired

thread_local char t_cuda_error[512] = "";

struct DeviceInfo {
    bool probed = false;
    bool is_sm100 = false;
    int sm_count = SM_COUNT_FALLBACK;
    uint32_t *status = nullptr;
    bool tc_attr_set[2][4] = {{false, false, false, false}, {false, false, false, false}};
    bool tc_tail_attr_set[2] = {false, false};
    bool stream_attr_set[4] = {false, false, false, false};
    bool tc2_attr_set[2] = {false, false};
    bool tcx_attr_set = false;
    bool tc8_attr_set = false;
    bool attn_attr_set[2] = {false, false};
};
DeviceInfo g_dev[MAX_DEVICES];
std::mutex g_init_mu;        // guards every lazily initialised field above and below (calls may come from several host threads)

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode_tiled = nullptr;

// ---- launch profile: CUDA events around every kernel launch, summed per kernel kind ----------
enum KernelKind { KIND_QUANTIZE = 0, KIND_DEQUANTIZE = 1, KIND_GEMM_TC = 2, KIND_GEMM_SIMT = 3,
                  KIND_GEMM_STREAM = 4, KIND_PREP = 5, KIND_GLUE = 6, KIND_COUNT = MX_KERNEL_KINDS };
struct ProfEntry { cudaEvent_t a, b; int kind; };
struct Profiler {
    bool on = false;
    std::vector<ProfEntry> entries;      // events in use since mx_profile_begin
    std::vector<ProfEntry> pool;         // events kept for reuse
    std::mutex mu;
};
Profiler g_prof;

struct ProfScope {
    cudaStream_t st;
    ProfEntry e{};
    bool live = false;
    ProfScope(int kind, cudaStream_t s) : st(s)
    {
        if (!g_prof.on) return;
        std::lock_guard<std::mutex> lk(g_prof.mu);
        if (!g_prof.pool.empty()) {
            e = g_prof.pool.back();
            g_prof.pool.pop_back();
        } else if (cudaEventCreate(&e.a) != cudaSuccess || cudaEventCreate(&e.b) != cudaSuccess) {
            return;
        }
        e.kind = kind;
        live = cudaEventRecord(e.a, st) == cudaSuccess;
    }
    ~ProfScope()
    {
        if (!live) return;
        cudaEventRecord(e.b, st);
        std::lock_guard<std::mutex> lk(g_prof.mu);
        g_prof.entries.push_back(e);
    }
};

mx_status_t cuda_fail(cudaError_t e, const char *what)
{
    snprintf(t_cuda_error, sizeof(t_cuda_error), "%s: %s", what, cudaGetErrorString(e));
    return MX_ERR_CUDA;
}

#define MX_CUDA(call)                                            \
    do {                                                         \
        cudaError_t e_ = (call);                                 \
        if (e_ != cudaSuccess) return cuda_fail(e_, #call);      \
    } while (0)

mx_status_t device_info(DeviceInfo **out)
{
    int dev = 0;
    MX_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return MX_ERR_CUDA;
    DeviceInfo &d = g_dev[dev];
    std::lock_guard<std::mutex> lk(g_init_mu);
    if (!d.probed) {
        int major = 0, sms = 0;
        MX_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
        MX_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        d.is_sm100 = (major == 10);
        d.sm_count = sms > 0 ? sms : SM_COUNT_FALLBACK;
        if (d.is_sm100) {
            void *p = nullptr;
            MX_CUDA(cudaGetSymbolAddress(&p, g_status_word));
            d.status = static_cast<uint32_t *>(p);
        }
        d.probed = true;
    }
    *out = &d;
    return d.is_sm100 ? MX_OK : MX_ERR_ARCH;
}

// block_rows == 2: two adjacent rows share the exponents (the paper's (16,2) block shape).
// Either storage form of the mantissas ...
bool format_ok_any(const mx_format_t &f)
{
    return (f.block == 16 || f.block == 32) && f.elem_bits >= 2 && f.elem_bits <= 8 &&
           f.exp_bits == 8 && (f.block_rows == 1 || f.block_rows == 2) && (f.packing == 0 || f.packing == 1);
}
// ... the container form only (what most kernels read and every kernel writes).
bool format_ok(const mx_format_t &f) { return format_ok_any(f) && f.packing == 0; }
size_t mant_row_bytes(int64_t K, const mx_format_t &f)
{
    return f.packing ? (size_t)(K * f.elem_bits / 8) : (f.elem_bits <= 4 ? (size_t)(K / 2) : (size_t)K);
}
bool format_1d(const mx_format_t &f) { return format_ok(f) && f.block_rows == 1; }
bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
size_t round256(size_t n) { return (n + 255u) & ~size_t(255); }

// CTAs of `kernel` (256 threads, no dynamic shared memory) that are resident per SM; looked up once.
template <typename K> int resident_ctas(K kernel)
{
    static std::mutex mu;
    static std::map<const void *, int> cache;
    std::lock_guard<std::mutex> lk(mu);
    const void *key = reinterpret_cast<const void *>(kernel);
    auto it = cache.find(key);
    if (it != cache.end()) return it->second;
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, 256, 0) != cudaSuccess || n < 1) n = 4;
    cache[key] = n;
    return n;
}

int grid_for(int64_t work_items, int threads, int sm_count, int ctas_per_sm)
{
    int64_t g = (work_items + threads - 1) / threads;
    const int64_t cap = (int64_t)sm_count * ctas_per_sm;
    if (g > cap) g = cap;
    if (g < 1) g = 1;
    return (int)g;
}

// Launch that may overlap the tail of the previous kernel in the stream (programmatic dependent
// launch): the kernel becomes resident early, sets up, and blocks in ptx::dep_wait() until its
// predecessor has completed.  Only for kernels that call dep_wait() before touching global memory.
template <typename... KArgs, typename... Args>
cudaError_t launch_dep(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                       Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    // the launch profile records events between kernels, which serialises them anyway: launch plainly
    cfg.numAttrs = g_prof.on ? 0 : 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- quantize launchers ---------------------------------------------------------------------
template <typename InT>
mx_status_t launch_quantize_rows(const InT *x, int64_t rows, int64_t K, int64_t ldx,
                                 const mx_format_t &f, mx::QuantOut out, const DeviceInfo &d,
                                 cudaStream_t st)
{
    const int64_t chunks = rows * (K / 8);
    if (chunks == 0) return MX_OK;
    if (f.block_rows == 2) {
        const int grid = grid_for((chunks + 1) / 2, 256, d.sm_count, 4);
        ProfScope prof(KIND_QUANTIZE, st);
        if (f.block == 16)
            MX_CUDA(launch_dep(mx::quantize_rows2_kernel<InT, 16>, dim3(grid), dim3(256), 0, st, x, rows, K, ldx, f.elem_bits, out));
        else
            MX_CUDA(launch_dep(mx::quantize_rows2_kernel<InT, 32>, dim3(grid), dim3(256), 0, st, x, rows, K, ldx, f.elem_bits, out));
        return MX_OK;
    }
    constexpr int UNROLL = 2;
    // at most one resident wave of CTAs: the grid-stride loop does the rest without a ragged second wave
    const int per_sm = f.block == 16 ? resident_ctas(mx::quantize_rows_kernel<InT, 16, UNROLL>)
                                     : resident_ctas(mx::quantize_rows_kernel<InT, 32, UNROLL>);
    const int grid = grid_for((chunks + UNROLL - 1) / UNROLL, 256, d.sm_count, per_sm);
    ProfScope prof(KIND_QUANTIZE, st);
    if (f.block == 16)
        MX_CUDA(launch_dep(mx::quantize_rows_kernel<InT, 16, UNROLL>, dim3(grid), dim3(256), 0, st, x, rows, K, ldx, f.elem_bits, out));
    else
        MX_CUDA(launch_dep(mx::quantize_rows_kernel<InT, 32, UNROLL>, dim3(grid), dim3(256), 0, st, x, rows, K, ldx, f.elem_bits, out));
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

mx_status_t quantize_rows_any(const void *x, mx_dtype_t dt, int64_t rows, int64_t K, int64_t ldx,
                              const mx_format_t &f, mx::QuantOut out, const DeviceInfo &d,
                              cudaStream_t st)
{
    if (dt == MX_F32)
        return launch_quantize_rows(static_cast<const float *>(x), rows, K, ldx, f, out, d, st);
    return launch_quantize_rows(static_cast<const __nv_bfloat16 *>(x), rows, K, ldx, f, out, d, st);
}

mx::PackedStrides dense_strides(int64_t K, const mx_format_t &f)
{
    mx::PackedStrides ps;
    ps.mant_ld = f.elem_bits <= 4 ? K / 2 : K;
    ps.exp_ld = K / f.block;
    ps.mant_batch = ps.exp_batch = ps.out_batch = 0;
    ps.exp_row_shift = f.block_rows == 2 ? 1 : 0;
    return ps;
}

// (mant, exps) -> bf16 [rows, ld] for `batch` items laid out by `ps`.
mx_status_t launch_dequant_bf16(const void *mant, const uint8_t *exps, int64_t rows, int64_t K,
                                const mx_format_t &f, __nv_bfloat16 *out, int64_t ld,
                                const mx::PackedStrides &ps, int64_t batch, const DeviceInfo &d,
                                cudaStream_t st)
{
    const int64_t chunks = rows * (K / 8);
    if (chunks == 0 || batch == 0) return MX_OK;
    ProfScope prof(KIND_DEQUANTIZE, st);
    const uint8_t *m = static_cast<const uint8_t *>(mant);
    const bool wide_ok = (K % 32) == 0 && (ps.mant_ld % 16) == 0 && (ps.mant_batch % 16) == 0;
    if (wide_ok) {                          // 32 elements per thread, 16-byte loads and stores
        constexpr int UNROLL = 2;
        const int64_t items = rows * (K / 32);
        const int per_sm = f.elem_bits <= 4 ? resident_ctas(mx::decode_bf16_kernel<true, UNROLL>)
                                            : resident_ctas(mx::decode_bf16_kernel<false, UNROLL>);
        const dim3 grid((unsigned)grid_for((items + UNROLL - 1) / UNROLL, 256, d.sm_count, per_sm), (unsigned)batch);
        if (f.elem_bits <= 4)
            MX_CUDA(launch_dep(mx::decode_bf16_kernel<true, UNROLL>, dim3(grid), dim3(256), 0, st, m, exps, rows, K, f.block, f.elem_bits, out, ld, ps));
        else
            MX_CUDA(launch_dep(mx::decode_bf16_kernel<false, UNROLL>, dim3(grid), dim3(256), 0, st, m, exps, rows, K, f.block, f.elem_bits, out, ld, ps));
    } else {
        const dim3 grid((unsigned)grid_for(chunks, 256, d.sm_count, 16), (unsigned)batch);
        mx::dequantize_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(m, exps, rows, K, f.block, f.elem_bits, out, ld, ps);
    }
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

mx_status_t launch_dequant_bf16(const void *mant, const uint8_t *exps, int64_t rows, int64_t K,
                                const mx_format_t &f, __nv_bfloat16 *out, int64_t ld,
                                const DeviceInfo &d, cudaStream_t st)
{
    if (f.packing) {                    // dense storage: w bits per element
        if (rows == 0 || K == 0) return MX_OK;
        ProfScope prof(KIND_DEQUANTIZE, st);
        MX_CUDA(launch_dep(mx::dequantize_dense_kernel<__nv_bfloat16>, dim3(grid_for(rows * (K / 8), 256, d.sm_count, 8)),
                           dim3(256), 0, st, static_cast<const uint8_t *>(mant), exps, rows, K, (int)f.block,
                           (int)f.elem_bits, f.block_rows == 2 ? 1 : 0, out, ld));
        MX_CUDA(cudaGetLastError());
        return MX_OK;
    }
    return launch_dequant_bf16(mant, exps, rows, K, f, out, ld, dense_strides(K, f), 1, d, st);
}

// Both operands of a product, (mant, exps) -> bf16 [rows, K]: one launch when both are in container form with
// whole 32-element items per row, else one launch each.
mx_status_t launch_dequant_pair(const void *a_mant, const uint8_t *a_exp, const mx_format_t &fa, int64_t M,
                                const void *w_mant, const uint8_t *w_exp, const mx_format_t &fw, int64_t N, int64_t K,
                                __nv_bfloat16 *a_hat, __nv_bfloat16 *w_hat, const DeviceInfo &d, cudaStream_t st)
{
    if (fa.packing || fw.packing || (K % 32) != 0) {
        const mx_status_t s = launch_dequant_bf16(a_mant, a_exp, M, K, fa, a_hat, K, d, st);
        if (s != MX_OK) return s;
        return launch_dequant_bf16(w_mant, w_exp, N, K, fw, w_hat, K, d, st);
    }
    mx::DecodePairJob j;
    j.a_mant = static_cast<const uint8_t *>(a_mant); j.a_exp = a_exp;
    j.w_mant = static_cast<const uint8_t *>(w_mant); j.w_exp = w_exp;
    j.M = M; j.N = N; j.K = K;
    j.block = fa.block; j.wa = fa.elem_bits; j.ww = fw.elem_bits;
    j.a_row_shift = fa.block_rows == 2 ? 1 : 0;
    j.w_row_shift = fw.block_rows == 2 ? 1 : 0;
    j.a_hat = a_hat; j.w_hat = w_hat;
    const bool na = fa.elem_bits <= 4, nw = fw.elem_bits <= 4;
    const int64_t items = (M + N) * (K / 32);
    ProfScope prof(KIND_DEQUANTIZE, st);
    const int per_sm = resident_ctas(mx::decode_pair_kernel<true, true>);
    const dim3 grid((unsigned)grid_for((items + 1) / 2, 256, d.sm_count, per_sm));
    if (na && nw) MX_CUDA(launch_dep(mx::decode_pair_kernel<true, true>, dim3(grid), dim3(256), 0, st, j));
    else if (na) MX_CUDA(launch_dep(mx::decode_pair_kernel<true, false>, dim3(grid), dim3(256), 0, st, j));
    else if (nw) MX_CUDA(launch_dep(mx::decode_pair_kernel<false, true>, dim3(grid), dim3(256), 0, st, j));
    else MX_CUDA(launch_dep(mx::decode_pair_kernel<false, false>, dim3(grid), dim3(256), 0, st, j));
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

// ---- tensor-core GEMM launcher ----------------------------------------------------------------
// Encoded tensor maps by (kind, base, extents): pure functions of their key, so entries never go stale.
typedef std::tuple<int, const void *, int64_t, int64_t, int64_t, int64_t, int64_t> MapKey;
std::map<MapKey, CUtensorMap> g_map_cache;
std::mutex g_map_mu;
bool cached_map(const MapKey &key, CUtensorMap *out)
{
    std::lock_guard<std::mutex> lk(g_map_mu);
    auto it = g_map_cache.find(key);
    if (it == g_map_cache.end()) return false;
    *out = it->second;
    return true;
}
void remember_map(const MapKey &key, const CUtensorMap &tm)
{
    std::lock_guard<std::mutex> lk(g_map_mu);
    if (g_map_cache.size() > 8192) g_map_cache.clear();
    g_map_cache[key] = tm;
}

// The driver's tensor-map encoder, looked up once.
mx_status_t ensure_encoder()
{
    std::lock_guard<std::mutex> lk(g_init_mu);
    if (g_encode_tiled) return MX_OK;
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    MX_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
    if (q != cudaDriverEntryPointSuccess || !fn) {
        snprintf(t_cuda_error, sizeof(t_cuda_error), "cuTensorMapEncodeTiled not available");
        return MX_ERR_CUDA;
    }
    g_encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
    return MX_OK;
}

// Sets a kernel's dynamic shared-memory limit the first time the kernel is used on a device.
template <typename K> mx_status_t smem_attr_once(bool &done, K kernel, int bytes)
{
    std::lock_guard<std::mutex> lk(g_init_mu);
    if (done) return MX_OK;
    MX_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    done = true;
    return MX_OK;
}

// bf16 [rows, K] (dense rows); batch > 1: `batch` such items `item_bytes` apart, as a rank-3 map.
mx_status_t encode_bf16_rows(CUtensorMap *tm, const void *base, int64_t rows, int64_t K, int box_rows,
                             int64_t batch = 1, size_t item_bytes = 0)
{
    {
        const mx_status_t es = ensure_encoder();
        if (es != MX_OK) return es;
    }
    // A map depends only on these seven numbers; a layer called again with the same workspace finds
    // its maps here instead of paying a driver call each (a few microseconds per product for small layers).
    const MapKey key = std::make_tuple(0, base, rows, K, (int64_t)box_rows, batch, (int64_t)item_bytes);
    if (cached_map(key, tm)) return MX_OK;
    const cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)rows, (cuuint64_t)batch};
    const cuuint64_t strides[2] = {(cuuint64_t)K * 2, (cuuint64_t)item_bytes};
    const cuuint32_t box[3] = {(cuuint32_t)mx::TC_BK, (cuuint32_t)box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = g_encode_tiled(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, batch > 1 ? 3 : 2, const_cast<void *>(base),
                                      dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                      CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(t_cuda_error, sizeof(t_cuda_error), "cuTensorMapEncodeTiled failed (%d)", (int)r);
        return MX_ERR_CUDA;
    }
    remember_map(key, *tm);
    return MX_OK;
}

struct QuantizedOut {            // MXInt result of the tensor-core product (see TcParams::yq_mant)
    uint8_t *mant = nullptr;
    uint8_t *exps = nullptr;
    uint32_t *nonfinite = nullptr;
    mx_format_t f{};
};

struct TcBatch {                 // several products of one shape in one launch (W_BF16 kernels)
    int64_t count = 1;
    size_t a_item = 0, w_item = 0;   // bytes between the items' bf16 operands
    int64_t y_batch = 0;             // floats between the items' outputs
    bool no_events = false;          // never bracket the launch with profile events (mx_gemm_static)
};

struct EpiTail {                 // element-wise tail fused into the product's epilogue (see TcParams::relu)
    int relu = 0;
    const float *residual = nullptr;
    int64_t ldr = 0;
    bool any() const { return relu != 0 || residual != nullptr; }
};

struct PackedW {                 // weight operand of the fused kernels (unused for W_BF16)
    const uint8_t *mant = nullptr;
    const uint8_t *exps = nullptr;
    int bits = 0, block = 0;
};

mx_status_t encode_f32_out(CUtensorMap *tm, float *y, int64_t M, int64_t N, int64_t ldy, int64_t batch = 1,
                           int64_t y_batch = 0)
{
    const MapKey key = std::make_tuple(1, static_cast<const void *>(y), M, N, ldy, batch, y_batch);
    if (cached_map(key, tm)) return MX_OK;
    const cuuint64_t dims[3] = {(cuuint64_t)N, (cuuint64_t)M, (cuuint64_t)batch};
    const cuuint64_t strides[2] = {(cuuint64_t)ldy * 4, (cuuint64_t)y_batch * 4};
    const cuuint32_t box[3] = {32, 32, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = g_encode_tiled(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, batch > 1 ? 3 : 2, y, dims, strides, box, estr,
                                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                      CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(t_cuda_error, sizeof(t_cuda_error), "cuTensorMapEncodeTiled (output) failed (%d)", (int)r);
        return MX_ERR_CUDA;
    }
    remember_map(key, *tm);
    return MX_OK;
}

// fp32 result, no fused tail, rows of y and the items of a batch 8-byte aligned: the epilogue may store from registers
// in the accumulator-fragment shape (TcParams::frag_store)
bool frag_store_ok(bool quantized, bool tail, const float *y, int64_t ldy, int64_t y_batch)
{
    return !quantized && !tail && y && (ldy % 2) == 0 && (y_batch % 2) == 0 && (reinterpret_cast<uintptr_t>(y) & 7u) == 0;
}

template <int BN, int WMODE>
mx_status_t launch_tc(const __nv_bfloat16 *a_hat, const __nv_bfloat16 *w_hat, const PackedW &pw,
                      int64_t M, int64_t N, int64_t K, const float *bias, float *y, int64_t ldy,
                      const QuantizedOut *yq, DeviceInfo &d, cudaStream_t st, const TcBatch &tb = TcBatch(),
                      const EpiTail &et = EpiTail())
{
    using Cfg = mx::TcCfg<BN>;
    CUtensorMap tm_a, tm_w;
    mx_status_t s = encode_bf16_rows(&tm_a, a_hat, M, K, mx::TC_BM, tb.count, tb.a_item);
    if (s != MX_OK) return s;
    if (WMODE == mx::W_BF16) {
        s = encode_bf16_rows(&tm_w, w_hat, N, K, BN, tb.count, tb.w_item);
        if (s != MX_OK) return s;
    } else {
        tm_w = tm_a;                     // not read by the fused kernels
    }
    CUtensorMap tm_y = tm_a;             // placeholder when the epilogue stores directly
    // the tiled store clips at the tensor's extent in units of 16 bytes: with N % 4 != 0 it would write up to three
    // floats past column N - 1 of every row (into the caller's row padding), so such shapes take the direct stores
    const bool tma_store = !yq && (ldy % 4) == 0 && (N % 4) == 0 && (tb.y_batch % 4) == 0;
    if (tma_store) {
        s = encode_f32_out(&tm_y, y, M, N, ldy, tb.count, tb.y_batch);
        if (s != MX_OK) return s;
    }
    constexpr int slot = BN == 256 ? 0 : 1;
    const bool tail = WMODE == mx::W_BF16 && et.any();
    s = tail ? smem_attr_once(d.tc_tail_attr_set[slot], mx::gemm_tc_kernel<BN, mx::W_BF16, true>, (int)Cfg::SMEM_BYTES)
             : smem_attr_once(d.tc_attr_set[slot][WMODE], mx::gemm_tc_kernel<BN, WMODE>, (int)Cfg::SMEM_BYTES);
    if (s != MX_OK) return s;
    if (et.any() && !tail) return MX_ERR_FORMAT;          // the in-kernel decode variants have no tail
    mx::TcParams p;
    p.y = y;
    p.bias = et.any() ? nullptr : bias;
    p.ex_bias = et.any() ? bias : nullptr;
    p.relu = et.relu;
    p.residual = et.residual;
    p.ldr = et.ldr;
    p.ldy = ldy;
    p.M = (int)M;
    p.N = (int)N;
    p.K = (int)K;
    p.tiles_m = (int)((M + mx::TC_BM - 1) / mx::TC_BM);
    p.tiles_n = (int)((N + BN - 1) / BN);
    p.status = d.status;
    p.tma_store = tma_store ? 1 : 0;
    p.frag_store = frag_store_ok(yq != nullptr, et.any(), y, ldy, tb.y_batch) && WMODE == mx::W_BF16 ? 1 : 0;
    p.w_mant = pw.mant;
    p.w_exp = pw.exps;
    p.w_bits = pw.bits;
    p.block = pw.block;
    p.yq_mant = yq ? yq->mant : nullptr;
    p.yq_exp = yq ? yq->exps : nullptr;
    p.yq_nonfinite = yq ? yq->nonfinite : nullptr;
    p.yq_bits = yq ? yq->f.elem_bits : 0;
    p.yq_block = yq ? yq->f.block : 0;
    p.yq_rows2 = yq && yq->f.block_rows == 2 ? 1 : 0;
    p.batch = (int)tb.count;
    p.y_batch = tb.y_batch;
    const int64_t tiles64 = (int64_t)p.tiles_m * p.tiles_n * tb.count;
    if (tiles64 > INT32_MAX / 2) return MX_ERR_SHAPE;
    const int tiles = (int)tiles64;
    const int grid = tiles < d.sm_count ? tiles : d.sm_count;
    const int threads = mx::tc_threads(BN, WMODE);
    if (tb.no_events) {
        mx::gemm_tc_kernel<BN, WMODE><<<grid, threads, Cfg::SMEM_BYTES, st>>>(tm_a, tm_w, tm_y, p);
        MX_CUDA(cudaGetLastError());
        return MX_OK;
    }
    ProfScope prof(KIND_GEMM_TC, st);
    if (tail) MX_CUDA(launch_dep(mx::gemm_tc_kernel<BN, mx::W_BF16, true>, dim3(grid), dim3(threads), Cfg::SMEM_BYTES, st, tm_a, tm_w, tm_y, p));
    else MX_CUDA(launch_dep(mx::gemm_tc_kernel<BN, WMODE>, dim3(grid), dim3(threads), Cfg::SMEM_BYTES, st, tm_a, tm_w, tm_y, p));
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

// The CTA-pair kernel: 256 x 256 tiles, one product per launch.
mx_status_t launch_tc2(const __nv_bfloat16 *a_hat, const __nv_bfloat16 *w_hat, int64_t M, int64_t N, int64_t K,
                       const float *bias, float *y, int64_t ldy, const QuantizedOut *yq, DeviceInfo &d, cudaStream_t st,
                       const EpiTail &et = EpiTail())
{
    using Cfg = mx::Tc2Cfg;
    CUtensorMap tm_a, tm_w;
    mx_status_t s = encode_bf16_rows(&tm_a, a_hat, M, K, mx::TC_BM);
    if (s != MX_OK) return s;
    s = encode_bf16_rows(&tm_w, w_hat, N, K, Cfg::BN / 2);
    if (s != MX_OK) return s;
    CUtensorMap tm_y = tm_a;
    const bool tma_store = !yq && (ldy % 4) == 0 && (N % 4) == 0;       // see launch_tc
    if (tma_store) {
        s = encode_f32_out(&tm_y, y, M, N, ldy);
        if (s != MX_OK) return s;
    }
    s = et.any() ? smem_attr_once(d.tc2_attr_set[1], mx::gemm_tc2_kernel<true>, (int)Cfg::SMEM_BYTES)
                 : smem_attr_once(d.tc2_attr_set[0], mx::gemm_tc2_kernel<false>, (int)Cfg::SMEM_BYTES);
    if (s != MX_OK) return s;
    mx::TcParams p{};
    p.y = y;
    p.bias = et.any() ? nullptr : bias;
    p.ex_bias = et.any() ? bias : nullptr;
    p.relu = et.relu;
    p.residual = et.residual;
    p.ldr = et.ldr;
    p.ldy = ldy;
    p.M = (int)M;
    p.N = (int)N;
    p.K = (int)K;
    p.tiles_m = (int)((M + 255) / 256);
    p.tiles_n = (int)((N + Cfg::BN - 1) / Cfg::BN);
    p.status = d.status;
    p.tma_store = tma_store ? 1 : 0;
    p.frag_store = frag_store_ok(yq != nullptr, et.any(), y, ldy, 0) ? 1 : 0;
    p.batch = 1;
    p.yq_mant = yq ? yq->mant : nullptr;
    p.yq_exp = yq ? yq->exps : nullptr;
    p.yq_nonfinite = yq ? yq->nonfinite : nullptr;
    p.yq_bits = yq ? yq->f.elem_bits : 0;
    p.yq_block = yq ? yq->f.block : 0;
    p.yq_rows2 = yq && yq->f.block_rows == 2 ? 1 : 0;
    const int tiles = p.tiles_m * p.tiles_n;
    const int pairs = tiles < d.sm_count / 2 ? tiles : d.sm_count / 2;
    ProfScope prof(KIND_GEMM_TC, st);
    if (et.any()) MX_CUDA(launch_dep(mx::gemm_tc2_kernel<true>, dim3(2 * pairs), dim3(Cfg::THREADS), Cfg::SMEM_BYTES, st, tm_a, tm_w, tm_y, p));
    else MX_CUDA(launch_dep(mx::gemm_tc2_kernel<false>, dim3(2 * pairs), dim3(Cfg::THREADS), Cfg::SMEM_BYTES, st, tm_a, tm_w, tm_y, p));
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

// The block-wise kernel (one tensor-memory accumulator per block, blocks added in fp32 registers):
// 128 x 128 tiles, fp32 result, one product per launch.
mx_status_t launch_tcx(const __nv_bfloat16 *a_hat, const __nv_bfloat16 *w_hat, int64_t M, int64_t N, int64_t K,
                       int block, const float *bias, float *y, int64_t ldy, DeviceInfo &d, cudaStream_t st)
{
    using Cfg = mx::TcxCfg;
    CUtensorMap tm_a, tm_w;
    mx_status_t s = encode_bf16_rows(&tm_a, a_hat, M, K, mx::TC_BM);
    if (s != MX_OK) return s;
    s = encode_bf16_rows(&tm_w, w_hat, N, K, Cfg::BN);
    if (s != MX_OK) return s;
    CUtensorMap tm_y = tm_a;
    const bool tma_store = (ldy % 4) == 0 && (N % 4) == 0;              // see launch_tc
    if (tma_store) {
        s = encode_f32_out(&tm_y, y, M, N, ldy);
        if (s != MX_OK) return s;
    }
    s = smem_attr_once(d.tcx_attr_set, mx::gemm_tcx_kernel, (int)Cfg::SMEM_BYTES);
    if (s != MX_OK) return s;
    mx::TcParams p{};
    p.y = y;
    p.bias = bias;
    p.ldy = ldy;
    p.M = (int)M;
    p.N = (int)N;
    p.K = (int)K;
    p.tiles_m = (int)((M + mx::TC_BM - 1) / mx::TC_BM);
    p.tiles_n = (int)((N + Cfg::BN - 1) / Cfg::BN);
    p.status = d.status;
    p.tma_store = tma_store ? 1 : 0;
    p.batch = 1;
    p.block = block;
    const int64_t tiles64 = (int64_t)p.tiles_m * p.tiles_n;
    if (tiles64 > INT32_MAX / 2) return MX_ERR_SHAPE;
    const int grid = tiles64 < d.sm_count ? (int)tiles64 : d.sm_count;
    ProfScope prof(KIND_GEMM_TC, st);
    MX_CUDA(launch_dep(mx::gemm_tcx_kernel, dim3(grid), dim3(Cfg::THREADS), Cfg::SMEM_BYTES, st, tm_a, tm_w, tm_y, p));
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

// ---- hardware block-scaled path (kind::mxf8f6f4): blocks of 32, widths <= 5 on both operands --------
bool mxf8_fits(const mx_format_t &fa, const mx_format_t &fw, int64_t K)
{
    return fa.block == 32 && fw.block == 32 && fa.elem_bits <= 5 && fw.elem_bits <= 5 && (K % 128) == 0 &&
           fa.packing == 0 && fw.packing == 0;
}
size_t mxf8_sf_bytes(int64_t rows, int64_t K) { return round256((size_t)((rows + 127) / 128) * (size_t)(K / 128) * 512); }
// E4M3 elements and scale chunks of both operands
size_t mxf8_operand_bytes(int64_t M, int64_t N, int64_t K)
{
    return round256((size_t)M * K) + mxf8_sf_bytes(M, K) + round256((size_t)N * K) + mxf8_sf_bytes(N, K);
}

mx_status_t encode_u8_sw128(CUtensorMap *tm, const void *base, int64_t rows, int64_t row_bytes, int box_rows)
{
    mx_status_t s = ensure_encoder();
    if (s != MX_OK) return s;
    const MapKey key = std::make_tuple(3, base, rows, row_bytes, (int64_t)box_rows, (int64_t)0, (int64_t)0);
    if (cached_map(key, tm)) return MX_OK;
    const cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
    const cuuint32_t box[2] = {128, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = g_encode_tiled(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box, estr,
                                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(t_cuda_error, sizeof(t_cuda_error), "cuTensorMapEncodeTiled (8-bit operand) failed (%d)", (int)r);
        return MX_ERR_CUDA;
    }
    remember_map(key, *tm);
    return MX_OK;
}

// Packed MXInt operands -> E4M3 + scale chunks in `ws` (mxf8_operand_bytes), then the block-scaled product.
mx_status_t run_tc8(const void *a_mant, const uint8_t *a_exp, const mx_format_t &fa, const void *w_mant, const uint8_t *w_exp,
                    const mx_format_t &fw, int64_t M, int64_t N, int64_t K, const float *bias, float *y, int64_t ldy,
                    uint8_t *ws, DeviceInfo &d, cudaStream_t st)
{
    using Cfg = mx::Tc8Cfg;
    uint8_t *a8 = ws;
    uint8_t *sfa = a8 + round256((size_t)M * K);
    uint8_t *w8 = sfa + mxf8_sf_bytes(M, K);
    uint8_t *sfw = w8 + round256((size_t)N * K);
    const int64_t chunks_a = (M + 127) / 128, chunks_w = (N + 127) / 128;
    {
        ProfScope prof(KIND_DEQUANTIZE, st);
        MX_CUDA(launch_dep(mx::pack_e4m3_kernel, dim3(grid_for(M * (K / 8), 256, d.sm_count, 8)), dim3(256), 0, st,
                           static_cast<const uint8_t *>(a_mant), a_exp, M, K, (int)fa.elem_bits, fa.block_rows == 2 ? 1 : 0,
                           a8, sfa, chunks_a));
    }
    {
        ProfScope prof(KIND_DEQUANTIZE, st);
        MX_CUDA(launch_dep(mx::pack_e4m3_kernel, dim3(grid_for(N * (K / 8), 256, d.sm_count, 8)), dim3(256), 0, st,
                           static_cast<const uint8_t *>(w_mant), w_exp, N, K, (int)fw.elem_bits, fw.block_rows == 2 ? 1 : 0,
                           w8, sfw, chunks_w));
    }
    CUtensorMap tm_a, tm_w;
    mx_status_t s = encode_u8_sw128(&tm_a, a8, M, K, mx::TC_BM);
    if (s != MX_OK) return s;
    s = encode_u8_sw128(&tm_w, w8, N, K, Cfg::BN);
    if (s != MX_OK) return s;
    CUtensorMap tm_y = tm_a;
    const bool tma_store = (ldy % 4) == 0 && (N % 4) == 0;              // see launch_tc
    if (tma_store) {
        s = encode_f32_out(&tm_y, y, M, N, ldy);
        if (s != MX_OK) return s;
    }
    s = smem_attr_once(d.tc8_attr_set, mx::gemm_tc8_kernel, (int)Cfg::SMEM_BYTES);
    if (s != MX_OK) return s;
    mx::TcParams p{};
    p.y = y;
    p.bias = bias;
    p.ldy = ldy;
    p.M = (int)M;
    p.N = (int)N;
    p.K = (int)K;
    p.tiles_m = (int)chunks_a;
    p.tiles_n = (int)chunks_w;
    p.status = d.status;
    p.tma_store = tma_store ? 1 : 0;
    p.batch = 1;
    const int64_t tiles64 = chunks_a * chunks_w;
    if (tiles64 > INT32_MAX / 2) return MX_ERR_SHAPE;
    const int grid = tiles64 < d.sm_count ? (int)tiles64 : d.sm_count;
    ProfScope prof(KIND_GEMM_TC, st);
    MX_CUDA(launch_dep(mx::gemm_tc8_kernel, dim3(grid), dim3(mx::TC_THREADS), Cfg::SMEM_BYTES, st, tm_a, tm_w, tm_y, p,
                       (const uint8_t *)sfa, (const uint8_t *)sfw, (int)chunks_a, (int)chunks_w));
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

bool wide_tile(int64_t M, int64_t N, const DeviceInfo &d)
{
    const int64_t tiles256 = ((M + 127) / 128) * ((N + 255) / 256);
    return tiles256 >= (int64_t)d.sm_count * 3 / 4;
}

// Pre-decoded bf16 weights (both operands fetched by TMA).
mx_status_t run_tc(const __nv_bfloat16 *a_hat, const __nv_bfloat16 *w_hat, int64_t M, int64_t N,
                   int64_t K, const float *bias, float *y, int64_t ldy, DeviceInfo &d, cudaStream_t st,
                   const QuantizedOut *yq = nullptr, const TcBatch &tb = TcBatch(), const EpiTail &et = EpiTail())
{
    const PackedW none;
    // CTA pairs (a third less shared-memory traffic per flop) when there is more than one wave of 256 x 256
    // tiles (+2 % on 2048 x 6144 x 2048, +14 % on 8192^3), or one nearly full wave of long tiles (K >= 4096:
    // 2048 x 2048 x 8192 runs in 49.5 instead of 56.5 us); a short single wave starts faster on the one-CTA
    // kernel (2048^3: 19.7 against 22.4 us).
    const int64_t pair_tiles = ((M + 255) / 256) * ((N + 255) / 256);
    const int pairs = d.sm_count / 2;
    if (tb.count == 1 && M > 128 && (pair_tiles > pairs || (K >= 4096 && 4 * pair_tiles >= 3 * pairs)))
        return launch_tc2(a_hat, w_hat, M, N, K, bias, y, ldy, yq, d, st, et);
    const int64_t tiles256 = ((M + 127) / 128) * ((N + 255) / 256) * tb.count;
    if (N > 128 && tiles256 >= (int64_t)d.sm_count * 3 / 4)
        return launch_tc<256, mx::W_BF16>(a_hat, w_hat, none, M, N, K, bias, y, ldy, yq, d, st, tb, et);
    return launch_tc<128, mx::W_BF16>(a_hat, w_hat, none, M, N, K, bias, y, ldy, yq, d, st, tb, et);
}

// Packed weights decoded inside the kernel.
mx_status_t run_tc_fused(const __nv_bfloat16 *a_hat, const void *w_mant, const uint8_t *w_exp,
                         const mx_format_t &fw, int64_t M, int64_t N, int64_t K, const float *bias,
                         float *y, int64_t ldy, DeviceInfo &d, cudaStream_t st, bool perm_a = false)
{
    PackedW pw;
    pw.mant = static_cast<const uint8_t *>(w_mant);
    pw.exps = w_exp;
    pw.bits = fw.elem_bits;
    pw.block = fw.block;
    const bool wide = wide_tile(M, N, d);
    if (perm_a) {                       // a_hat was written in the permuted K order: nibbles, K % 64 == 0
        if (wide) return launch_tc<256, mx::W_NIBBLE_PERM>(a_hat, nullptr, pw, M, N, K, bias, y, ldy, nullptr, d, st);
        return launch_tc<128, mx::W_NIBBLE_PERM>(a_hat, nullptr, pw, M, N, K, bias, y, ldy, nullptr, d, st);
    }
    if (fw.elem_bits <= 4) {
        if (wide) return launch_tc<256, mx::W_NIBBLE>(a_hat, nullptr, pw, M, N, K, bias, y, ldy, nullptr, d, st);
        return launch_tc<128, mx::W_NIBBLE>(a_hat, nullptr, pw, M, N, K, bias, y, ldy, nullptr, d, st);
    }
    if (wide) return launch_tc<256, mx::W_INT8>(a_hat, nullptr, pw, M, N, K, bias, y, ldy, nullptr, d, st);
    return launch_tc<128, mx::W_INT8>(a_hat, nullptr, pw, M, N, K, bias, y, ldy, nullptr, d, st);
}

// The fused kernels read weight rows with 16-byte loads and exponent pairs with 2-byte loads.
bool fused_ok(int64_t K, const uint8_t *w_exp)
{
    return (K % 32) == 0 && (reinterpret_cast<uintptr_t>(w_exp) & 1u) == 0;
}

size_t tc_operand_bytes(int64_t M, int64_t N, int64_t K)
{
    return round256((size_t)M * K * 2) + round256((size_t)N * K * 2);
}
size_t tc_workspace(int64_t M, int64_t N, int64_t K) { return tc_operand_bytes(M, N, K); }

size_t fused_workspace(int64_t M, int64_t K) { return round256((size_t)M * K * 2); }
size_t packed_workspace(int64_t M, int64_t K, const mx_format_t &fa)
{
    return round256(mx_mant_bytes(M, K, fa)) + round256(mx_exp_bytes(M, K, fa));
}

mx_status_t check_gemm_args(const void *a, const void *a_exp, const mx_format_t &fa, const void *w,
                            const void *w_exp, const mx_format_t &fw, int64_t M, int64_t N, int64_t K,
                            const float *bias, const float *y, int64_t ldy)
{
    if (!a || !w || !w_exp || !y) return MX_ERR_NULL;
    (void)a_exp;
    if (!format_ok_any(fa) || !format_ok_any(fw) || fa.block != fw.block) return MX_ERR_FORMAT;
    if (M <= 0 || N <= 0 || K <= 0 || (K % fa.block) != 0 || ldy < N) return MX_ERR_SHAPE;
    if ((M % fa.block_rows) != 0 || (N % fw.block_rows) != 0) return MX_ERR_SHAPE;     // whole two-row blocks
    if (M > INT32_MAX / 2 || N > INT32_MAX / 2 || K > INT32_MAX / 2) return MX_ERR_SHAPE;
    if (!aligned16(a) || !aligned16(w) || !aligned16(y) || (bias && !aligned16(bias))) return MX_ERR_ALIGN;
    return MX_OK;
}

// ---- decode: few tokens, weights streamed once ------------------------------------------------
// Tensor maps over packed weight matrices are cached: weights are static, so after the first
// call a layer costs a map lookup instead of a driver call.
struct WeightMaps { CUtensorMap mant, exps; };
std::map<std::tuple<const void *, const void *, int64_t, int64_t>, WeightMaps> g_wmap_cache;
std::mutex g_wmap_mu;

mx_status_t encode_u8_rows(CUtensorMap *out, const void *base, int64_t rows, int64_t row_bytes, int box_bytes,
                           CUtensorMapSwizzle swz)
{
    const cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)box_bytes, 16};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = g_encode_tiled(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides,
                                      box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(t_cuda_error, sizeof(t_cuda_error), "cuTensorMapEncodeTiled (packed weights) failed (%d)", (int)r);
        return MX_ERR_CUDA;
    }
    return MX_OK;
}

mx_status_t packed_weight_maps(const void *w_mant, const void *w_exp, int64_t N, int64_t K, CUtensorMap *out2)
{
    std::lock_guard<std::mutex> lk(g_wmap_mu);
    const auto key = std::make_tuple(w_mant, w_exp, N, K);
    auto it = g_wmap_cache.find(key);
    if (it == g_wmap_cache.end()) {
        const mx_status_t es = ensure_encoder();
        if (es != MX_OK) return es;
        WeightMaps wm;
        mx_status_t s = encode_u8_rows(&wm.mant, w_mant, N, K / 2, 128, CU_TENSOR_MAP_SWIZZLE_128B);
        if (s != MX_OK) return s;
        s = encode_u8_rows(&wm.exps, w_exp, N, K / 32, 16, CU_TENSOR_MAP_SWIZZLE_NONE);
        if (s != MX_OK) return s;
        if (g_wmap_cache.size() > 4096) g_wmap_cache.clear();
        it = g_wmap_cache.emplace(key, wm).first;
    }
    out2[0] = it->second.mant;
    out2[1] = it->second.exps;
    return MX_OK;
}

size_t stream_table_bytes(int32_t n_layers)
{
    return round256((size_t)n_layers * sizeof(mx::StreamLayer)) + round256((size_t)n_layers * 2 * sizeof(CUtensorMap)) +
           round256((size_t)n_layers * sizeof(mx::QuantJob));
}

bool stream_layer_ok(const mx_linear_args_t &a)
{
    return a.M >= 1 && a.M <= 16 && a.fw.block == 32 && a.fa.block == 32 && a.fw.elem_bits <= 4 &&
           (a.K % 128) == 0 && a.fa.packing == 0 && a.fw.packing == 0;
}

size_t stream_act_bytes(const mx_linear_args_t &a)
{
    return round256(mx_mant_bytes(a.M, a.K, a.fa)) + round256(mx_exp_bytes(a.M, a.K, a.fa));
}

bool same_activation(const mx_linear_args_t &a, const mx_linear_args_t &b)
{
    return a.x == b.x && a.dt == b.dt && a.M == b.M && a.K == b.K && a.ldx == b.ldx &&
           a.fa.block == b.fa.block && a.fa.elem_bits == b.fa.elem_bits && a.fa.block_rows == b.fa.block_rows;
}

template <int NT, bool BULK>
mx_status_t launch_stream(const mx::StreamParams &sp, size_t smem, int grid, DeviceInfo &d, cudaStream_t st)
{
    const mx_status_t as = smem_attr_once(d.stream_attr_set[(NT - 1) * 2 + (BULK ? 1 : 0)],
                                          mx::gemv_stream_kernel<NT, BULK>, 227 * 1024);
    if (as != MX_OK) return as;
    ProfScope prof(KIND_GEMM_STREAM, st);
    MX_CUDA(launch_dep(mx::gemv_stream_kernel<NT, BULK>, dim3(grid), dim3(mx::StreamCfg<NT, BULK>::THREADS), smem, st, sp));
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}


// Both operands of one layer in the tensor-core form: activations quantized straight to exact
// bf16, packed weights decoded to bf16.  One launch when K % 32 == 0, else two.
mx_status_t tc_prepare(const mx_linear_args_t &a, __nv_bfloat16 *a_hat, __nv_bfloat16 *w_hat, DeviceInfo &d,
                       cudaStream_t st)
{
    const int64_t M = a.M, N = a.N, K = a.K;
    mx::QuantOut out{nullptr, nullptr, a_hat, K, nullptr};
    if ((K % 32) != 0 || a.fw.packing) {
        mx_status_t s = quantize_rows_any(a.x, a.dt, M, K, a.ldx, a.fa, out, d, st);
        if (s != MX_OK) return s;
        return launch_dequant_bf16(a.w_mant, a.w_exp, N, K, a.fw, w_hat, K, d, st);
    }
    // one launch for both sides; every warp takes its share of each (see the kernel)
    mx::PrepJob job;
    job.x = a.x; job.M = M; job.K = K; job.ldx = a.ldx; job.wa = a.fa.elem_bits; job.block = a.fa.block;
    job.a_hat = a_hat;
    job.w_mant = static_cast<const uint8_t *>(a.w_mant); job.w_exp = a.w_exp; job.N = N; job.ww = a.fw.elem_bits;
    job.w_hat = w_hat;
    job.w_row_shift = a.fw.block_rows == 2 ? 1 : 0;
    job.a_rows2 = a.fa.block_rows == 2 ? 1 : 0;
    const bool f32 = a.dt == MX_F32, nib = a.fw.elem_bits <= 4;
    // CTAs of 128 threads (8 K registers): small enough to become resident beside a persistent product CTA of the
    // previous call, where they wait in griddepcontrol.wait and start the moment that grid completes
    constexpr int PT = 128;
    const int need_q = grid_for((M * (K / 8) + 1) / 2, PT, 1 << 20, 1);
    const int need_d = grid_for((N * (K / 32) + 1) / 2, PT, 1 << 20, 1);
    const int per_sm = (256 / PT) * (f32 ? (nib ? resident_ctas(mx::prep_operands_kernel<float, true>)
                                            : resident_ctas(mx::prep_operands_kernel<float, false>))
                                     : (nib ? resident_ctas(mx::prep_operands_kernel<__nv_bfloat16, true>)
                                            : resident_ctas(mx::prep_operands_kernel<__nv_bfloat16, false>)));
    const int total = d.sm_count * per_sm;            // at most one resident wave
    const int grid = need_q + need_d < total ? need_q + need_d : total;
    ProfScope prof(KIND_PREP, st);
    if (f32) {
        if (nib) MX_CUDA(launch_dep(mx::prep_operands_kernel<float, true>, dim3(grid), dim3(PT), 0, st, job));
        else MX_CUDA(launch_dep(mx::prep_operands_kernel<float, false>, dim3(grid), dim3(PT), 0, st, job));
    } else {
        if (nib) MX_CUDA(launch_dep(mx::prep_operands_kernel<__nv_bfloat16, true>, dim3(grid), dim3(PT), 0, st, job));
        else MX_CUDA(launch_dep(mx::prep_operands_kernel<__nv_bfloat16, false>, dim3(grid), dim3(PT), 0, st, job));
    }
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

}  // namespace

// =================================================================================================
extern "C" {

static mx_status_t grouped_impl(const mx_linear_args_t *layers, int32_t n_layers,
                                const uint8_t *const *packed_exps, void *workspace, size_t workspace_bytes,
                                void *stream);

size_t mx_mant_bytes(int64_t rows, int64_t K, mx_format_t f)
{
    if (!format_ok_any(f) || rows < 0 || K < 0 || (K % f.block) != 0) return 0;
    return (size_t)rows * mant_row_bytes(K, f);
}

size_t mx_exp_bytes(int64_t rows, int64_t K, mx_format_t f)
{
    if (!format_ok_any(f) || rows < 0 || K < 0 || (K % f.block) != 0 || (rows % f.block_rows) != 0) return 0;
    return (size_t)(rows / f.block_rows) * (size_t)(K / f.block);
}

double mx_format_bits(mx_format_t f)
{
    if (f.block <= 0 || f.block_rows <= 0 || f.exp_bits <= 0 || f.elem_bits < 2) return 0.0;
    return (double)f.exp_bits / ((double)f.block * (double)f.block_rows) + (double)(f.elem_bits - 1) + 1.0;
}

size_t mx_workspace_bytes_ex(int64_t M, int64_t N, int64_t K, mx_format_t fa, mx_format_t fw,
                             mx_algo_t algo)
{
    if (!format_ok_any(fa) || !format_ok_any(fw) || M <= 0 || N <= 0 || K <= 0) return 0;
    const size_t pk = packed_workspace(M, K, fa);          // mx_linear with the CUDA-core kernel
    switch (algo) {
    case MX_ALGO_SIMT: return pk;
    case MX_ALGO_STREAM: return stream_table_bytes(1) + round256(mx_mant_bytes(M, K, fa)) +
                                round256(mx_exp_bytes(M, K, fa));
    case MX_ALGO_AUTO: {            // mx_linear may stream (M <= 16), mx_gemm uses the tensor cores
        const size_t st = mx_workspace_bytes_ex(M, N, K, fa, fw, MX_ALGO_STREAM);
        const size_t tc = tc_workspace(M, N, K);
        return st > tc ? st : tc;
    }
    case MX_ALGO_TCGEN05:
    case MX_ALGO_TCGEN05_BLOCKWISE: return tc_workspace(M, N, K);
    case MX_ALGO_TCGEN05_FUSED: return (K % 32) == 0 ? fused_workspace(M, K) : tc_workspace(M, N, K);
    case MX_ALGO_TCGEN05_MXF8:      // E4M3 operands + scale chunks; mx_linear also keeps the packed activations
        return mxf8_fits(fa, fw, K) ? mxf8_operand_bytes(M, N, K) + pk : 0;
    default: return 0;
    }
}

size_t mx_workspace_bytes(int64_t M, int64_t N, int64_t K, mx_format_t fa, mx_format_t fw)
{
    return mx_workspace_bytes_ex(M, N, K, fa, fw, MX_ALGO_AUTO);
}

const char *mx_status_string(mx_status_t s)
{
    switch (s) {
    case MX_OK: return "ok";
    case MX_ERR_NULL: return "null pointer";
    case MX_ERR_SHAPE: return "bad shape";
    case MX_ERR_FORMAT: return "unsupported MXInt format";
    case MX_ERR_ALIGN: return "misaligned pointer or stride";
    case MX_ERR_WORKSPACE: return "workspace missing or too small";
    case MX_ERR_CUDA: return "CUDA error";
    case MX_ERR_TIMEOUT: return "device-side wait timed out";
    case MX_ERR_ARCH: return "device is not sm_100";
    }
    return "unknown status";
}

const char *mx_last_cuda_error(void) { return t_cuda_error; }

mx_status_t mx_quantize(const void *x, mx_dtype_t dt, int64_t rows, int64_t K, int64_t stride_row,
                        int64_t stride_k, mx_format_t f, void *mant_out, uint8_t *exp_out,
                        uint32_t *nonfinite_count, void *stream)
{
    if (!format_ok(f) || (dt != MX_F32 && dt != MX_BF16)) return MX_ERR_FORMAT;
    if (rows < 0 || K < 0 || (K % f.block) != 0 || (rows % f.block_rows) != 0) return MX_ERR_SHAPE;
    if (rows == 0 || K == 0) return MX_OK;               // empty tensor: nothing to do
    if (f.block_rows != 1 && stride_k != 1) return MX_ERR_FORMAT;   // two-row blocks: rows contiguous along K only
    if (!x || !mant_out || !exp_out) return MX_ERR_NULL;
    if (stride_k == 0 || (stride_k == 1 && stride_row < K)) return MX_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(mant_out)) return MX_ERR_ALIGN;
    if (stride_k == 1 && (stride_row % 8) != 0) return MX_ERR_ALIGN;
    DeviceInfo *d = nullptr;
    mx_status_t s = device_info(&d);
    if (s != MX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    mx::QuantOut out{static_cast<uint8_t *>(mant_out), exp_out, nullptr, 0, nonfinite_count};
    if (stride_k == 1) return quantize_rows_any(x, dt, rows, K, stride_row, f, out, *d, st);
    if (stride_row == 1 && (K % 32) == 0 && (reinterpret_cast<uintptr_t>(mant_out) & 15u) == 0) {
        // a transposed view: blocks along the slow axis of a row-major tensor
        const int64_t tiles = ((rows + 31) / 32) * ((K + 255) / 256);
        const int tgrid = (int)(tiles < (int64_t)d->sm_count * 4 ? tiles : (int64_t)d->sm_count * 4);
        ProfScope prof(KIND_QUANTIZE, st);
        if (dt == MX_F32)
            mx::quantize_transposed_kernel<float><<<tgrid, 256, 0, st>>>(static_cast<const float *>(x), rows, K, stride_k,
                                                                         f.block, f.elem_bits, out);
        else
            mx::quantize_transposed_kernel<__nv_bfloat16><<<tgrid, 256, 0, st>>>(static_cast<const __nv_bfloat16 *>(x), rows, K,
                                                                                 stride_k, f.block, f.elem_bits, out);
        MX_CUDA(cudaGetLastError());
        return MX_OK;
    }
    const int grid = grid_for(rows * (K / f.block), 256, d->sm_count, 8);
    ProfScope prof(KIND_QUANTIZE, st);
    if (dt == MX_F32)
        mx::quantize_strided_kernel<float><<<grid, 256, 0, st>>>(
            static_cast<const float *>(x), rows, K, stride_row, stride_k, f.block, f.elem_bits, out);
    else
        mx::quantize_strided_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(
            static_cast<const __nv_bfloat16 *>(x), rows, K, stride_row, stride_k, f.block, f.elem_bits, out);
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

static mx_status_t repack_impl(const void *src, int64_t rows, int64_t K, mx_format_t f, void *dst, bool to_dense, void *stream)
{
    f.packing = 0;
    if (!format_ok(f)) return MX_ERR_FORMAT;
    if (rows < 0 || K < 0 || (K % f.block) != 0) return MX_ERR_SHAPE;
    if (rows == 0 || K == 0) return MX_OK;
    if (!src || !dst) return MX_ERR_NULL;
    if (!aligned16(to_dense ? src : dst)) return MX_ERR_ALIGN;
    DeviceInfo *d = nullptr;
    mx_status_t s = device_info(&d);
    if (s != MX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int grid = grid_for(rows * (K / 8), 256, d->sm_count, 8);
    ProfScope prof(KIND_QUANTIZE, st);
    if (to_dense)
        MX_CUDA(launch_dep(mx::dense_pack_kernel, dim3(grid), dim3(256), 0, st, static_cast<const uint8_t *>(src), rows, K,
                           (int)f.elem_bits, static_cast<uint8_t *>(dst)));
    else
        MX_CUDA(launch_dep(mx::dense_unpack_kernel, dim3(grid), dim3(256), 0, st, static_cast<const uint8_t *>(src), rows, K,
                           (int)f.elem_bits, static_cast<uint8_t *>(dst)));
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

mx_status_t mx_pack_dense(const void *mant, int64_t rows, int64_t K, mx_format_t f, void *dense_out, void *stream)
{
    return repack_impl(mant, rows, K, f, dense_out, true, stream);
}

mx_status_t mx_unpack_dense(const void *dense, int64_t rows, int64_t K, mx_format_t f, void *mant_out, void *stream)
{
    return repack_impl(dense, rows, K, f, mant_out, false, stream);
}

mx_status_t mx_cast(const void *mant_in, const uint8_t *exp_in, mx_format_t f_in, int64_t rows, int64_t K,
                    mx_format_t f_out, void *mant_out, uint8_t *exp_out, uint32_t *nonfinite_count, void *stream)
{
    if (!format_1d(f_in) || !format_1d(f_out)) return MX_ERR_FORMAT;
    if (rows < 0 || K < 0 || (K % f_in.block) != 0 || (K % f_out.block) != 0) return MX_ERR_SHAPE;
    if (rows == 0 || K == 0) return MX_OK;
    if (!mant_in || !exp_in || !mant_out || !exp_out) return MX_ERR_NULL;
    if (!aligned16(mant_in) || !aligned16(mant_out)) return MX_ERR_ALIGN;
    DeviceInfo *d = nullptr;
    mx_status_t s = device_info(&d);
    if (s != MX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    mx::QuantOut out{static_cast<uint8_t *>(mant_out), exp_out, nullptr, 0, nonfinite_count};
    const int grid = grid_for(rows * (K / 8), 256, d->sm_count, 8);
    const uint8_t *mi = static_cast<const uint8_t *>(mant_in);
    ProfScope prof(KIND_QUANTIZE, st);
    if (f_out.block == 16)
        MX_CUDA(launch_dep(mx::cast_rows_kernel<16>, dim3(grid), dim3(256), 0, st, mi, exp_in, (int)f_in.block,
                           (int)f_in.elem_bits, rows, K, (int)f_out.elem_bits, out));
    else
        MX_CUDA(launch_dep(mx::cast_rows_kernel<32>, dim3(grid), dim3(256), 0, st, mi, exp_in, (int)f_in.block,
                           (int)f_in.elem_bits, rows, K, (int)f_out.elem_bits, out));
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

mx_status_t mx_dequantize(const void *mant, const uint8_t *exps, int64_t rows, int64_t K,
                          mx_format_t f, void *out, mx_dtype_t dt, int64_t ld_out, void *stream)
{
    if (!mant || !exps || !out) return MX_ERR_NULL;
    if (!format_ok_any(f) || (dt != MX_F32 && dt != MX_BF16)) return MX_ERR_FORMAT;
    if (rows < 0 || K < 0 || (K % f.block) != 0 || ld_out < K || (rows % f.block_rows) != 0) return MX_ERR_SHAPE;
    if (!aligned16(mant) || !aligned16(out) || (ld_out % 8) != 0) return MX_ERR_ALIGN;
    if (rows == 0 || K == 0) return MX_OK;
    DeviceInfo *d = nullptr;
    mx_status_t s = device_info(&d);
    if (s != MX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (f.packing && dt == MX_F32) {
        ProfScope prof(KIND_DEQUANTIZE, st);
        MX_CUDA(launch_dep(mx::dequantize_dense_kernel<float>, dim3(grid_for(rows * (K / 8), 256, d->sm_count, 8)), dim3(256), 0,
                           st, static_cast<const uint8_t *>(mant), exps, rows, K, (int)f.block, (int)f.elem_bits,
                           f.block_rows == 2 ? 1 : 0, static_cast<float *>(out), ld_out));
        MX_CUDA(cudaGetLastError());
        return MX_OK;
    }
    if (dt == MX_BF16)
        return launch_dequant_bf16(mant, exps, rows, K, f, static_cast<__nv_bfloat16 *>(out), ld_out, *d, st);
    ProfScope prof(KIND_DEQUANTIZE, st);
    mx::dequantize_kernel<float><<<grid_for(rows * (K / 8), 256, d->sm_count, 16), 256, 0, st>>>(
        static_cast<const uint8_t *>(mant), exps, rows, K, f.block, f.elem_bits,
        static_cast<float *>(out), ld_out, dense_strides(K, f));
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

mx_status_t mx_gemm_ex(const void *a_mant, const uint8_t *a_exp, mx_format_t fa, const void *w_mant,
                       const uint8_t *w_exp, mx_format_t fw, int64_t M, int64_t N, int64_t K,
                       const float *bias, float *y, int64_t ldy, void *workspace,
                       size_t workspace_bytes, mx_algo_t algo, void *stream)
{
    mx_status_t s = check_gemm_args(a_mant, a_exp, fa, w_mant, w_exp, fw, M, N, K, bias, y, ldy);
    if (s != MX_OK) return s;
    if (!a_exp) return MX_ERR_NULL;
    {
        mx_linear_args_t one;
        one.x = a_mant; one.dt = MX_F32; one.M = M; one.K = K; one.ldx = K; one.fa = fa;
        one.w_mant = w_mant; one.w_exp = w_exp; one.fw = fw; one.N = N; one.bias = bias; one.y = y; one.ldy = ldy;
        const bool can_stream = stream_layer_ok(one) && (reinterpret_cast<uintptr_t>(w_exp) & 3u) == 0 &&
                                workspace && workspace_bytes >= stream_table_bytes(1);
        if (algo == MX_ALGO_AUTO) algo = can_stream ? MX_ALGO_STREAM : MX_ALGO_TCGEN05;
        if (algo == MX_ALGO_STREAM) return grouped_impl(&one, 1, &a_exp, workspace, workspace_bytes, stream);
    }
    if (algo == MX_ALGO_TCGEN05_MXF8) {
        if (!mxf8_fits(fa, fw, K)) return MX_ERR_FORMAT;
        if (!workspace || workspace_bytes < mxf8_operand_bytes(M, N, K)) return MX_ERR_WORKSPACE;
        if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MX_ERR_ALIGN;
        DeviceInfo *d8 = nullptr;
        s = device_info(&d8);
        if (s != MX_OK) return s;
        return run_tc8(a_mant, a_exp, fa, w_mant, w_exp, fw, M, N, K, bias, y, ldy, static_cast<uint8_t *>(workspace), *d8,
                       static_cast<cudaStream_t>(stream));
    }
    if (algo != MX_ALGO_SIMT && algo != MX_ALGO_TCGEN05_FUSED && algo != MX_ALGO_TCGEN05 &&
        algo != MX_ALGO_TCGEN05_BLOCKWISE)
        return MX_ERR_FORMAT;
    // dense storage is read by the decode pass in front of the tensor-core kernels only
    if ((fa.packing || fw.packing) && algo != MX_ALGO_TCGEN05 && algo != MX_ALGO_TCGEN05_BLOCKWISE) return MX_ERR_FORMAT;
    DeviceInfo *d = nullptr;
    s = device_info(&d);
    if (s != MX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (algo == MX_ALGO_SIMT) {
        dim3 grid((unsigned)((N + 15) / 16), (unsigned)((M + 15) / 16));
        ProfScope prof(KIND_GEMM_SIMT, st);
        mx::gemm_simt_kernel<<<grid, 256, 0, st>>>(static_cast<const uint8_t *>(a_mant), a_exp,
                                                   fa.elem_bits, static_cast<const uint8_t *>(w_mant),
                                                   w_exp, fw.elem_bits, M, N, K, fa.block, bias, y, ldy,
                                                   fa.block_rows == 2 ? 1 : 0, fw.block_rows == 2 ? 1 : 0);
        MX_CUDA(cudaGetLastError());
        return MX_OK;
    }
    const bool fused = algo == MX_ALGO_TCGEN05_FUSED && (K % 32) == 0 && fw.block_rows == 1;
    if (fused && !fused_ok(K, w_exp)) return MX_ERR_ALIGN;
    if (!workspace || workspace_bytes < (fused ? fused_workspace(M, K) : tc_workspace(M, N, K)))
        return MX_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MX_ERR_ALIGN;
    __nv_bfloat16 *a_hat = static_cast<__nv_bfloat16 *>(workspace);
    if (fused) {
        s = launch_dequant_bf16(a_mant, a_exp, M, K, fa, a_hat, K, *d, st);
        if (s != MX_OK) return s;
        return run_tc_fused(a_hat, w_mant, w_exp, fw, M, N, K, bias, y, ldy, *d, st);
    }
    __nv_bfloat16 *w_hat = reinterpret_cast<__nv_bfloat16 *>(static_cast<uint8_t *>(workspace) +
                                                             round256((size_t)M * K * 2));
    s = launch_dequant_pair(a_mant, a_exp, fa, M, w_mant, w_exp, fw, N, K, a_hat, w_hat, *d, st);
    if (s != MX_OK) return s;
    if (algo == MX_ALGO_TCGEN05_BLOCKWISE) return launch_tcx(a_hat, w_hat, M, N, K, fa.block, bias, y, ldy, *d, st);
    return run_tc(a_hat, w_hat, M, N, K, bias, y, ldy, *d, st);
}

mx_status_t mx_gemm(const void *a_mant, const uint8_t *a_exp, mx_format_t fa, const void *w_mant,
                    const uint8_t *w_exp, mx_format_t fw, int64_t M, int64_t N, int64_t K,
                    const float *bias, float *y, int64_t ldy, void *workspace, size_t workspace_bytes,
                    void *stream)
{
    return mx_gemm_ex(a_mant, a_exp, fa, w_mant, w_exp, fw, M, N, K, bias, y, ldy, workspace,
                      workspace_bytes, MX_ALGO_AUTO, stream);
}

mx_status_t mx_linear_ex(const void *x, mx_dtype_t dt, int64_t M, int64_t K, int64_t ldx,
                         mx_format_t fa, const void *w_mant, const uint8_t *w_exp, mx_format_t fw,
                         int64_t N, const float *bias, float *y, int64_t ldy, void *workspace,
                         size_t workspace_bytes, mx_algo_t algo, void *stream)
{
    mx_status_t s = check_gemm_args(x, nullptr, fa, w_mant, w_exp, fw, M, N, K, bias, y, ldy);
    if (s != MX_OK) return s;
    if (dt != MX_F32 && dt != MX_BF16) return MX_ERR_FORMAT;
    if (fa.packing) return MX_ERR_FORMAT;                 // the activations are produced here: container form
    if (ldx < K) return MX_ERR_SHAPE;
    if ((ldx % 8) != 0) return MX_ERR_ALIGN;
    mx_linear_args_t one;
    one.x = x; one.dt = dt; one.M = M; one.K = K; one.ldx = ldx; one.fa = fa;
    one.w_mant = w_mant; one.w_exp = w_exp; one.fw = fw; one.N = N; one.bias = bias; one.y = y; one.ldy = ldy;
    if (fw.packing && algo != MX_ALGO_AUTO && algo != MX_ALGO_TCGEN05 && algo != MX_ALGO_TCGEN05_BLOCKWISE)
        return MX_ERR_FORMAT;
    if (algo == MX_ALGO_AUTO)
        algo = (stream_layer_ok(one) && (reinterpret_cast<uintptr_t>(w_exp) & 3u) == 0) ? MX_ALGO_STREAM
                                                                                     : MX_ALGO_TCGEN05;
    if (algo == MX_ALGO_STREAM) return mx_linear_grouped(&one, 1, workspace, workspace_bytes, stream);
    if (algo != MX_ALGO_SIMT && algo != MX_ALGO_TCGEN05_FUSED && algo != MX_ALGO_TCGEN05 &&
        algo != MX_ALGO_TCGEN05_BLOCKWISE && algo != MX_ALGO_TCGEN05_MXF8)
        return MX_ERR_FORMAT;
    DeviceInfo *d = nullptr;
    s = device_info(&d);
    if (s != MX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!workspace) return MX_ERR_WORKSPACE;
    if (algo == MX_ALGO_TCGEN05_MXF8) {
        if (!mxf8_fits(fa, fw, K)) return MX_ERR_FORMAT;
        if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MX_ERR_ALIGN;
        if (workspace_bytes < mxf8_operand_bytes(M, N, K) + packed_workspace(M, K, fa)) return MX_ERR_WORKSPACE;
        uint8_t *ws8 = static_cast<uint8_t *>(workspace);
        uint8_t *a_mant = ws8 + mxf8_operand_bytes(M, N, K);
        uint8_t *a_exp = a_mant + round256(mx_mant_bytes(M, K, fa));
        mx::QuantOut qo{a_mant, a_exp, nullptr, 0, nullptr};
        s = quantize_rows_any(x, dt, M, K, ldx, fa, qo, *d, st);
        if (s != MX_OK) return s;
        return run_tc8(a_mant, a_exp, fa, w_mant, w_exp, fw, M, N, K, bias, y, ldy, ws8, *d, st);
    }
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MX_ERR_ALIGN;
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    if (algo == MX_ALGO_SIMT) {
        if (workspace_bytes < packed_workspace(M, K, fa)) return MX_ERR_WORKSPACE;
        uint8_t *a_mant = ws;
        uint8_t *a_exp = ws + round256(mx_mant_bytes(M, K, fa));
        mx::QuantOut out{a_mant, a_exp, nullptr, 0, nullptr};
        s = quantize_rows_any(x, dt, M, K, ldx, fa, out, *d, st);
        if (s != MX_OK) return s;
        return mx_gemm_ex(a_mant, a_exp, fa, w_mant, w_exp, fw, M, N, K, bias, y, ldy, nullptr, 0,
                          MX_ALGO_SIMT, stream);
    }
    const bool fused = algo == MX_ALGO_TCGEN05_FUSED && (K % 32) == 0 && fw.block_rows == 1;
    if (fused && !fused_ok(K, w_exp)) return MX_ERR_ALIGN;
    if (workspace_bytes < (fused ? fused_workspace(M, K) : tc_workspace(M, N, K))) return MX_ERR_WORKSPACE;
    __nv_bfloat16 *a_hat = reinterpret_cast<__nv_bfloat16 *>(ws);
    // the activations' mantissas and exponents go straight to the MMA operand form (exact bf16)
    mx::QuantOut out{nullptr, nullptr, a_hat, K, nullptr};
    if (fused) {
        // 4-bit weights and whole K steps: the lean in-kernel decode, which wants both operands in
        // its own K order inside every group of 8
        const bool perm = fw.elem_bits <= 4 && (K % 64) == 0;
        out.xhat_perm = perm ? 1 : 0;
        s = quantize_rows_any(x, dt, M, K, ldx, fa, out, *d, st);
        if (s != MX_OK) return s;
        return run_tc_fused(a_hat, w_mant, w_exp, fw, M, N, K, bias, y, ldy, *d, st, perm);
    }
    __nv_bfloat16 *w_hat = reinterpret_cast<__nv_bfloat16 *>(ws + round256((size_t)M * K * 2));
    s = tc_prepare(one, a_hat, w_hat, *d, st);
    if (s != MX_OK) return s;
    if (algo == MX_ALGO_TCGEN05_BLOCKWISE) return launch_tcx(a_hat, w_hat, M, N, K, fa.block, bias, y, ldy, *d, st);
    return run_tc(a_hat, w_hat, M, N, K, bias, y, ldy, *d, st);
}

mx_status_t mx_linear(const void *x, mx_dtype_t dt, int64_t M, int64_t K, int64_t ldx, mx_format_t fa,
                      const void *w_mant, const uint8_t *w_exp, mx_format_t fw, int64_t N,
                      const float *bias, float *y, int64_t ldy, void *workspace, size_t workspace_bytes,
                      void *stream)
{
    return mx_linear_ex(x, dt, M, K, ldx, fa, w_mant, w_exp, fw, N, bias, y, ldy, workspace,
                        workspace_bytes, MX_ALGO_AUTO, stream);
}

// ---- the layer with an MXInt result -------------------------------------------------------------
static mx_status_t check_quantized_out(mx_format_t fy, int64_t M, int64_t N, const void *y_mant, const uint8_t *y_exp)
{
    if (!y_mant || !y_exp) return MX_ERR_NULL;
    if (!format_ok(fy)) return MX_ERR_FORMAT;
    if ((N % fy.block) != 0 || (M % fy.block_rows) != 0) return MX_ERR_SHAPE;
    if (!aligned16(y_mant)) return MX_ERR_ALIGN;
    return MX_OK;
}

// Tensor-core product of packed operands with an fp32 (y) or MXInt (fy, y_mant, y_exp) result and an
// optional element-wise tail.
static mx_status_t gemm_tc_impl(const void *a_mant, const uint8_t *a_exp, mx_format_t fa, const void *w_mant,
                                const uint8_t *w_exp, mx_format_t fw, int64_t M, int64_t N, int64_t K,
                                const float *bias, const EpiTail &et, float *y, int64_t ldy, mx_format_t fy,
                                void *y_mant, uint8_t *y_exp, uint32_t *nonfinite_count, void *workspace,
                                size_t workspace_bytes, void *stream)
{
    // the output pointer checks (non-null, 16-byte aligned) apply to the mantissa array of an MXInt result
    mx_status_t s = check_gemm_args(a_mant, a_exp, fa, w_mant, w_exp, fw, M, N, K, bias,
                                    y ? y : static_cast<const float *>(y_mant), y ? ldy : N);
    if (s != MX_OK) return s;
    if (!a_exp) return MX_ERR_NULL;
    if (!y) {
        s = check_quantized_out(fy, M, N, y_mant, y_exp);
        if (s != MX_OK) return s;
    }
    DeviceInfo *d = nullptr;
    s = device_info(&d);
    if (s != MX_OK) return s;
    if (!workspace || workspace_bytes < tc_workspace(M, N, K)) return MX_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MX_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    __nv_bfloat16 *a_hat = static_cast<__nv_bfloat16 *>(workspace);
    __nv_bfloat16 *w_hat = reinterpret_cast<__nv_bfloat16 *>(static_cast<uint8_t *>(workspace) +
                                                             round256((size_t)M * K * 2));
    s = launch_dequant_pair(a_mant, a_exp, fa, M, w_mant, w_exp, fw, N, K, a_hat, w_hat, *d, st);
    if (s != MX_OK) return s;
    if (y) return run_tc(a_hat, w_hat, M, N, K, bias, y, ldy, *d, st, nullptr, TcBatch(), et);
    QuantizedOut yq;
    yq.mant = static_cast<uint8_t *>(y_mant);
    yq.exps = y_exp;
    yq.nonfinite = nonfinite_count;
    yq.f = fy;
    return run_tc(a_hat, w_hat, M, N, K, bias, nullptr, N, *d, st, &yq, TcBatch(), et);
}

// The same for the layer: activations quantized on the fly.
// The operand pass with LayerNorm in front of the activation quantizer (see prep_ln_operands_kernel).
static mx_status_t tc_prepare_ln(const mx_linear_args_t &a, const mx_prologue_t &ln, __nv_bfloat16 *a_hat,
                                 __nv_bfloat16 *w_hat, DeviceInfo &d, cudaStream_t st)
{
    mx::PrepLnJob j;
    j.x = static_cast<const float *>(a.x); j.M = a.M; j.K = a.K; j.ldx = a.ldx;
    j.gamma = ln.ln_gamma; j.beta = ln.ln_beta; j.eps = ln.ln_eps;
    j.wa = a.fa.elem_bits; j.block = a.fa.block; j.a_hat = a_hat;
    j.w_mant = static_cast<const uint8_t *>(a.w_mant); j.w_exp = a.w_exp; j.N = a.N; j.ww = a.fw.elem_bits;
    j.w_hat = w_hat; j.w_row_shift = a.fw.block_rows == 2 ? 1 : 0;
    const int per = (int)((a.K + mx::GLUE_THREADS - 1) / mx::GLUE_THREADS);
    const bool nib = a.fw.elem_bits <= 4;
    const unsigned g = (unsigned)(a.M < (int64_t)d.sm_count * 8 ? a.M : (int64_t)d.sm_count * 8);
    ProfScope prof(KIND_PREP, st);
#define MX_LAUNCH_LN(P)                                                                                                  \
    do {                                                                                                                 \
        if (nib) MX_CUDA(launch_dep(mx::prep_ln_operands_kernel<P, true>, dim3(g), dim3(mx::GLUE_THREADS), 0, st, j));   \
        else MX_CUDA(launch_dep(mx::prep_ln_operands_kernel<P, false>, dim3(g), dim3(mx::GLUE_THREADS), 0, st, j));      \
    } while (0)
    if (per <= 4) MX_LAUNCH_LN(4);
    else if (per <= 8) MX_LAUNCH_LN(8);
    else if (per <= 16) MX_LAUNCH_LN(16);
    else MX_LAUNCH_LN(32);
#undef MX_LAUNCH_LN
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

static mx_status_t linear_tc_impl(const void *x, mx_dtype_t dt, int64_t M, int64_t K, int64_t ldx, mx_format_t fa,
                                  const void *w_mant, const uint8_t *w_exp, mx_format_t fw, int64_t N,
                                  const float *bias, const EpiTail &et, float *y, int64_t ldy, mx_format_t fy,
                                  void *y_mant, uint8_t *y_exp, uint32_t *nonfinite_count, void *workspace,
                                  size_t workspace_bytes, void *stream, const mx_prologue_t *ln = nullptr)
{
    mx_status_t s = check_gemm_args(x, nullptr, fa, w_mant, w_exp, fw, M, N, K, bias,
                                    y ? y : static_cast<const float *>(y_mant), y ? ldy : N);
    if (s != MX_OK) return s;
    if (dt != MX_F32 && dt != MX_BF16) return MX_ERR_FORMAT;
    if (fa.packing) return MX_ERR_FORMAT;
    if (ldx < K) return MX_ERR_SHAPE;
    if ((ldx % 8) != 0) return MX_ERR_ALIGN;
    if (!y) {
        s = check_quantized_out(fy, M, N, y_mant, y_exp);
        if (s != MX_OK) return s;
    }
    const bool with_ln = ln && ln->layernorm;
    if (with_ln) {
        // rows normalised in registers: fp32 input, rows of at most 8192 values, one-row container formats
        if (dt != MX_F32 || fa.block_rows != 1 || fw.packing) return MX_ERR_FORMAT;
        if ((K % 32) != 0 || K > mx::GLUE_THREADS * mx::GLUE_MAX_PER_THREAD) return MX_ERR_SHAPE;
    }
    DeviceInfo *d = nullptr;
    s = device_info(&d);
    if (s != MX_OK) return s;
    if (!workspace || workspace_bytes < tc_workspace(M, N, K)) return MX_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MX_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    __nv_bfloat16 *a_hat = reinterpret_cast<__nv_bfloat16 *>(ws);
    __nv_bfloat16 *w_hat = reinterpret_cast<__nv_bfloat16 *>(ws + round256((size_t)M * K * 2));
    mx_linear_args_t one;
    one.x = x; one.dt = dt; one.M = M; one.K = K; one.ldx = ldx; one.fa = fa;
    one.w_mant = w_mant; one.w_exp = w_exp; one.fw = fw; one.N = N; one.bias = bias; one.y = y; one.ldy = y ? ldy : N;
    if (with_ln) {
        s = tc_prepare_ln(one, *ln, a_hat, w_hat, *d, st);
    } else {
        s = tc_prepare(one, a_hat, w_hat, *d, st);
    }
    if (s != MX_OK) return s;
    if (y) return run_tc(a_hat, w_hat, M, N, K, bias, y, ldy, *d, st, nullptr, TcBatch(), et);
    QuantizedOut yq;
    yq.mant = static_cast<uint8_t *>(y_mant);
    yq.exps = y_exp;
    yq.nonfinite = nonfinite_count;
    yq.f = fy;
    return run_tc(a_hat, w_hat, M, N, K, bias, nullptr, N, *d, st, &yq, TcBatch(), et);
}

mx_status_t mx_gemm_q(const void *a_mant, const uint8_t *a_exp, mx_format_t fa, const void *w_mant,
                      const uint8_t *w_exp, mx_format_t fw, int64_t M, int64_t N, int64_t K,
                      const float *bias, mx_format_t fy, void *y_mant, uint8_t *y_exp,
                      uint32_t *nonfinite_count, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!y_mant) return MX_ERR_NULL;
    return gemm_tc_impl(a_mant, a_exp, fa, w_mant, w_exp, fw, M, N, K, bias, EpiTail(), nullptr, 0, fy, y_mant, y_exp,
                        nonfinite_count, workspace, workspace_bytes, stream);
}

mx_status_t mx_linear_q(const void *x, mx_dtype_t dt, int64_t M, int64_t K, int64_t ldx, mx_format_t fa,
                        const void *w_mant, const uint8_t *w_exp, mx_format_t fw, int64_t N,
                        const float *bias, mx_format_t fy, void *y_mant, uint8_t *y_exp,
                        uint32_t *nonfinite_count, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!y_mant) return MX_ERR_NULL;
    return linear_tc_impl(x, dt, M, K, ldx, fa, w_mant, w_exp, fw, N, bias, EpiTail(), nullptr, 0, fy, y_mant, y_exp,
                          nonfinite_count, workspace, workspace_bytes, stream);
}

// ---- the product with a fused element-wise tail ---------------------------------------------------
static mx_status_t tail_of(const mx_epilogue_t *ep, int64_t N, const float *y, const void *y_mant, const float **bias,
                           EpiTail *et)
{
    if ((y != nullptr) == (y_mant != nullptr)) return MX_ERR_NULL;        // exactly one kind of result
    *bias = nullptr;
    *et = EpiTail();
    if (!ep) return MX_OK;
    *bias = ep->bias;
    et->relu = ep->relu ? 1 : 0;
    et->residual = ep->residual;
    et->ldr = ep->ldr;
    if (ep->residual && ep->ldr < N) return MX_ERR_SHAPE;
    if (ep->residual && (reinterpret_cast<uintptr_t>(ep->residual) & 3u) != 0) return MX_ERR_ALIGN;
    return MX_OK;
}

mx_status_t mx_gemm_fused(const void *a_mant, const uint8_t *a_exp, mx_format_t fa, const void *w_mant,
                          const uint8_t *w_exp, mx_format_t fw, int64_t M, int64_t N, int64_t K,
                          const mx_epilogue_t *ep, float *y, int64_t ldy, mx_format_t fy, void *y_mant,
                          uint8_t *y_exp, void *workspace, size_t workspace_bytes, void *stream)
{
    const float *bias;
    EpiTail et;
    const mx_status_t s = tail_of(ep, N, y, y_mant, &bias, &et);
    if (s != MX_OK) return s;
    return gemm_tc_impl(a_mant, a_exp, fa, w_mant, w_exp, fw, M, N, K, bias, et, y, ldy, fy, y_mant, y_exp, nullptr,
                        workspace, workspace_bytes, stream);
}

mx_status_t mx_linear_fused(const void *x, mx_dtype_t dt, int64_t M, int64_t K, int64_t ldx, mx_format_t fa,
                            const mx_prologue_t *pro, const void *w_mant, const uint8_t *w_exp, mx_format_t fw,
                            int64_t N, const mx_epilogue_t *ep, float *y, int64_t ldy, mx_format_t fy, void *y_mant,
                            uint8_t *y_exp, void *workspace, size_t workspace_bytes, void *stream)
{
    const float *bias;
    EpiTail et;
    const mx_status_t s = tail_of(ep, N, y, y_mant, &bias, &et);
    if (s != MX_OK) return s;
    return linear_tc_impl(x, dt, M, K, ldx, fa, w_mant, w_exp, fw, N, bias, et, y, ldy, fy, y_mant, y_exp, nullptr,
                          workspace, workspace_bytes, stream, pro);
}

// ---- decode: few tokens, weights streamed once ------------------------------------------------
size_t mx_linear_grouped_workspace_bytes(const mx_linear_args_t *layers, int32_t n_layers)
{
    if (!layers || n_layers <= 0) return 0;
    size_t total = stream_table_bytes(n_layers);
    for (int i = 0; i < n_layers; ++i) {
        if (!format_ok(layers[i].fa) || !format_ok(layers[i].fw)) return 0;
        bool seen = false;
        for (int j = 0; j < i && !seen; ++j) seen = same_activation(layers[i], layers[j]);
        if (!seen) total += stream_act_bytes(layers[i]);
    }
    return total;
}

// packed_exps == nullptr: layers[i].x are floating-point activations, quantized here.
// packed_exps != nullptr: layers[i].x are mantissas already in format fa, packed_exps[i] their exponents.
static mx_status_t grouped_impl(const mx_linear_args_t *layers, int32_t n_layers,
                                const uint8_t *const *packed_exps, void *workspace, size_t workspace_bytes,
                                void *stream)
{
    if (!layers) return MX_ERR_NULL;
    if (n_layers <= 0) return MX_ERR_SHAPE;
    int max_t = 0, max_nb = 0, min_nb = INT32_MAX;
    for (int i = 0; i < n_layers; ++i) {
        const mx_linear_args_t &a = layers[i];
        mx_status_t s = check_gemm_args(a.x, nullptr, a.fa, a.w_mant, a.w_exp, a.fw, a.M, a.N, a.K, a.bias,
                                        a.y, a.ldy);
        if (s != MX_OK) return s;
        if (!packed_exps && a.dt != MX_F32 && a.dt != MX_BF16) return MX_ERR_FORMAT;
        if (packed_exps && !packed_exps[i]) return MX_ERR_NULL;
        if (!packed_exps && a.ldx < a.K) return MX_ERR_SHAPE;
        if ((!packed_exps && (a.ldx % 8) != 0) || (reinterpret_cast<uintptr_t>(a.w_exp) & 3u) != 0) return MX_ERR_ALIGN;
        if (!stream_layer_ok(a)) return a.M > 16 || (a.K % 128) != 0 ? MX_ERR_SHAPE : MX_ERR_FORMAT;
        max_t = a.M > max_t ? (int)a.M : max_t;
        const int nb = (int)(a.K / 32);
        max_nb = nb > max_nb ? nb : max_nb;
        min_nb = nb < min_nb ? nb : min_nb;
    }
    const size_t need = packed_exps ? stream_table_bytes(n_layers) : mx_linear_grouped_workspace_bytes(layers, n_layers);
    if (!workspace || workspace_bytes < need) return MX_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MX_ERR_ALIGN;
    const int nt = max_t > 8 ? 2 : 1;
    // weights staged by bulk copies need 16-byte aligned exponent chunks: K % 512 == 0 everywhere
    bool bulk = true;
    for (int i = 0; i < n_layers; ++i)
        bulk = bulk && (layers[i].K % 512) == 0 && (reinterpret_cast<uintptr_t>(layers[i].w_exp) & 15u) == 0 &&
               layers[i].fw.block_rows == 1;
    auto smem_of = [&](bool b) {
        return nt == 2 ? (b ? mx::StreamCfg<2, true>::smem_bytes(max_nb) : mx::StreamCfg<2, false>::smem_bytes(max_nb))
                       : (b ? mx::StreamCfg<1, true>::smem_bytes(max_nb) : mx::StreamCfg<1, false>::smem_bytes(max_nb));
    };
    size_t smem = smem_of(bulk);
    if (bulk && smem > 227u * 1024u) {
        bulk = false;
        smem = smem_of(false);
    }
    if (smem > 227u * 1024u) return MX_ERR_SHAPE;                  // tokens x K too large to stage
    DeviceInfo *d = nullptr;
    mx_status_t s = device_info(&d);
    if (s != MX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    // quantize every distinct activation tensor once, build the device layer table
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    size_t off = stream_table_bytes(n_layers);
    const size_t tmap_off = round256((size_t)n_layers * sizeof(mx::StreamLayer));
    const size_t job_off = tmap_off + round256((size_t)n_layers * 2 * sizeof(CUtensorMap));
    std::vector<mx::QuantJob> jobs;
    bool any_dt[2] = {false, false};
    int64_t max_chunks = 0;
    std::vector<mx::StreamLayer> table((size_t)n_layers);
    std::vector<CUtensorMap> tmaps(bulk ? (size_t)n_layers * 2 : 0);
    std::vector<uint8_t *> act_ptr((size_t)n_layers, nullptr);
    int total_tiles = 0;
    for (int i = 0; i < n_layers; ++i) {
        const mx_linear_args_t &a = layers[i];
        for (int j = 0; j < i && !act_ptr[i] && !packed_exps; ++j)
            if (same_activation(a, layers[j])) act_ptr[i] = act_ptr[j];
        if (!act_ptr[i] && !packed_exps) {
            act_ptr[i] = ws + off;
            off += stream_act_bytes(a);
            mx::QuantJob job;
            job.x = a.x;
            job.rows = a.M;
            job.K = a.K;
            job.ldx = a.ldx;
            job.w = a.fa.elem_bits;
            job.block = a.fa.block;
            job.dt = a.dt == MX_F32 ? 0 : 1;
            job.out = mx::QuantOut{act_ptr[i], act_ptr[i] + round256(mx_mant_bytes(a.M, a.K, a.fa)), nullptr, 0, nullptr};
            if (a.fa.block_rows == 2) {
                // pairs of tokens share their exponents: the two-row quantizer, one launch for this tensor
                s = quantize_rows_any(a.x, a.dt, a.M, a.K, a.ldx, a.fa, job.out, *d, st);
                if (s != MX_OK) return s;
            } else {
                jobs.push_back(job);
                any_dt[job.dt] = true;
                const int64_t chunks = a.M * (a.K / 8);
                max_chunks = chunks > max_chunks ? chunks : max_chunks;
            }
        }
        mx::StreamLayer &L = table[i];
        L.w_mant = static_cast<const uint8_t *>(a.w_mant);
        L.w_exp = a.w_exp;
        L.a_mant = packed_exps ? static_cast<const uint8_t *>(a.x) : act_ptr[i];
        L.a_exp = packed_exps ? packed_exps[i] : act_ptr[i] + round256(mx_mant_bytes(a.M, a.K, a.fa));
        L.bias = a.bias;
        L.y = a.y;
        L.ldy = a.ldy;
        L.N = (int)a.N;
        L.K = (int)a.K;
        L.T = (int)a.M;
        L.a_bits = a.fa.elem_bits;
        L.w_bits = a.fw.elem_bits;
        L.w_rows2 = a.fw.block_rows == 2 ? 1 : 0;
        L.a_rows2 = a.fa.block_rows == 2 ? 1 : 0;
        L.tile_begin = total_tiles;
        L.n_tiles = (int)((a.N + 15) / 16);
        total_tiles += L.n_tiles;
        if (bulk) {
            s = packed_weight_maps(a.w_mant, a.w_exp, a.N, a.K, &tmaps[(size_t)i * 2]);
            if (s != MX_OK) return s;
        }
    }
    if (bulk)
        MX_CUDA(cudaMemcpyAsync(ws + tmap_off, tmaps.data(), (size_t)n_layers * 2 * sizeof(CUtensorMap),
                                cudaMemcpyHostToDevice, st));
    MX_CUDA(cudaMemcpyAsync(ws, table.data(), (size_t)n_layers * sizeof(mx::StreamLayer),
                            cudaMemcpyHostToDevice, st));
    // all distinct activation tensors are quantized by one launch per input type
    if (!jobs.empty()) {
        MX_CUDA(cudaMemcpyAsync(ws + job_off, jobs.data(), jobs.size() * sizeof(mx::QuantJob), cudaMemcpyHostToDevice, st));
        const mx::QuantJob *dj = reinterpret_cast<const mx::QuantJob *>(ws + job_off);
        const dim3 qgrid((unsigned)grid_for((max_chunks + 1) / 2, 256, d->sm_count, 8), (unsigned)jobs.size());
        if (any_dt[0]) {
            ProfScope prof(KIND_QUANTIZE, st);
            MX_CUDA(launch_dep(mx::quantize_multi_kernel<float, 0>, dim3(qgrid), dim3(256), 0, st, dj));
        }
        if (any_dt[1]) {
            ProfScope prof(KIND_QUANTIZE, st);
            MX_CUDA(launch_dep(mx::quantize_multi_kernel<__nv_bfloat16, 1>, dim3(qgrid), dim3(256), 0, st, dj));
        }
        MX_CUDA(cudaGetLastError());
    }

    const int ctas_per_sm = (int)((227u * 1024u) / (smem + 1024)) < 4 ? (int)((227u * 1024u) / (smem + 1024)) : 4;
    const int max_ctas = d->sm_count * (ctas_per_sm < 1 ? 1 : ctas_per_sm);
    const int warps = bulk ? 16 : 8;
    int split = 1;                         // cut K over warps only when row tiles alone cannot fill the GPU
    const int unit = bulk ? 16 : 4;        // blocks per row a warp's K piece must be a multiple of
    if (total_tiles < max_ctas * warps) {
        for (int cand = 8; cand > 1 && split == 1; cand >>= 1)
            if (min_nb % (unit * cand) == 0 && (cand <= 4 || total_tiles * 4 < max_ctas * warps)) split = cand;
    }
    const int tpr = warps / split;
    const int rounds = (total_tiles + tpr - 1) / tpr;
    const int grid = rounds < max_ctas ? rounds : max_ctas;
    mx::StreamParams sp;
    sp.layers = reinterpret_cast<const mx::StreamLayer *>(ws);
    sp.n_layers = n_layers;
    sp.total_tiles = total_tiles;
    sp.split = split;
    sp.max_nb = max_nb;
    sp.status = d->status;
    sp.tmaps = reinterpret_cast<const CUtensorMap *>(ws + tmap_off);
    if (bulk)
        return nt == 2 ? launch_stream<2, true>(sp, smem, grid, *d, st) : launch_stream<1, true>(sp, smem, grid, *d, st);
    return nt == 2 ? launch_stream<2, false>(sp, smem, grid, *d, st) : launch_stream<1, false>(sp, smem, grid, *d, st);
}

mx_status_t mx_linear_grouped(const mx_linear_args_t *layers, int32_t n_layers, void *workspace,
                              size_t workspace_bytes, void *stream)
{
    return grouped_impl(layers, n_layers, nullptr, workspace, workspace_bytes, stream);
}

// ---- batched product (per-head attention matmuls) ------------------------------------------------
size_t mx_gemm_batched_workspace_bytes(int64_t M, int64_t N, int64_t K, int64_t batch)
{
    if (M <= 0 || N <= 0 || K <= 0 || batch <= 0) return 0;
    return (size_t)batch * (round256((size_t)M * K * 2) + round256((size_t)N * K * 2));
}

mx_status_t mx_gemm_batched(const void *a_mant, const uint8_t *a_exp, mx_format_t fa, int64_t lda,
                            int64_t stride_a, const void *w_mant, const uint8_t *w_exp, mx_format_t fw,
                            int64_t ldw, int64_t stride_w, int64_t M, int64_t N, int64_t K, int64_t batch,
                            float *y, int64_t ldy, int64_t stride_y, void *workspace,
                            size_t workspace_bytes, void *stream)
{
    mx_status_t s = check_gemm_args(a_mant, a_exp, fa, w_mant, w_exp, fw, M, N, K, nullptr, y, ldy);
    if (s != MX_OK) return s;
    if (!a_exp) return MX_ERR_NULL;
    if (fa.packing || fw.packing) return MX_ERR_FORMAT;
    if (batch <= 0 || lda < K || ldw < K || stride_a < 0 || stride_w < 0 || stride_y < 0) return MX_ERR_SHAPE;
    // row and batch strides must keep whole blocks and whole container bytes together
    if ((lda % fa.block) || (ldw % fw.block) || (stride_a % fa.block) || (stride_w % fw.block) ||
        (lda % 8) || (ldw % 8) || (stride_a % 8) || (stride_w % 8) || (stride_y % 4))
        return MX_ERR_ALIGN;
    if (!workspace || workspace_bytes < mx_gemm_batched_workspace_bytes(M, N, K, batch)) return MX_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MX_ERR_ALIGN;
    DeviceInfo *d = nullptr;
    s = device_info(&d);
    if (s != MX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t a_item = round256((size_t)M * K * 2), w_item = round256((size_t)N * K * 2);
    __nv_bfloat16 *a_hat = static_cast<__nv_bfloat16 *>(workspace);
    __nv_bfloat16 *w_hat = reinterpret_cast<__nv_bfloat16 *>(static_cast<uint8_t *>(workspace) + (size_t)batch * a_item);
    // two-row blocks: an item must start on an even row of the packed tensor
    if ((fa.block_rows == 2 && ((stride_a / lda) & 1)) || (fw.block_rows == 2 && ((stride_w / ldw) & 1))) return MX_ERR_ALIGN;
    auto strides = [](const mx_format_t &f, int64_t ld, int64_t bstride, size_t out_item) {
        mx::PackedStrides ps;
        ps.mant_ld = f.elem_bits <= 4 ? ld / 2 : ld;
        ps.exp_ld = ld / f.block;
        ps.mant_batch = f.elem_bits <= 4 ? bstride / 2 : bstride;
        ps.exp_row_shift = f.block_rows == 2 ? 1 : 0;   // rows 2i, 2i+1 read one row of exponent bytes
        // an item starts (bstride / ld) rows down and (bstride % ld) elements into the row
        ps.exp_batch = ((bstride / ld) >> ps.exp_row_shift) * (ld / f.block) + (bstride % ld) / f.block;
        ps.out_batch = (int64_t)(out_item / 2);
        return ps;
    };
    // one decode launch per operand and one product launch cover every batch item
    s = launch_dequant_bf16(a_mant, a_exp, M, K, fa, a_hat, K, strides(fa, lda, stride_a, a_item), batch, *d, st);
    if (s != MX_OK) return s;
    s = launch_dequant_bf16(w_mant, w_exp, N, K, fw, w_hat, K, strides(fw, ldw, stride_w, w_item), batch, *d, st);
    if (s != MX_OK) return s;
    TcBatch tb;
    tb.count = batch;
    tb.a_item = a_item;
    tb.w_item = w_item;
    tb.y_batch = stride_y;
    return run_tc(a_hat, w_hat, M, N, K, nullptr, y, ldy, *d, st, nullptr, tb);
}

// ---- fused attention ---------------------------------------------------------------------------
extern "C++" {
// The fused attention kernel on operands already in bf16 operand form: q_hat, k_hat [seq, hid], v_hat [hid, seq].
template <int D>
static mx_status_t launch_attention_d(const __nv_bfloat16 *q_hat, const __nv_bfloat16 *k_hat, const __nv_bfloat16 *v_hat,
                                      int64_t seq, int64_t heads, float scale, int causal, mx_format_t fp, float *ctx,
                                      int64_t ldc, void *p_mant_out, uint8_t *p_exp_out, DeviceInfo *d, cudaStream_t st)
{
    using Cfg = mx::AttnCfgT<D>;
    const int64_t hid = heads * D;
    CUtensorMap tm_q, tm_k, tm_v;
    mx_status_t s = encode_bf16_rows(&tm_q, q_hat, seq, hid, 128);
    if (s != MX_OK) return s;
    s = encode_bf16_rows(&tm_k, k_hat, seq, hid, 128);
    if (s != MX_OK) return s;
    s = encode_bf16_rows(&tm_v, v_hat, hid, seq, D);
    if (s != MX_OK) return s;
    s = smem_attr_once(d->attn_attr_set[D == 128 ? 0 : 1], mx::attention_kernel<D>, (int)Cfg::SMEM_BYTES);
    if (s != MX_OK) return s;
    mx::AttnParams ap;
    ap.ctx = ctx;
    ap.ldc = ldc;
    ap.seq = (int)seq;
    ap.heads = (int)heads;
    ap.scale = scale;
    ap.causal = causal ? 1 : 0;
    ap.p_bits = fp.elem_bits;
    ap.p_block = fp.block;
    ap.p_mant = static_cast<uint8_t *>(p_mant_out);
    ap.p_exp = p_exp_out;
    ap.status = d->status;
    const int64_t items = ((seq + Cfg::BQ - 1) / Cfg::BQ) * heads;
    const int grid = items < d->sm_count ? (int)items : d->sm_count;
    ProfScope prof(KIND_GEMM_TC, st);
    MX_CUDA(launch_dep(mx::attention_kernel<D>, dim3(grid), dim3(Cfg::THREADS), Cfg::SMEM_BYTES, st, tm_q, tm_k, tm_v, ap));
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

static mx_status_t launch_attention(const __nv_bfloat16 *q_hat, const __nv_bfloat16 *k_hat, const __nv_bfloat16 *v_hat,
                                    int64_t seq, int64_t heads, int64_t head_dim, float scale, int causal, mx_format_t fp,
                                    float *ctx, int64_t ldc, void *p_mant_out, uint8_t *p_exp_out, DeviceInfo *d,
                                    cudaStream_t st)
{
    if (head_dim == 64)
        return launch_attention_d<64>(q_hat, k_hat, v_hat, seq, heads, scale, causal, fp, ctx, ldc, p_mant_out, p_exp_out, d, st);
    return launch_attention_d<128>(q_hat, k_hat, v_hat, seq, heads, scale, causal, fp, ctx, ldc, p_mant_out, p_exp_out, d, st);
}

}  // extern "C++"

size_t mx_attention_workspace_bytes(int64_t seq, int64_t heads, int64_t head_dim)
{
    if (seq <= 0 || heads <= 0 || head_dim <= 0) return 0;
    return 3 * round256((size_t)seq * heads * head_dim * 2);
}

mx_status_t mx_attention(const void *q_mant, const uint8_t *q_exp, const void *k_mant, const uint8_t *k_exp, mx_format_t fqk,
                         const void *vt_mant, const uint8_t *vt_exp, mx_format_t fv, int64_t seq, int64_t heads,
                         int64_t head_dim, float scale, int causal, mx_format_t fp, float *ctx, int64_t ldc,
                         void *p_mant_out, uint8_t *p_exp_out, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!q_mant || !q_exp || !k_mant || !k_exp || !vt_mant || !vt_exp || !ctx) return MX_ERR_NULL;
    if ((p_mant_out == nullptr) != (p_exp_out == nullptr)) return MX_ERR_NULL;
    if (!format_1d(fqk) || !format_1d(fv) || !format_1d(fp)) return MX_ERR_FORMAT;
    const int64_t hid = heads * head_dim;
    if (seq <= 0 || heads <= 0 || (head_dim != 128 && head_dim != 64) || (seq % 32) != 0 || ldc < hid ||
        seq > INT32_MAX / 4 || hid > INT32_MAX / 4 || !(scale > 0.f))
        return MX_ERR_SHAPE;
    if (!aligned16(q_mant) || !aligned16(k_mant) || !aligned16(vt_mant) || !aligned16(ctx) || (ldc % 4) != 0 ||
        (p_mant_out && !aligned16(p_mant_out)))
        return MX_ERR_ALIGN;
    if (!workspace || workspace_bytes < mx_attention_workspace_bytes(seq, heads, head_dim)) return MX_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MX_ERR_ALIGN;
    DeviceInfo *d = nullptr;
    mx_status_t s = device_info(&d);
    if (s != MX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t one = round256((size_t)seq * hid * 2);
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    __nv_bfloat16 *q_hat = reinterpret_cast<__nv_bfloat16 *>(ws), *k_hat = reinterpret_cast<__nv_bfloat16 *>(ws + one),
                  *v_hat = reinterpret_cast<__nv_bfloat16 *>(ws + 2 * one);
    s = launch_dequant_bf16(q_mant, q_exp, seq, hid, fqk, q_hat, hid, *d, st);
    if (s != MX_OK) return s;
    s = launch_dequant_bf16(k_mant, k_exp, seq, hid, fqk, k_hat, hid, *d, st);
    if (s != MX_OK) return s;
    s = launch_dequant_bf16(vt_mant, vt_exp, hid, seq, fv, v_hat, seq, *d, st);
    if (s != MX_OK) return s;
    return launch_attention(q_hat, k_hat, v_hat, seq, heads, head_dim, scale, causal, fp, ctx, ldc, p_mant_out, p_exp_out, d, st);
}

mx_status_t mx_attention_fp(const void *q, const void *k, const void *v, mx_dtype_t dt, int64_t ldq, int64_t ldk,
                            int64_t ldv, mx_format_t fqk, mx_format_t fv, int64_t seq, int64_t heads, int64_t head_dim,
                            float scale, int causal, mx_format_t fp, float *ctx, int64_t ldc, void *workspace,
                            size_t workspace_bytes, void *stream)
{
    if (!q || !k || !v || !ctx) return MX_ERR_NULL;
    if (dt != MX_F32 && dt != MX_BF16) return MX_ERR_FORMAT;
    if (!format_1d(fqk) || !format_1d(fv) || !format_1d(fp) || fqk.packing || fv.packing) return MX_ERR_FORMAT;
    const int64_t hid = heads * head_dim;
    if (seq <= 0 || heads <= 0 || (head_dim != 128 && head_dim != 64) || (seq % 32) != 0 || ldc < hid || ldq < hid ||
        ldk < hid || ldv < hid || seq > INT32_MAX / 4 || hid > INT32_MAX / 4 || !(scale > 0.f))
        return MX_ERR_SHAPE;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(ctx) || (ldc % 4) != 0 || (ldq % 8) != 0 ||
        (ldk % 8) != 0 || (ldv % 8) != 0)
        return MX_ERR_ALIGN;
    if (!workspace || workspace_bytes < mx_attention_workspace_bytes(seq, heads, head_dim)) return MX_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MX_ERR_ALIGN;
    DeviceInfo *d = nullptr;
    mx_status_t s = device_info(&d);
    if (s != MX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t one = round256((size_t)seq * hid * 2);
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    __nv_bfloat16 *q_hat = reinterpret_cast<__nv_bfloat16 *>(ws), *k_hat = reinterpret_cast<__nv_bfloat16 *>(ws + one),
                  *v_hat = reinterpret_cast<__nv_bfloat16 *>(ws + 2 * one);
    // one launch for the three operands: q and k in blocks along the head dimension, v in blocks along the tokens
    // (the slow axis of v) and written transposed, [hid, seq]; all straight to the operand form
    {
        mx::AttnOperandsJob j;
        j.q = q; j.k = k; j.v = v;
        j.seq = seq; j.hid = hid; j.ldq = ldq; j.ldk = ldk; j.ldv = ldv;
        j.block_qk = fqk.block; j.w_qk = fqk.elem_bits; j.block_v = fv.block; j.w_v = fv.elem_bits;
        j.q_hat = q_hat; j.k_hat = k_hat; j.v_hat = v_hat;
        const int64_t row_items = seq * ((hid + 255) / 256), tiles = ((hid + 31) / 32) * ((seq + 255) / 256);
        const int64_t want = (row_items + 7) / 8 > tiles ? (row_items + 7) / 8 : tiles;      // 8 warps per CTA
        const int per_sm = dt == MX_F32 ? resident_ctas(mx::attention_operands_kernel<float>)
                                        : resident_ctas(mx::attention_operands_kernel<__nv_bfloat16>);
        const int64_t cap = (int64_t)d->sm_count * per_sm;
        const int grid = (int)(want < cap ? want : cap);
        ProfScope prof(KIND_QUANTIZE, st);
        if (dt == MX_F32) MX_CUDA(launch_dep(mx::attention_operands_kernel<float>, dim3(grid), dim3(256), 0, st, j));
        else MX_CUDA(launch_dep(mx::attention_operands_kernel<__nv_bfloat16>, dim3(grid), dim3(256), 0, st, j));
        MX_CUDA(cudaGetLastError());
    }
    return launch_attention(q_hat, k_hat, v_hat, seq, heads, head_dim, scale, causal, fp, ctx, ldc, nullptr, nullptr, d, st);
}

// ---- fp32 glue of the transformer block ---------------------------------------------------------
mx_status_t mx_layernorm(const float *x, int64_t ldx, const float *gamma, const float *beta, float eps,
                         int64_t rows, int64_t cols, float *y, int64_t ldy, void *stream)
{
    if (!x || !y) return MX_ERR_NULL;
    if (rows < 0 || cols <= 0 || ldx < cols || ldy < cols || cols > mx::GLUE_THREADS * mx::GLUE_MAX_PER_THREAD)
        return MX_ERR_SHAPE;
    if (rows == 0) return MX_OK;
    DeviceInfo *d = nullptr;
    mx_status_t s = device_info(&d);
    if (s != MX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int per = (int)((cols + mx::GLUE_THREADS - 1) / mx::GLUE_THREADS);
    const unsigned g = (unsigned)rows;
    ProfScope prof(KIND_GLUE, st);
    if (per <= 4) mx::layernorm_kernel<4><<<g, mx::GLUE_THREADS, 0, st>>>(x, ldx, gamma, beta, eps, (int)cols, y, ldy);
    else if (per <= 8) mx::layernorm_kernel<8><<<g, mx::GLUE_THREADS, 0, st>>>(x, ldx, gamma, beta, eps, (int)cols, y, ldy);
    else if (per <= 16) mx::layernorm_kernel<16><<<g, mx::GLUE_THREADS, 0, st>>>(x, ldx, gamma, beta, eps, (int)cols, y, ldy);
    else mx::layernorm_kernel<32><<<g, mx::GLUE_THREADS, 0, st>>>(x, ldx, gamma, beta, eps, (int)cols, y, ldy);
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

mx_status_t mx_softmax(float *s_inout, int64_t ld, int64_t rows, int64_t cols, float scale, int causal,
                       int64_t rows_per_batch, void *stream)
{
    if (!s_inout) return MX_ERR_NULL;
    if (rows < 0 || cols <= 0 || ld < cols || cols > mx::GLUE_THREADS * mx::GLUE_MAX_PER_THREAD ||
        (causal && rows_per_batch <= 0))
        return MX_ERR_SHAPE;
    if (rows == 0) return MX_OK;
    DeviceInfo *d = nullptr;
    mx_status_t s = device_info(&d);
    if (s != MX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int per = (int)((cols + mx::GLUE_THREADS - 1) / mx::GLUE_THREADS);
    const unsigned g = (unsigned)rows;
    ProfScope prof(KIND_GLUE, st);
    if (per <= 4) mx::softmax_kernel<4><<<g, mx::GLUE_THREADS, 0, st>>>(s_inout, ld, (int)cols, scale, causal, rows_per_batch);
    else if (per <= 8) mx::softmax_kernel<8><<<g, mx::GLUE_THREADS, 0, st>>>(s_inout, ld, (int)cols, scale, causal, rows_per_batch);
    else if (per <= 16) mx::softmax_kernel<16><<<g, mx::GLUE_THREADS, 0, st>>>(s_inout, ld, (int)cols, scale, causal, rows_per_batch);
    else mx::softmax_kernel<32><<<g, mx::GLUE_THREADS, 0, st>>>(s_inout, ld, (int)cols, scale, causal, rows_per_batch);
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

mx_status_t mx_softmax_q(const float *s_in, int64_t ld, int64_t rows, int64_t cols, float scale, int causal,
                         int64_t rows_per_batch, mx_format_t fp, void *p_mant, uint8_t *p_exp, void *stream)
{
    if (!s_in || !p_mant || !p_exp) return MX_ERR_NULL;
    if (!format_1d(fp)) return MX_ERR_FORMAT;
    if (rows < 0 || cols <= 0 || ld < cols || cols > mx::GLUE_THREADS * mx::GLUE_MAX_PER_THREAD ||
        (cols % fp.block) != 0 || (causal && rows_per_batch <= 0))
        return MX_ERR_SHAPE;
    if (!aligned16(s_in) || !aligned16(p_mant) || (ld % 4) != 0) return MX_ERR_ALIGN;
    if (rows == 0) return MX_OK;
    DeviceInfo *d = nullptr;
    mx_status_t st_ = device_info(&d);
    if (st_ != MX_OK) return st_;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int per8 = (int)((cols / 8 + mx::GLUE_THREADS - 1) / mx::GLUE_THREADS);      // 1..4
    const unsigned g = (unsigned)rows;
    uint8_t *pm = static_cast<uint8_t *>(p_mant);
    ProfScope prof(KIND_GLUE, st);
#define MX_SOFTMAX_Q(P8)                                                                                         \
    do {                                                                                                         \
        if (fp.block == 16)                                                                                      \
            mx::softmax_q_kernel<P8, 16><<<g, mx::GLUE_THREADS, 0, st>>>(s_in, ld, (int)cols, scale, causal,     \
                                                                         rows_per_batch, fp.elem_bits, pm, p_exp); \
        else                                                                                                     \
            mx::softmax_q_kernel<P8, 32><<<g, mx::GLUE_THREADS, 0, st>>>(s_in, ld, (int)cols, scale, causal,     \
                                                                         rows_per_batch, fp.elem_bits, pm, p_exp); \
    } while (0)
    if (per8 <= 1) MX_SOFTMAX_Q(1);
    else if (per8 <= 2) MX_SOFTMAX_Q(2);
    else MX_SOFTMAX_Q(4);
#undef MX_SOFTMAX_Q
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

mx_status_t mx_relu_add(const float *a, const float *b, float *y, int64_t n, int relu, void *stream)
{
    if (!a || !y) return MX_ERR_NULL;
    if (n < 0) return MX_ERR_SHAPE;
    if (!aligned16(a) || !aligned16(y) || (b && !aligned16(b))) return MX_ERR_ALIGN;
    if (n == 0) return MX_OK;
    DeviceInfo *d = nullptr;
    mx_status_t s = device_info(&d);
    if (s != MX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    ProfScope prof(KIND_GLUE, st);
    mx::relu_add_kernel<<<grid_for((n + 3) / 4, mx::GLUE_THREADS, d->sm_count, 8), mx::GLUE_THREADS, 0, st>>>(a, b, y, n, relu);
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

// ---- Block Minifloat / Block Logarithm ---------------------------------------------------------
static bool alt_format_ok(const mx_alt_format_t &f)
{
    if (f.block != 16 && f.block != 32) return false;
    if (f.kind == MX_ELEM_BMF)
        return f.elem_exp_bits >= 1 && f.elem_exp_bits <= 5 && f.elem_man_bits >= 1 &&
               1 + f.elem_exp_bits + f.elem_man_bits <= 8;
    if (f.kind == MX_ELEM_BL) return f.elem_exp_bits >= 1 && f.elem_exp_bits <= 5 && f.elem_man_bits == 0;
    return false;
}
static mx::AltFormat alt_of(const mx_alt_format_t &f)
{
    return mx::AltFormat{f.kind, f.block, f.elem_exp_bits, f.elem_man_bits};
}

mx_status_t mx_alt_quantize(const void *x, mx_dtype_t dt, int64_t rows, int64_t K, int64_t ldx, mx_alt_format_t f,
                            uint8_t *codes, uint8_t *shared, uint32_t *nonfinite_count, void *stream)
{
    if (!alt_format_ok(f) || (dt != MX_F32 && dt != MX_BF16)) return MX_ERR_FORMAT;
    if (rows < 0 || K < 0 || (K % f.block) != 0 || ldx < K) return MX_ERR_SHAPE;
    if (rows == 0 || K == 0) return MX_OK;
    if (!x || !codes || !shared) return MX_ERR_NULL;
    if (!aligned16(x) || !aligned16(codes) || (ldx % 8) != 0) return MX_ERR_ALIGN;
    DeviceInfo *d = nullptr;
    mx_status_t s = device_info(&d);
    if (s != MX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t items = rows * ((K / 8 + 31) / 32);
    const int grid = grid_for(items * 32, 256, d->sm_count, 8);
    const mx::AltFormat af = alt_of(f);
    ProfScope prof(KIND_QUANTIZE, st);
    if (dt == MX_F32) {
        const float *xf = static_cast<const float *>(x);
        if (f.block == 16) MX_CUDA(launch_dep(mx::alt_quantize_kernel<float, 16>, dim3(grid), dim3(256), 0, st, xf, rows, K, ldx, af, codes, shared, nonfinite_count));
        else MX_CUDA(launch_dep(mx::alt_quantize_kernel<float, 32>, dim3(grid), dim3(256), 0, st, xf, rows, K, ldx, af, codes, shared, nonfinite_count));
    } else {
        const __nv_bfloat16 *xb = static_cast<const __nv_bfloat16 *>(x);
        if (f.block == 16) MX_CUDA(launch_dep(mx::alt_quantize_kernel<__nv_bfloat16, 16>, dim3(grid), dim3(256), 0, st, xb, rows, K, ldx, af, codes, shared, nonfinite_count));
        else MX_CUDA(launch_dep(mx::alt_quantize_kernel<__nv_bfloat16, 32>, dim3(grid), dim3(256), 0, st, xb, rows, K, ldx, af, codes, shared, nonfinite_count));
    }
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

static mx_status_t alt_decode_any(const uint8_t *codes, const uint8_t *shared, int64_t rows, int64_t K,
                                  const mx_alt_format_t &f, void *out, mx_dtype_t dt, int64_t ld_out, DeviceInfo &d,
                                  cudaStream_t st)
{
    const int grid = grid_for(rows * (K / 8), 256, d.sm_count, 8);
    const mx::AltFormat af = alt_of(f);
    ProfScope prof(KIND_DEQUANTIZE, st);
    if (dt == MX_F32)
        MX_CUDA(launch_dep(mx::alt_decode_kernel<float>, dim3(grid), dim3(256), 0, st, codes, shared, rows, K, af,
                           static_cast<float *>(out), ld_out));
    else
        MX_CUDA(launch_dep(mx::alt_decode_kernel<__nv_bfloat16>, dim3(grid), dim3(256), 0, st, codes, shared, rows, K, af,
                           static_cast<__nv_bfloat16 *>(out), ld_out));
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

mx_status_t mx_alt_dequantize(const uint8_t *codes, const uint8_t *shared, int64_t rows, int64_t K, mx_alt_format_t f,
                              void *out, mx_dtype_t dt, int64_t ld_out, void *stream)
{
    if (!codes || !shared || !out) return MX_ERR_NULL;
    if (!alt_format_ok(f) || (dt != MX_F32 && dt != MX_BF16)) return MX_ERR_FORMAT;
    if (rows < 0 || K < 0 || (K % f.block) != 0 || ld_out < K) return MX_ERR_SHAPE;
    if (!aligned16(codes) || !aligned16(out) || (ld_out % 8) != 0) return MX_ERR_ALIGN;
    if (rows == 0 || K == 0) return MX_OK;
    DeviceInfo *d = nullptr;
    mx_status_t s = device_info(&d);
    if (s != MX_OK) return s;
    return alt_decode_any(codes, shared, rows, K, f, out, dt, ld_out, *d, static_cast<cudaStream_t>(stream));
}

size_t mx_alt_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K)
{
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    return tc_operand_bytes(M, N, K);
}

mx_status_t mx_alt_gemm(const uint8_t *a_codes, const uint8_t *a_shared, mx_alt_format_t fa, const uint8_t *w_codes,
                        const uint8_t *w_shared, mx_alt_format_t fw, int64_t M, int64_t N, int64_t K, const float *bias,
                        float *y, int64_t ldy, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!a_codes || !a_shared || !w_codes || !w_shared || !y) return MX_ERR_NULL;
    if (!alt_format_ok(fa) || !alt_format_ok(fw) || fa.block != fw.block) return MX_ERR_FORMAT;
    if (M <= 0 || N <= 0 || K <= 0 || (K % fa.block) != 0 || ldy < N) return MX_ERR_SHAPE;
    if (M > INT32_MAX / 2 || N > INT32_MAX / 2 || K > INT32_MAX / 2) return MX_ERR_SHAPE;
    if (!aligned16(a_codes) || !aligned16(w_codes) || !aligned16(y) || (bias && !aligned16(bias))) return MX_ERR_ALIGN;
    if (!workspace || workspace_bytes < tc_operand_bytes(M, N, K)) return MX_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MX_ERR_ALIGN;
    DeviceInfo *d = nullptr;
    mx_status_t s = device_info(&d);
    if (s != MX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    __nv_bfloat16 *a_hat = static_cast<__nv_bfloat16 *>(workspace);
    __nv_bfloat16 *w_hat = reinterpret_cast<__nv_bfloat16 *>(static_cast<uint8_t *>(workspace) + round256((size_t)M * K * 2));
    s = alt_decode_any(a_codes, a_shared, M, K, fa, a_hat, MX_BF16, K, *d, st);
    if (s != MX_OK) return s;
    s = alt_decode_any(w_codes, w_shared, N, K, fw, w_hat, MX_BF16, K, *d, st);
    if (s != MX_OK) return s;
    return run_tc(a_hat, w_hat, M, N, K, bias, y, ldy, *d, st);
}

// ---- product without any allocation ---------------------------------------------------------
// Scratch for mx_gemm_static: a fixed array in the library's device image.  In host code the
// name below is only a handle for the runtime, never a device address; the address a kernel can
// use comes from cudaGetSymbolAddress, looked up once per device with that device current.
static __device__ __align__(256) unsigned char g_static_scratch[MX_STATIC_SCRATCH_BYTES];
static void *g_static_scratch_addr[MAX_DEVICES] = {nullptr};

mx_status_t mx_gemm_static(const void *a_mant, const uint8_t *a_exp, mx_format_t fa,
                           const void *w_mant, const uint8_t *w_exp, mx_format_t fw, int64_t M,
                           int64_t N, int64_t K, const float *bias, float *y, int64_t ldy,
                           void *stream)
{
    mx_status_t s = check_gemm_args(a_mant, a_exp, fa, w_mant, w_exp, fw, M, N, K, bias, y, ldy);
    if (s != MX_OK) return s;
    if (!a_exp) return MX_ERR_NULL;
    if (fa.block_rows != 1 || fw.block_rows != 1 || fa.packing || fw.packing) return MX_ERR_FORMAT;
    const size_t need = tc_operand_bytes(M, N, K);
    if (need > (size_t)MX_STATIC_SCRATCH_BYTES) {
        snprintf(t_cuda_error, sizeof(t_cuda_error),
                 "mx_gemm_static: M=%lld N=%lld K=%lld needs %zu bytes of scratch, the built-in array holds %zu",
                 (long long)M, (long long)N, (long long)K, need, (size_t)MX_STATIC_SCRATCH_BYTES);
        return MX_ERR_WORKSPACE;
    }
    DeviceInfo *d = nullptr;
    s = device_info(&d);
    if (s != MX_OK) return s;
    int dev = 0;
    MX_CUDA(cudaGetDevice(&dev));
    {
        std::lock_guard<std::mutex> lk(g_init_mu);
        if (!g_static_scratch_addr[dev]) {          // set-up: first call on this device
            void *p = nullptr;
            MX_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
            g_static_scratch_addr[dev] = p;
        }
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t *scratch = static_cast<uint8_t *>(g_static_scratch_addr[dev]);
    __nv_bfloat16 *a_hat = reinterpret_cast<__nv_bfloat16 *>(scratch);
    __nv_bfloat16 *w_hat = reinterpret_cast<__nv_bfloat16 *>(scratch + round256((size_t)M * K * 2));
    // Decode both operands into the scratch (every byte the product reads is written here first,
    // so nothing left by an earlier call is ever observed), then the tensor-core product.
    // Launches are issued directly: no event, no buffer and no handle is created on this path.
    mx::dequantize_kernel<__nv_bfloat16><<<grid_for(M * (K / 8), 256, d->sm_count, 16), 256, 0, st>>>(
        static_cast<const uint8_t *>(a_mant), a_exp, M, K, fa.block, fa.elem_bits, a_hat, K, dense_strides(K, fa));
    MX_CUDA(cudaGetLastError());
    mx::dequantize_kernel<__nv_bfloat16><<<grid_for(N * (K / 8), 256, d->sm_count, 16), 256, 0, st>>>(
        static_cast<const uint8_t *>(w_mant), w_exp, N, K, fw.block, fw.elem_bits, w_hat, K, dense_strides(K, fw));
    MX_CUDA(cudaGetLastError());
    TcBatch opt;
    opt.no_events = true;
    return launch_tc<128, mx::W_BF16>(a_hat, w_hat, PackedW(), M, N, K, bias, y, ldy, nullptr, *d, st, opt);
}

mx_status_t mx_profile_begin(void)
{
    std::lock_guard<std::mutex> lk(g_prof.mu);
    for (const ProfEntry &e : g_prof.entries) g_prof.pool.push_back(e);
    g_prof.entries.clear();
    g_prof.on = true;
    return MX_OK;
}

mx_status_t mx_profile_end(double *ms_per_kind, int64_t *launches_per_kind)
{
    if (!ms_per_kind || !launches_per_kind) return MX_ERR_NULL;
    std::lock_guard<std::mutex> lk(g_prof.mu);
    g_prof.on = false;
    for (int k = 0; k < MX_KERNEL_KINDS; ++k) {
        ms_per_kind[k] = 0.0;
        launches_per_kind[k] = 0;
    }
    mx_status_t rc = MX_OK;
    for (const ProfEntry &e : g_prof.entries) {
        float ms = 0.f;
        cudaError_t err = cudaEventSynchronize(e.b);
        if (err == cudaSuccess) err = cudaEventElapsedTime(&ms, e.a, e.b);
        if (err != cudaSuccess) rc = cuda_fail(err, "mx_profile_end");
        if (e.kind >= 0 && e.kind < MX_KERNEL_KINDS) {
            ms_per_kind[e.kind] += ms;
            launches_per_kind[e.kind] += 1;
        }
        g_prof.pool.push_back(e);
    }
    g_prof.entries.clear();
    return rc;
}

// One warp waits, with the library's bounded wait, on a barrier that nothing ever arrives on.
__global__ void wait_probe_kernel(uint32_t *status, uint64_t limit_ns)
{
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        mx::ptx::mbar_init(mx::ptx::smem_u32(&bar), 1);
        abort_flag = 0;
        mx::ptx::fence_mbar_init();
    }
    __syncthreads();
    const bool ok = mx::ptx::mbar_wait_bounded(mx::ptx::smem_u32(&bar), 0u, &abort_flag, limit_ns);
    if (!ok && threadIdx.x == 0) atomicOr(status, mx::STATUS_TIMEOUT_BIT);
}

mx_status_t mx_selftest_wait_expiry(uint32_t limit_us, void *stream)
{
    if (limit_us == 0 || limit_us > 100000u) return MX_ERR_SHAPE;       // at most 0.1 s
    DeviceInfo *d = nullptr;
    mx_status_t s = device_info(&d);
    if (s != MX_OK) return s;
    wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(d->status, (uint64_t)limit_us * 1000ull);
    MX_CUDA(cudaGetLastError());
    return MX_OK;
}

mx_status_t mx_poll_status(void *stream)
{
    DeviceInfo *d = nullptr;
    mx_status_t s = device_info(&d);
    if (s != MX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    MX_CUDA(cudaStreamSynchronize(st));
    uint32_t word = 0;
    MX_CUDA(cudaMemcpy(&word, d->status, sizeof(word), cudaMemcpyDeviceToHost));
    if (word != 0) {
        const uint32_t zero = 0;
        MX_CUDA(cudaMemcpy(d->status, &zero, sizeof(zero), cudaMemcpyHostToDevice));
    }
    return (word & mx::STATUS_TIMEOUT_BIT) ? MX_ERR_TIMEOUT : MX_OK;
}

}  // extern "C"
