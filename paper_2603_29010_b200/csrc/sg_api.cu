// Host side of libsolgemm: argument validation, tensor-map construction, tile-shape choice,
// launches, the Speed-of-Light calculator and the status helpers declared in include/solgemm.h.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <algorithm>
#include <vector>

#include "solgemm.h"
#include "sg_kernel.cuh"
#include "sg_variants.h"
#include "sg_transpose.cuh"
#include "sg_gemv.cuh"
#include "sg_splitk.cuh"

namespace {

using namespace sg;

// ------------------------------------------------------------------------------------------ errors
thread_local char t_err[512] = "";

sg_status_t fail(sg_status_t st, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(t_err, sizeof t_err, fmt, ap);
    va_end(ap);
    return st;
}

#define SG_CUDA(call)                                                                              \
    do {                                                                                           \
        cudaError_t e_ = (call);                                                                   \
        if (e_ != cudaSuccess) return fail(SG_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e_));  \
    } while (0)

// ------------------------------------------------------------------------------------------ per-device state
__device__ uint32_t g_status_words[8 + 64];   // 8 status words, then scratch for experimental time stamps

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
using EncodeIm2colFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const int*, const int*, cuuint32_t, cuuint32_t,
                                    const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct DeviceState {
    bool ready = false;
    sg_status_t init_status = SG_OK;
    char init_error[256] = "";
    int sm_count = 0;
    int max_pairs = 0;               // CTA pairs that can be resident at once
    uint32_t* status_dev = nullptr;  // device address of g_status_words on this device
    void* scratch = nullptr;         // caller-registered scratch for K-split tail tiles (sg_set_scratch)
    size_t scratch_bytes = 0;
};

constexpr size_t kScratchFlagBytes = 8192;     // 1024 arrival counters + 1024 consumed counters
constexpr int kScratchMaxBuffers = 1024;

constexpr int kMaxDevices = 64;
DeviceState g_dev[kMaxDevices];
std::mutex g_mutex;
EncodeTiledFn g_encode_tiled = nullptr;
EncodeIm2colFn g_encode_im2col = nullptr;
std::atomic<int64_t> g_launches{0};
std::atomic<int> g_tune_tile_n{-1}, g_tune_pair{-1}, g_tune_tail{-1};
// sg_set_option: planner overrides for measurements and tests (-1 = the planner decides / the default)
std::atomic<int64_t> g_opt[SG_OPT_COUNT_];
struct OptInit {
    OptInit() { for (auto& o : g_opt) o.store(-1); }
} g_opt_init;
inline int64_t opt(int which) { return g_opt[which].load(std::memory_order_relaxed); }
thread_local char t_last_kernel[128] = "";      // the kernel function this thread launched last (sg_last_kernel_name)
void note_kernel(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(t_last_kernel, sizeof t_last_kernel, fmt, ap);
    va_end(ap);
}
thread_local int32_t t_last_plan[6] = {0, 0, 0, 0, 0, 0};   // tile_n, cta_pair, tail split, tile-list length, first split position, grid

KernelEntry kernel_for(int bn, bool pair, int out, int epi_warps, int variant = 0) {
    switch (variant) {
        case 1: return kernel_variant_1(bn, pair, out, epi_warps);
        case 2: return kernel_variant_2(bn, pair, out, epi_warps);
        case 3: return kernel_variant_3(bn, pair, out, epi_warps);
        case 4: return kernel_variant_4(bn, pair, out, epi_warps);
        case 5: return kernel_variant_5(bn, pair, out, epi_warps);
        case 6: return kernel_variant_6(bn, pair, out, epi_warps);
        case 7: return kernel_variant_7(bn, pair, out, epi_warps);
        case 8: return kernel_variant_8(bn, pair, out, epi_warps);
        case 9: return kernel_variant_9(bn, pair, out, epi_warps);
        default: return kernel_variant_0(bn, pair, out, epi_warps);
    }
}

// transpose kernels by (input, output) type: 0 fp32, 1 bf16, 2 fp16
struct TransposeEntry {
    void (*tma)(const TransposeTmaParams);
    void (*plain)(const TransposeParams);
    int smem, ctas_per_sm;
    const char* in_name;
    const char* out_name;
};
template <typename TI, typename TO>
TransposeEntry transpose_entry_for(const char* in_name, const char* out_name) {
    return TransposeEntry{transpose_tma_kernel<TI, TO>, transpose_kernel<TI, TO>, TransposeCfg<TI, TO>::SMEM_BYTES,
                          TransposeCfg<TI, TO>::CTAS_PER_SM, in_name, out_name};
}
TransposeEntry transpose_entry(int ti, int to) {
#define SG_TR_ROW(TI, NI)                                                                                   \
    return to == 0 ? transpose_entry_for<TI, float>(NI, "float")                                            \
                   : (to == 1 ? transpose_entry_for<TI, __nv_bfloat16>(NI, "__nv_bfloat16") : transpose_entry_for<TI, __half>(NI, "__half"));
    if (ti == 0) { SG_TR_ROW(float, "float") }
    if (ti == 1) { SG_TR_ROW(__nv_bfloat16, "__nv_bfloat16") }
    SG_TR_ROW(__half, "__half")
#undef SG_TR_ROW
}
inline int transpose_type_index(int32_t dt) { return dt == SG_F32 ? 0 : (dt == SG_BF16 ? 1 : 2); }

sg_status_t device_state(DeviceState** out) {
    int dev = 0;
    SG_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return fail(SG_ERR_CUDA, "device index %d out of range", dev);
    DeviceState& d = g_dev[dev];
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!d.ready) {
        d.ready = true;
        d.init_status = SG_OK;
        auto bad = [&](sg_status_t st, const char* what, const char* detail) {
            d.init_status = st;
            snprintf(d.init_error, sizeof d.init_error, "%s: %s", what, detail);
        };
        cudaDeviceProp prop;
        cudaError_t e = cudaGetDeviceProperties(&prop, dev);
        if (e != cudaSuccess) {
            bad(SG_ERR_CUDA, "cudaGetDeviceProperties", cudaGetErrorString(e));
        } else if (prop.major != 10 || prop.minor != 0) {
            char buf[64];
            snprintf(buf, sizeof buf, "compute capability %d.%d", prop.major, prop.minor);
            bad(SG_ERR_ARCH, "this library runs on compute capability 10.0 (B200) only, found", buf);
        } else {
            d.sm_count = prop.multiProcessorCount;
            if (!g_encode_tiled) {
                cudaDriverEntryPointQueryResult q;
                void* fn = nullptr;
                e = cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &q);
                if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !fn)
                    bad(SG_ERR_CUDA, "driver entry point", "cuTensorMapEncodeTiled not found");
                g_encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
                fn = nullptr;
                e = cudaGetDriverEntryPointByVersion("cuTensorMapEncodeIm2col", &fn, 12000, cudaEnableDefault, &q);
                if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !fn)
                    bad(SG_ERR_CUDA, "driver entry point", "cuTensorMapEncodeIm2col not found");
                g_encode_im2col = reinterpret_cast<EncodeIm2colFn>(fn);
            }
            if (d.init_status == SG_OK) {
                e = cudaGetSymbolAddress(reinterpret_cast<void**>(&d.status_dev), g_status_words);
                if (e != cudaSuccess) bad(SG_ERR_CUDA, "cudaGetSymbolAddress", cudaGetErrorString(e));
            }
            const int bns[3] = {64, 128, 256};
            for (int i = 0; i < 3 && d.init_status == SG_OK; ++i)
                for (int pair = 0; pair < 2 && d.init_status == SG_OK; ++pair)
                    for (int f32 = 0; f32 < 3 && d.init_status == SG_OK; ++f32)
                        for (int ew = 4; ew <= 8 && d.init_status == SG_OK; ew += 4)
                            for (int variant = 0; variant < 10 && d.init_status == SG_OK; ++variant) {
                                if ((variant == 6 || variant == 7) && pair) continue;      // the short-A variants have no two-CTA form
                                KernelEntry k = kernel_for(bns[i], pair != 0, f32, ew, variant);
                                e = cudaFuncSetAttribute(k.fn, cudaFuncAttributeMaxDynamicSharedMemorySize, k.smem);
                                if (e != cudaSuccess) bad(SG_ERR_CUDA, "cudaFuncSetAttribute(shared memory)", cudaGetErrorString(e));
                            }
            if (d.init_status == SG_OK) {
                cudaError_t e2 = cudaSuccess;
                for (int ti = 0; ti < 3 && e2 == cudaSuccess; ++ti)
                    for (int to = 0; to < 3 && e2 == cudaSuccess; ++to) {
                        const TransposeEntry te = transpose_entry(ti, to);
                        e2 = cudaFuncSetAttribute(te.tma, cudaFuncAttributeMaxDynamicSharedMemorySize, te.smem);
                    }
                if (e2 != cudaSuccess) bad(SG_ERR_CUDA, "cudaFuncSetAttribute(transpose shared memory)", cudaGetErrorString(e2));
            }
            if (d.init_status == SG_OK) {
                // how many 2-CTA clusters fit at once (some GPCs may not pair up all of their SMs)
                KernelEntry k = kernel_for(256, true, 0, 8);
                cudaLaunchConfig_t cfg = {};
                cfg.gridDim = dim3(2 * d.sm_count);
                cfg.blockDim = dim3(k.threads);
                cfg.dynamicSmemBytes = k.smem;
                cudaLaunchAttribute attr;
                attr.id = cudaLaunchAttributeClusterDimension;
                attr.val.clusterDim.x = 2;
                attr.val.clusterDim.y = 1;
                attr.val.clusterDim.z = 1;
                cfg.attrs = &attr;
                cfg.numAttrs = 1;
                int clusters = 0;
                e = cudaOccupancyMaxActiveClusters(&clusters, k.fn, &cfg);
                if (e != cudaSuccess || clusters <= 0) {
                    cudaGetLastError();
                    clusters = d.sm_count / 2;
                }
                d.max_pairs = clusters < d.sm_count / 2 ? clusters : d.sm_count / 2;
            }
        }
    }
    if (d.init_status != SG_OK) return fail(d.init_status, "%s", d.init_error);
    *out = &d;
    return SG_OK;
}

// ------------------------------------------------------------------------------------------ tensor maps
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// 3-D tiled map over a row-major [batch][rows][inner] tensor with 128-byte swizzled boxes.
sg_status_t make_tiled_map(CUtensorMap* map, CUtensorMapDataType dt, int esize, const void* base, uint64_t inner,
                           uint64_t rows, uint64_t batch, uint64_t row_stride_elems, uint64_t batch_stride_elems,
                           uint32_t box_inner, uint32_t box_rows, const char* what,
                           CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B) {
    cuuint64_t dims[3] = {inner, rows, batch};
    cuuint64_t strides[2] = {row_stride_elems * esize, batch_stride_elems * esize};
    if (batch <= 1) strides[1] = strides[0] * (rows > 0 ? rows : 1);
    cuuint32_t box[3] = {box_inner, box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode_tiled(map, dt, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return fail(SG_ERR_CUDA, "cuTensorMapEncodeTiled(%s) failed with CUresult %d (dims %llu x %llu x %llu, strides %llu, %llu)",
                    what, static_cast<int>(r), (unsigned long long)inner, (unsigned long long)rows,
                    (unsigned long long)batch, (unsigned long long)strides[0], (unsigned long long)strides[1]);
    return SG_OK;
}

// ------------------------------------------------------------------------------------------ validation
struct Checked {
    bool f32_out;
    int esize_out;
    int out_kind;                 // kernel template value: 0 bf16, 1 fp32, 2 fp16
    bool in_f16;
    int in_fp8;                   // operand kind: 0 sixteen-bit, 1 e4m3, 2 e5m2, 3 fp32 storage read as tf32, 4 int8
    int esize_in, bk;             // bytes per input element; K elements per 128-byte stage row
    CUtensorMapDataType tm_in, tm_out;
};

sg_status_t check_common(int32_t in_dtype, int32_t out_dtype, int32_t epi, float alpha, float beta, float a0, float a1,
                         int32_t reserved, Checked* c) {
    if (in_dtype != SG_BF16 && in_dtype != SG_F16 && in_dtype != SG_FP8_E4M3 && in_dtype != SG_FP8_E5M2 && in_dtype != SG_F32 &&
        in_dtype != SG_INT8)
        return fail(SG_ERR_UNSUPPORTED, "in_dtype %d: inputs must be SG_BF16, SG_F16, SG_F32 (tf32), SG_FP8_E4M3, SG_FP8_E5M2 or SG_INT8", in_dtype);
    if (out_dtype != SG_BF16 && out_dtype != SG_F32 && out_dtype != SG_F16)
        return fail(out_dtype == SG_FP8_E4M3 || out_dtype == SG_FP8_E5M2 || out_dtype == SG_INT8 ? SG_ERR_UNSUPPORTED : SG_ERR_INVALID_ARG,
                    "out_dtype %d: outputs must be SG_BF16, SG_F16 or SG_F32", out_dtype);
    if (epi < SG_EPI_NONE || epi > SG_EPI_CLIP) return fail(SG_ERR_INVALID_ARG, "epi %d is not a sg_epilogue_t", epi);
    if (!std::isfinite(alpha) || !std::isfinite(beta)) return fail(SG_ERR_INVALID_ARG, "alpha and beta must be finite");
    if ((epi == SG_EPI_LEAKY_RELU || epi == SG_EPI_ELU) && !std::isfinite(a0)) return fail(SG_ERR_INVALID_ARG, "epi_arg0 (slope) must be finite");
    if (epi == SG_EPI_CLIP && !(a0 <= a1)) return fail(SG_ERR_INVALID_ARG, "clip needs epi_arg0 <= epi_arg1");
    if (reserved != 0) return fail(SG_ERR_INVALID_ARG, "reserved field must be 0");
    c->f32_out = (out_dtype == SG_F32);
    c->esize_out = c->f32_out ? 4 : 2;
    c->out_kind = out_dtype == SG_F32 ? 1 : (out_dtype == SG_F16 ? 2 : 0);
    c->in_f16 = (in_dtype == SG_F16);
    c->in_fp8 = in_dtype == SG_FP8_E4M3 ? 1 : (in_dtype == SG_FP8_E5M2 ? 2 : (in_dtype == SG_F32 ? 3 : (in_dtype == SG_INT8 ? 4 : 0)));
    c->esize_in = c->in_fp8 == 3 ? 4 : (c->in_fp8 ? 1 : 2);
    c->bk = 128 / c->esize_in;                      // one 128-byte swizzled row of K per stage row
    c->tm_in = c->in_fp8 == 3 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                              : (c->in_fp8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                                           : (c->in_f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16));
    c->tm_out = out_dtype == SG_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                    : (out_dtype == SG_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16);
    return SG_OK;
}

sg_status_t check_gemm_desc(const sg_gemm_desc_t* d, bool grouped, Checked* c) {
    if (!d) return fail(SG_ERR_NULL_POINTER, "desc is NULL");
    sg_status_t st = check_common(d->in_dtype, d->out_dtype, d->epi, d->alpha, d->beta, d->epi_arg0, d->epi_arg1, d->reserved, c);
    if (st != SG_OK) return st;
    if ((!grouped && d->M < 0) || d->N < 0 || d->K < 0) return fail(SG_ERR_INVALID_ARG, "M, N, K must be >= 0");
    if ((!grouped && d->M > INT32_MAX) || d->N > INT32_MAX || d->K > INT32_MAX)
        return fail(SG_ERR_UNSUPPORTED, "extents above 2^31-1 are not supported");
    if (d->layout_a != SG_ROW_MAJOR && d->layout_a != SG_COL_MAJOR) return fail(SG_ERR_INVALID_ARG, "layout_a %d is not a sg_layout_t", d->layout_a);
    if (d->layout_b != SG_ROW_MAJOR && d->layout_b != SG_COL_MAJOR) return fail(SG_ERR_INVALID_ARG, "layout_b %d is not a sg_layout_t", d->layout_b);
    const int64_t M = grouped ? 1 : d->M;
    // leading dimension >= the contiguous extent: K for a K-contiguous operand, M (resp. N) otherwise
    const int64_t a_inner = d->layout_a == SG_ROW_MAJOR ? d->K : M;
    const int64_t b_inner = d->layout_b == SG_COL_MAJOR ? d->K : d->N;
    if (d->lda < (a_inner > 1 ? a_inner : 1) && M > 0 && d->K > 0)
        return fail(SG_ERR_INVALID_ARG, "lda %lld is smaller than A's contiguous extent %lld", (long long)d->lda, (long long)a_inner);
    if (d->ldb < (b_inner > 1 ? b_inner : 1) && d->N > 0 && d->K > 0)
        return fail(SG_ERR_INVALID_ARG, "ldb %lld is smaller than B's contiguous extent %lld", (long long)d->ldb, (long long)b_inner);
    if (d->ldd < (d->N > 1 ? d->N : 1)) return fail(SG_ERR_INVALID_ARG, "ldd %lld < N %lld", (long long)d->ldd, (long long)d->N);
    if (d->beta != 0.0f && d->ldc < (d->N > 1 ? d->N : 1)) return fail(SG_ERR_INVALID_ARG, "ldc %lld < N %lld", (long long)d->ldc, (long long)d->N);
    if ((d->lda * c->esize_in) % 16 || (d->ldb * c->esize_in) % 16) return fail(SG_ERR_ALIGNMENT, "lda and ldb must be multiples of 16 bytes");
    if (c->in_fp8 && (d->layout_a != SG_ROW_MAJOR || d->layout_b != SG_COL_MAJOR))
        return fail(SG_ERR_UNSUPPORTED, "8-bit and tf32 inputs are implemented for the K-contiguous pair (A row-major, B column-major) only");
    if ((d->ldd * c->esize_out) % 16) return fail(SG_ERR_ALIGNMENT, "ldd must be a multiple of 16 bytes");
    if (d->beta != 0.0f && (d->ldc * c->esize_out) % 16) return fail(SG_ERR_ALIGNMENT, "ldc must be a multiple of 16 bytes");
    return SG_OK;
}

sg_status_t check_ptrs(const void* A, const void* B, const void* C, const void* bias, const void* D, int64_t K, float beta,
                       int32_t epi, const char* who) {
    if (!D) return fail(SG_ERR_NULL_POINTER, "%s: D is NULL", who);
    if (K > 0 && (!A || !B)) return fail(SG_ERR_NULL_POINTER, "%s: A or B is NULL", who);
    if (beta != 0.0f && !C) return fail(SG_ERR_NULL_POINTER, "%s: beta != 0 needs C", who);
    if (epi == SG_EPI_BIAS && !bias) return fail(SG_ERR_NULL_POINTER, "%s: SG_EPI_BIAS needs bias", who);
    if (!aligned16(D) || (K > 0 && (!aligned16(A) || !aligned16(B))) || (beta != 0.0f && !aligned16(C)))
        return fail(SG_ERR_ALIGNMENT, "%s: base pointers must be 16-byte aligned", who);
    if (bias && (reinterpret_cast<uintptr_t>(bias) & 1u)) return fail(SG_ERR_ALIGNMENT, "%s: bias must be 2-byte aligned", who);
    return SG_OK;
}

// ------------------------------------------------------------------------------------------ tile shape
struct Shape {
    int bn;
    bool pair;
    int epi_warps;
};

// Tile-shape choice.  Cost = waves of tiles over the SMs x tile width x a measured per-area factor
// (wide two-CTA tiles move the fewest operand bytes per FLOP; narrow tiles are bound by shared-memory
// and L2 reads, not by the tensor pipe).  Two-CTA tiles pay a fixed cluster set-up cost, so they are
// used only when the K loop is long and there is at least one full wave of them.
// Modelled cost of sharing one tile's K loop between ks work items through the scratch (us): every part parks its
// partial sums and finishes a share of the columns from the other parts' (measured: conv weight gradient and
// skinny long-K products).
inline double ksplit_exchange_us(int64_t ks) { return ks > 1 ? 6.0 + 0.5 * static_cast<double>(ks - 1) : 0.0; }
// The same for the two-pass form (every part parks all its sums and exits; a second kernel adds them up): flat in ks.
constexpr int kTwoPassMinKb = 4;           // k-blocks per part at least
constexpr double kGemvSmallMacs = 160.0e6;         // products of at most this many multiply-adds run on the warp-level MMA
                                                    // kernel when its CTAs all fit on the GPU at once (see try_gemv)
// Modelled time (us) of a two-pass K split with `ks` parts per tile: the longer of the parts' tensor time and of streaming
// the operands from HBM (a CTA pulls about 38 GB/s, all of them together about 5.5 TB/s), plus a fixed 3 us for the
// second kernel, plus writing and re-reading the parked sums.  Fitted to 256 x 256 x {8192 .. 131072}, 512 x 512 x 16384,
// 1024 x 1024 x 8192 and 128 x 4096 x 16384 with the number of parts forced to 2 .. 74.
inline double two_pass_us(int64_t tiles, int64_t ks, int bn, bool pair, int64_t num_kb, double t_kb, double t_fixed,
                          double operand_bytes) {
    const double ctas = static_cast<double>(tiles * ks * (pair ? 2 : 1));
    const double rate = std::min(5.5e6, ctas * 0.038e6);                     // bytes per us
    const double parked = static_cast<double>(tiles * ks) * (pair ? 2.0 : 1.0) * 128.0 * bn * 4.0;
    return std::max(t_kb * static_cast<double>((num_kb + ks - 1) / ks) + t_fixed, operand_bytes / rate) + 3.0 + 2.0 * parked / 8.0e6;
}
constexpr double kUsPerKBlock = 0.25;      // one 64-deep k-block of a 128 x 256 tile per SM

bool ksplit_allowed(const DeviceState& d) {
    const int tail_mode = g_tune_tail.load();
    return d.scratch != nullptr && tail_mode != 0 && tail_mode != 1 && opt(SG_OPT_TAIL_KSPLIT) != 0;
}

// What choose_shape needs to know for problems bound by memory traffic rather than by the tensor pipe: operand and
// output element sizes and whether the activation is one of the transcendental ones (epi < 0: terms not applied).
struct MemHint {
    int epi = -1;
    int esize_in = 2;
    int esize_out = 2;
    double operand_bytes = 0.0;      // bytes of A and B as stored (0: (rows + N) K esize_in per problem)
};

inline bool heavy_activation(int epi) {
    return epi == SG_EPI_GELU || epi == SG_EPI_SILU || epi == SG_EPI_SIGMOID || epi == SG_EPI_TANH || epi == SG_EPI_MISH ||
           epi == SG_EPI_ELU;
}

Shape choose_shape(const DeviceState& d, const std::vector<int64_t>& rows_per_problem, int64_t batch_mult, int64_t N,
                   int64_t K, int min_b_rows = 1, MemHint mem = MemHint{}, bool two_pass_ok = false) {
    const int force_bn = g_tune_tile_n.load();
    const int force_pair = g_tune_pair.load();
    const int bns[3] = {256, 128, 64};
    // [pair][bn index]: time per output area relative to two-CTA 256-wide tiles, measured on the 4096^3 GEMM and the
    // benchmark convolution with every tiling forced (narrow tiles re-read the A panel for fewer columns and are bound
    // by operand traffic)
    const double factor[2][3] = {{1.18, 1.56, 2.90}, {1.00, 1.50, 3.30}};
    auto tiles_for = [&](int tile_m, int bn) {
        int64_t tiles = 0;
        for (int64_t r : rows_per_problem) tiles += ((r + tile_m - 1) / tile_m) * ((N + bn - 1) / bn);
        return tiles * batch_mult;
    };
    int64_t max_rows = 0;
    for (int64_t r : rows_per_problem) max_rows = r > max_rows ? r : max_rows;
    const int64_t num_kb = (K + 63) / 64;
    const bool can_split = ksplit_allowed(d) && num_kb >= 2;
    const bool full_wave_of_pairs = d.max_pairs > 0 && tiles_for(256, 256) >= d.max_pairs;
    // pairs: for long K loops, when there is a whole wave of 256 x 256 tiles -- or, for problems with less than a wave
    // of tiles whose K loop can be shared between SMs, when a pair's 256 rows are not mostly padding
    const bool pair_only = K >= 1024 && full_wave_of_pairs;
    const bool pair_possible = pair_only || (K >= 1024 && d.max_pairs > 0 && can_split && max_rows > 128);
    // Eight epilogue warps drain an accumulator twice as fast; that pays when the K loop is too short to hide
    // the epilogue (short K, heavy activations) and costs a little when it is long.
    const int64_t forced_ew = opt(SG_OPT_EPI_WARPS);
    const int epi_warps = (forced_ew == 4 || forced_ew == 8) ? static_cast<int>(forced_ew) : (K <= 1024 ? 8 : 4);
    Shape best{256, false, epi_warps};
    double best_cost = 1e300;
    for (int pi = 0; pi < 2; ++pi) {
        if (force_pair >= 0 ? pi != force_pair : (pi == 1 ? !pair_possible : pair_only)) continue;
        for (int bi = 0; bi < 3; ++bi) {
            const int bn = bns[bi];
            if (force_bn > 0 && bn != force_bn) continue;
            if (bn / (pi ? 2 : 1) < min_b_rows) continue;       // an N-contiguous B is loaded in blocks of 64 rows
            const int64_t tiles = tiles_for(pi ? 256 : 128, bn);
            const int64_t slots = pi ? d.max_pairs : d.sm_count;
            if (slots <= 0) continue;
            const int64_t waves = (tiles + slots - 1) / slots;
            // time of one k-block of a tile on its SM(s), and the K-independent part of a tile (pipeline fill,
            // epilogue drain), which weighs more when K is short
            const double t_kb = kUsPerKBlock * bn / 256.0 * factor[pi][bi];
            const double t_fixed = kUsPerKBlock * bn / 256.0 * 96.0 / 64.0;
            double cost = static_cast<double>(waves) * (t_kb * static_cast<double>(num_kb > 0 ? num_kb : 1) + t_fixed);
            // One row of tiles (M <= 128: a weight matrix streamed past a few activations): what bounds the time is
            // how many of B's bytes are in flight -- `active` CTAs x stages x the B share of a stage -- against the
            // memory latency under load (~1.9 us); the A share of every stage is mostly padding.  Parts of a K-split
            // tile stream at ~4.7 TB/s at best and start ~2 us later.  Fitted to 8..128 x {2048..14336} x {4096..14336}
            // with every tiling forced, e.g. 16 x 8192 x 8192: 256-wide tiles in 4 column slices 45 us, in 4 K ranges
            // 36 us, 128-wide 35 us, 64-wide 31 us.
            auto stream_us = [&](int64_t active, bool k_ranges) {
                // with at most 64 (32) rows only that many rows of A are loaded per stage, and up to 16 stages fit
                const double a_bytes = k_ranges || max_rows > 64 ? 16384.0 : (max_rows > 32 ? 8192.0 : 4096.0);
                const double stages = std::min(a_bytes < 16384.0 ? 16.0 : 8.0, std::floor(192.0 * 1024.0 / (a_bytes + 128.0 * bn)));
                const double in_flight = static_cast<double>(std::min<int64_t>(active, slots)) * stages * 128.0 * bn;
                const double b_bytes = static_cast<double>(N) * static_cast<double>(K) * mem.esize_in * static_cast<double>(batch_mult) *
                                       static_cast<double>(rows_per_problem.size());
                return b_bytes / std::min(k_ranges ? 4.7e6 : 7.0e6, in_flight / 1.9) + (k_ranges ? 2.0 : 0.0);
            };
            const bool one_tile_row = mem.epi >= 0 && !pi && max_rows <= 128;
            if (one_tile_row) cost = std::max(cost, stream_us(tiles, false));
            if (can_split && tiles * 2 <= slots) {
                // less than half a wave: plan_tail may cut every tile's K loop into ranges run by different SMs
                const bool two_pass = two_pass_ok && opt(SG_OPT_TWO_PASS_SPLIT_K) != 0;
                int64_t ks_max = slots / tiles;
                if (!two_pass && ks_max > 16) ks_max = 16;
                if (ks_max > num_kb / (two_pass ? kTwoPassMinKb : 1)) ks_max = num_kb / (two_pass ? kTwoPassMinKb : 1);
                double operand_bytes = mem.operand_bytes;
                if (operand_bytes <= 0.0) {
                    for (int64_t r : rows_per_problem) operand_bytes += static_cast<double>(r + N) * static_cast<double>(K) * mem.esize_in;
                    operand_bytes *= static_cast<double>(batch_mult);
                }
                for (int64_t ks = 2; ks <= ks_max; ++ks) {
                    double t;
                    if (two_pass) {
                        t = two_pass_us(tiles, ks, bn, pi != 0, num_kb, t_kb, t_fixed, operand_bytes);
                    } else {
                        t = t_kb * static_cast<double>((num_kb + ks - 1) / ks) + t_fixed + ksplit_exchange_us(ks);
                        if (one_tile_row) t = std::max(t, stream_us(tiles * ks, true) + ksplit_exchange_us(ks));
                    }
                    if (t < cost) cost = t;
                }
            }
            if (mem.epi >= 0 && !pi && tiles_for(128, 256) >= d.sm_count) {
                // Memory-bound problems with at least a wave of tiles (short K, many small problems): the time is the traffic -- each operand once
                // from HBM (~7 TB/s), every tile's operand panels from the L2 (~14 TB/s over all SMs) -- plus what
                // cannot overlap with it: the last tile's epilogue (measured: 1.7 us for a 128 x 256 tile under a
                // transcendental activation, 0.5 us otherwise) and ~0.2 us per tile an SM walks through.  Narrower
                // tiles shorten that end; measured on 128 problems of 256 x 256 x 512 with GELU: 18.8 us with 256-wide
                // tiles, 17.7 us with 128-wide ones (19.8 with 64: L2 traffic), and the reverse order without activation.
                double hbm_bytes = 0.0;
                for (int64_t r : rows_per_problem)
                    hbm_bytes += static_cast<double>(r + N) * static_cast<double>(K) * mem.esize_in +
                                 static_cast<double>(r) * static_cast<double>(N) * mem.esize_out;
                hbm_bytes *= static_cast<double>(batch_mult);
                const double l2_bytes = static_cast<double>(tiles) * (128.0 + bn) * static_cast<double>(K) * mem.esize_in;
                const double t_traffic = std::max(hbm_bytes / 7.0e6, l2_bytes / 14.0e6);
                const double t_end = (heavy_activation(mem.epi) ? 1.7 : 0.5) * bn / 256.0 + 0.2 * static_cast<double>(waves);
                if (t_traffic + t_end > cost) cost = t_traffic + t_end;
            }
            if (cost < best_cost) {
                best_cost = cost;
                best = Shape{bn, pi != 0, epi_warps};
            }
        }
    }
    return best;
}

// Wave quantisation: when the tiles do not fill a whole number of waves, the tiles of the last wave are
// cut into `split` column slices so that the idle SMs of that wave take a share.  Narrow slices cost more
// per output area (same factors as in choose_shape), so a split is used only when it shortens the tail.
// Sets p->split_begin, p->split and p->num_tiles (the length of the tile list) from the full-width count.
void plan_tail(const DeviceState& d, Shape& s, int64_t full_tiles, Params* p, int min_b_rows = 1, bool allow_ksplit = true,
               bool two_pass_ok = false, double operand_bytes = 0.0) {
    const int64_t slots = s.pair ? d.max_pairs : d.sm_count;
    const double factor[2][3] = {{1.00, 1.10, 1.60}, {1.00, 1.26, 2.57}};   // relative to the full width: [pair][log2(split)]
    int best_split = 1, best_ksplit = 1, early_ks = 0;
    const int64_t rem = full_tiles % slots;
    const int forced = static_cast<int>(opt(SG_OPT_TAIL_SPLIT));      // 1, 2 or 4
    const int env_k = static_cast<int>(opt(SG_OPT_TAIL_KSPLIT));      // 0 = off, >= 2: that many K ranges
    const int tail_mode = g_tune_tail.load();      // -1 auto, 0 none, 1 column slices, 2 K ranges
    const int forced_k = tail_mode == 2 ? 4 : (tail_mode == 0 || tail_mode == 1 ? 0 : env_k);
    if (rem != 0 && tail_mode != 0) {
        double best = 1.0;      // cost of the unsplit tail wave, in units of one full-width tile
        for (int k = 1; k <= 2; ++k) {
            const int split = 1 << k;
            if (s.bn / split < 64 || s.bn / split / (s.pair ? 2 : 1) < min_b_rows) break;
            const int64_t waves = (rem * split + slots - 1) / slots;
            const double cost = static_cast<double>(waves) / split * factor[s.pair ? 1 : 0][k];
            if (cost < best - 0.05) {
                best = cost;
                best_split = split;
            }
        }
        if (forced == 1 || forced == 2 || forced == 4) {
            best_split = (s.bn / forced >= 64 && s.bn / forced / (s.pair ? 2 : 1) >= min_b_rows) ? forced : 1;
            best = 0.9;
        }
        // K ranges through the registered scratch: ksplit SM groups share one tail tile's K loop; every part parks its
        // fp32 partial sums and finishes a share of the tile's columns from all parts' sums (this is also what serves
        // skinny problems with a long K: when there is less than one wave of tiles, every tile is a "tail" tile).
        // A k-block of a tile takes about 0.25 us; a split is planned when it saves a fifth of the tail's time.
        if (allow_ksplit && d.scratch && forced_k != 0 && p->num_kb >= 2 && rem * 2 <= slots) {
            int64_t ks_max = slots / rem;
            if (ks_max > 16) ks_max = 16;
            if (ks_max > p->num_kb) ks_max = p->num_kb;
            const size_t buf_bytes = static_cast<size_t>(s.pair ? 2 : 1) * 128 * s.bn * sizeof(float);
            size_t max_buffers = d.scratch_bytes > kScratchFlagBytes ? (d.scratch_bytes - kScratchFlagBytes) / buf_bytes : 0;
            if (max_buffers > static_cast<size_t>(kScratchMaxBuffers)) max_buffers = kScratchMaxBuffers;
            while (ks_max >= 2 && static_cast<size_t>(rem * ks_max) > max_buffers) --ks_max;      // every part parks a tile
            int64_t ks = 0;
            if (forced_k >= 2) {
                ks = forced_k < ks_max ? forced_k : ks_max;
            } else if (rem <= kScratchMaxBuffers) {
                const double t_tile = kUsPerKBlock * p->num_kb * best;      // us: the tail as planned so far (whole or sliced)
                double best_time = t_tile * 0.8;
                for (int64_t k = 2; k <= ks_max; ++k) {
                    const double t = kUsPerKBlock * p->num_kb / static_cast<double>(k) + ksplit_exchange_us(k);
                    if (t < best_time) {
                        best_time = t;
                        ks = k;
                    }
                }
            }
            if (ks >= 2 && rem <= kScratchMaxBuffers) {
                best_ksplit = static_cast<int>(ks);
                best_split = 1;
            }
        }
        // K ranges with early donors (see decode_tile): with at least one whole wave before the partial one, the tiles
        // of the last wave are cut into ks K ranges of which all but the last run FIRST, on CTAs of their own, and park
        // their sums; the CTA that runs the last range at the very end has them put into its accumulator beforehand, by
        // epilogue warps that would otherwise idle.  Nobody waits for a peer and nothing is exchanged after the last MMA,
        // so the tail costs 1 / ks of a tile -- against column slices, which are bound by operand traffic and take
        // almost a whole tile's time however narrow they are.  (Needs two whole waves: the accumulator is filled while
        // the CTA works on the item before the last.)
        const int early_opt = static_cast<int>(opt(SG_OPT_EARLY_DONORS));      // -1 auto, 0 off, k >= 2: k ranges
        const int64_t waves = full_tiles / slots;
        if (allow_ksplit && d.scratch && tail_mode != 0 && tail_mode != 1 && early_opt != 0 && forced_k <= 0 && waves >= 2 &&
            rem * 2 <= slots && p->num_kb >= 16) {
            const size_t buf_bytes = static_cast<size_t>(s.pair ? 2 : 1) * 128 * s.bn * sizeof(float);
            size_t max_buffers = d.scratch_bytes > kScratchFlagBytes ? (d.scratch_bytes - kScratchFlagBytes) / buf_bytes : 0;
            if (max_buffers > static_cast<size_t>(kScratchMaxBuffers)) max_buffers = kScratchMaxBuffers;
            int64_t ks_max = slots / rem;
            if (ks_max > 4) ks_max = 4;
            while (ks_max >= 2 && (p->num_kb / ks_max < 8 || static_cast<size_t>(rem * ks_max) > max_buffers)) --ks_max;
            const double t_tile = kUsPerKBlock * p->num_kb * (s.bn / 256.0) * (s.pair ? 1.5 : 1.18);      // one whole tile, us
            double best_time = t_tile * (best_ksplit > 1 ? 1.0 / best_ksplit : best) + (best_ksplit > 1 ? ksplit_exchange_us(best_ksplit) : 0.0);
            int64_t ks = 0;
            // Measured against column slices (the kernel variant that keeps the K-range code in runs its tiles 2 - 3 %
            // slower than the plain one, which eats the better balance on short K loops): 4096 x 4096 x 8192 188.7 ->
            // 184.2 us, 2560 x 4096 x 8192 123.2 -> 120.1, 4096^3 93.4 -> 93.8, 4096 x 4096 x 2048 49.2 -> 49.9.  So the
            // planner takes this road for K loops of 96 k-blocks or more only.
            for (int64_t k = 2; k <= ks_max && p->num_kb >= 96; ++k) {
                const double t = t_tile / static_cast<double>(k) + 0.5;
                if (t < best_time * 0.9) {
                    best_time = t;
                    ks = k;
                }
            }
            if (early_opt >= 2 && early_opt <= ks_max) ks = early_opt;
            if (ks >= 2 && rem <= kScratchMaxBuffers) {
                early_ks = static_cast<int>(ks);
                best_ksplit = early_ks;
                best_split = 1;
            }
        }
    }
    // raster bands: keep a band's A panels (band_m x TILE_M rows x K) within about 32 MB of L2
    const int64_t panel_bytes = static_cast<int64_t>(s.pair ? 256 : 128) * (p->K > 0 ? p->K : 1) * 2;
    int64_t band = (32ll << 20) / panel_bytes;
    const int64_t forced_band = opt(SG_OPT_BAND_M);
    if (forced_band > 0) band = forced_band;
    p->band_m = static_cast<int32_t>(band < 1 ? 1 : (band > 4096 ? 4096 : band));
    const int parts = best_ksplit > 1 ? best_ksplit : best_split;
    p->split = best_split;
    p->ksplit = best_ksplit;
    p->split_begin = static_cast<int32_t>(parts > 1 ? full_tiles - rem : full_tiles);
    p->num_tiles = static_cast<int32_t>(parts > 1 ? full_tiles - rem + rem * parts : full_tiles);
    p->sk_early = 0;
    p->sk_park_all = 0;
    // Two-pass K split: fewer tiles than half the SMs (a skinny problem with a long K loop).  Every tile's K loop is cut
    // into as many ranges as there are SMs to go round; each part parks its sums and exits, a second kernel adds them up
    // and runs the epilogue (launch() enqueues it).  No part waits for another, and the cost of the exchange does not grow
    // with the number of parts.
    if (two_pass_ok && allow_ksplit && d.scratch && opt(SG_OPT_TWO_PASS_SPLIT_K) != 0 && tail_mode != 0 && tail_mode != 1 &&
        tail_mode != 2 && forced_k <= 0 && full_tiles * 2 <= slots && p->num_kb >= 2 * kTwoPassMinKb) {
        const size_t buf_bytes = static_cast<size_t>(s.pair ? 2 : 1) * 128 * s.bn * sizeof(float);
        size_t max_buffers = d.scratch_bytes > kScratchFlagBytes ? (d.scratch_bytes - kScratchFlagBytes) / buf_bytes : 0;
        int64_t ks_max = slots / full_tiles;
        if (ks_max > p->num_kb / kTwoPassMinKb) ks_max = p->num_kb / kTwoPassMinKb;
        while (ks_max >= 2 && static_cast<size_t>(full_tiles * ks_max) > max_buffers) --ks_max;
        if (operand_bytes <= 0.0)
            operand_bytes = (static_cast<double>(p->M) + p->N) * static_cast<double>(p->K) * (128.0 / p->bk_elems) *
                            static_cast<double>(p->batch > 0 ? p->batch : 1);
        const int pi = s.pair ? 1 : 0, bi = s.bn == 256 ? 0 : (s.bn == 128 ? 1 : 2);
        const double shape_factor[2][3] = {{1.18, 1.56, 2.90}, {1.00, 1.50, 3.30}};      // as in choose_shape
        const double t_kb = kUsPerKBlock * s.bn / 256.0 * shape_factor[pi][bi];
        const double t_fixed = kUsPerKBlock * s.bn / 256.0 * 96.0 / 64.0;
        // the unsplit launch as the yardstick: a split has to be a tenth faster to be taken
        const double ctas1 = static_cast<double>(full_tiles * (s.pair ? 2 : 1));
        int64_t ks = 0;
        double best_t = 0.9 * std::max(t_kb * static_cast<double>(p->num_kb) + t_fixed, operand_bytes / std::min(5.5e6, ctas1 * 0.038e6));
        for (int64_t k = 2; k <= ks_max; ++k) {
            const double t = two_pass_us(full_tiles, k, s.bn, s.pair, p->num_kb, t_kb, t_fixed, operand_bytes);
            if (t < best_t) {
                best_t = t;
                ks = k;
            }
        }
        const int64_t forced_parts = opt(SG_OPT_TWO_PASS_SPLIT_K);
        if (forced_parts >= 2) ks = forced_parts < ks_max ? forced_parts : ks_max;
        if (ks >= 2) {
            p->sk_park_all = 1;
            p->split = 1;
            p->ksplit = static_cast<int32_t>(ks);
            p->split_begin = 0;
            p->num_tiles = static_cast<int32_t>(full_tiles * ks);
            p->band_m = INT32_MAX;      // tiles in plain column-major order: the second pass decodes them the same way
            p->sk_partials = reinterpret_cast<float*>(static_cast<uint8_t*>(d.scratch) + kScratchFlagBytes);
            p->sk_flags = static_cast<uint32_t*>(d.scratch);
            p->sk_consumed_off = kScratchMaxBuffers;
            p->sk_arrivals = s.epi_warps * (s.pair ? 2 : 1);
            return;
        }
    }
    if (early_ks > 1) {
        // list: R (ks - 1) donor parts, the whole waves' tiles, R owner parts
        p->sk_early = static_cast<int32_t>(rem * (early_ks - 1));
        p->split_begin = static_cast<int32_t>(p->sk_early + (full_tiles - rem));
        p->num_tiles = static_cast<int32_t>(p->split_begin + rem);
    }
    if (best_ksplit > 1) {
        p->sk_flags = static_cast<uint32_t*>(d.scratch);
        p->sk_consumed_off = kScratchMaxBuffers;
        p->sk_partials = reinterpret_cast<float*>(static_cast<uint8_t*>(d.scratch) + kScratchFlagBytes);
        p->sk_arrivals = s.epi_warps * (s.pair ? 2 : 1);
    }
}

// Magic numbers of sg::fast_div for a divisor 1 <= d < 2^31 (exact for dividends below 2^31: with
// 2^sh = q d + r and mul = q + 1, n mul / 2^sh exceeds n / d by less than 2^-ceil(log2 d) <= 1 / d).
FastDiv make_fastdiv(int64_t d) {
    if (d < 1) d = 1;
    int l = 0;
    while ((int64_t{1} << l) < d) ++l;
    FastDiv f;
    f.sh = static_cast<uint32_t>(31 + l);
    f.mul = static_cast<uint32_t>((uint64_t{1} << f.sh) / static_cast<uint64_t>(d) + 1);
    return f;
}

sg_status_t launch(const DeviceState& d, const Shape& s, int out_kind, const Params& p_in, cudaStream_t stream) {
    Params p = p_in;
    p.split_log2 = p.split >= 4 ? 2 : (p.split >= 2 ? 1 : 0);
    if (p.mode != MODE_GROUPED && p.tiles_m > 0 && p.band_m > p.tiles_m) p.band_m = p.tiles_m;   // same walk, one divisor
    p.div_per = make_fastdiv(static_cast<int64_t>(p.tiles_m) * p.tiles_n);
    p.div_band_tiles = make_fastdiv(static_cast<int64_t>(p.band_m) * p.tiles_n);
    p.div_band_m = make_fastdiv(p.band_m);
    p.div_pq = make_fastdiv(static_cast<int64_t>(p.P) * p.Q);
    p.div_q = make_fastdiv(p.Q);
    // plain dense, convolution-forward and grouped problems run the variant of the kernel specialised for them
    // (same instructions, the other modes and options compiled out)
    const bool no_lean = opt(SG_OPT_GENERAL_KERNEL) > 0;
    int variant = 0;
    if (!no_lean && !p.in_fp8) {
        const bool plain_k = !p.a_mn_major && !p.b_mn_major && !p.d_remap && p.nphases <= 1;
        const bool plain = plain_k && p.ksplit <= 1;
        if (p.mode == MODE_DENSE && plain) variant = p.ex_any ? 4 : (p.a_rows == 64 ? 6 : (p.a_rows == 32 ? 7 : 1));
        else if (p.mode == MODE_CONV && plain && !p.ex_any) variant = 2;
        else if (p.mode == MODE_DENSE && plain_k && !p.ex_any && p.a_rows == 128) variant = 8;      // dense with K ranges
        else if (p.mode == MODE_CONV && plain_k && !p.ex_any) variant = 9;                          // convolution with K ranges
        else if (p.mode == MODE_GROUPED && plain && !p.ex_any) variant = 3;
        else if (p.mode == MODE_CONV && !p.a_mn_major && p.b_mn_major && p.ksplit <= 1 && !p.ex_any) variant = 5;
    }
    // L2 warm-up at kernel entry: measured to pay for short K loops, where a launch is mostly its start and its end
    // (128 problems of 256 x 256 x 512: 17.6 -> 17.1 us with 4 k-blocks), and to cost a little on long ones
    // (4096^3: 94.6 -> 95.3 us with 8)
    if (p.warm_kb < 0) p.warm_kb = p.num_kb <= 16 ? 4 : 0;
    KernelEntry k = kernel_for(s.bn, s.pair, out_kind, s.epi_warps, variant);
    const int ctas_per_tile = s.pair ? 2 : 1;
    const int slots = s.pair ? d.max_pairs : d.sm_count;
    const int tiles = p.num_tiles < slots ? p.num_tiles : slots;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(tiles * ctas_per_tile);
    cfg.blockDim = dim3(k.threads);
    cfg.dynamicSmemBytes = k.smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = ctas_per_tile;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // programmatic dependent launch: this kernel's set-up may overlap the previous kernel's tail (the kernel
    // itself waits for that kernel before it touches global memory)
    const bool pdl = !(opt(SG_OPT_NO_PDL) > 0);
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 2 : 1;
    SG_CUDA(cudaLaunchKernelEx(&cfg, k.fn, p));
    g_launches.fetch_add(1);
    note_kernel("sg::contract_kernel<%d, %s, %d, %d, %d>", s.bn, s.pair ? "true" : "false", out_kind, s.epi_warps, variant);
    if (p.sk_park_all) {
        // second pass of a two-pass K split: add the parked parts up and run the epilogue
        SplitKReduceParams r;
        memset(&r, 0, sizeof r);
        r.partials = p.sk_partials;
        r.status = p.status;
        r.nparts = p.ksplit;
        r.kctas = ctas_per_tile;
        r.bn = s.bn;
        r.tiles_m = p.tiles_m;
        r.tiles_n = p.tiles_n;
        r.M = p.M;
        r.N = p.N;
        r.batch = p.batch;
        r.D = p.D;
        r.C = p.C;
        r.bias = p.bias;
        r.ldd = p.ldd; r.strideD = p.strideD; r.ldc = p.ldc; r.strideC = p.strideC; r.strideBias = p.strideBias;
        r.alpha = p.alpha; r.beta = p.beta; r.epi_arg0 = p.epi_arg0; r.epi_arg1 = p.epi_arg1;
        r.epi = p.epi;
        r.in_f16 = p.in_f16;
        r.bias_f32 = p.in_fp8 == 3 ? 1 : 0;
        const int ch = out_kind == 1 ? 32 : 64;
        const int64_t full_tiles = static_cast<int64_t>(p.num_tiles) / p.ksplit;
        cudaLaunchConfig_t rc = {};
        r.pw = p.ksplit <= 4 ? 1 : (p.ksplit <= 8 ? 2 : (p.ksplit <= 16 ? 4 : 8));
        const int64_t forced_pw = opt(SG_OPT_SPLIT_K_REDUCE_WARPS);
        if (forced_pw == 1 || forced_pw == 2 || forced_pw == 4 || forced_pw == 8) r.pw = static_cast<int32_t>(forced_pw);
        rc.gridDim = dim3(static_cast<unsigned>(full_tiles * ctas_per_tile * (s.bn / ch) * 4 * r.pw));
        rc.blockDim = dim3(256);
        rc.stream = stream;
        rc.attrs = &attr[1];
        rc.numAttrs = pdl ? 1 : 0;
        using ReduceFn = void (*)(const SplitKReduceParams);
        static const ReduceFn reduce_fns[3][4] = {
            {splitk_reduce_kernel<0, 1>, splitk_reduce_kernel<0, 2>, splitk_reduce_kernel<0, 4>, splitk_reduce_kernel<0, 8>},
            {splitk_reduce_kernel<1, 1>, splitk_reduce_kernel<1, 2>, splitk_reduce_kernel<1, 4>, splitk_reduce_kernel<1, 8>},
            {splitk_reduce_kernel<2, 1>, splitk_reduce_kernel<2, 2>, splitk_reduce_kernel<2, 4>, splitk_reduce_kernel<2, 8>}};
        const int pwi = r.pw == 1 ? 0 : (r.pw == 2 ? 1 : (r.pw == 4 ? 2 : 3));
        cudaError_t e = cudaLaunchKernelEx(&rc, reduce_fns[out_kind][pwi], r);
        if (e != cudaSuccess) return fail(SG_ERR_CUDA, "split-K second pass launch: %s", cudaGetErrorString(e));
        g_launches.fetch_add(1);
    }
    t_last_plan[0] = s.bn;
    t_last_plan[1] = s.pair ? 1 : 0;
    t_last_plan[2] = p.ksplit > 1 ? -p.ksplit : p.split;
    t_last_plan[3] = p.num_tiles;
    t_last_plan[4] = p.split_begin;
    t_last_plan[5] = tiles * ctas_per_tile;
    return SG_OK;
}

constexpr uint64_t kWaitLimitNs = 2000000000ull;   // 2 s: far beyond any legitimate wait inside one launch

void base_params(Params* p, const DeviceState& d, float alpha, float beta, int32_t epi, float a0, float a1) {
    memset(p, 0, sizeof *p);
    p->alpha = alpha;
    p->beta = beta;
    p->epi = epi;
    p->epi_arg0 = a0;
    p->epi_arg1 = a1;
    p->status = d.status_dev;
    const int64_t warm = opt(SG_OPT_L2_WARM_KBLOCKS);
    p->warm_kb = warm >= 0 ? static_cast<int32_t>(warm > 64 ? 64 : warm) : -1;      // -1: launch() decides from the K loop's length
    const int64_t limit = opt(SG_OPT_WAIT_LIMIT_NS);
    p->timeout_ns = limit > 0 ? static_cast<uint64_t>(limit) : kWaitLimitNs;
}

// Validates the optional extended epilogue chain and copies it into the kernel parameters.
sg_status_t apply_ex(Params* p, const sg_epilogue_ex_t* ex, int64_t N, int esize_out, const char* who) {
    if (!ex) return SG_OK;
    if (ex->reserved0 != 0) return fail(SG_ERR_INVALID_ARG, "%s: ex->reserved0 must be 0", who);
    if (!std::isfinite(ex->post_scale)) return fail(SG_ERR_INVALID_ARG, "%s: post_scale must be finite", who);
    if ((reinterpret_cast<uintptr_t>(ex->row_scale) | reinterpret_cast<uintptr_t>(ex->row_bias)) % 4)
        return fail(SG_ERR_ALIGNMENT, "%s: row_scale and row_bias must be 4-byte aligned", who);
    if (reinterpret_cast<uintptr_t>(ex->col_scale) % 16) return fail(SG_ERR_ALIGNMENT, "%s: col_scale must be 16-byte aligned", who);
    if (ex->aux_load) {
        if (ex->ld_aux_load < N) return fail(SG_ERR_INVALID_ARG, "%s: ld_aux_load smaller than N", who);
        if (reinterpret_cast<uintptr_t>(ex->aux_load) % 16 || (ex->ld_aux_load * esize_out) % 16)
            return fail(SG_ERR_ALIGNMENT, "%s: aux_load base and leading dimension must be multiples of 16 bytes", who);
    }
    if (ex->aux_store) {
        if (ex->ld_aux_store < N) return fail(SG_ERR_INVALID_ARG, "%s: ld_aux_store smaller than N", who);
        if (reinterpret_cast<uintptr_t>(ex->aux_store) % 16 || (ex->ld_aux_store * esize_out) % 16)
            return fail(SG_ERR_ALIGNMENT, "%s: aux_store base and leading dimension must be multiples of 16 bytes", who);
    }
    p->row_scale = static_cast<const float*>(ex->row_scale);
    p->col_scale = static_cast<const float*>(ex->col_scale);
    p->row_bias = static_cast<const float*>(ex->row_bias);
    p->post_scale = ex->post_scale;
    p->aux_load = ex->aux_load;
    p->ld_aux_load = ex->ld_aux_load;
    p->aux_store = ex->aux_store;
    p->ld_aux_store = ex->ld_aux_store;
    p->ex_any = (ex->row_scale || ex->col_scale || ex->row_bias || ex->aux_load || ex->aux_store || ex->post_scale != 1.0f) ? 1 : 0;
    return SG_OK;
}

sg_status_t run_dense(const sg_gemm_desc_t* desc, int64_t batch, int64_t sA, int64_t sB, int64_t sC, int64_t sD,
                      int64_t sBias, const void* A, const void* B, const void* C, const void* bias, void* D,
                      void* stream, const char* who, const sg_epilogue_ex_t* ex = nullptr) {
    Checked c;
    sg_status_t st = check_gemm_desc(desc, false, &c);
    if (st != SG_OK) return st;
    if (batch < 0) return fail(SG_ERR_INVALID_ARG, "%s: batch must be >= 0", who);
    if (batch > 65535 * 16) return fail(SG_ERR_UNSUPPORTED, "%s: batch too large", who);
    if (desc->M == 0 || desc->N == 0 || batch == 0) return SG_OK;
    st = check_ptrs(A, B, C, bias, D, desc->K, desc->beta, desc->epi, who);
    if (st != SG_OK) return st;
    if (c.in_fp8 == 3 && bias && (reinterpret_cast<uintptr_t>(bias) & 3u))
        return fail(SG_ERR_ALIGNMENT, "%s: an fp32 bias must be 4-byte aligned", who);
    bool ex_any = false;
    {
        Params scratch_params;          // the chain's rules are checked before any device is touched
        scratch_params.ex_any = 0;
        st = apply_ex(&scratch_params, ex, desc->N, c.esize_out, who);
        if (st != SG_OK) return st;
        ex_any = ex != nullptr && scratch_params.ex_any != 0;
    }
    if (batch > 1) {
        if (sA < 0 || sB < 0 || sC < 0 || sD < 0 || sBias < 0) return fail(SG_ERR_INVALID_ARG, "%s: negative batch stride", who);
        if ((sA * c.esize_in) % 16 || (sB * c.esize_in) % 16 || (sD * c.esize_out) % 16 || (desc->beta != 0.0f && (sC * c.esize_out) % 16))
            return fail(SG_ERR_ALIGNMENT, "%s: batch strides must be multiples of 16 bytes", who);
        if (sD < (desc->M - 1) * desc->ldd + desc->N) return fail(SG_ERR_INVALID_ARG, "%s: strideD smaller than one output", who);
    }
    DeviceState* d = nullptr;
    st = device_state(&d);
    if (st != SG_OK) return st;

    Params p;
    base_params(&p, *d, desc->alpha, desc->beta, desc->epi, desc->epi_arg0, desc->epi_arg1);
    p.in_f16 = c.in_f16 ? 1 : 0;
    p.in_fp8 = c.in_fp8;
    p.bk_elems = c.bk;
    const int min_b_rows = desc->layout_b == SG_ROW_MAJOR ? 64 : 1;
    Shape s = choose_shape(*d, std::vector<int64_t>{desc->M}, batch, desc->N, desc->K, min_b_rows,
                           MemHint{desc->epi, c.esize_in, c.esize_out}, !ex_any);
    const int tile_m = s.pair ? 256 : 128;
    p.mode = MODE_DENSE;
    p.a_mn_major = desc->layout_a == SG_COL_MAJOR ? 1 : 0;
    p.b_mn_major = desc->layout_b == SG_ROW_MAJOR ? 1 : 0;
    p.M = static_cast<int32_t>(desc->M);
    p.N = static_cast<int32_t>(desc->N);
    p.K = static_cast<int32_t>(desc->K);
    p.batch = static_cast<int32_t>(batch);
    p.tiles_m = static_cast<int32_t>((desc->M + tile_m - 1) / tile_m);
    p.tiles_n = static_cast<int32_t>((desc->N + s.bn - 1) / s.bn);
    const int64_t tiles = static_cast<int64_t>(p.tiles_m) * p.tiles_n * batch;
    if (tiles > INT32_MAX / 4) return fail(SG_ERR_UNSUPPORTED, "%s: too many tiles", who);
    p.num_kb = static_cast<int32_t>((desc->K + c.bk - 1) / c.bk);
    plan_tail(*d, s, tiles, &p, min_b_rows, true, !ex_any);
    st = apply_ex(&p, ex, desc->N, c.esize_out, who);
    if (st != SG_OK) return st;
    // a few rows against a large matrix: load only 32 or 64 rows of A per stage (kernel variants 6 and 7), which
    // leaves room for more stages of B
    const bool no_short_a = opt(SG_OPT_NO_SHORT_A) > 0;
    p.a_rows = 128;
    if (!no_short_a && !s.pair && !p.in_fp8 && !p.a_mn_major && !p.b_mn_major && p.ksplit <= 1 && !p.ex_any && desc->M <= 64)
        p.a_rows = desc->M <= 32 ? 32 : 64;
    p.bias = bias;
    p.C = desc->beta != 0.0f ? C : nullptr;
    p.ldc = desc->ldc;
    p.strideC = sC;
    p.strideBias = sBias;
    p.D = D;
    p.ldd = desc->ldd;
    p.strideD = sD;
    if (desc->K > 0) {
        // K-contiguous operand: boxes of 64 k x tile rows.  M/N-contiguous operand (column-major A, row-major B):
        // the map is over [k][rows] and every load is a box of 64 rows x 64 k.
        if (p.a_mn_major)
            st = make_tiled_map(&p.tmA, c.tm_in, c.esize_in, A, desc->M, desc->K, batch, desc->lda, sA, 64, 64, "A");
        else
            st = make_tiled_map(&p.tmA, c.tm_in, c.esize_in, A, desc->K, desc->M, batch, desc->lda, sA, c.bk, p.a_rows, "A");
        if (st != SG_OK) return st;
        if (p.b_mn_major) {
            st = make_tiled_map(&p.tmB, c.tm_in, c.esize_in, B, desc->N, desc->K, batch, desc->ldb, sB, 64, 64, "B");
            p.tmB2 = p.tmB;
        } else {
            st = make_tiled_map(&p.tmB, c.tm_in, c.esize_in, B, desc->K, desc->N, batch, desc->ldb, sB, c.bk,
                                s.pair ? s.bn / 2 : s.bn, "B");
            if (st != SG_OK) return st;
            st = make_tiled_map(&p.tmB2, c.tm_in, c.esize_in, B, desc->K, desc->N, batch, desc->ldb, sB, c.bk,
                                (s.pair ? s.bn / 2 : s.bn) / p.split, "B (narrow)");
        }
        if (st != SG_OK) return st;
    }
    st = make_tiled_map(&p.tmD, c.tm_out, c.esize_out, D,
                        desc->N, desc->M, batch, desc->ldd, sD, c.f32_out ? 32 : 64, 32, "D");
    if (st != SG_OK) return st;
    if (desc->K == 0) { p.tmA = p.tmD; p.tmB = p.tmD; p.tmB2 = p.tmD; }   // never used for loads; keeps the prefetch harmless
    return launch(*d, s, c.out_kind, p, static_cast<cudaStream_t>(stream));
}

// ------------------------------------------------------------------------------------------ grouped
struct GroupedLayout {
    size_t off_maps, off_tile_start, off_M, off_bias, off_C, off_D, total;
};

size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

GroupedLayout grouped_layout(int32_t groups) {
    GroupedLayout L;
    size_t o = 0;
    L.off_maps = o;        o = round_up(o + static_cast<size_t>(groups) * 4 * sizeof(CUtensorMap), 128);
    L.off_tile_start = o;  o = round_up(o + (static_cast<size_t>(groups) + 1) * 4, 128);
    L.off_M = o;           o = round_up(o + static_cast<size_t>(groups) * 4, 128);
    L.off_bias = o;        o = round_up(o + static_cast<size_t>(groups) * 8, 128);
    L.off_C = o;           o = round_up(o + static_cast<size_t>(groups) * 8, 128);
    L.off_D = o;           o = round_up(o + static_cast<size_t>(groups) * 8, 128);
    L.total = o;
    return L;
}

// Copies a block of host bytes that travels in the kernel's parameter space into device memory,
// so that the table reaches the workspace in stream order without a staging allocation.
constexpr int kBlobBytes = 3840;
struct Blob {
    uint8_t bytes[kBlobBytes];
};
__global__ void scatter_blob_kernel(const __grid_constant__ Blob blob, uint8_t* dst, int n) {
    const uint32_t* src = reinterpret_cast<const uint32_t*>(blob.bytes);
    uint32_t* out = reinterpret_cast<uint32_t*>(dst);
    for (int i = threadIdx.x; i < n / 4; i += blockDim.x) out[i] = src[i];
}

sg_status_t upload(const std::vector<uint8_t>& host, void* dev, cudaStream_t stream) {
    for (size_t off = 0; off < host.size(); off += kBlobBytes) {
        Blob b;
        const size_t n = host.size() - off < static_cast<size_t>(kBlobBytes) ? host.size() - off : kBlobBytes;
        memcpy(b.bytes, host.data() + off, n);
        scatter_blob_kernel<<<1, 256, 0, stream>>>(b, static_cast<uint8_t*>(dev) + off, static_cast<int>(round_up(n, 4)));
        SG_CUDA(cudaGetLastError());
        g_launches.fetch_add(1);
    }
    return SG_OK;
}

// ------------------------------------------------------------------------------------------ matrix-vector products
// A GEMM with N <= 8 (the matrix is A) or M <= 8 (the matrix is B; fp32 inputs: 4) whose matrix is K-contiguous and whose vectors are
// contiguous runs as a stream over the matrix (sg_gemv.cuh) instead of through the tensor-core tiles.  *taken is false
// when the call does not have that form (the general path then validates and runs it).
template <typename T>
cudaError_t launch_gemv(const GemvParams& gp, int rb, int ctas, cudaStream_t stream) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(static_cast<unsigned>(ctas), 1, 1);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(gp.ksplit);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;      // (the kernel waits for its predecessor itself)
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = opt(SG_OPT_NO_PDL) > 0 ? 1 : 2;
    const int nv = gp.nvec <= 1 ? 1 : (gp.nvec == 2 ? 2 : 4);
#define SG_GEMV_CASE(RB_)                                                             \
    case RB_:                                                                         \
        return nv == 1   ? cudaLaunchKernelEx(&cfg, gemv_kernel<T, RB_, 1>, gp)       \
               : nv == 2 ? cudaLaunchKernelEx(&cfg, gemv_kernel<T, RB_, 2>, gp)       \
                         : cudaLaunchKernelEx(&cfg, gemv_kernel<T, RB_, 4>, gp);
    switch (rb) {
        SG_GEMV_CASE(4)
        SG_GEMV_CASE(2)
        default:
            SG_GEMV_CASE(1)
    }
#undef SG_GEMV_CASE
}

sg_status_t try_gemv(const sg_gemm_desc_t* desc, const void* A, const void* B, const void* C, const void* bias, void* D,
                     void* stream, bool* taken) {
    *taken = false;
    if (!desc || desc->K < 1 || desc->K > INT32_MAX || desc->M < 1 || desc->N < 1) return SG_OK;
    if (opt(SG_OPT_NO_GEMV) > 0) return SG_OK;      // tests: the same product through the tiles
    // up to 32 vectors of 16-bit inputs (four of fp32); the matrix is the operand with more rows
    if (desc->in_dtype != SG_BF16 && desc->in_dtype != SG_F16 && desc->in_dtype != SG_F32) return SG_OK;
    const int es = desc->in_dtype == SG_F32 ? 4 : 2;
    const bool no_mma = opt(SG_OPT_GEMV_NO_MMA) > 0;      // FMA kernel only (<= 4 vectors)
    // More than eight vectors (16-bit operands, K % 8 == 0) run on the same warp-level MMA kernel in GROUPS of 8, 16 or 32
    // vectors along the grid: a CTA takes 16 rows of the operand with more rows ("the matrix") and one group of rows of
    // the other, straight from the L2 into MMA fragments -- one memory round trip, no tensor-memory allocation, no
    // barrier set-up, no staging, no TMA store -- and the CTAs that share 16 rows of the matrix are neighbours in launch
    // order.  That has less start and end than the tiles and, with groups of eight, as many loads of the matrix in
    // flight as the plain matrix-vector form; it pays as long as all CTAs are resident at once (4, 3 or 2 per SM for
    // groups of 8, 16 or 32: registers), beyond which the tiles' operand reuse wins.  Measured against the tiles (us):
    //   nine to 32 rows against a matrix, groups of 8: 9 x 4096 x 4096 10.2 / 19.3, 16 x 4096 x 4096 10.2 / 14.6,
    //   24 x 3072 x 3072 7.9 / 12.2, 32 x 2048 x 2048 5.7 / 10.0, 24 x 2048 x 4096 8.4 / 11.9, 32 x 1024 x 8192 9.9 / 11.3,
    //   16 x 1024 x 1024 2.9 / 6.0 -- but (more CTAs than fit) 32 x 4096 x 4096 15.4 / 15.2, 16 x 8192 x 4096 17.9 / 16.5,
    //   20 x 8192 x 2048 13.4 / 10.2, 16 x 8192 x 8192 31.5 / 28.6;
    //   small products, the smallest group size that fits: 256^3 2.7-2.9 / 3.6, 128^3 1.8 / 3.2, 384^3 3.4 / 4.1,
    //   256 x 256 x 1024 3.9-4.1 / 6.5, 256 x 256 x 2048 5.1 / 7.9, 384 x 384 x 1024 4.6 / 6.5, 64 x 64 x 4096 4.0 / 7.0,
    //   512 x 64 x 512 2.5 / 4.5 -- but 400^3 5.4 / 4.5, 512^3 6.5 / 4.5, 512 x 512 x 128 5.2 / 3.3, 256 x 1024 x 256
    //   6.5 / 3.7 (more CTAs than fit) and 256 x 256 x 4096 11.6 / 10.4, 160 x 160 x 8192 12.3 / 9.6 (long K: taken up to
    //   160 M multiply-adds; SG_OPT_GEMV_SMALL_LOG2 pins that limit and lifts the residency rule).
    // A tile shape forced through sg_set_tuning keeps a product on the tiles; SG_OPT_GEMV_MAX_VECTORS > 0 restores the
    // plain limit on the number of vectors and nothing else.
    const bool small_forced = opt(SG_OPT_GEMV_SMALL_LOG2) >= 0;
    const double small_macs = small_forced ? std::ldexp(1.0, static_cast<int>(std::min<int64_t>(40, opt(SG_OPT_GEMV_SMALL_LOG2)))) : kGemvSmallMacs;
    const bool groups_ok = es == 2 && !no_mma && desc->K % 8 == 0 && opt(SG_OPT_GEMV_MAX_VECTORS) <= 0 &&
                           g_tune_tile_n.load() <= 0 && g_tune_pair.load() < 0;
    const int64_t few = std::min(desc->M, desc->N), many = std::max(desc->M, desc->N);
    int group_blocks = 0;            // 1, 2 or 4 blocks of eight vectors per CTA when the grouped form is taken
    if (groups_ok && few > 8) {
        const bool is_small = static_cast<double>(desc->M) * static_cast<double>(desc->N) * static_cast<double>(desc->K) <= small_macs;
        const bool few_rows = few <= 32 && static_cast<double>(many) * static_cast<double>(desc->K) * es <= 48.0e6;
        DeviceState* ds = nullptr;
        if ((is_small || few_rows) && device_state(&ds) == SG_OK && ds) {
            const int64_t row_blocks = (many + 15) / 16;
            const int per_sm[3] = {4, 3, 2};
            // (groups of 32 only with the 32-byte row pieces: with 16-byte pieces they measured slower than the tiles)
            const bool wide_ok = desc->K % 16 == 0 && (desc->lda * 2) % 32 == 0 && (desc->ldb * 2) % 32 == 0;
            // Which group size, where several fit: groups of eight keep the most loads in flight (long K loops, few
            // CTAs); with more than two CTAs per SM of them and a short K loop larger groups are quicker -- fewer CTAs,
            // less re-reading (256^3: 2.72 us in groups of 32, 2.90 in groups of 8; 256 x 256 x 2048: 5.8 against 5.1).
            const bool small_first = row_blocks * ((few + 7) / 8) <= 2 * static_cast<int64_t>(ds->sm_count) || desc->K > 1024;
            for (int i = 0; i < 3 && !group_blocks; ++i) {
                const int b = small_first ? i : 2 - i;
                if (!is_small && b > 0) continue;        // a few rows against a matrix: groups of eight or the tiles
                if (b == 2 && !wide_ok && !small_forced) continue;
                const int64_t ctas = row_blocks * ((few + (8 << b) - 1) / (8 << b));
                if (ctas <= per_sm[b] * static_cast<int64_t>(ds->sm_count) || (small_forced && is_small && b == 2)) group_blocks = 1 << b;
            }
        }
    }
    const bool grouped = group_blocks > 0;
    const int64_t plain_vec = (es == 2 && !no_mma && desc->K % 8 == 0) ? (opt(SG_OPT_GEMV_MAX_VECTORS) > 0 ? std::max<int64_t>(4, std::min<int64_t>(32, opt(SG_OPT_GEMV_MAX_VECTORS))) : 8) : 4;
    const bool mat_a = grouped ? desc->M >= desc->N : (desc->N <= plain_vec && desc->M >= desc->N);
    if (!grouped && !mat_a && desc->M > plain_vec) return SG_OK;
    // the matrix K-contiguous, the vectors contiguous (a K x 1 row-major B with ldb = 1 is as good as a column-major one)
    const bool a_kc = desc->layout_a == SG_ROW_MAJOR, b_kc = desc->layout_b == SG_COL_MAJOR;
    const void* W = mat_a ? A : B;
    const void* x = mat_a ? B : A;
    const int64_t ld = mat_a ? desc->lda : desc->ldb;
    const int64_t R = mat_a ? desc->M : desc->N;
    const int64_t nvec = mat_a ? desc->N : desc->M;
    const int64_t x_stride = mat_a ? desc->ldb : desc->lda;
    if (mat_a ? !(a_kc && (b_kc || (nvec == 1 && desc->ldb == 1))) : !(b_kc && (a_kc || (nvec == 1 && desc->lda == 1)))) return SG_OK;
    if (R > INT32_MAX || ld < desc->K || (ld * es) % 16 || !W || !x || !aligned16(W) || !aligned16(x)) return SG_OK;
    if (nvec > 1 && (x_stride < desc->K || (x_stride * es) % 16)) return SG_OK;
    *taken = true;

    Checked c;
    sg_status_t st = check_common(desc->in_dtype, desc->out_dtype, desc->epi, desc->alpha, desc->beta, desc->epi_arg0,
                                  desc->epi_arg1, desc->reserved, &c);
    if (st != SG_OK) return st;
    if (desc->layout_a != SG_ROW_MAJOR && desc->layout_a != SG_COL_MAJOR) return fail(SG_ERR_INVALID_ARG, "layout_a %d is not a sg_layout_t", desc->layout_a);
    if (desc->layout_b != SG_ROW_MAJOR && desc->layout_b != SG_COL_MAJOR) return fail(SG_ERR_INVALID_ARG, "layout_b %d is not a sg_layout_t", desc->layout_b);
    if (!D) return fail(SG_ERR_NULL_POINTER, "sg_gemm: D is NULL");
    if (desc->beta != 0.0f && !C) return fail(SG_ERR_NULL_POINTER, "sg_gemm: beta != 0 needs C");
    if (desc->epi == SG_EPI_BIAS && !bias) return fail(SG_ERR_NULL_POINTER, "sg_gemm: SG_EPI_BIAS needs bias");
    if (desc->ldd < desc->N) return fail(SG_ERR_INVALID_ARG, "ldd %lld < N %lld", (long long)desc->ldd, (long long)desc->N);
    if (desc->beta != 0.0f && desc->ldc < desc->N) return fail(SG_ERR_INVALID_ARG, "ldc %lld < N %lld", (long long)desc->ldc, (long long)desc->N);
    const uintptr_t out_mask = static_cast<uintptr_t>(c.esize_out - 1), in_mask = static_cast<uintptr_t>(es - 1);
    if ((reinterpret_cast<uintptr_t>(D) & out_mask) || (desc->beta != 0.0f && (reinterpret_cast<uintptr_t>(C) & out_mask)) ||
        (bias && (reinterpret_cast<uintptr_t>(bias) & in_mask)))
        return fail(SG_ERR_ALIGNMENT, "sg_gemm: D, C and bias must be aligned to their element size");
    DeviceState* d = nullptr;
    st = device_state(&d);
    if (st != SG_OK) return st;

    GemvParams gp;
    memset(&gp, 0, sizeof gp);
    gp.W = W;
    gp.x = x;
    gp.C = desc->beta != 0.0f ? C : nullptr;
    gp.bias = bias;
    gp.D = D;
    gp.status = d->status_dev;
    gp.ld = ld;
    gp.x_stride = x_stride;
    gp.c_row_stride = mat_a ? desc->ldc : 1;
    gp.c_vec_stride = mat_a ? 1 : desc->ldc;
    gp.d_row_stride = mat_a ? desc->ldd : 1;
    gp.d_vec_stride = mat_a ? 1 : desc->ldd;
    gp.R = static_cast<int32_t>(R);
    gp.K = static_cast<int32_t>(desc->K);
    gp.nvec = static_cast<int32_t>(nvec);
    gp.bias_row_stride = mat_a ? 0 : 1;
    gp.bias_vec_stride = mat_a ? 1 : 0;
    gp.out_kind = c.out_kind;
    gp.epi = desc->epi;
    gp.alpha = desc->alpha;
    gp.beta = desc->beta;
    gp.a0 = desc->epi_arg0;
    gp.a1 = desc->epi_arg1;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const int64_t want = 2 * static_cast<int64_t>(d->sm_count);
    if (es == 2 && !no_mma && desc->K % 8 == 0 && nvec >= 2) {
        // two to 32 vectors: warp-level MMAs, 16 rows per CTA, K ranges in units of 256 elements (one step of
        // the CTA's eight warps), at least four steps per warp and rank
        const int64_t blocks = (R + 15) / 16;
        const int64_t ks_max = std::max<int64_t>(1, std::min<int64_t>(8, desc->K / 1024));
        // K ranges only until there are two CTAs per SM: more (to even out the 16-row units over the SMs) measured
        // slower (8192 x 8192: 30 -> 33 us)
        const int64_t want_mma = 2 * static_cast<int64_t>(d->sm_count);
        // blocks of eight vectors per CTA: the grouped form's choice; else (a pinned vector limit) as few as hold them all
        int nvb = grouped ? (group_blocks == 1 ? 0 : (group_blocks == 2 ? 1 : 2)) : (nvec <= 8 ? 0 : (nvec <= 16 ? 1 : 2));
        if (opt(SG_OPT_GEMV_VECTOR_BLOCKS) == 1 || opt(SG_OPT_GEMV_VECTOR_BLOCKS) == 2 || opt(SG_OPT_GEMV_VECTOR_BLOCKS) == 4)
            nvb = opt(SG_OPT_GEMV_VECTOR_BLOCKS) == 1 ? 0 : (opt(SG_OPT_GEMV_VECTOR_BLOCKS) == 2 ? 1 : 2);
        const int64_t vgroups = (nvec + (8 << nvb) - 1) / (8 << nvb);
        int64_t ks = 1;
        if (vgroups > 1) {
            // several groups: K ranges only while all CTAs stay resident at once
            const int64_t resident = (nvb == 0 ? 4 : (nvb == 1 ? 3 : 2)) * static_cast<int64_t>(d->sm_count);
            while (ks < 8 && ks * 2 <= ks_max && blocks * vgroups * ks * 2 <= resident) ks *= 2;
        } else {
            while (ks < 8 && ks * 2 <= ks_max && blocks * ks < want_mma) ks *= 2;
        }
        const bool no_wide = opt(SG_OPT_GEMV_NO_WIDE) > 0;
        const bool wide = !no_wide && desc->K % 16 == 0 && (ld * 2) % 32 == 0 && (x_stride * 2) % 32 == 0 &&
                          reinterpret_cast<uintptr_t>(W) % 32 == 0 && reinterpret_cast<uintptr_t>(x) % 32 == 0;
        const int64_t unit = wide ? 512 : 256;      // K elements per step of the CTA's eight warps
        int64_t kchunk = (desc->K + ks - 1) / ks;
        kchunk = (kchunk + unit - 1) / unit * unit;
        ks = (desc->K + kchunk - 1) / kchunk;
        gp.kchunk = static_cast<int32_t>(kchunk);
        gp.ksplit = static_cast<int32_t>(ks);
        const int64_t ctas = blocks * ks;
        if (ctas > INT32_MAX) return fail(SG_ERR_UNSUPPORTED, "sg_gemm: too many rows for the matrix-vector path");
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof cfg);
        if (vgroups > 65535 || (vgroups > 1 && blocks > 65535))
            return fail(SG_ERR_UNSUPPORTED, "sg_gemm: too many vectors or rows for the matrix-vector path");
        cfg.gridDim = vgroups > 1 ? dim3(static_cast<unsigned>(ks), static_cast<unsigned>(vgroups), static_cast<unsigned>(blocks))
                                  : dim3(static_cast<unsigned>(ctas), 1, 1);
        cfg.blockDim = dim3(256, 1, 1);
        cfg.stream = cs;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = static_cast<unsigned>(ks);
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // (the kernel waits for its predecessor itself)
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = opt(SG_OPT_NO_PDL) > 0 ? 1 : 2;
        using GemvMmaFn = void (*)(const GemvParams);
        static const GemvMmaFn table[2][2][3] = {
            {{gemv_mma_kernel<__nv_bfloat16, false, 1>, gemv_mma_kernel<__nv_bfloat16, false, 2>, gemv_mma_kernel<__nv_bfloat16, false, 4>},
             {gemv_mma_kernel<__nv_bfloat16, true, 1>, gemv_mma_kernel<__nv_bfloat16, true, 2>, gemv_mma_kernel<__nv_bfloat16, true, 4>}},
            {{gemv_mma_kernel<__half, false, 1>, gemv_mma_kernel<__half, false, 2>, gemv_mma_kernel<__half, false, 4>},
             {gemv_mma_kernel<__half, true, 1>, gemv_mma_kernel<__half, true, 2>, gemv_mma_kernel<__half, true, 4>}}};
        cudaError_t e = cudaLaunchKernelEx(&cfg, table[desc->in_dtype == SG_F16 ? 1 : 0][wide ? 1 : 0][nvb], gp);
        if (e != cudaSuccess) return fail(SG_ERR_CUDA, "matrix-vector (MMA) kernel launch: %s", cudaGetErrorString(e));
        g_launches.fetch_add(1);
        note_kernel("sg::gemv_mma_kernel<%s, %s, %d>", desc->in_dtype == SG_F16 ? "__half" : "__nv_bfloat16", wide ? "true" : "false",
                    1 << nvb);
        t_last_plan[0] = 0;
        t_last_plan[1] = 0;
        t_last_plan[2] = -static_cast<int32_t>(ks);
        t_last_plan[3] = 16;
        t_last_plan[4] = 0;
        t_last_plan[5] = static_cast<int32_t>(ctas * vgroups);
        return SG_OK;
    }
    // Geometry: at least two CTAs per SM where the problem has that much work; K ranges (CTAs of one cluster, at
    // most 8) when the rows alone do not give that many, each range at least two sweeps of the 256 threads.
    const int64_t sweep = 256 * (16 / es);
    const int64_t ks_max = std::max<int64_t>(1, std::min<int64_t>(8, desc->K / (2 * sweep)));
    const int64_t forced_rb = opt(SG_OPT_GEMV_ROWS);    // 1, 2, 4
    int rb = (forced_rb == 1 || forced_rb == 2 || forced_rb == 4) ? static_cast<int>(forced_rb) : 4;
    int64_t ks = 1;
    for (;; rb >>= 1) {
        const int64_t blocks = (R + rb - 1) / rb;
        ks = std::min<int64_t>(ks_max, std::max<int64_t>(1, (want + blocks - 1) / blocks));
        if (blocks * ks >= want || rb == 1 || forced_rb > 0) break;
    }
    int64_t kchunk = (desc->K + ks - 1) / ks;
    kchunk = (kchunk + sweep - 1) / sweep * sweep;
    ks = (desc->K + kchunk - 1) / kchunk;
    gp.kchunk = static_cast<int32_t>(kchunk);
    gp.ksplit = static_cast<int32_t>(ks);
    const int64_t ctas = (R + rb - 1) / rb * ks;
    if (ctas > INT32_MAX) return fail(SG_ERR_UNSUPPORTED, "sg_gemm: too many rows for the matrix-vector path");
    cudaError_t e = desc->in_dtype == SG_F32   ? launch_gemv<float>(gp, rb, static_cast<int>(ctas), cs)
                    : desc->in_dtype == SG_F16 ? launch_gemv<__half>(gp, rb, static_cast<int>(ctas), cs)
                                               : launch_gemv<__nv_bfloat16>(gp, rb, static_cast<int>(ctas), cs);
    if (e != cudaSuccess) return fail(SG_ERR_CUDA, "matrix-vector kernel launch: %s", cudaGetErrorString(e));
    g_launches.fetch_add(1);
    note_kernel("sg::gemv_kernel<%s, %d, %d>", desc->in_dtype == SG_F32 ? "float" : (desc->in_dtype == SG_F16 ? "__half" : "__nv_bfloat16"),
                rb, static_cast<int>(nvec <= 1 ? 1 : (nvec == 2 ? 2 : 4)));
    t_last_plan[0] = 0;              // no tensor-core tiles: rows per CTA and K ranges instead
    t_last_plan[1] = 0;
    t_last_plan[2] = -static_cast<int32_t>(ks);
    t_last_plan[3] = rb;
    t_last_plan[4] = 0;
    t_last_plan[5] = static_cast<int32_t>(ctas);
    return SG_OK;
}


}  // namespace

// ============================================================================================ C ABI
extern "C" {

const char* sg_status_string(sg_status_t s) {
    switch (s) {
        case SG_OK: return "SG_OK";
        case SG_ERR_INVALID_ARG: return "SG_ERR_INVALID_ARG";
        case SG_ERR_NULL_POINTER: return "SG_ERR_NULL_POINTER";
        case SG_ERR_ALIGNMENT: return "SG_ERR_ALIGNMENT";
        case SG_ERR_UNSUPPORTED: return "SG_ERR_UNSUPPORTED";
        case SG_ERR_ARCH: return "SG_ERR_ARCH";
        case SG_ERR_WORKSPACE: return "SG_ERR_WORKSPACE";
        case SG_ERR_CUDA: return "SG_ERR_CUDA";
        case SG_ERR_TIMEOUT: return "SG_ERR_TIMEOUT";
    }
    return "SG_ERR_UNKNOWN";
}

const char* sg_last_error(void) { return t_err; }

int64_t sg_launch_count(void) { return g_launches.load(); }

const char* sg_last_kernel_name(void) { return t_last_kernel; }

sg_status_t sg_set_option(int32_t option, int64_t value) {
    if (option < 0 || option >= SG_OPT_COUNT_) return fail(SG_ERR_INVALID_ARG, "sg_set_option: option %d is not a sg_option_t", option);
    if (value < -1) return fail(SG_ERR_INVALID_ARG, "sg_set_option: value must be >= -1");
    g_opt[option].store(value);
    return SG_OK;
}

sg_status_t sg_test_set_status_word(uint32_t value, void* cuda_stream) {
    DeviceState* d = nullptr;
    sg_status_t st = device_state(&d);
    if (st != SG_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    SG_CUDA(cudaMemcpyAsync(d->status_dev, &value, sizeof value, cudaMemcpyHostToDevice, stream));
    SG_CUDA(cudaStreamSynchronize(stream));
    return SG_OK;
}

#ifdef SG_DEBUG_STAMPS
// Diagnostic builds only (-DSG_DEBUG_STAMPS, never the product library, hence not in solgemm.h): choose the CTA that
// records time stamps in later launches, and copy out the 32 time-stamp words it recorded in the last one.
sg_status_t sg_debug_select_cta(uint32_t cta) {
    DeviceState* d = nullptr;
    sg_status_t st = device_state(&d);
    if (st != SG_OK) return st;
    const uint64_t v = cta;
    SG_CUDA(cudaDeviceSynchronize());
    SG_CUDA(cudaMemcpy(reinterpret_cast<uint64_t*>(d->status_dev + 8) + 31, &v, sizeof v, cudaMemcpyHostToDevice));
    return SG_OK;
}
sg_status_t sg_debug_stamps(uint64_t* out32) {
    DeviceState* d = nullptr;
    sg_status_t st = device_state(&d);
    if (st != SG_OK) return st;
    SG_CUDA(cudaDeviceSynchronize());
    SG_CUDA(cudaMemcpy(out32, d->status_dev + 8, 32 * sizeof(uint64_t), cudaMemcpyDeviceToHost));
    return SG_OK;
}
#endif

sg_status_t sg_set_scratch(void* scratch_dev, size_t bytes) {
    DeviceState* d = nullptr;
    sg_status_t st = device_state(&d);
    if (st != SG_OK) return st;
    if (!scratch_dev || bytes == 0) {
        d->scratch = nullptr;
        d->scratch_bytes = 0;
        return SG_OK;
    }
    if (reinterpret_cast<uintptr_t>(scratch_dev) & 255u) return fail(SG_ERR_WORKSPACE, "sg_set_scratch: scratch must be 256-byte aligned");
    if (bytes < kScratchFlagBytes + (1u << 20)) return fail(SG_ERR_WORKSPACE, "sg_set_scratch: at least %zu bytes are needed", kScratchFlagBytes + (1u << 20));
    SG_CUDA(cudaMemset(scratch_dev, 0, kScratchFlagBytes));      // counters start at zero (synchronous)
    d->scratch = scratch_dev;
    d->scratch_bytes = bytes;
    return SG_OK;
}

sg_status_t sg_last_launch_plan(int32_t* plan6) {
    if (!plan6) return fail(SG_ERR_NULL_POINTER, "plan6 is NULL");
    for (int i = 0; i < 6; ++i) plan6[i] = t_last_plan[i];
    return SG_OK;
}

sg_status_t sg_set_tuning(int32_t tile_n, int32_t cta_pair) {
    if (tile_n != -1 && tile_n != 64 && tile_n != 128 && tile_n != 256) return fail(SG_ERR_INVALID_ARG, "tile_n must be -1, 64, 128 or 256");
    if (cta_pair < -1 || cta_pair > 1) return fail(SG_ERR_INVALID_ARG, "cta_pair must be -1, 0 or 1");
    g_tune_tile_n.store(tile_n);
    g_tune_pair.store(cta_pair);
    return SG_OK;
}

sg_status_t sg_last_kernel_clock(double* sm_mhz, void* cuda_stream) {
    if (!sm_mhz) return fail(SG_ERR_NULL_POINTER, "sm_mhz is NULL");
    DeviceState* d = nullptr;
    sg_status_t st = device_state(&d);
    if (st != SG_OK) return st;
    uint64_t w[2] = {0, 0};
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    SG_CUDA(cudaMemcpyAsync(w, d->status_dev + 4, sizeof w, cudaMemcpyDeviceToHost, stream));
    SG_CUDA(cudaStreamSynchronize(stream));
    *sm_mhz = w[1] > 0 ? static_cast<double>(w[0]) / static_cast<double>(w[1]) * 1e3 : 0.0;
    return SG_OK;
}

sg_status_t sg_set_tail_mode(int32_t mode) {
    if (mode < -1 || mode > 2) return fail(SG_ERR_INVALID_ARG, "tail mode must be -1 (auto), 0, 1 or 2");
    g_tune_tail.store(mode);
    return SG_OK;
}

sg_status_t sg_gemm(const sg_gemm_desc_t* desc, const void* A, const void* B, const void* C, const void* bias, void* D,
                    void* cuda_stream) {
    bool taken = false;
    const sg_status_t st = try_gemv(desc, A, B, C, bias, D, cuda_stream, &taken);
    if (taken) return st;
    return run_dense(desc, 1, 0, 0, 0, 0, 0, A, B, C, bias, D, cuda_stream, "sg_gemm");
}

// ---- sg_gemm with operands in host memory -------------------------------------------------------------------
namespace {
constexpr int kHostMaxChunks = 16;
struct HostPipe {
    bool ready = false;
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t fork = nullptr, back = nullptr, arrived[kHostMaxChunks] = {}, done[kHostMaxChunks] = {};
};
HostPipe g_host_pipe[kMaxDevices];

struct HostLayout {
    size_t off_a, off_b, off_bias, off_c, off_d, total;
    int64_t a_outer, b_outer;      // rows of the stored A / B arrays (the non-contiguous extent)
};
HostLayout host_layout(const sg_gemm_desc_t* d, const Checked& c) {
    HostLayout L;
    L.a_outer = d->layout_a == SG_ROW_MAJOR ? d->M : d->K;
    L.b_outer = d->layout_b == SG_COL_MAJOR ? d->N : d->K;
    size_t o = 0;
    L.off_a = o;    o = round_up(o + static_cast<size_t>(L.a_outer) * d->lda * c.esize_in, 256);
    L.off_b = o;    o = round_up(o + static_cast<size_t>(L.b_outer) * d->ldb * c.esize_in, 256);
    L.off_bias = o; o = round_up(o + static_cast<size_t>(d->N) * 4, 256);
    L.off_c = o;    o = round_up(o + (d->beta != 0.0f ? static_cast<size_t>(d->M) * d->ldc * c.esize_out : 0), 256);
    L.off_d = o;    o = round_up(o + static_cast<size_t>(d->M) * d->ldd * c.esize_out, 256);
    L.total = o;
    return L;
}
}  // namespace

sg_status_t sg_gemm_host_staging_size(const sg_gemm_desc_t* desc, size_t* bytes) {
    if (!bytes) return fail(SG_ERR_NULL_POINTER, "bytes is NULL");
    Checked c;
    sg_status_t st = check_gemm_desc(desc, false, &c);
    if (st != SG_OK) return st;
    *bytes = host_layout(desc, c).total;
    return SG_OK;
}

sg_status_t sg_gemm_host(const sg_gemm_desc_t* desc, const void* A_host, const void* B_host, const void* C_host,
                         const void* bias_host, void* D_host, void* staging_dev, size_t staging_bytes, int32_t chunks,
                         void* cuda_stream) {
    Checked c;
    sg_status_t st = check_gemm_desc(desc, false, &c);
    if (st != SG_OK) return st;
    if (desc->M == 0 || desc->N == 0) return SG_OK;
    if (!D_host || (desc->K > 0 && (!A_host || !B_host))) return fail(SG_ERR_NULL_POINTER, "sg_gemm_host: A_host, B_host or D_host is NULL");
    if (desc->beta != 0.0f && !C_host) return fail(SG_ERR_NULL_POINTER, "sg_gemm_host: beta != 0 needs C_host");
    if (desc->epi == SG_EPI_BIAS && !bias_host) return fail(SG_ERR_NULL_POINTER, "sg_gemm_host: SG_EPI_BIAS needs bias_host");
    const HostLayout L = host_layout(desc, c);
    if (!staging_dev) return fail(SG_ERR_WORKSPACE, "sg_gemm_host: staging_dev is NULL");
    if (reinterpret_cast<uintptr_t>(staging_dev) & 255u) return fail(SG_ERR_WORKSPACE, "sg_gemm_host: staging_dev must be 256-byte aligned");
    if (staging_bytes < L.total) return fail(SG_ERR_WORKSPACE, "sg_gemm_host: staging has %zu bytes, %zu needed", staging_bytes, L.total);
    if (chunks <= 0) chunks = 4;
    if (chunks > kHostMaxChunks) chunks = kHostMaxChunks;

    int dev = 0;
    SG_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return fail(SG_ERR_CUDA, "device index %d out of range", dev);
    HostPipe& hp = g_host_pipe[dev];
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (!hp.ready) {
            SG_CUDA(cudaStreamCreateWithFlags(&hp.s_in, cudaStreamNonBlocking));
            SG_CUDA(cudaStreamCreateWithFlags(&hp.s_out, cudaStreamNonBlocking));
            SG_CUDA(cudaEventCreateWithFlags(&hp.fork, cudaEventDisableTiming));
            SG_CUDA(cudaEventCreateWithFlags(&hp.back, cudaEventDisableTiming));
            for (int i = 0; i < kHostMaxChunks; ++i) {
                SG_CUDA(cudaEventCreateWithFlags(&hp.arrived[i], cudaEventDisableTiming));
                SG_CUDA(cudaEventCreateWithFlags(&hp.done[i], cudaEventDisableTiming));
            }
            hp.ready = true;
        }
    }
    cudaStream_t main_stream = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* base = static_cast<uint8_t*>(staging_dev);
    uint8_t* dA = base + L.off_a;
    uint8_t* dB = base + L.off_b;
    uint8_t* dBias = base + L.off_bias;
    uint8_t* dC = base + L.off_c;
    uint8_t* dD = base + L.off_d;
    const size_t es_in = static_cast<size_t>(c.esize_in), es_out = static_cast<size_t>(c.esize_out);
    const size_t bias_es = c.in_fp8 == 3 ? 4 : 2;
    // row blocks of A and D: multiples of the 256-row tile
    int64_t rows = (desc->M + chunks - 1) / chunks;
    rows = (rows + 255) / 256 * 256;
    if (rows < 256) rows = 256;
    const int nblocks = static_cast<int>((desc->M + rows - 1) / rows);

    // the staging buffers may still be in use by work enqueued on the caller's stream before this call
    SG_CUDA(cudaEventRecord(hp.fork, main_stream));
    SG_CUDA(cudaStreamWaitEvent(hp.s_in, hp.fork, 0));
    SG_CUDA(cudaStreamWaitEvent(hp.s_out, hp.fork, 0));
    if (desc->K > 0) {
        const size_t b_inner = static_cast<size_t>(desc->layout_b == SG_COL_MAJOR ? desc->K : desc->N) * es_in;
        SG_CUDA(cudaMemcpy2DAsync(dB, desc->ldb * es_in, B_host, desc->ldb * es_in, b_inner, static_cast<size_t>(L.b_outer),
                                  cudaMemcpyHostToDevice, hp.s_in));
    }
    if (bias_host) SG_CUDA(cudaMemcpyAsync(dBias, bias_host, static_cast<size_t>(desc->N) * bias_es, cudaMemcpyHostToDevice, hp.s_in));
    for (int i = 0; i < nblocks; ++i) {
        const int64_t r0 = i * rows, r1 = std::min<int64_t>(desc->M, r0 + rows);
        if (desc->K > 0) {
            if (desc->layout_a == SG_ROW_MAJOR) {
                SG_CUDA(cudaMemcpy2DAsync(dA + r0 * desc->lda * es_in, desc->lda * es_in,
                                          static_cast<const uint8_t*>(A_host) + r0 * desc->lda * es_in, desc->lda * es_in,
                                          static_cast<size_t>(desc->K) * es_in, static_cast<size_t>(r1 - r0), cudaMemcpyHostToDevice, hp.s_in));
            } else {
                SG_CUDA(cudaMemcpy2DAsync(dA + r0 * es_in, desc->lda * es_in, static_cast<const uint8_t*>(A_host) + r0 * es_in,
                                          desc->lda * es_in, static_cast<size_t>(r1 - r0) * es_in, static_cast<size_t>(desc->K),
                                          cudaMemcpyHostToDevice, hp.s_in));
            }
        }
        if (desc->beta != 0.0f)
            SG_CUDA(cudaMemcpy2DAsync(dC + r0 * desc->ldc * es_out, desc->ldc * es_out,
                                      static_cast<const uint8_t*>(C_host) + r0 * desc->ldc * es_out, desc->ldc * es_out,
                                      static_cast<size_t>(desc->N) * es_out, static_cast<size_t>(r1 - r0), cudaMemcpyHostToDevice, hp.s_in));
        SG_CUDA(cudaEventRecord(hp.arrived[i], hp.s_in));
    }
    for (int i = 0; i < nblocks; ++i) {
        const int64_t r0 = i * rows, r1 = std::min<int64_t>(desc->M, r0 + rows);
        SG_CUDA(cudaStreamWaitEvent(main_stream, hp.arrived[i], 0));
        sg_gemm_desc_t blk = *desc;
        blk.M = r1 - r0;
        const uint8_t* a_blk = dA + (desc->layout_a == SG_ROW_MAJOR ? r0 * desc->lda : r0) * es_in;
        st = sg_gemm(&blk, a_blk, dB, desc->beta != 0.0f ? dC + r0 * desc->ldc * es_out : nullptr, bias_host ? dBias : nullptr,
                     dD + r0 * desc->ldd * es_out, main_stream);
        if (st != SG_OK) return st;
        SG_CUDA(cudaEventRecord(hp.done[i], main_stream));
        SG_CUDA(cudaStreamWaitEvent(hp.s_out, hp.done[i], 0));
        SG_CUDA(cudaMemcpy2DAsync(static_cast<uint8_t*>(D_host) + r0 * desc->ldd * es_out, desc->ldd * es_out,
                                  dD + r0 * desc->ldd * es_out, desc->ldd * es_out, static_cast<size_t>(desc->N) * es_out,
                                  static_cast<size_t>(r1 - r0), cudaMemcpyDeviceToHost, hp.s_out));
    }
    SG_CUDA(cudaEventRecord(hp.back, hp.s_out));
    SG_CUDA(cudaStreamWaitEvent(main_stream, hp.back, 0));
    return SG_OK;
}

sg_status_t sg_gemm_ex(const sg_gemm_desc_t* desc, const sg_epilogue_ex_t* ex, const void* A, const void* B, const void* C,
                       const void* bias, void* D, void* cuda_stream) {
    return run_dense(desc, 1, 0, 0, 0, 0, 0, A, B, C, bias, D, cuda_stream, "sg_gemm_ex", ex);
}

sg_status_t sg_batched_gemm(const sg_gemm_desc_t* desc, int64_t batch, int64_t strideA, int64_t strideB, int64_t strideC,
                            int64_t strideD, int64_t strideBias, const void* A, const void* B, const void* C,
                            const void* bias, void* D, void* cuda_stream) {
    return run_dense(desc, batch, strideA, strideB, strideC, strideD, strideBias, A, B, C, bias, D, cuda_stream,
                     "sg_batched_gemm");
}

sg_status_t sg_grouped_gemm_workspace_size(int32_t groups, size_t* bytes) {
    if (!bytes) return fail(SG_ERR_NULL_POINTER, "bytes is NULL");
    if (groups < 0) return fail(SG_ERR_INVALID_ARG, "groups must be >= 0");
    *bytes = grouped_layout(groups > 0 ? groups : 1).total;
    return SG_OK;
}

sg_status_t sg_grouped_gemm(const sg_gemm_desc_t* common, int32_t groups, const int64_t* M_host,
                            const void* const* A_ptrs_host, const void* const* B_ptrs_host,
                            const void* const* C_ptrs_host, const void* const* bias_ptrs_host, void* const* D_ptrs_host,
                            void* workspace_dev, size_t workspace_bytes, void* cuda_stream) {
    Checked c;
    sg_status_t st = check_gemm_desc(common, true, &c);
    if (st != SG_OK) return st;
    if (groups < 0) return fail(SG_ERR_INVALID_ARG, "groups must be >= 0");
    if (groups == 0 || common->N == 0) return SG_OK;
    if (!M_host || !A_ptrs_host || !B_ptrs_host || !D_ptrs_host) return fail(SG_ERR_NULL_POINTER, "sg_grouped_gemm: a host array is NULL");
    if (common->beta != 0.0f && !C_ptrs_host) return fail(SG_ERR_NULL_POINTER, "sg_grouped_gemm: beta != 0 needs C_ptrs_host");
    if (common->epi == SG_EPI_BIAS && !bias_ptrs_host) return fail(SG_ERR_NULL_POINTER, "sg_grouped_gemm: SG_EPI_BIAS needs bias_ptrs_host");
    int64_t total_rows = 0;
    std::vector<int64_t> rows(groups);
    for (int g = 0; g < groups; ++g) {
        if (M_host[g] < 0 || M_host[g] > INT32_MAX) return fail(SG_ERR_INVALID_ARG, "sg_grouped_gemm: M[%d] = %lld", g, (long long)M_host[g]);
        rows[g] = M_host[g];
        total_rows += M_host[g];
        if (M_host[g] == 0) continue;
        st = check_ptrs(A_ptrs_host[g], B_ptrs_host[g], C_ptrs_host ? C_ptrs_host[g] : nullptr,
                        bias_ptrs_host ? bias_ptrs_host[g] : nullptr, D_ptrs_host[g], common->K, common->beta, common->epi,
                        "sg_grouped_gemm");
        if (st != SG_OK) return st;
        if (bias_ptrs_host && !bias_ptrs_host[g]) return fail(SG_ERR_NULL_POINTER, "sg_grouped_gemm: bias pointer of group %d is NULL", g);
    }
    if (total_rows == 0) return SG_OK;
    const GroupedLayout L = grouped_layout(groups);
    if (!workspace_dev) return fail(SG_ERR_WORKSPACE, "sg_grouped_gemm: workspace is NULL");
    if (reinterpret_cast<uintptr_t>(workspace_dev) & 127u) return fail(SG_ERR_WORKSPACE, "sg_grouped_gemm: workspace must be 128-byte aligned");
    if (workspace_bytes < L.total) return fail(SG_ERR_WORKSPACE, "sg_grouped_gemm: workspace has %zu bytes, %zu needed", workspace_bytes, L.total);

    DeviceState* d = nullptr;
    st = device_state(&d);
    if (st != SG_OK) return st;
    const int min_b_rows = common->layout_b == SG_ROW_MAJOR ? 64 : 1;
    Shape s = choose_shape(*d, rows, 1, common->N, common->K, min_b_rows);
    const int tile_m = s.pair ? 256 : 128;
    const int tiles_n = static_cast<int>((common->N + s.bn - 1) / s.bn);

    Params p;
    base_params(&p, *d, common->alpha, common->beta, common->epi, common->epi_arg0, common->epi_arg1);
    p.in_f16 = c.in_f16 ? 1 : 0;
    p.in_fp8 = c.in_fp8;
    p.bk_elems = c.bk;
    int64_t tiles = 0;
    for (int g = 0; g < groups; ++g) tiles += ((rows[g] + tile_m - 1) / tile_m) * tiles_n;
    if (tiles > INT32_MAX / 4) return fail(SG_ERR_UNSUPPORTED, "sg_grouped_gemm: too many tiles");
    p.K = static_cast<int32_t>(common->K);
    p.num_kb = static_cast<int32_t>((common->K + c.bk - 1) / c.bk);
    plan_tail(*d, s, tiles, &p, min_b_rows);

    std::vector<uint8_t> host(L.total, 0);
    CUtensorMap* maps = reinterpret_cast<CUtensorMap*>(host.data() + L.off_maps);
    int32_t* tile_start = reinterpret_cast<int32_t*>(host.data() + L.off_tile_start);
    int32_t* gM = reinterpret_cast<int32_t*>(host.data() + L.off_M);
    const void** gbias = reinterpret_cast<const void**>(host.data() + L.off_bias);
    const void** gC = reinterpret_cast<const void**>(host.data() + L.off_C);
    void** gD = reinterpret_cast<void**>(host.data() + L.off_D);
    tiles = 0;
    for (int g = 0; g < groups; ++g) {
        tile_start[g] = static_cast<int32_t>(tiles);
        gM[g] = static_cast<int32_t>(rows[g]);
        gbias[g] = bias_ptrs_host ? bias_ptrs_host[g] : nullptr;
        gC[g] = (common->beta != 0.0f && C_ptrs_host) ? C_ptrs_host[g] : nullptr;
        gD[g] = D_ptrs_host[g];
        if (rows[g] == 0) continue;
        tiles += ((rows[g] + tile_m - 1) / tile_m) * tiles_n;
        const uint32_t b_box = static_cast<uint32_t>(s.pair ? s.bn / 2 : s.bn);
        if (common->K > 0) {
            if (common->layout_a == SG_COL_MAJOR) {
                // A_g stored [K][M_g] with the common leading dimension: 64 x 64 boxes, consumed M-contiguous
                if (common->lda < rows[g]) return fail(SG_ERR_INVALID_ARG, "sg_grouped_gemm: lda %lld is smaller than M[%d] = %lld",
                                                       (long long)common->lda, g, (long long)rows[g]);
                st = make_tiled_map(&maps[4 * g], c.tm_in, c.esize_in, A_ptrs_host[g], rows[g], common->K, 1, common->lda, 0, 64, 64, "A_g");
            } else {
                st = make_tiled_map(&maps[4 * g], c.tm_in, c.esize_in, A_ptrs_host[g], common->K, rows[g], 1,
                                    common->lda, 0, c.bk, 128, "A_g");
            }
            if (st != SG_OK) return st;
            if (common->layout_b == SG_ROW_MAJOR) {
                st = make_tiled_map(&maps[4 * g + 1], c.tm_in, c.esize_in, B_ptrs_host[g], common->N, common->K, 1,
                                    common->ldb, 0, 64, 64, "B_g");
                maps[4 * g + 3] = maps[4 * g + 1];
            } else {
                st = make_tiled_map(&maps[4 * g + 1], c.tm_in, c.esize_in, B_ptrs_host[g], common->K, common->N, 1,
                                    common->ldb, 0, c.bk, b_box, "B_g");
                if (st != SG_OK) return st;
                st = make_tiled_map(&maps[4 * g + 3], c.tm_in, c.esize_in, B_ptrs_host[g], common->K, common->N, 1,
                                    common->ldb, 0, c.bk, b_box / p.split, "B_g (narrow)");
            }
            if (st != SG_OK) return st;
        }
        st = make_tiled_map(&maps[4 * g + 2], c.tm_out,
                            c.esize_out, D_ptrs_host[g], common->N, rows[g], 1, common->ldd, 0, c.f32_out ? 32 : 64, 32, "D_g");
        if (st != SG_OK) return st;
    }
    tile_start[groups] = static_cast<int32_t>(tiles);

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    st = upload(host, workspace_dev, stream);
    if (st != SG_OK) return st;

    uint8_t* ws = static_cast<uint8_t*>(workspace_dev);
    p.mode = MODE_GROUPED;
    p.a_mn_major = common->layout_a == SG_COL_MAJOR ? 1 : 0;
    p.b_mn_major = common->layout_b == SG_ROW_MAJOR ? 1 : 0;
    p.gmaps = reinterpret_cast<const CUtensorMap*>(ws + L.off_maps);
    p.g_tile_start = reinterpret_cast<const int32_t*>(ws + L.off_tile_start);
    p.g_M = reinterpret_cast<const int32_t*>(ws + L.off_M);
    p.g_bias = bias_ptrs_host ? reinterpret_cast<const void* const*>(ws + L.off_bias) : nullptr;
    p.g_C = common->beta != 0.0f ? reinterpret_cast<const void* const*>(ws + L.off_C) : nullptr;
    p.g_D = reinterpret_cast<void* const*>(ws + L.off_D);
    p.ldc = common->ldc;
    p.ldd = common->ldd;
    p.N = static_cast<int32_t>(common->N);
    p.K = static_cast<int32_t>(common->K);
    p.batch = groups;
    p.tiles_n = tiles_n;
    p.num_kb = static_cast<int32_t>((common->K + c.bk - 1) / c.bk);
    return launch(*d, s, c.out_kind, p, stream);
}

// ---- grouped GEMM without any device allocation by anyone -----------------------------------------------
// Scratch for the tensor maps and tile table of up to SG_STATIC_MAX_GROUPS groups.  In host code this name is
// only a handle for the runtime: the address a kernel can use comes from cudaGetSymbolAddress, per device.
constexpr size_t kStaticWsBytes = 36 * 1024;
static __device__ __align__(256) unsigned char g_static_grouped_ws[kStaticWsBytes];
static void* g_static_ws_ptr[kMaxDevices] = {nullptr};

sg_status_t sg_grouped_gemm_static(const sg_gemm_desc_t* common, int32_t groups, const int64_t* M_host,
                                   const void* const* A_ptrs_host, const void* const* B_ptrs_host,
                                   const void* const* C_ptrs_host, const void* const* bias_ptrs_host,
                                   void* const* D_ptrs_host, void* cuda_stream) {
    if (groups > SG_STATIC_MAX_GROUPS)
        return fail(SG_ERR_WORKSPACE, "sg_grouped_gemm_static: %d groups exceed the built-in scratch for %d groups; "
                    "use sg_grouped_gemm with a caller-provided workspace", groups, SG_STATIC_MAX_GROUPS);
    if (groups > 0 && grouped_layout(groups).total > kStaticWsBytes)
        return fail(SG_ERR_WORKSPACE, "sg_grouped_gemm_static: internal scratch too small for %d groups", groups);
    int dev = 0;
    SG_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return fail(SG_ERR_CUDA, "device index %d out of range", dev);
    void* ws = nullptr;
    {
        // first call on this device: resolve the device address of the scratch array (the current device is `dev`)
        std::lock_guard<std::mutex> lock(g_mutex);
        if (!g_static_ws_ptr[dev]) {
            void* ptr = nullptr;
            cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_grouped_ws);
            if (e != cudaSuccess || !ptr)
                return fail(SG_ERR_CUDA, "cudaGetSymbolAddress(static scratch): %s", cudaGetErrorString(e));
            g_static_ws_ptr[dev] = ptr;
        }
        ws = g_static_ws_ptr[dev];
    }
    // Every table entry the kernel reads is rewritten by this call's stream-ordered upload, so nothing left by
    // an earlier call can be seen; the existing entry point does the rest and allocates no device memory.
    return sg_grouped_gemm(common, groups, M_host, A_ptrs_host, B_ptrs_host, C_ptrs_host, bias_ptrs_host, D_ptrs_host, ws,
                           kStaticWsBytes, cuda_stream);
}

sg_status_t sg_conv2d_fprop(const sg_conv2d_desc_t* desc, const void* X, const void* Wf, const void* Cin, const void* bias,
                            void* Y, void* cuda_stream) {
    return sg_conv2d_fprop_ex(desc, nullptr, X, Wf, Cin, bias, Y, cuda_stream);
}

sg_status_t sg_conv2d_fprop_ex(const sg_conv2d_desc_t* desc, const sg_epilogue_ex_t* ex, const void* X, const void* Wf,
                               const void* Cin, const void* bias, void* Y, void* cuda_stream) {
    if (!desc) return fail(SG_ERR_NULL_POINTER, "desc is NULL");
    Checked c;
    sg_status_t st = check_common(desc->in_dtype, desc->out_dtype, desc->epi, desc->alpha, desc->beta, desc->epi_arg0, desc->epi_arg1,
                                  desc->reserved, &c);
    if (st != SG_OK) return st;
    if (desc->N < 0 || desc->H < 0 || desc->W < 0 || desc->C < 0 || desc->K < 0 || desc->R < 1 || desc->S < 1)
        return fail(SG_ERR_INVALID_ARG, "sg_conv2d_fprop: extents must be >= 0 and the filter at least 1x1");
    if (desc->stride_h < 1 || desc->stride_w < 1 || desc->dil_h < 1 || desc->dil_w < 1 || desc->pad_h < 0 || desc->pad_w < 0)
        return fail(SG_ERR_INVALID_ARG, "sg_conv2d_fprop: strides and dilations must be >= 1, pads >= 0");
    const int64_t span_h = desc->H + 2 * desc->pad_h - desc->dil_h * (desc->R - 1) - 1;
    const int64_t span_w = desc->W + 2 * desc->pad_w - desc->dil_w * (desc->S - 1) - 1;
    const int64_t P = span_h < 0 ? 0 : span_h / desc->stride_h + 1;
    const int64_t Q = span_w < 0 ? 0 : span_w / desc->stride_w + 1;
    const int64_t Mg = desc->N * P * Q;
    if (Mg == 0 || desc->K == 0) return SG_OK;
    if (Mg > INT32_MAX || desc->C * desc->R * desc->S > INT32_MAX || desc->K > INT32_MAX || desc->H > 65535 || desc->W > 65535)
        return fail(SG_ERR_UNSUPPORTED, "sg_conv2d_fprop: extents too large");
    if ((desc->C * c.esize_in) % 16 || (desc->K * c.esize_out) % 16)
        return fail(SG_ERR_ALIGNMENT, "sg_conv2d_fprop: C (input type) and K (output type) must span multiples of 16 bytes");
    if (desc->pad_h > 127 || desc->pad_w > 127 || (desc->R - 1) * desc->dil_h > 255 || (desc->S - 1) * desc->dil_w > 255 ||
        desc->pad_h - (desc->R - 1) * desc->dil_h < -128 || desc->pad_w - (desc->S - 1) * desc->dil_w < -128 ||
        desc->stride_h > 8 || desc->stride_w > 8)
        return fail(SG_ERR_UNSUPPORTED, "sg_conv2d_fprop: pad / filter extent / stride outside the im2col TMA limits");
    const int64_t Kg = desc->C * desc->R * desc->S;
    st = check_ptrs(X, Wf, Cin, bias, Y, Kg, desc->beta, desc->epi, "sg_conv2d_fprop");
    if (st != SG_OK) return st;
    if (c.in_fp8 == 3 && bias && (reinterpret_cast<uintptr_t>(bias) & 3u))
        return fail(SG_ERR_ALIGNMENT, "sg_conv2d_fprop: an fp32 bias must be 4-byte aligned");
    bool ex_any = false;
    {
        Params scratch_params;
        scratch_params.ex_any = 0;
        st = apply_ex(&scratch_params, ex, desc->K, c.esize_out, "sg_conv2d_fprop_ex");
        if (st != SG_OK) return st;
        ex_any = ex != nullptr && scratch_params.ex_any != 0;
    }
    if (desc->C == 0) return fail(SG_ERR_UNSUPPORTED, "sg_conv2d_fprop: C == 0");

    DeviceState* d = nullptr;
    st = device_state(&d);
    if (st != SG_OK) return st;
    Params p;
    base_params(&p, *d, desc->alpha, desc->beta, desc->epi, desc->epi_arg0, desc->epi_arg1);
    p.in_f16 = c.in_f16 ? 1 : 0;
    p.in_fp8 = c.in_fp8;
    p.bk_elems = c.bk;
    const double conv_bytes = (static_cast<double>(desc->N) * desc->H * desc->W * desc->C + static_cast<double>(desc->K) * Kg) * c.esize_in;
    MemHint conv_hint;
    conv_hint.operand_bytes = conv_bytes;
    Shape s = choose_shape(*d, std::vector<int64_t>{Mg}, 1, desc->K, Kg, 1, conv_hint, !ex_any);
    const int tile_m = s.pair ? 256 : 128;
    p.mode = MODE_CONV;
    p.M = static_cast<int32_t>(Mg);
    p.N = static_cast<int32_t>(desc->K);
    p.K = static_cast<int32_t>(Kg);
    p.batch = 1;
    p.tiles_m = static_cast<int32_t>((Mg + tile_m - 1) / tile_m);
    p.tiles_n = static_cast<int32_t>((desc->K + s.bn - 1) / s.bn);
    p.cblocks = static_cast<int32_t>((desc->C + c.bk - 1) / c.bk);
    p.num_kb = static_cast<int32_t>(desc->R * desc->S) * p.cblocks;
    plan_tail(*d, s, static_cast<int64_t>(p.tiles_m) * p.tiles_n, &p, 1, true, !ex_any, conv_bytes);
    p.bias = bias;
    p.C = desc->beta != 0.0f ? Cin : nullptr;
    p.ldc = desc->K;
    p.D = Y;
    p.ldd = desc->K;
    p.P = static_cast<int32_t>(P);
    p.Q = static_cast<int32_t>(Q);
    p.stride_h = desc->stride_h; p.stride_w = desc->stride_w;
    p.pad_h = desc->pad_h; p.pad_w = desc->pad_w;
    p.dil_h = desc->dil_h; p.dil_w = desc->dil_w;
    p.S = static_cast<int32_t>(desc->S);

    // A: im2col view of X [N,H,W,C]: 128 output pixels x 64 channels per load; the bounding box of
    // base pixels starts at -pad and ends where the last filter tap still touches the padded image.
    {
        cuuint64_t dims[4] = {static_cast<cuuint64_t>(desc->C), static_cast<cuuint64_t>(desc->W),
                              static_cast<cuuint64_t>(desc->H), static_cast<cuuint64_t>(desc->N)};
        const cuuint64_t es = static_cast<cuuint64_t>(c.esize_in);
        cuuint64_t strides[3] = {static_cast<cuuint64_t>(desc->C) * es, static_cast<cuuint64_t>(desc->W * desc->C) * es,
                                 static_cast<cuuint64_t>(desc->H * desc->W * desc->C) * es};
        int lower[2] = {-desc->pad_w, -desc->pad_h};
        int upper[2] = {static_cast<int>(desc->pad_w - (desc->S - 1) * desc->dil_w),
                        static_cast<int>(desc->pad_h - (desc->R - 1) * desc->dil_h)};
        cuuint32_t estr[4] = {1, static_cast<cuuint32_t>(desc->stride_w), static_cast<cuuint32_t>(desc->stride_h), 1};
        CUresult r = g_encode_im2col(&p.tmA, c.tm_in, 4, const_cast<void*>(X), dims, strides, lower, upper,
                                     static_cast<cuuint32_t>(c.bk), 128, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail(SG_ERR_CUDA, "cuTensorMapEncodeIm2col(X) failed with CUresult %d", static_cast<int>(r));
    }
    // B: filter [K][R*S][C] -> rows = output channels, one tap and 64 input channels per load
    {
        cuuint64_t dims[3] = {static_cast<cuuint64_t>(desc->C), static_cast<cuuint64_t>(desc->R * desc->S),
                              static_cast<cuuint64_t>(desc->K)};
        cuuint64_t strides[2] = {static_cast<cuuint64_t>(desc->C) * c.esize_in, static_cast<cuuint64_t>(Kg) * c.esize_in};
        cuuint32_t box[3] = {static_cast<cuuint32_t>(c.bk), 1, static_cast<cuuint32_t>(s.pair ? s.bn / 2 : s.bn)};
        cuuint32_t estr[3] = {1, 1, 1};
        CUresult r = g_encode_tiled(&p.tmB, c.tm_in, 3, const_cast<void*>(Wf), dims, strides, box, estr,
                                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail(SG_ERR_CUDA, "cuTensorMapEncodeTiled(Wf) failed with CUresult %d", static_cast<int>(r));
        box[2] /= static_cast<cuuint32_t>(p.split);
        r = g_encode_tiled(&p.tmB2, c.tm_in, 3, const_cast<void*>(Wf), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail(SG_ERR_CUDA, "cuTensorMapEncodeTiled(Wf, narrow) failed with CUresult %d", static_cast<int>(r));
    }
    st = make_tiled_map(&p.tmD, c.tm_out, c.esize_out, Y,
                        desc->K, Mg, 1, desc->K, 0, c.f32_out ? 32 : 64, 32, "Y");
    if (st != SG_OK) return st;
    st = apply_ex(&p, ex, desc->K, c.esize_out, "sg_conv2d_fprop_ex");
    if (st != SG_OK) return st;
    return launch(*d, s, c.out_kind, p, static_cast<cudaStream_t>(cuda_stream));
}

}  // extern "C"

namespace {

// Checks shared by the two gradient entry points; P, Q are the forward output extents.
sg_status_t grad_geometry(const sg_conv2d_desc_t* desc, const char* who, Checked* c, int64_t* P, int64_t* Q) {
    if (!desc) return fail(SG_ERR_NULL_POINTER, "desc is NULL");
    sg_status_t st = check_common(desc->in_dtype, desc->out_dtype, desc->epi, desc->alpha, desc->beta, desc->epi_arg0,
                                  desc->epi_arg1, desc->reserved, c);
    if (st != SG_OK) return st;
    if (desc->epi != SG_EPI_NONE) return fail(SG_ERR_INVALID_ARG, "%s: epi must be SG_EPI_NONE", who);
    if (c->in_fp8) return fail(SG_ERR_UNSUPPORTED, "%s: 8-bit and tf32 inputs are not supported (an operand is read N-contiguous)", who);
    if (desc->N < 0 || desc->H < 0 || desc->W < 0 || desc->C < 0 || desc->K < 0 || desc->R < 1 || desc->S < 1)
        return fail(SG_ERR_INVALID_ARG, "%s: extents must be >= 0 and the filter at least 1x1", who);
    if (desc->stride_h < 1 || desc->stride_w < 1 || desc->dil_h < 1 || desc->dil_w < 1 || desc->pad_h < 0 || desc->pad_w < 0)
        return fail(SG_ERR_INVALID_ARG, "%s: strides and dilations must be >= 1, pads >= 0", who);
    const int64_t span_h = desc->H + 2 * desc->pad_h - desc->dil_h * (desc->R - 1) - 1;
    const int64_t span_w = desc->W + 2 * desc->pad_w - desc->dil_w * (desc->S - 1) - 1;
    *P = span_h < 0 ? 0 : span_h / desc->stride_h + 1;
    *Q = span_w < 0 ? 0 : span_w / desc->stride_w + 1;
    if (desc->N * desc->H * desc->W > INT32_MAX || desc->N * *P * *Q > INT32_MAX || desc->C * desc->R * desc->S > INT32_MAX ||
        desc->K * desc->R * desc->S > INT32_MAX || desc->H > 65535 || desc->W > 65535)
        return fail(SG_ERR_UNSUPPORTED, "%s: extents too large", who);
    if ((desc->R - 1) * desc->dil_h > 255 || (desc->S - 1) * desc->dil_w > 255 || desc->pad_h > 127 || desc->pad_w > 127 ||
        desc->stride_h > 8 || desc->stride_w > 8)
        return fail(SG_ERR_UNSUPPORTED, "%s: pad / filter extent / stride outside the im2col TMA limits", who);
    return SG_OK;
}

}  // namespace

namespace {

// One spatial dimension of one output phase of the data gradient.  Output positions h = a + stride * i (i < out_n)
// receive the filter taps r with (a + pad - r * dil) divisible by the stride; for those p = i + (a + pad - r * dil) /
// stride.  The taps form an arithmetic progression; walked from the largest r down, the offsets grow by dd per tap,
// i.e. the phase is a stride-1 correlation of dY with a mirrored, thinned filter:
//   p = i + lower + m * dd,   filter tap r = tap_hi - m * tap_step,   m = 0 .. taps - 1.
struct PhaseDim {
    int64_t out_n = 0;
    int taps = 0, tap_hi = 0, tap_step = 1, dd = 1;
    int64_t lower = 0;
};
PhaseDim phase_dim(int64_t a, int64_t extent, int64_t pad, int64_t dil, int64_t filt, int64_t stride) {
    PhaseDim d;
    d.out_n = a < extent ? (extent - a + stride - 1) / stride : 0;
    int first = -1, second = -1, last = -1;
    for (int r = 0; r < filt; ++r) {
        const int64_t x = a + pad - r * dil;
        if (((x % stride) + stride) % stride != 0) continue;
        if (first < 0) first = r;
        else if (second < 0) second = r;
        last = r;
        ++d.taps;
    }
    if (d.taps == 0) return d;
    d.tap_hi = last;
    d.tap_step = d.taps > 1 ? second - first : 1;
    d.dd = d.taps > 1 ? static_cast<int>(dil * d.tap_step / stride) : 1;
    const int64_t x = a + pad - static_cast<int64_t>(last) * dil;       // divisible by the stride
    d.lower = x >= 0 ? x / stride : -((-x) / stride);
    return d;
}

}  // namespace

extern "C" sg_status_t sg_conv2d_dgrad(const sg_conv2d_desc_t* desc, const void* dY, const void* Wf, const void* Cin, void* dX,
                                       void* cuda_stream) {
    const char* who = "sg_conv2d_dgrad";
    Checked c;
    int64_t P = 0, Q = 0;
    sg_status_t st = grad_geometry(desc, who, &c, &P, &Q);
    if (st != SG_OK) return st;
    if (desc->N * desc->H * desc->W == 0 || desc->C == 0) return SG_OK;
    if ((desc->K * c.esize_in) % 16 || (desc->C * c.esize_in) % 16 || (desc->C * c.esize_out) % 16)
        return fail(SG_ERR_ALIGNMENT, "%s: K and C must span multiples of 16 bytes", who);
    const bool no_sum = P == 0 || Q == 0 || desc->K == 0;       // nothing to sum anywhere: dX = beta * Cin
    st = check_ptrs(dY, Wf, Cin, nullptr, dX, no_sum ? 0 : desc->K, desc->beta, desc->epi, who);
    if (st != SG_OK) return st;
    const bool strided = desc->stride_h != 1 || desc->stride_w != 1;
    // every output phase (h mod stride_h, w mod stride_w) is one launch; a stride-1 gradient has one phase
    std::vector<std::pair<PhaseDim, PhaseDim>> phases;
    std::vector<std::pair<int, int>> phase_ab;
    for (int a = 0; a < desc->stride_h; ++a)
        for (int b = 0; b < desc->stride_w; ++b) {
            PhaseDim ph = phase_dim(a, desc->H, desc->pad_h, desc->dil_h, desc->R, desc->stride_h);
            PhaseDim pw = phase_dim(b, desc->W, desc->pad_w, desc->dil_w, desc->S, desc->stride_w);
            if (ph.out_n == 0 || pw.out_n == 0) continue;
            for (const PhaseDim* d : {&ph, &pw}) {
                const int64_t in_extent = d == &ph ? P : Q;
                const int64_t upper = d->out_n - in_extent + d->lower;
                if (d->taps > 0 && (d->lower < -128 || d->lower > 127 || upper < -128 || upper > 127 ||
                                    static_cast<int64_t>(d->taps - 1) * d->dd > 255))
                    return fail(SG_ERR_UNSUPPORTED, "%s: pad / filter extent / stride outside the im2col TMA limits", who);
            }
            phases.emplace_back(ph, pw);
            phase_ab.emplace_back(a, b);
        }

    DeviceState* d = nullptr;
    st = device_state(&d);
    if (st != SG_OK) return st;
    if (strided && !no_sum && phases.size() >= 2 && phases.size() <= static_cast<size_t>(kMaxPhases)) {
        // All phases in one launch: their tiles are one list (longest K loops first), so the phases share the waves
        // of the machine instead of each paying its own partial last wave and its own launch.
        std::vector<size_t> order(phases.size());
        for (size_t i = 0; i < order.size(); ++i) order[i] = i;
        std::sort(order.begin(), order.end(), [&](size_t x, size_t y) {
            const int64_t kx = static_cast<int64_t>(phases[x].first.taps) * phases[x].second.taps;
            const int64_t ky = static_cast<int64_t>(phases[y].first.taps) * phases[y].second.taps;
            return kx != ky ? kx > ky : x < y;
        });
        std::vector<int64_t> rows;
        int64_t k_sum = 0;
        for (size_t i : order) {
            rows.push_back(desc->N * phases[i].first.out_n * phases[i].second.out_n);
            k_sum += desc->K * std::max<int64_t>(1, static_cast<int64_t>(phases[i].first.taps) * phases[i].second.taps);
        }
        Params p;
        base_params(&p, *d, desc->alpha, desc->beta, desc->epi, 0.0f, 0.0f);
        p.in_f16 = c.in_f16 ? 1 : 0;
        p.bk_elems = c.bk;
        Shape s = choose_shape(*d, rows, 1, desc->C, k_sum / static_cast<int64_t>(order.size()), 64);
        const int tile_m = s.pair ? 256 : 128;
        p.mode = MODE_CONV;
        p.b_mn_major = 1;
        p.filt_s = static_cast<int32_t>(desc->S);
        p.N = static_cast<int32_t>(desc->C);
        p.batch = 1;
        p.tiles_m = 1;
        p.tiles_n = static_cast<int32_t>((desc->C + s.bn - 1) / s.bn);
        p.cblocks = static_cast<int32_t>((desc->K + c.bk - 1) / c.bk);
        p.stride_h = 1; p.stride_w = 1;
        p.d_remap = 1;
        p.remap_sh = desc->stride_h; p.remap_sw = desc->stride_w;
        p.remap_H = static_cast<int32_t>(desc->H); p.remap_W = static_cast<int32_t>(desc->W);
        p.C = desc->beta != 0.0f ? Cin : nullptr;
        p.ldc = desc->C;
        p.D = dX;
        p.ldd = desc->C;
        st = make_tiled_map(&p.tmD, c.tm_out, c.esize_out, dX, desc->C, desc->N * desc->H * desc->W, 1, desc->C, 0,
                            c.f32_out ? 32 : 64, 32, "dX");
        if (st != SG_OK) return st;
        p.nphases = static_cast<int32_t>(order.size());
        int64_t tiles = 0;
        for (size_t j = 0; j < order.size(); ++j) {
            const PhaseDim& ph = phases[order[j]].first;
            const PhaseDim& pw = phases[order[j]].second;
            ConvPhase& f = p.ph[j];
            const int64_t taps = static_cast<int64_t>(ph.taps) * pw.taps;
            f.tile_start = static_cast<int32_t>(tiles);
            f.M = static_cast<int32_t>(rows[j]);
            f.num_kb = static_cast<int32_t>(taps * p.cblocks);
            f.P = static_cast<int32_t>(ph.out_n); f.Q = static_cast<int32_t>(pw.out_n);
            f.pad_h = static_cast<int32_t>(-ph.lower); f.pad_w = static_cast<int32_t>(-pw.lower);
            f.dil_h = ph.dd; f.dil_w = pw.dd;
            f.S = pw.taps > 0 ? pw.taps : 1;
            f.tapb_r0 = ph.tap_hi; f.tapb_rs = -ph.tap_step;
            f.tapb_s0 = pw.tap_hi; f.tapb_ss = -pw.tap_step;
            f.remap_h0 = phase_ab[order[j]].first; f.remap_w0 = phase_ab[order[j]].second;
            f.div_pq = make_fastdiv(ph.out_n * pw.out_n);
            f.div_q = make_fastdiv(pw.out_n);
            tiles += ((rows[j] + tile_m - 1) / tile_m) * p.tiles_n;
            if (f.num_kb > p.num_kb) p.num_kb = f.num_kb;
            if (f.M > p.M) p.M = f.M;
            if (taps == 0) {
                p.tmPh[j] = p.tmD;
                continue;
            }
            cuuint64_t dims[4] = {static_cast<cuuint64_t>(desc->K), static_cast<cuuint64_t>(Q), static_cast<cuuint64_t>(P),
                                  static_cast<cuuint64_t>(desc->N)};
            const cuuint64_t es = static_cast<cuuint64_t>(c.esize_in);
            cuuint64_t strides[3] = {static_cast<cuuint64_t>(desc->K) * es, static_cast<cuuint64_t>(Q * desc->K) * es,
                                     static_cast<cuuint64_t>(P * Q * desc->K) * es};
            int lower[2] = {static_cast<int>(pw.lower), static_cast<int>(ph.lower)};
            int upper[2] = {static_cast<int>(pw.out_n - Q + pw.lower), static_cast<int>(ph.out_n - P + ph.lower)};
            cuuint32_t estr[4] = {1, 1, 1, 1};
            CUresult r = g_encode_im2col(&p.tmPh[j], c.tm_in, 4, const_cast<void*>(dY), dims, strides, lower, upper,
                                         static_cast<cuuint32_t>(c.bk), 128, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) return fail(SG_ERR_CUDA, "cuTensorMapEncodeIm2col(dY) failed with CUresult %d", static_cast<int>(r));
        }
        if (tiles > INT32_MAX / 4) return fail(SG_ERR_UNSUPPORTED, "%s: too many tiles", who);
        p.K = p.num_kb * c.bk;
        p.tmA = p.tmPh[0];
        {
            const cuuint64_t es = static_cast<cuuint64_t>(c.esize_in);
            cuuint64_t fdims[3] = {static_cast<cuuint64_t>(desc->C), static_cast<cuuint64_t>(desc->R * desc->S),
                                   static_cast<cuuint64_t>(desc->K)};
            cuuint64_t fstrides[2] = {static_cast<cuuint64_t>(desc->C) * es, static_cast<cuuint64_t>(desc->C * desc->R * desc->S) * es};
            cuuint32_t box[3] = {64, 1, 64};
            cuuint32_t e3[3] = {1, 1, 1};
            CUresult r = g_encode_tiled(&p.tmB, c.tm_in, 3, const_cast<void*>(Wf), fdims, fstrides, box, e3, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) return fail(SG_ERR_CUDA, "cuTensorMapEncodeTiled(Wf) failed with CUresult %d", static_cast<int>(r));
            p.tmB2 = p.tmB;
        }
        plan_tail(*d, s, tiles, &p, 64, false);
        return launch(*d, s, c.out_kind, p, static_cast<cudaStream_t>(cuda_stream));
    }
    for (size_t i = 0; i < phases.size(); ++i) {
        const PhaseDim& ph = phases[i].first;
        const PhaseDim& pw = phases[i].second;
        const int64_t Mg = desc->N * ph.out_n * pw.out_n;       // rows: this phase's input pixels
        const int64_t taps = static_cast<int64_t>(ph.taps) * pw.taps;
        const bool empty = no_sum || taps == 0;
        const int64_t Kg = desc->K * (taps > 0 ? taps : 1);     // contraction: taps x output channels of the forward pass
        Params p;
        base_params(&p, *d, desc->alpha, desc->beta, desc->epi, 0.0f, 0.0f);
        p.in_f16 = c.in_f16 ? 1 : 0;
        p.bk_elems = c.bk;
        Shape s = choose_shape(*d, std::vector<int64_t>{Mg}, 1, desc->C, Kg, 64);
        const int tile_m = s.pair ? 256 : 128;
        p.mode = MODE_CONV;
        p.b_mn_major = 1;
        p.num_taps = static_cast<int32_t>(taps);
        p.tapb_r0 = ph.tap_hi; p.tapb_rs = -ph.tap_step;
        p.tapb_s0 = pw.tap_hi; p.tapb_ss = -pw.tap_step;
        p.filt_s = static_cast<int32_t>(desc->S);
        p.M = static_cast<int32_t>(Mg);
        p.N = static_cast<int32_t>(desc->C);
        p.K = static_cast<int32_t>(Kg);
        p.batch = 1;
        p.tiles_m = static_cast<int32_t>((Mg + tile_m - 1) / tile_m);
        p.tiles_n = static_cast<int32_t>((desc->C + s.bn - 1) / s.bn);
        p.cblocks = static_cast<int32_t>((desc->K + c.bk - 1) / c.bk);
        p.num_kb = empty ? 0 : p.num_taps * p.cblocks;
        plan_tail(*d, s, static_cast<int64_t>(p.tiles_m) * p.tiles_n, &p, 64);
        p.C = desc->beta != 0.0f ? Cin : nullptr;
        p.ldc = desc->C;
        p.D = dX;
        p.ldd = desc->C;
        // the "image" the kernel walks is dY [N,P,Q,K]; its output pixels are this phase's pixels of dX
        p.P = static_cast<int32_t>(ph.out_n);
        p.Q = static_cast<int32_t>(pw.out_n);
        p.stride_h = 1; p.stride_w = 1;
        p.pad_h = static_cast<int32_t>(-ph.lower); p.pad_w = static_cast<int32_t>(-pw.lower);
        p.dil_h = ph.dd; p.dil_w = pw.dd;
        p.S = pw.taps > 0 ? pw.taps : 1;
        if (strided) {
            p.d_remap = 1;
            p.remap_h0 = phase_ab[i].first; p.remap_sh = desc->stride_h;
            p.remap_w0 = phase_ab[i].second; p.remap_sw = desc->stride_w;
            p.remap_H = static_cast<int32_t>(desc->H); p.remap_W = static_cast<int32_t>(desc->W);
        }
        st = make_tiled_map(&p.tmD, c.tm_out, c.esize_out, dX, desc->C, desc->N * desc->H * desc->W, 1, desc->C, 0,
                            c.f32_out ? 32 : 64, 32, "dX");
        if (st != SG_OK) return st;
        if (empty) {
            p.tmA = p.tmD; p.tmB = p.tmD; p.tmB2 = p.tmD;
        } else {
            cuuint64_t dims[4] = {static_cast<cuuint64_t>(desc->K), static_cast<cuuint64_t>(Q), static_cast<cuuint64_t>(P),
                                  static_cast<cuuint64_t>(desc->N)};
            const cuuint64_t es = static_cast<cuuint64_t>(c.esize_in);
            cuuint64_t strides[3] = {static_cast<cuuint64_t>(desc->K) * es, static_cast<cuuint64_t>(Q * desc->K) * es,
                                     static_cast<cuuint64_t>(P * Q * desc->K) * es};
            int lower[2] = {static_cast<int>(pw.lower), static_cast<int>(ph.lower)};
            int upper[2] = {static_cast<int>(pw.out_n - Q + pw.lower), static_cast<int>(ph.out_n - P + ph.lower)};
            cuuint32_t estr[4] = {1, 1, 1, 1};
            CUresult r = g_encode_im2col(&p.tmA, c.tm_in, 4, const_cast<void*>(dY), dims, strides, lower, upper,
                                         static_cast<cuuint32_t>(c.bk), 128, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS)
                return fail(SG_ERR_CUDA, "cuTensorMapEncodeIm2col(dY) failed with CUresult %d (corners %d..%d, %d..%d)",
                            static_cast<int>(r), lower[0], upper[0], lower[1], upper[1]);
            // filter [K][R*S][C] read with C contiguous: boxes of 64 c x 1 tap x 64 k
            cuuint64_t fdims[3] = {static_cast<cuuint64_t>(desc->C), static_cast<cuuint64_t>(desc->R * desc->S),
                                   static_cast<cuuint64_t>(desc->K)};
            cuuint64_t fstrides[2] = {static_cast<cuuint64_t>(desc->C) * es, static_cast<cuuint64_t>(desc->C * desc->R * desc->S) * es};
            cuuint32_t box[3] = {64, 1, 64};
            cuuint32_t e3[3] = {1, 1, 1};
            r = g_encode_tiled(&p.tmB, c.tm_in, 3, const_cast<void*>(Wf), fdims, fstrides, box, e3, CU_TENSOR_MAP_INTERLEAVE_NONE,
                               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) return fail(SG_ERR_CUDA, "cuTensorMapEncodeTiled(Wf) failed with CUresult %d", static_cast<int>(r));
            p.tmB2 = p.tmB;
        }
        st = launch(*d, s, c.out_kind, p, static_cast<cudaStream_t>(cuda_stream));
        if (st != SG_OK) return st;
    }
    return SG_OK;
}

extern "C" sg_status_t sg_conv2d_wgrad(const sg_conv2d_desc_t* desc, const void* dY, const void* X, const void* Cin, void* dW,
                                       void* cuda_stream) {
    const char* who = "sg_conv2d_wgrad";
    Checked c;
    int64_t P = 0, Q = 0;
    sg_status_t st = grad_geometry(desc, who, &c, &P, &Q);
    if (st != SG_OK) return st;
    if (desc->K == 0 || desc->C == 0) return SG_OK;
    const int64_t taps = desc->R * desc->S;
    const int64_t pixels = desc->N * P * Q;               // contraction: output pixels of the forward pass
    if ((desc->K * c.esize_in) % 16 || (desc->C * c.esize_in) % 16 || (desc->C * c.esize_out) % 16)
        return fail(SG_ERR_ALIGNMENT, "%s: K and C must span multiples of 16 bytes", who);
    if (desc->pad_h - (desc->R - 1) * desc->dil_h < -128 || desc->pad_w - (desc->S - 1) * desc->dil_w < -128)
        return fail(SG_ERR_UNSUPPORTED, "%s: filter extent outside the im2col TMA limits", who);
    st = check_ptrs(dY, X, Cin, nullptr, dW, pixels, desc->beta, desc->epi, who);
    if (st != SG_OK) return st;

    DeviceState* d = nullptr;
    st = device_state(&d);
    if (st != SG_OK) return st;
    Params p;
    base_params(&p, *d, desc->alpha, desc->beta, desc->epi, 0.0f, 0.0f);
    p.in_f16 = c.in_f16 ? 1 : 0;
    p.bk_elems = c.bk;
    // one product per filter tap: dW[:, tap, :] (K x C) = dY^T (K x pixels) . X shifted by the tap (pixels x C)
    const double wgrad_bytes = (static_cast<double>(pixels) * desc->K + static_cast<double>(desc->N) * desc->H * desc->W * desc->C) * c.esize_in;
    MemHint wgrad_hint;
    wgrad_hint.operand_bytes = wgrad_bytes;
    Shape s = choose_shape(*d, std::vector<int64_t>{desc->K}, taps, desc->C, pixels, 64, wgrad_hint, true);
    const int tile_m = s.pair ? 256 : 128;
    p.mode = MODE_WGRAD;
    p.a_mn_major = 1;
    p.b_mn_major = 1;
    p.num_taps = static_cast<int32_t>(taps);
    p.M = static_cast<int32_t>(desc->K);
    p.N = static_cast<int32_t>(desc->C);
    p.K = static_cast<int32_t>(pixels);
    p.batch = static_cast<int32_t>(taps);
    p.tiles_m = static_cast<int32_t>((desc->K + tile_m - 1) / tile_m);
    p.tiles_n = static_cast<int32_t>((desc->C + s.bn - 1) / s.bn);
    p.num_kb = static_cast<int32_t>((pixels + 63) / 64);
    plan_tail(*d, s, static_cast<int64_t>(p.tiles_m) * p.tiles_n * taps, &p, 64, true, true, wgrad_bytes);
    p.C = desc->beta != 0.0f ? Cin : nullptr;
    p.ldc = taps * desc->C;
    p.strideC = desc->C;
    p.D = dW;
    p.ldd = taps * desc->C;
    p.strideD = desc->C;
    p.P = static_cast<int32_t>(P);
    p.Q = static_cast<int32_t>(Q);
    p.stride_h = desc->stride_h; p.stride_w = desc->stride_w;
    p.pad_h = desc->pad_h; p.pad_w = desc->pad_w;
    p.dil_h = desc->dil_h; p.dil_w = desc->dil_w;
    p.S = static_cast<int32_t>(desc->S);
    st = make_tiled_map(&p.tmD, c.tm_out, c.esize_out, dW, desc->C, desc->K, taps, taps * desc->C, desc->C,
                        c.f32_out ? 32 : 64, 32, "dW");
    if (st != SG_OK) return st;
    if (pixels == 0) {
        p.tmA = p.tmD; p.tmB = p.tmD; p.tmB2 = p.tmD;
    } else {
        st = make_tiled_map(&p.tmA, c.tm_in, c.esize_in, dY, desc->K, pixels, 1, desc->K, 0, 64, 64, "dY");
        if (st != SG_OK) return st;
        cuuint64_t dims[4] = {static_cast<cuuint64_t>(desc->C), static_cast<cuuint64_t>(desc->W), static_cast<cuuint64_t>(desc->H),
                              static_cast<cuuint64_t>(desc->N)};
        const cuuint64_t es = static_cast<cuuint64_t>(c.esize_in);
        cuuint64_t strides[3] = {static_cast<cuuint64_t>(desc->C) * es, static_cast<cuuint64_t>(desc->W * desc->C) * es,
                                 static_cast<cuuint64_t>(desc->H * desc->W * desc->C) * es};
        int lower[2] = {-desc->pad_w, -desc->pad_h};
        int upper[2] = {static_cast<int>(desc->pad_w - (desc->S - 1) * desc->dil_w),
                        static_cast<int>(desc->pad_h - (desc->R - 1) * desc->dil_h)};
        cuuint32_t estr[4] = {1, static_cast<cuuint32_t>(desc->stride_w), static_cast<cuuint32_t>(desc->stride_h), 1};
        CUresult r = g_encode_im2col(&p.tmB, c.tm_in, 4, const_cast<void*>(X), dims, strides, lower, upper, 64, 64, estr,
                                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail(SG_ERR_CUDA, "cuTensorMapEncodeIm2col(X) failed with CUresult %d", static_cast<int>(r));
        p.tmB2 = p.tmB;
    }
    return launch(*d, s, c.out_kind, p, static_cast<cudaStream_t>(cuda_stream));
}

extern "C" {

sg_status_t sg_transpose(const sg_transpose_desc_t* desc, const void* in, void* out, void* cuda_stream) {
    if (!desc) return fail(SG_ERR_NULL_POINTER, "desc is NULL");
    if (desc->reserved != 0 || desc->reserved2 != 0) return fail(SG_ERR_INVALID_ARG, "reserved fields must be 0");
    if ((desc->in_dtype != SG_BF16 && desc->in_dtype != SG_F32 && desc->in_dtype != SG_F16) ||
        (desc->out_dtype != SG_BF16 && desc->out_dtype != SG_F32 && desc->out_dtype != SG_F16))
        return fail(SG_ERR_INVALID_ARG, "sg_transpose: dtypes must be SG_BF16, SG_F16 or SG_F32");
    const TransposeEntry te = transpose_entry(transpose_type_index(desc->in_dtype), transpose_type_index(desc->out_dtype));
    if (desc->batch < 0 || desc->rows < 0 || desc->cols < 0) return fail(SG_ERR_INVALID_ARG, "sg_transpose: extents must be >= 0");
    if (desc->batch == 0 || desc->rows == 0 || desc->cols == 0) return SG_OK;
    const int es_in = desc->in_dtype == SG_F32 ? 4 : 2, es_out = desc->out_dtype == SG_F32 ? 4 : 2;
    if (desc->ld_in < desc->cols || desc->ld_out < desc->rows) return fail(SG_ERR_INVALID_ARG, "sg_transpose: ld_in >= cols and ld_out >= rows are required");
    if (desc->batch > 1 && (desc->stride_in < (desc->rows - 1) * desc->ld_in + desc->cols ||
                            desc->stride_out < (desc->cols - 1) * desc->ld_out + desc->rows))
        return fail(SG_ERR_INVALID_ARG, "sg_transpose: batch strides smaller than one matrix");
    if (!in || !out) return fail(SG_ERR_NULL_POINTER, "sg_transpose: in or out is NULL");
    if (!aligned16(in) || !aligned16(out)) return fail(SG_ERR_ALIGNMENT, "sg_transpose: base pointers must be 16-byte aligned");
    if ((desc->ld_in * es_in) % 16 || (desc->ld_out * es_out) % 16 ||
        (desc->batch > 1 && ((desc->stride_in * es_in) % 16 || (desc->stride_out * es_out) % 16)))
        return fail(SG_ERR_ALIGNMENT, "sg_transpose: leading dimensions and batch strides must be multiples of 16 bytes");
    const int64_t tiles_r = (desc->rows + 63) / 64, tiles_c = (desc->cols + 63) / 64;
    if (tiles_r * tiles_c * desc->batch > INT32_MAX || tiles_r > INT32_MAX || tiles_c > INT32_MAX)
        return fail(SG_ERR_UNSUPPORTED, "sg_transpose: too many tiles");
    DeviceState* d = nullptr;
    sg_status_t st = device_state(&d);
    if (st != SG_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // Extents that are multiples of 16 bytes in both types (every tile edge then falls on a 16-byte boundary of its
    // row): the persistent TMA kernel.  Ragged extents take the plain-store kernel below.
    if ((desc->cols * es_in) % 16 == 0 && (desc->rows * es_out) % 16 == 0 && desc->rows <= INT32_MAX && desc->cols <= INT32_MAX &&
        desc->batch <= INT32_MAX && opt(SG_OPT_TRANSPOSE_PLAIN) <= 0) {
        const int vi = 16 / es_in, vo = 16 / es_out;
        const int TR = 16 * vo, TC = 16 * vi;
        const int64_t tr = (desc->rows + TR - 1) / TR, tc = (desc->cols + TC - 1) / TC;
        if (tr * tc * desc->batch > INT32_MAX) return fail(SG_ERR_UNSUPPORTED, "sg_transpose: too many tiles");
        TransposeTmaParams tp;
        memset(&tp, 0, sizeof tp);
        auto map_type = [](int32_t dt) {
            return dt == SG_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : (dt == SG_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16);
        };
        const CUtensorMapDataType dt_in = map_type(desc->in_dtype), dt_out = map_type(desc->out_dtype);
        st = make_tiled_map(&tp.tm_in, dt_in, es_in, in, desc->cols, desc->rows, desc->batch, desc->ld_in, desc->stride_in, TC, TR,
                            "transpose input", CU_TENSOR_MAP_SWIZZLE_NONE);
        if (st != SG_OK) return st;
        st = make_tiled_map(&tp.tm_out, dt_out, es_out, out, desc->rows, desc->cols, desc->batch, desc->ld_out, desc->stride_out, TR, TC,
                            "transpose output", CU_TENSOR_MAP_SWIZZLE_NONE);
        if (st != SG_OK) return st;
        tp.tiles_r = static_cast<int32_t>(tr);
        tp.tiles_c = static_cast<int32_t>(tc);
        tp.num_tiles = static_cast<int32_t>(tr * tc * desc->batch);
        tp.status = d->status_dev;
        const int64_t limit = opt(SG_OPT_WAIT_LIMIT_NS);
        tp.timeout_ns = limit > 0 ? static_cast<uint64_t>(limit) : kWaitLimitNs;
        cudaLaunchConfig_t cfg = {};
        const int64_t slots = static_cast<int64_t>(d->sm_count) * te.ctas_per_sm;
        cfg.gridDim = dim3(static_cast<unsigned>(tp.num_tiles < slots ? tp.num_tiles : slots));
        cfg.blockDim = dim3(288);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = opt(SG_OPT_NO_PDL) > 0 ? 0 : 1;
        cfg.dynamicSmemBytes = te.smem;
        const cudaError_t e = cudaLaunchKernelEx(&cfg, te.tma, tp);
        if (e != cudaSuccess) return fail(SG_ERR_CUDA, "transpose kernel launch: %s", cudaGetErrorString(e));
        g_launches.fetch_add(1);
        note_kernel("sg::transpose_tma_kernel<%s, %s>", te.in_name, te.out_name);
        return SG_OK;
    }
    TransposeParams tp;
    tp.in = in;
    tp.out = out;
    tp.rows = desc->rows; tp.cols = desc->cols;
    tp.ld_in = desc->ld_in; tp.ld_out = desc->ld_out;
    tp.stride_in = desc->stride_in; tp.stride_out = desc->stride_out;
    tp.tiles_r = static_cast<int32_t>(tiles_r); tp.tiles_c = static_cast<int32_t>(tiles_c);
    const dim3 grid(static_cast<unsigned>(tiles_r * tiles_c * desc->batch));
    te.plain<<<grid, 256, 0, stream>>>(tp);
    SG_CUDA(cudaGetLastError());
    g_launches.fetch_add(1);
    note_kernel("sg::transpose_kernel<%s, %s>", te.in_name, te.out_name);
    return SG_OK;
}

sg_status_t sg_poll_status(void* cuda_stream) {
    DeviceState* d = nullptr;
    sg_status_t st = device_state(&d);
    if (st != SG_OK) return st;
    uint32_t words[8] = {0};
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    SG_CUDA(cudaMemcpyAsync(words, d->status_dev, sizeof words, cudaMemcpyDeviceToHost, stream));
    SG_CUDA(cudaStreamSynchronize(stream));
    if (words[0] == 0) return SG_OK;
    SG_CUDA(cudaMemsetAsync(d->status_dev, 0, sizeof words, stream));
    if (d->scratch) SG_CUDA(cudaMemsetAsync(d->scratch, 0, kScratchFlagBytes, stream));   // an aborted K-split may leave counters set
    SG_CUDA(cudaStreamSynchronize(stream));
    static const char* roles[] = {"?", "producer", "mma", "epilogue", "setup"};
    const uint32_t role = words[0] >> 24;
    return fail(SG_ERR_TIMEOUT, "device-side wait expired: role %s, barrier %u, tile %u, parity %u, block %u",
                roles[role < 5 ? role : 0], words[0] & 0xFFFFFF, words[1], words[2], words[3]);
}

sg_status_t sg_sol_bound(int32_t op, const void* desc, int64_t batch_or_groups, const int64_t* M_host, int32_t eb_in,
                         int32_t eb_out, int32_t has_bias, const sg_hw_t* hw, sg_sol_t* out) {
    if (!desc || !hw || !out) return fail(SG_ERR_NULL_POINTER, "sg_sol_bound: desc, hw and out are required");
    if (eb_in <= 0 || eb_out <= 0 || has_bias < 0 || has_bias > 2) return fail(SG_ERR_INVALID_ARG, "sg_sol_bound: bad element size or has_bias");
    if (!(hw->peak_flops > 0.0) || !(hw->peak_bytes_per_s > 0.0)) return fail(SG_ERR_INVALID_ARG, "sg_sol_bound: peaks must be positive");
    int64_t macs = 0, elems_in = 0, elems_out = 0;   // inputs counted in input-type elements, C and D in output-type elements
    if (op == SG_OP_GEMM || op == SG_OP_BATCHED || op == SG_OP_GROUPED) {
        const sg_gemm_desc_t* g = static_cast<const sg_gemm_desc_t*>(desc);
        if (g->N < 0 || g->K < 0) return fail(SG_ERR_INVALID_ARG, "sg_sol_bound: negative extent");
        const bool reads_c = g->beta != 0.0f;
        if (op == SG_OP_GROUPED) {
            if (!M_host || batch_or_groups < 0) return fail(SG_ERR_INVALID_ARG, "sg_sol_bound: grouped needs M_host and groups >= 0");
            for (int64_t i = 0; i < batch_or_groups; ++i) {
                const int64_t m = M_host[i];
                if (m < 0) return fail(SG_ERR_INVALID_ARG, "sg_sol_bound: negative M");
                macs += m * g->N * g->K;
                elems_in += m * g->K + g->K * g->N + (has_bias ? g->N : 0);
                elems_out += m * g->N * (reads_c ? 2 : 1);
            }
        } else {
            const int64_t b = (op == SG_OP_BATCHED) ? batch_or_groups : 1;
            if (g->M < 0 || b < 0) return fail(SG_ERR_INVALID_ARG, "sg_sol_bound: negative extent");
            macs = b * g->M * g->N * g->K;
            elems_in = b * (g->M * g->K + g->K * g->N);
            if (has_bias == 1) elems_in += b * g->N;
            if (has_bias == 2) elems_in += g->N;
            elems_out = b * g->M * g->N * (reads_c ? 2 : 1);
        }
    } else if (op == SG_OP_CONV2D || op == SG_OP_CONV2D_DGRAD || op == SG_OP_CONV2D_WGRAD) {
        const sg_conv2d_desc_t* cv = static_cast<const sg_conv2d_desc_t*>(desc);
        if (cv->N < 0 || cv->H < 0 || cv->W < 0 || cv->C < 0 || cv->K < 0 || cv->R < 1 || cv->S < 1 || cv->stride_h < 1 ||
            cv->stride_w < 1 || cv->dil_h < 1 || cv->dil_w < 1 || cv->pad_h < 0 || cv->pad_w < 0)
            return fail(SG_ERR_INVALID_ARG, "sg_sol_bound: bad convolution descriptor");
        const int64_t sh = cv->H + 2 * cv->pad_h - cv->dil_h * (cv->R - 1) - 1;
        const int64_t sw = cv->W + 2 * cv->pad_w - cv->dil_w * (cv->S - 1) - 1;
        const int64_t P = sh < 0 ? 0 : sh / cv->stride_h + 1;
        const int64_t Q = sw < 0 ? 0 : sw / cv->stride_w + 1;
        macs = cv->N * P * Q * cv->K * cv->C * cv->R * cv->S;
        const int64_t x = cv->N * cv->H * cv->W * cv->C, w = cv->K * cv->R * cv->S * cv->C, y = cv->N * P * Q * cv->K;
        const int64_t rw = cv->beta != 0.0f ? 2 : 1;            // the output tensor is also read when beta != 0
        if (op == SG_OP_CONV2D) {
            elems_in = x + w + (has_bias ? cv->K : 0);
            elems_out = y * rw;
        } else if (op == SG_OP_CONV2D_DGRAD) {                   // reads dY and the filter, writes dX
            elems_in = y + w;
            elems_out = x * rw;
        } else {                                                 // reads dY and X, writes dW
            elems_in = y + x;
            elems_out = w * rw;
        }
    } else if (op == SG_OP_TRANSPOSE) {
        const sg_transpose_desc_t* t = static_cast<const sg_transpose_desc_t*>(desc);
        if (t->batch < 0 || t->rows < 0 || t->cols < 0) return fail(SG_ERR_INVALID_ARG, "sg_sol_bound: negative extent");
        elems_in = elems_out = t->batch * t->rows * t->cols;
        eb_in = t->in_dtype == SG_F32 ? 4 : 2;
        eb_out = t->out_dtype == SG_F32 ? 4 : 2;
    } else {
        return fail(SG_ERR_INVALID_ARG, "sg_sol_bound: op %d is not a sg_op_t", op);
    }
    out->flops = 2 * macs;
    out->bytes = elems_in * eb_in + elems_out * eb_out;
    const double sm_ratio = (hw->sm_clock_mhz > 0.0 && hw->sm_clock_max_mhz > 0.0) ? hw->sm_clock_mhz / hw->sm_clock_max_mhz : 1.0;
    const double mem_ratio = (hw->mem_clock_mhz > 0.0 && hw->mem_clock_max_mhz > 0.0) ? hw->mem_clock_mhz / hw->mem_clock_max_mhz : 1.0;
    out->eff_peak_flops = hw->peak_flops * sm_ratio;
    out->eff_bytes_per_s = hw->peak_bytes_per_s * mem_ratio;
    out->t_compute_s = static_cast<double>(out->flops) / out->eff_peak_flops;
    out->t_mem_s = static_cast<double>(out->bytes) / out->eff_bytes_per_s;
    out->t_sol_s = out->t_compute_s > out->t_mem_s ? out->t_compute_s : out->t_mem_s;
    out->ai = out->bytes > 0 ? static_cast<double>(out->flops) / static_cast<double>(out->bytes) : INFINITY;
    out->ridge = out->eff_peak_flops / out->eff_bytes_per_s;
    out->compute_bound = out->ai > out->ridge ? 1 : 0;
    out->reserved = 0;
    return SG_OK;
}

}  // extern "C"
