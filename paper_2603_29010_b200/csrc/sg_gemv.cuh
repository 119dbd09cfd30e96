// Matrix-vector products with the fused epilogue: out[r][v] = act(alpha * sum_k W[r][k] x_v[k] + beta * C + bias), for
// up to 32 vectors x_v at once.  The GEMM with N <= 8 (or M <= 8) of the paper's workload list (single-token
// decode): every matrix element is used once per vector, so the kernels are a stream over W bound by HBM, and the
// tcgen05 tiles (128 rows for at most eight useful ones, operands staged in shared memory) have nothing to offer.
// Two kernels: gemv_kernel (CUDA-core FMAs: one vector; fp32 inputs or a ragged K: up to four) and gemv_mma_kernel
// (warp-level MMAs: two to eight vectors of 16-bit inputs, and nine to 32 against matrices small enough that the
// tiles' fixed cost would decide the time).
//
// Work split of gemv_kernel: a CTA of 256 threads takes RB consecutive rows and one K range; each thread walks the
// range in 16-byte vectors (one vector of x serves RB vectors of W, so RB independent loads are in flight per thread
// and iteration), sums in fp32, and the CTA reduces with shuffles and shared memory.  K ranges of one row block are
// the CTAs of one thread-block cluster: rank 0 adds the other ranks' partial sums in rank order through distributed
// shared memory (no global scratch, no atomics; the result depends only on the launch geometry).
#pragma once
#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cstdint>

namespace sg {

struct GemvParams {
    const void* W;        // [R][ld], K contiguous
    const void* x;        // nvec vectors [K], contiguous, x_stride elements apart
    const void* C;        // residual (output type) or null
    const void* bias;     // input type (fp32 for fp32 inputs) or null
    void* D;
    const uint32_t* status;   // the library's device status word: while it is set (an expired wait of an earlier launch,
                              // not yet reported by sg_poll_status) nothing is stored
    int64_t ld;           // elements between rows of W
    int64_t x_stride;
    int64_t c_row_stride, c_vec_stride, d_row_stride, d_vec_stride;   // element (row r, vector v) of C and D
    int32_t R, K;
    int32_t nvec;         // gemv_kernel: 1..4; gemv_mma_kernel: any number, in groups of 8, 16 or 32 along gridDim.y
    int32_t kchunk;       // K elements per cluster rank (a multiple of 256 vectors)
    int32_t ksplit;       // CTAs per cluster
    int32_t bias_row_stride, bias_vec_stride;   // (0, 1): one bias per vector (the matrix is A); (1, 0): one per row
    int32_t out_kind;     // 0 bf16, 1 fp32, 2 fp16
    int32_t epi;
    float alpha, beta, a0, a1;
};

__device__ __forceinline__ uint4 ldg_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// 16 bytes of input elements as fp32 values; fp32 inputs are read the way the tensor cores read them (tf32: the low
// 13 fraction bits dropped), so that both paths of the library compute the same product.
template <typename T> struct GemvVec;
template <> struct GemvVec<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ void cvt(const uint4& u, float (&f)[8]) {
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    static __device__ __forceinline__ float one(const __nv_bfloat16* p) { return __bfloat162float(*p); }
    static __device__ __forceinline__ float exact(const __nv_bfloat16* p) { return __bfloat162float(*p); }
};
template <> struct GemvVec<__half> {
    static constexpr int N = 8;
    static __device__ __forceinline__ void cvt(const uint4& u, float (&f)[8]) {
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 v = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
            f[2 * i] = v.x;
            f[2 * i + 1] = v.y;
        }
    }
    static __device__ __forceinline__ float one(const __half* p) { return __half2float(*p); }
    static __device__ __forceinline__ float exact(const __half* p) { return __half2float(*p); }
};
template <> struct GemvVec<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ void cvt(const uint4& u, float (&f)[4]) {
        f[0] = __uint_as_float(u.x & 0xFFFFE000u);
        f[1] = __uint_as_float(u.y & 0xFFFFE000u);
        f[2] = __uint_as_float(u.z & 0xFFFFE000u);
        f[3] = __uint_as_float(u.w & 0xFFFFE000u);
    }
    static __device__ __forceinline__ float one(const float* p) { return __uint_as_float(__float_as_uint(*p) & 0xFFFFE000u); }
    static __device__ __forceinline__ float exact(const float* p) { return *p; }      // the bias is not an MMA operand
};

__device__ __forceinline__ float gemv_load_out(const void* base, int64_t i, int out_kind) {
    if (out_kind == 1) return reinterpret_cast<const float*>(base)[i];
    if (out_kind == 2) return __half2float(reinterpret_cast<const __half*>(base)[i]);
    return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(base)[i]);
}
__device__ __forceinline__ void gemv_store_out(void* base, int64_t i, int out_kind, float v) {
    if (out_kind == 1) reinterpret_cast<float*>(base)[i] = v;
    else if (out_kind == 2) reinterpret_cast<__half*>(base)[i] = __float2half_rn(v);
    else reinterpret_cast<__nv_bfloat16*>(base)[i] = __float2bfloat16_rn(v);
}

// Four rows per CTA and a register budget that lets four CTAs of 16-bit inputs share an SM measured best (more,
// smaller CTAs balance better over the SMs than eight rows per CTA; deeper unrolling did not help).
// NV = vectors handled at once (1, 2 or 4; three vectors run as four with the last one repeated and not stored);
// with several vectors a budget of 85 registers (three CTAs per SM) measured best: two leave too few loads in
// flight, four spill.
template <typename T, int RB, int NV>
__global__ void __launch_bounds__(256, (sizeof(T) == 2 && RB == 4 && NV == 1) ? 4 : (NV > 1 ? 3 : 1)) gemv_kernel(const GemvParams p) {
    namespace cg = cooperative_groups;
    constexpr int V = GemvVec<T>::N;
    constexpr int WARPS = 8;
    constexpr int NACC = RB * NV;
    __shared__ float warp_part[WARPS][NACC];
    __shared__ float cta_part[NACC];
    // Programmatic dependent launch: the CTAs of this launch may become resident while the previous kernel of the stream
    // is still finishing; nothing of global memory is touched before that kernel has completed.
    grid_dependency_wait();
    grid_launch_dependents();
    // fetched now, looked at before the stores at the very end: the load's latency hides behind the sweep
    const uint32_t sticky = p.status != nullptr ? *reinterpret_cast<const volatile uint32_t*>(p.status) : 0u;

    const int ks = p.ksplit;
    const int rank = static_cast<int>(blockIdx.x % static_cast<unsigned>(ks));      // = rank in the (ks, 1, 1) cluster
    const int64_t r0 = static_cast<int64_t>(blockIdx.x / static_cast<unsigned>(ks)) * RB;
    const int kbeg = rank * p.kchunk;
    const int kend = min(p.K, kbeg + p.kchunk);
    const int kvec_end = kbeg < kend ? kbeg + ((kend - kbeg) / V) * V : kbeg;

    const T* x[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) x[v] = reinterpret_cast<const T*>(p.x) + static_cast<int64_t>(min(v, p.nvec - 1)) * p.x_stride;
    const T* w[RB];
#pragma unroll
    for (int i = 0; i < RB; ++i) {
        // rows past the end read the last row again (a valid address); their sums are never stored
        const int64_t r = min(r0 + i, static_cast<int64_t>(p.R) - 1);
        w[i] = reinterpret_cast<const T*>(p.W) + r * p.ld;
    }
    float acc[RB][NV];
#pragma unroll
    for (int i = 0; i < RB; ++i) {
#pragma unroll
        for (int v = 0; v < NV; ++v) acc[i][v] = 0.0f;
    }

#pragma unroll 2
    for (int k = kbeg + static_cast<int>(threadIdx.x) * V; k < kvec_end; k += 256 * V) {
        uint4 wv[RB], xv[NV];
#pragma unroll
        for (int i = 0; i < RB; ++i) wv[i] = ldg_stream16(w[i] + k);
#pragma unroll
        for (int v = 0; v < NV; ++v) xv[v] = __ldg(reinterpret_cast<const uint4*>(x[v] + k));
        float wf[RB][V];
#pragma unroll
        for (int i = 0; i < RB; ++i) GemvVec<T>::cvt(wv[i], wf[i]);
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            float xf[V];
            GemvVec<T>::cvt(xv[v], xf);
#pragma unroll
            for (int i = 0; i < RB; ++i) {
#pragma unroll
                for (int j = 0; j < V; ++j) acc[i][v] = fmaf(wf[i][j], xf[j], acc[i][v]);
            }
        }
    }
    // the last K % V elements (only the last rank has any)
    {
        const int kt = kvec_end + static_cast<int>(threadIdx.x);
        if (kt < kend) {
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                const float xv = GemvVec<T>::one(x[v] + kt);
#pragma unroll
                for (int i = 0; i < RB; ++i) acc[i][v] = fmaf(GemvVec<T>::one(w[i] + kt), xv, acc[i][v]);
            }
        }
    }

#pragma unroll
    for (int i = 0; i < RB; ++i) {
#pragma unroll
        for (int v = 0; v < NV; ++v) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) acc[i][v] += __shfl_xor_sync(0xFFFFFFFFu, acc[i][v], off);
        }
    }
    const int warp = static_cast<int>(threadIdx.x) >> 5, lane = static_cast<int>(threadIdx.x) & 31;
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < RB; ++i) {
#pragma unroll
            for (int v = 0; v < NV; ++v) warp_part[warp][i * NV + v] = acc[i][v];
        }
    }
    __syncthreads();
    if (threadIdx.x < NACC) {
        float s = 0.0f;
#pragma unroll
        for (int wi = 0; wi < WARPS; ++wi) s += warp_part[wi][threadIdx.x];
        cta_part[threadIdx.x] = s;
    }
    if (ks > 1) cg::this_cluster().sync();
    if (rank == 0 && threadIdx.x < NACC) {
        float s = cta_part[threadIdx.x];
        if (ks > 1) {
            cg::cluster_group cluster = cg::this_cluster();
            for (int r = 1; r < ks; ++r) s += *cluster.map_shared_rank(&cta_part[threadIdx.x], r);
        }
        const int64_t row = r0 + static_cast<int>(threadIdx.x) / NV;
        const int vec = static_cast<int>(threadIdx.x) % NV;
        if (row < p.R && vec < p.nvec) {
            float v[1] = {p.alpha * s};
            if (p.beta != 0.0f) v[0] = fmaf(p.beta, gemv_load_out(p.C, row * p.c_row_stride + vec * p.c_vec_stride, p.out_kind), v[0]);
            if (p.bias != nullptr)
                v[0] += GemvVec<T>::exact(reinterpret_cast<const T*>(p.bias) + row * p.bias_row_stride + vec * p.bias_vec_stride);
            if (p.epi >= EPI_RELU) apply_act_chunk<false, 1>(v, p.epi, p.a0, p.a1);
            if (!sticky) gemv_store_out(p.D, row * p.d_row_stride + vec * p.d_vec_stride, p.out_kind, v[0]);
        }
    }
    if (ks > 1) cg::this_cluster().sync();      // keep every rank's shared memory alive until rank 0 has read it
}

// Two to eight vectors of 16-bit inputs: the multiply-adds of the kernel above would saturate the FMA pipe (8 vectors =
// 64 FMAs per 16 bytes of W), so the products go through warp-level tensor-core MMAs (m16n8k16, fp32 accumulation):
// a warp owns 16 rows x 8 vectors, needs four accumulator registers per thread, and one MMA consumes what 16 rows x
// 16 k took 256 FMAs-lanes.  tcgen05 has no shape for this (its tiles are 64 or 128 rows fed from shared memory);
// the kernel stays a stream over W bound by HBM.
// Fragment trick: the MMA sums over k, so any permutation of k applied to both operands gives the same result.  Thread
// (g = lane / 4, t = lane % 4) loads 16 bytes = 8 consecutive k of rows g and g + 8 and of vector g, all at
// k0 + 8 t, and feeds word pairs (0, 1) and (2, 3) of those loads to two MMAs: the MMA's "k = 2t, 2t+1" and
// "k = 2t+8, 2t+9" slots then hold the same physical k on the A and on the B side.  The four lanes of a row read 64
// contiguous bytes; the eight warps of a CTA interleave their steps, so a CTA reads 512 contiguous bytes per row.
template <typename T> struct GemvMma;
template <> struct GemvMma<__nv_bfloat16> {
    static __device__ __forceinline__ void mma(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                     : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    }
};
template <> struct GemvMma<__half> {
    static __device__ __forceinline__ void mma(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                     : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    }
};

// 256-bit global load (sm_100): 32 contiguous bytes per thread, so the four lanes of a row fetch a whole 128-byte line
// with one instruction (with 16-byte loads a warp-wide load covers 16 row pieces of 64 bytes: twice the number of
// memory transactions per byte).
struct U8 {
    uint32_t w[8];
};
__device__ __forceinline__ U8 ldg_stream32(const void* p) {
    U8 v;
    asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]), "=r"(v.w[4]), "=r"(v.w[5]), "=r"(v.w[6]), "=r"(v.w[7])
                 : "l"(p));
    return v;
}
__device__ __forceinline__ U8 ldg_cached32(const void* p) {
    U8 v;
    asm volatile("ld.global.nc.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]), "=r"(v.w[4]), "=r"(v.w[5]), "=r"(v.w[6]), "=r"(v.w[7])
                 : "l"(p));
    return v;
}

// kWide = false: 16-byte pieces; requires K % 8 == 0 and kchunk % 256 == 0.
// kWide = true: 32-byte pieces; requires K % 16 == 0, kchunk % 512 == 0 and 32-byte aligned rows and vectors.
// NVB: blocks of eight vectors (1, 2 or 4: up to 8, 16 or 32 vectors).  Every block is one more MMA per piece of W on
// the same A fragment and four more accumulator registers; thread group g loads vectors g, g + 8, g + 16, g + 24.
// Grid: x = ceil(R / 16) row blocks x ksplit ranks; y = groups of 8 NVB vectors (more than one group: a small GEMM whose
// every CTA reads 16 rows of one operand and 8 NVB rows of the other once -- no shared-memory staging, no tensor
// memory, one memory round trip: what a product of a few hundred rows and columns needs is latency, not tiles).
template <typename T, bool kWide, int NVB = 1>
__global__ void __launch_bounds__(256) gemv_mma_kernel(const GemvParams p) {
    namespace cg = cooperative_groups;
    constexpr int WARPS = 8;
    constexpr int PE = kWide ? 16 : 8;        // elements per thread and step
    constexpr int U = (kWide ? 2 : 4) / (NVB == 4 ? 2 : 1);   // steps in flight per warp (fewer with 32 vectors: registers)
    constexpr int STEP = 4 * PE;              // elements of K a warp covers per step
    constexpr int NV = 8 * NVB;               // vector slots
    __shared__ float warp_part[WARPS][16 * NV];   // 16 rows x NV vectors per warp
    __shared__ float cta_part[16 * NV];
    // Programmatic dependent launch: the CTAs of this launch may become resident while the previous kernel of the stream
    // is still finishing; nothing of global memory is touched before that kernel has completed.
    grid_dependency_wait();
    grid_launch_dependents();
    // fetched now, looked at before the stores at the very end: the load's latency hides behind the sweep
    const uint32_t sticky = p.status != nullptr ? *reinterpret_cast<const volatile uint32_t*>(p.status) : 0u;

    const int ks = p.ksplit;
    // x = row blocks x ranks with one group of vectors; with several groups x = ranks, y = groups, z = row blocks, so
    // that the CTAs that read the same 16 rows of W are neighbours in launch order and find them in the L2
    const bool grouped = gridDim.y > 1;
    const int rank = grouped ? static_cast<int>(blockIdx.x) : static_cast<int>(blockIdx.x % static_cast<unsigned>(ks));
    const int64_t r0 = static_cast<int64_t>(grouped ? blockIdx.z : blockIdx.x / static_cast<unsigned>(ks)) * 16;
    const int kbeg = rank * p.kchunk;
    const int kend = min(p.K, kbeg + p.kchunk);
    const int warp = static_cast<int>(threadIdx.x) >> 5, lane = static_cast<int>(threadIdx.x) & 31;
    const int g = lane >> 2, t = lane & 3;
    const int v0 = static_cast<int>(blockIdx.y) * NV;        // first vector of this CTA's group

    const T* wlo = reinterpret_cast<const T*>(p.W) + min(r0 + g, static_cast<int64_t>(p.R) - 1) * p.ld;
    const T* whi = reinterpret_cast<const T*>(p.W) + min(r0 + g + 8, static_cast<int64_t>(p.R) - 1) * p.ld;
    const T* xv[NVB];
    float c[NVB][4];
#pragma unroll
    for (int j = 0; j < NVB; ++j) {
        xv[j] = reinterpret_cast<const T*>(p.x) + static_cast<int64_t>(min(v0 + g + 8 * j, p.nvec - 1)) * p.x_stride;
        c[j][0] = c[j][1] = c[j][2] = c[j][3] = 0.0f;
    }

    // The loop bounds are the same for all lanes of a warp (mma.sync must be executed by the whole warp).  Main loop:
    // U steps whose pieces all lie inside the K range, loads without conditions; then single steps in which a lane
    // whose piece lies past the end contributes zeros.
    int kw = kbeg + warp * STEP;
    for (; kw + (U - 1) * WARPS * STEP + STEP <= kend; kw += U * WARPS * STEP) {
        const int k0 = kw + t * PE;
        if constexpr (kWide) {
            U8 lo[U], hi[U], xx[U][NVB];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                lo[u] = ldg_stream32(wlo + k0 + u * WARPS * STEP);
                hi[u] = ldg_stream32(whi + k0 + u * WARPS * STEP);
#pragma unroll
                for (int b = 0; b < NVB; ++b) xx[u][b] = ldg_cached32(xv[b] + k0 + u * WARPS * STEP);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
#pragma unroll
                for (int b = 0; b < NVB; ++b) {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        GemvMma<T>::mma(c[b], lo[u].w[2 * j], hi[u].w[2 * j], lo[u].w[2 * j + 1], hi[u].w[2 * j + 1],
                                        xx[u][b].w[2 * j], xx[u][b].w[2 * j + 1]);
                }
            }
        } else {
            uint4 lo[U], hi[U], xx[U][NVB];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                lo[u] = ldg_stream16(wlo + k0 + u * WARPS * STEP);
                hi[u] = ldg_stream16(whi + k0 + u * WARPS * STEP);
#pragma unroll
                for (int b = 0; b < NVB; ++b) xx[u][b] = __ldg(reinterpret_cast<const uint4*>(xv[b] + k0 + u * WARPS * STEP));
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
#pragma unroll
                for (int b = 0; b < NVB; ++b) {
                    GemvMma<T>::mma(c[b], lo[u].x, hi[u].x, lo[u].y, hi[u].y, xx[u][b].x, xx[u][b].y);
                    GemvMma<T>::mma(c[b], lo[u].z, hi[u].z, lo[u].w, hi[u].w, xx[u][b].z, xx[u][b].w);
                }
            }
        }
    }
    for (; kw < kend; kw += WARPS * STEP) {
        const int k = kw + t * PE;
        const bool valid = k < kend;        // pieces are whole: K, kbeg and k are multiples of PE
        if constexpr (kWide) {
            U8 lo, hi, xx[NVB];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                lo.w[j] = hi.w[j] = 0u;
#pragma unroll
                for (int b = 0; b < NVB; ++b) xx[b].w[j] = 0u;
            }
            if (valid) {
                lo = ldg_stream32(wlo + k);
                hi = ldg_stream32(whi + k);
#pragma unroll
                for (int b = 0; b < NVB; ++b) xx[b] = ldg_cached32(xv[b] + k);
            }
#pragma unroll
            for (int b = 0; b < NVB; ++b) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    GemvMma<T>::mma(c[b], lo.w[2 * j], hi.w[2 * j], lo.w[2 * j + 1], hi.w[2 * j + 1], xx[b].w[2 * j], xx[b].w[2 * j + 1]);
            }
        } else {
            uint4 lo = make_uint4(0u, 0u, 0u, 0u), hi = lo, xx[NVB];
#pragma unroll
            for (int b = 0; b < NVB; ++b) xx[b] = lo;
            if (valid) {
                lo = ldg_stream16(wlo + k);
                hi = ldg_stream16(whi + k);
#pragma unroll
                for (int b = 0; b < NVB; ++b) xx[b] = __ldg(reinterpret_cast<const uint4*>(xv[b] + k));
            }
#pragma unroll
            for (int b = 0; b < NVB; ++b) {
                GemvMma<T>::mma(c[b], lo.x, hi.x, lo.y, hi.y, xx[b].x, xx[b].y);
                GemvMma<T>::mma(c[b], lo.z, hi.z, lo.w, hi.w, xx[b].z, xx[b].w);
            }
        }
    }
    // accumulator fragment of block b: c0 (row g, vector 8b + 2t), c1 (g, 8b + 2t+1), c2 (g+8, 8b + 2t), c3 (g+8, 8b + 2t+1)
#pragma unroll
    for (int b = 0; b < NVB; ++b) {
        warp_part[warp][g * NV + 8 * b + 2 * t] = c[b][0];
        warp_part[warp][g * NV + 8 * b + 2 * t + 1] = c[b][1];
        warp_part[warp][(g + 8) * NV + 8 * b + 2 * t] = c[b][2];
        warp_part[warp][(g + 8) * NV + 8 * b + 2 * t + 1] = c[b][3];
    }
    __syncthreads();
    for (int i = static_cast<int>(threadIdx.x); i < 16 * NV; i += 256) {
        float s = 0.0f;
#pragma unroll
        for (int wi = 0; wi < WARPS; ++wi) s += warp_part[wi][i];
        cta_part[i] = s;
    }
    if (ks > 1) cg::this_cluster().sync();
    for (int i = static_cast<int>(threadIdx.x); rank == 0 && i < 16 * NV; i += 256) {
        float s = cta_part[i];
        if (ks > 1) {
            cg::cluster_group cluster = cg::this_cluster();
            for (int r = 1; r < ks; ++r) s += *cluster.map_shared_rank(&cta_part[i], r);
        }
        const int64_t row = r0 + i / NV;
        const int vec = v0 + i % NV;
        if (row < p.R && vec < p.nvec) {
            float v[1] = {p.alpha * s};
            if (p.beta != 0.0f) v[0] = fmaf(p.beta, gemv_load_out(p.C, row * p.c_row_stride + vec * p.c_vec_stride, p.out_kind), v[0]);
            if (p.bias != nullptr)
                v[0] += GemvVec<T>::exact(reinterpret_cast<const T*>(p.bias) + row * p.bias_row_stride + vec * p.bias_vec_stride);
            if (p.epi >= EPI_RELU) apply_act_chunk<false, 1>(v, p.epi, p.a0, p.a1);
            if (!sticky) gemv_store_out(p.D, row * p.d_row_stride + vec * p.d_vec_stride, p.out_kind, v[0]);
        }
    }
    if (ks > 1) cg::this_cluster().sync();
}

}  // namespace sg
