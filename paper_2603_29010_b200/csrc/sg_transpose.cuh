// Batched 2-D transpose with fused dtype conversion: out[b][c][r] = convert(in[b][r][c]).  A pure HBM-bound stage.
//
// transpose_tma_kernel (the path for 16-byte-multiple extents): persistent CTAs, one per SM.  A producer thread streams
// input tiles through a ring of shared-memory stages with TMA loads (cp.async.bulk.tensor, full / empty mbarriers);
// 256 consumer threads each move one block of the tile -- VO rows x VI columns, VI = elements per 16 bytes of the
// input type, VO of the output type -- with 16-byte shared-memory loads along the input rows, transpose it in
// registers (the conversion happens there), and write it with 16-byte stores into one of two output tiles, which a
// TMA store sends to memory (clipped at the tensor's extents).  Rows of both tiles are 256 bytes, so the bank group
// of an access is its 16-byte chunk index mod 8; the eight threads of a quarter warp are given blocks on a diagonal
// (distinct row-block AND distinct column-block indices mod 8), which makes the loads and the stores conflict-free
// without padding or swizzling.
// transpose_kernel (ragged extents): 64 x 64 element tiles through a padded shared-memory tile, plain 16-byte
// global accesses and element-wise edges.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cstdint>
#include "sg_ptx.cuh"

namespace sg {

struct TransposeParams {
    const void* in;
    void* out;
    int64_t rows, cols, ld_in, ld_out, stride_in, stride_out;
    int32_t tiles_r, tiles_c;
};

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <> __device__ __forceinline__ float to_f32<__half>(__half v) { return __half2float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }
template <> __device__ __forceinline__ __half from_f32<__half>(float v) { return __float2half_rn(v); }

// 16 bytes of consecutive elements (4 fp32 or 8 bf16) as one aligned vector access
template <typename T, int V>
__device__ __forceinline__ void load_vec(const T* p, float (&v)[V]) {
    if constexpr (sizeof(T) == 4) {
        const float4 x = *reinterpret_cast<const float4*>(p);
        v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
    } else {
        const uint4 x = *reinterpret_cast<const uint4*>(p);
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if constexpr (sizeof(T) == 2 && !__is_same(T, __nv_bfloat16)) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
                v[2 * i] = f.x;
                v[2 * i + 1] = f.y;
            } else {
                v[2 * i] = __uint_as_float(w[i] << 16);
                v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
            }
        }
    }
}
template <typename T, int V>
__device__ __forceinline__ void store_vec(T* p, const float (&v)[V]) {
    if constexpr (sizeof(T) == 4) {
        *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
    } else {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if constexpr (!__is_same(T, __nv_bfloat16)) {
                const __half2 h = __floats2half2_rn(v[2 * i], v[2 * i + 1]);
                w[i] = *reinterpret_cast<const uint32_t*>(&h);
            } else {
                const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
                w[i] = *reinterpret_cast<const uint32_t*>(&h);
            }
        }
        *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

template <typename TI, typename TO>
__global__ void __launch_bounds__(256) transpose_kernel(const TransposeParams p) {
    constexpr int T = 64;
    constexpr int VI = 16 / sizeof(TI);          // elements per 16-byte load
    constexpr int VO = 16 / sizeof(TO);          // elements per 16-byte store
    __shared__ float tile[T][T + 1];
    const int per_batch = p.tiles_r * p.tiles_c;
    const int b = blockIdx.x / per_batch;
    const int rem = blockIdx.x - b * per_batch;
    const int tr = rem / p.tiles_c;
    const int tc = rem - tr * p.tiles_c;
    const int64_t r0 = static_cast<int64_t>(tr) * T, c0 = static_cast<int64_t>(tc) * T;
    const TI* in = static_cast<const TI*>(p.in) + b * p.stride_in;
    TO* out = static_cast<TO*>(p.out) + b * p.stride_out;

    // read: T / VI threads cover one 64-element row with 16-byte loads
    {
        constexpr int TPR = T / VI;              // threads per row
        constexpr int RPP = 256 / TPR;           // rows per pass
        const int lc = (threadIdx.x % TPR) * VI;
        const int lr = threadIdx.x / TPR;
#pragma unroll
        for (int pass = 0; pass < T / RPP; ++pass) {
            const int r = lr + pass * RPP;
            const int64_t gr = r0 + r, gc = c0 + lc;
            float v[VI];
#pragma unroll
            for (int i = 0; i < VI; ++i) v[i] = 0.0f;
            if (gr < p.rows) {
                const TI* src = in + gr * p.ld_in + gc;
                if (gc + VI <= p.cols) {
                    load_vec<TI, VI>(src, v);
                } else {
                    for (int i = 0; i < VI; ++i) if (gc + i < p.cols) v[i] = to_f32<TI>(src[i]);
                }
            }
#pragma unroll
            for (int i = 0; i < VI; ++i) tile[r][lc + i] = v[i];
        }
    }
    __syncthreads();
    // write: an output row is an input column; T / VO threads cover the 64 input rows of one input column
    {
        constexpr int TPR = T / VO;
        constexpr int RPP = 256 / TPR;
        const int orr = (threadIdx.x % TPR) * VO;    // first of VO consecutive input rows
        const int occ = threadIdx.x / TPR;           // input column within the pass
#pragma unroll
        for (int pass = 0; pass < T / RPP; ++pass) {
            const int c = occ + pass * RPP;
            const int64_t gc = c0 + c, gr = r0 + orr;
            if (gc < p.cols && gr < p.rows) {
                float v[VO];
#pragma unroll
                for (int i = 0; i < VO; ++i) v[i] = tile[orr + i][c];
                TO* dst = out + gc * p.ld_out + gr;
                if (gr + VO <= p.rows) {
                    store_vec<TO, VO>(dst, v);
                } else {
                    for (int i = 0; i < VO; ++i) if (gr + i < p.rows) dst[i] = from_f32<TO>(v[i]);
                }
            }
        }
    }
}


// ---------------------------------------------------------------------------------------------- TMA kernel
struct TransposeTmaParams {
    CUtensorMap tm_in;       // [batch][rows][cols] input, box {TC, TR, 1}, no swizzle
    CUtensorMap tm_out;      // [batch][cols][rows] output, box {TR, TC, 1}, no swizzle
    int32_t tiles_r, tiles_c, num_tiles;
    uint32_t* status;        // device status words (word 0 is set when a wait runs out)
    uint64_t timeout_ns;     // bound of every wait
};

template <typename TI, typename TO>
struct TransposeCfg {
    static constexpr int VI = 16 / sizeof(TI);           // input elements per 16 bytes
    static constexpr int VO = 16 / sizeof(TO);           // output elements per 16 bytes
    static constexpr int TR = 16 * VO;                   // tile rows: the output tile's rows are 256 bytes
    static constexpr int TC = 16 * VI;                   // tile columns: the input tile's rows are 256 bytes
    static constexpr int IN_BYTES = TR * 256;
    static constexpr int OUT_BYTES = TC * 256;
    // 96 KB of loads in flight per SM.  Where both tiles are 16 KB (fp32 -> fp32: the shortest iterations) two CTAs share
    // an SM, three stages each, so that one CTA's barrier and store issue overlap the other's copying.
    static constexpr int CTAS_PER_SM = (IN_BYTES <= 16384 && OUT_BYTES <= 16384) ? 2 : 1;
    static constexpr int STAGES = (IN_BYTES <= 16384 && CTAS_PER_SM == 1) ? 6 : 3;
    static constexpr int OFF_OUT = STAGES * IN_BYTES;
    static constexpr int OUT_BUFS = 3;
    static constexpr int OFF_BAR = OFF_OUT + OUT_BUFS * OUT_BYTES;
    static constexpr int SMEM_BYTES = OFF_BAR + 2 * STAGES * 8 + 16;
    static constexpr int CONSUMERS = 256;
    static constexpr int THREADS = CONSUMERS + 32;
};

// AND-reduction of a predicate over the `count` threads that use named barrier `id` (also a barrier).
__device__ __forceinline__ bool bar_and(uint32_t id, uint32_t count, bool pred) {
    uint32_t out;
    asm volatile(
        "{\n"
        ".reg .pred p, q;\n"
        "setp.ne.u32 q, %3, 0;\n"
        "bar.red.and.pred p, %1, %2, q;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(out)
        : "r"(id), "r"(count), "r"(static_cast<uint32_t>(pred))
        : "memory");
    return out != 0;
}
__device__ __forceinline__ void bar_sync(uint32_t id, uint32_t count) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

// Bounded mbarrier wait; `abort_flag` (shared memory) is raised by whoever runs out of time so that everybody leaves.
static __device__ __noinline__ bool transpose_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                                   const TransposeTmaParams& p, uint32_t which) {
    const uint64_t t0 = global_timer_ns();
    uint32_t it = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++it & 63u) == 0) {
            if (*abort_flag != 0u) return false;
            if (global_timer_ns() - t0 > p.timeout_ns) {
                *abort_flag = 1u;
                if (atomicCAS(p.status, 0u, (5u << 24) | which) == 0u) {
                    volatile uint32_t* st = p.status;
                    st[1] = 0;
                    st[2] = parity;
                    st[3] = blockIdx.x;
                }
                return false;
            }
        }
    }
    return true;
}

template <typename TI, typename TO>
__global__ void __launch_bounds__(TransposeCfg<TI, TO>::THREADS, TransposeCfg<TI, TO>::CTAS_PER_SM) transpose_tma_kernel(const __grid_constant__ TransposeTmaParams p) {
    using Cfg = TransposeCfg<TI, TO>;
    constexpr int VI = Cfg::VI, VO = Cfg::VO, STAGES = Cfg::STAGES;
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bar_base = smem_base + Cfg::OFF_BAR;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + Cfg::OFF_BAR + 2 * STAGES * 8);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), Cfg::CONSUMERS);
        }
        *abort_flag = 0u;
        fence_barrier_init();
    }
    if (threadIdx.x == 32) {
        prefetch_tensormap(&p.tm_in);
        prefetch_tensormap(&p.tm_out);
    }
    __syncthreads();
    grid_dependency_wait();
    grid_launch_dependents();

    // Tile t -> (batch, tile row, tile column): consecutive tiles, which run at the same time on neighbouring SMs, are
    // neighbours along the input rows.  (Walking the tiles in two-dimensional groups, so that the writes join up as
    // well, measured no better on large matrices and worse on matrices with few rows of tiles.)
    const int per_batch = p.tiles_r * p.tiles_c;
    auto coords = [&](int t, int& b, int& r0, int& c0) {
        b = t / per_batch;
        const int rem = t - b * per_batch;
        const int tr = rem / p.tiles_c;
        r0 = tr * Cfg::TR;
        c0 = (rem - tr * p.tiles_c) * Cfg::TC;
    };

    if (threadIdx.x >= Cfg::CONSUMERS) {
        // ------------------------------------------------------------ producer (one lane)
        if (threadIdx.x == Cfg::CONSUMERS) {
            int stage = 0;
            uint32_t phase = 0;
            for (int t = blockIdx.x; t < p.num_tiles; t += gridDim.x) {
                int b, r0, c0;
                coords(t, b, r0, c0);                 // before the wait: the load goes out the moment the stage is free
                if (!transpose_wait(empty_bar(stage), phase ^ 1u, abort_flag, p, 100 + stage)) break;
                mbar_arrive_expect_tx(full_bar(stage), Cfg::IN_BYTES);
                tma_load_3d<false>(smem_base + stage * Cfg::IN_BYTES, &p.tm_in, full_bar(stage), c0, r0, b);
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
        return;
    }

    // ---------------------------------------------------------------- consumers
    // block of this thread: row block rb (VO rows), column block cb (VI columns); see the header comment
    const int tq = threadIdx.x & 7, g = threadIdx.x >> 3;
    const int rb = 8 * (g & 1) + tq;
    const int cb = 8 * ((g >> 1) & 1) + ((tq + (g >> 2)) & 7);
    int stage = 0, obuf = 0;
    uint32_t phase = 0;
    // One CTA-wide barrier per tile.  Three output tiles are in rotation: after issuing the store of tile i thread 0
    // waits until the store of tile i - 1 has read its tile, and only then joins the barrier of tile i + 1 -- so whoever
    // passes that barrier knows that the tile used for i + 2 (the one of i - 1) is free.
    for (int t = blockIdx.x; t < p.num_tiles; t += gridDim.x) {
        int tb, tr0, tc0;
        coords(t, tb, tr0, tc0);
        const bool ok = transpose_wait(full_bar(stage), phase, abort_flag, p, stage);
        if (ok) {
            float v[VO][VI];
            const uint8_t* src = smem + stage * Cfg::IN_BYTES + (rb * VO) * 256 + cb * 16;
#pragma unroll
            for (int i = 0; i < VO; ++i) {
                float row[VI];
                load_vec<TI, VI>(reinterpret_cast<const TI*>(src + i * 256), row);
#pragma unroll
                for (int j = 0; j < VI; ++j) v[i][j] = row[j];
            }
            mbar_arrive(empty_bar(stage));            // this thread has read its share of the stage
            uint8_t* dst = smem + Cfg::OFF_OUT + obuf * Cfg::OUT_BYTES + (cb * VI) * 256 + rb * 16;
#pragma unroll
            for (int j = 0; j < VI; ++j) {
                float col[VO];
#pragma unroll
                for (int i = 0; i < VO; ++i) col[i] = v[i][j];
                store_vec<TO, VO>(reinterpret_cast<TO*>(dst + j * 256), col);
            }
            fence_proxy_async_smem();
        }
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        if (!bar_and(1, Cfg::CONSUMERS, ok)) break;   // everybody leaves together when a wait ran out
        if (threadIdx.x == 0) {
            tma_store_3d(&p.tm_out, smem_base + Cfg::OFF_OUT + obuf * Cfg::OUT_BYTES, tr0, tc0, tb);
            tma_store_commit();
            tma_store_wait_read<1>();
        }
        if (++obuf == Cfg::OUT_BUFS) obuf = 0;
    }
    if (threadIdx.x == 0) tma_store_wait_read<0>();   // shared memory must outlive the stores' reads
    if (*abort_flag != 0u) {
        // a wait ran out: give loads still in flight time to land before the CTA's shared memory goes away
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
}

}  // namespace sg
