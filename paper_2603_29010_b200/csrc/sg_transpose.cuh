// Batched 2-D transpose with fused dtype conversion: out[b][c][r] = convert(in[b][r][c]).
// A pure HBM-bound stage: 64 x 64 element tiles go through a padded shared-memory tile so that both the
// global reads (along cols) and the global writes (along rows) are contiguous 8- or 16-byte accesses.
#pragma once
#include <cuda_bf16.h>
#include <cstdint>

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
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

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
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
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
            const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
            w[i] = *reinterpret_cast<const uint32_t*>(&h);
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

}  // namespace sg
