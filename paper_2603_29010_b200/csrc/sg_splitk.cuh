// Second pass of a two-pass K split: sums the partial tiles that the contraction kernel's parts parked in the scratch
// and runs the epilogue on the totals.
//
// Problems with few output tiles and a long K loop (a skinny GEMM, the convolution weight gradient) are cut into many
// K ranges -- as many as there are SMs to go round -- each run by its own CTA (or CTA pair) of the contraction kernel,
// which stores its raw fp32 sums and exits: no flags, no waiting for a peer.  This kernel, launched behind it on the
// same stream, adds the parts up in part order (reproducible for a given plan), applies alpha, beta C, the bias and
// the activation exactly as the fused epilogue does, and writes D.  (The DSL's `splits=` / `.with_split_k`, Appendix A.1.)
//
// Layout of a parked CTA tile (128 rows x BN columns, see the contraction kernel): units of 32 rows x CH columns
// (CH = 64 for 16-bit outputs, 32 for fp32), unit (chunk c, lane quarter q) at float offset (4 c + q) 32 CH, inside it
// column group i (a multiple of 4) of row `lane` at i * 32 + 4 * lane: a warp reads 512 contiguous bytes per access.
#pragma once
#include "sg_kernel.cuh"

namespace sg {

struct SplitKReduceParams {
    const float* partials;      // [tile][part][CTA of the tile][128 x BN] fp32
    const uint32_t* status;     // device status word 0: non-zero makes this launch a no-op, like the first pass
    int32_t nparts, kctas, bn;
    int32_t pw;                 // warps of a block that share the parts of one column slice: 1, 2, 4 or 8
    int32_t tiles_m, tiles_n;   // tiles of one problem; tile r of a problem is (r % tiles_m, r / tiles_m)
    int32_t M, N, batch;
    void* D;
    const void* C;
    const void* bias;
    int64_t ldd, strideD, ldc, strideC, strideBias;
    float alpha, beta, epi_arg0, epi_arg1;
    int32_t epi, in_f16, bias_f32;
};

// A unit = (tile, CTA of the tile, chunk, lane quarter) has 8 column slices of CH / 8 columns (two groups of 4, or one
// for fp32 outputs).  grid: pw blocks per unit, each with 8 / pw slices; the pw warps of a slice share the parts (warp g
// adds parts g, g + pw, ..., lane = row), their sums are added in warp order through shared memory (a fixed order:
// reproducible), and the first of them runs the epilogue.  The host picks pw from the number of parts: few parts want few,
// fat blocks (launching blocks is not free), many parts want the parallelism.
template <int kOut, int PW>
__global__ void __launch_bounds__(256) splitk_reduce_kernel(const SplitKReduceParams p) {
    constexpr bool kOutF32 = (kOut == 1);
    constexpr bool kOutF16 = (kOut == 2);
    constexpr int CH = kOutF32 ? 32 : 64;
    constexpr int NV = CH / 8;                       // columns per block: 8 (two groups of 4) or 4
    __shared__ float part_sums[8][NV][32];
    grid_dependency_wait();                          // the first pass has finished and its sums are visible
    grid_launch_dependents();
    if (*reinterpret_cast<const volatile uint32_t*>(p.status) != 0u) return;
    const int chunks = p.bn / CH;
    int u = blockIdx.x;
    const int lane = threadIdx.x & 31, j = threadIdx.x >> 5;
    constexpr int pw = PW;
    const int g = j & (pw - 1);                      // which share of the parts this warp adds
    const int w = (u & (pw - 1)) * (8 / pw) + j / pw;   // column slice inside the chunk
    u /= pw;
    const int q = u & 3; u >>= 2;
    const int c = u % chunks; u /= chunks;
    const int cta = u % p.kctas;
    const int tile = u / p.kctas;
    const int per = p.tiles_m * p.tiles_n;
    const int b = tile / per;
    const int r = tile - b * per;
    const int tn = r / p.tiles_m, tm = r - tn * p.tiles_m;
    const int row = (tm * p.kctas + cta) * 128 + q * 32 + lane;
    const int col0 = tn * p.bn + c * CH + w * NV;
    const bool exists = (tm * p.kctas + cta) * 128 + q * 32 < p.M && col0 < p.N;      // else nobody parked this slice

    const size_t tile_elems = static_cast<size_t>(128) * p.bn;
    const float* src = p.partials + (static_cast<size_t>(tile) * p.nparts * p.kctas + cta) * tile_elems +
                       static_cast<size_t>(c * 4 + q) * (CH * 32) + static_cast<size_t>(w * NV) * 32 + lane * 4;
    float v[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) v[i] = 0.0f;
    const size_t part_stride = static_cast<size_t>(p.kctas) * tile_elems;
    if (exists) {
#pragma unroll 4
        for (int h = g; h < p.nparts; h += PW) {
#pragma unroll
            for (int i = 0; i < NV; i += 4) {
                const float4 y = __ldcg(reinterpret_cast<const float4*>(src + static_cast<size_t>(h) * part_stride + i * 32));
                v[i] += y.x; v[i + 1] += y.y; v[i + 2] += y.z; v[i + 3] += y.w;
            }
        }
    }
#pragma unroll
    for (int i = 0; i < NV; ++i) part_sums[j][i][lane] = v[i];
    __syncthreads();
    if (g != 0 || !exists) return;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        float t = part_sums[j][i][lane];
#pragma unroll
        for (int k = 1; k < PW; ++k) t += part_sums[j + k][i][lane];
        v[i] = t;
    }
    if (row >= p.M || col0 >= p.N) return;
    if (p.alpha != 1.0f) {
#pragma unroll
        for (int i = 0; i < NV; ++i) v[i] *= p.alpha;
    }
    const int valid = min(NV, p.N - col0);
    if (p.beta != 0.0f) {
        if constexpr (kOutF32) {
            const float* cp = reinterpret_cast<const float*>(p.C) + static_cast<int64_t>(b) * p.strideC + static_cast<int64_t>(row) * p.ldc + col0;
            for (int i = 0; i < valid; ++i) v[i] += p.beta * cp[i];
        } else {
            const uint16_t* cp = reinterpret_cast<const uint16_t*>(p.C) + static_cast<int64_t>(b) * p.strideC + static_cast<int64_t>(row) * p.ldc + col0;
            for (int i = 0; i < valid; ++i) v[i] += p.beta * half_bits_to_float(cp[i], kOutF16);
        }
    }
    if (p.bias != nullptr) {
        if (p.bias_f32) {
            const float* bp = reinterpret_cast<const float*>(p.bias) + static_cast<int64_t>(b) * p.strideBias + col0;
            for (int i = 0; i < valid; ++i) v[i] += bp[i];
        } else {
            const uint16_t* bp = reinterpret_cast<const uint16_t*>(p.bias) + static_cast<int64_t>(b) * p.strideBias + col0;
            for (int i = 0; i < valid; ++i) v[i] += half_bits_to_float(bp[i], p.in_f16 != 0);
        }
    }
    if (p.epi >= EPI_RELU) apply_act_chunk<kOut == 0, NV>(v, p.epi, p.epi_arg0, p.epi_arg1);
    if constexpr (kOutF32) {
        float* dp = reinterpret_cast<float*>(p.D) + static_cast<int64_t>(b) * p.strideD + static_cast<int64_t>(row) * p.ldd + col0;
        if (valid == NV && (reinterpret_cast<uintptr_t>(dp) & 15u) == 0) {
            *reinterpret_cast<float4*>(dp) = make_float4(v[0], v[1], v[2], v[3]);
        } else {
            for (int i = 0; i < valid; ++i) dp[i] = v[i];
        }
    } else {
        uint16_t* dp = reinterpret_cast<uint16_t*>(p.D) + static_cast<int64_t>(b) * p.strideD + static_cast<int64_t>(row) * p.ldd + col0;
        if (valid == NV && (reinterpret_cast<uintptr_t>(dp) & 15u) == 0) {
            *reinterpret_cast<uint4*>(dp) = make_uint4(pack2<kOutF16>(v[0], v[1]), pack2<kOutF16>(v[2], v[3]),
                                                       pack2<kOutF16>(v[4], v[5]), pack2<kOutF16>(v[6], v[7]));
        } else {
            for (int i = 0; i < valid; ++i) dp[i] = static_cast<uint16_t>(pack2<kOutF16>(v[i], 0.0f) & 0xFFFFu);
        }
    }
}

}  // namespace sg
