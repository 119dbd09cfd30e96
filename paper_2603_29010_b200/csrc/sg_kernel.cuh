// The persistent, warp-specialised tcgen05 contraction kernel shared by sg_gemm, sg_batched_gemm,
// sg_grouped_gemm and sg_conv2d_fprop.
//
// One CTA (or a pair of CTAs on neighbouring SMs) owns one output tile at a time and walks a static
// round-robin list of tiles.  Inside the CTA the work is split by warp:
//
//   warp 0      producer   one lane issues TMA loads of the A and B k-blocks into a ring of
//                          shared-memory stages (128-byte swizzled rows of 64 bf16)
//   warp 1      MMA        allocates TMEM; one lane issues tcgen05.mma (bf16 x bf16 -> fp32 in
//                          TMEM) for every k-block and commits to mbarriers
//   warps 2-5   epilogue   tcgen05.ld TMEM -> registers, v = alpha*acc + beta*C + bias, activation,
//                          cast, swizzled st.shared, one TMA store per 32-row x 128-byte chunk
//
// Two accumulator buffers live in TMEM, so the epilogue of tile i overlaps the main loop of tile
// i+1.  Every mbarrier wait is bounded: when one expires the kernel records where, raises a flag all
// roles poll, lets outstanding copies land, frees TMEM and returns.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include "sg_ptx.cuh"

namespace sg {

enum : int32_t { MODE_DENSE = 0, MODE_GROUPED = 1, MODE_CONV = 2, MODE_WGRAD = 3 };
enum : int32_t { EPI_NONE = 0, EPI_BIAS = 1, EPI_RELU = 2, EPI_GELU = 3, EPI_SILU = 4, EPI_SIGMOID = 5, EPI_TANH = 6,
                 EPI_MISH = 7, EPI_HARDSWISH = 8, EPI_LEAKY_RELU = 9, EPI_ELU = 10, EPI_CLIP = 11 };

// status word 0: 0 = fine, else (role << 24 | detail); words 1..3 hold tile / barrier / block of the first failure
enum : uint32_t { ROLE_PRODUCER = 1, ROLE_MMA = 2, ROLE_EPILOGUE = 3, ROLE_SETUP = 4 };

// Division by a divisor fixed per launch: q = (n * mul) >> sh is floor(n / d) for every 0 <= n < 2^31 when
// sh = 31 + ceil(log2 d) and mul = floor(2^sh / d) + 1 (the host fills these in).  A 32-bit integer division
// is a chain of some thirty dependent instructions; the tile decode runs four of them before a CTA's first load.
struct FastDiv {
    uint32_t mul, sh;
};
__device__ __forceinline__ int fast_div(int n, FastDiv d) {
    return static_cast<int>((static_cast<uint64_t>(static_cast<uint32_t>(n)) * d.mul) >> d.sh);
}

// One output phase of a strided convolution data gradient run inside one launch (see sg_conv2d_dgrad): the phases are
// consecutive ranges of the tile list, each with its own rows, K loop, im2col window and pixel map.
struct ConvPhase {
    int32_t tile_start;                 // first (full-width) tile of the phase in the tile list
    int32_t M, num_kb;                  // rows (pixels of the phase) and k-blocks (taps x channel blocks)
    int32_t P, Q, pad_h, pad_w, dil_h, dil_w, S;
    int32_t tapb_r0, tapb_rs, tapb_s0, tapb_ss;
    int32_t remap_h0, remap_w0;
    FastDiv div_pq, div_q;
};
constexpr int kMaxPhases = 4;

struct alignas(64) Params {
    CUtensorMap tmA, tmB, tmD;          // dense / batched / conv operands (3-D; conv A is a 4-D im2col map)
    CUtensorMap tmB2;                   // B with the narrower box of split tail tiles
    const CUtensorMap* gmaps;           // grouped: A_g, B_g, D_g, B2_g maps at [4g] .. [4g+3]
    const int32_t* g_tile_start;        // grouped: first tile of group g, [groups + 1]
    const int32_t* g_M;                 // grouped: rows of group g
    const void* const* g_bias;          // grouped: per-group bias pointers (or null)
    const void* const* g_C;             // grouped: per-group C pointers (or null)
    void* const* g_D;                   // grouped: per-group D pointers
    void* D;                            // out dtype, row-major (+ b * strideD); used for ragged column tails only
    int64_t ldd, strideD;               // elements
    const void* bias;                   // bf16 [N] (+ b * strideBias)
    const void* C;                      // out dtype, row-major (+ b * strideC)
    int64_t ldc, strideC, strideBias;   // elements
    int32_t M, N, K, batch;             // batch = number of problems (dense) or groups (grouped)
    int32_t tiles_m, tiles_n, num_tiles, num_kb;
    int32_t split_begin, split;         // tiles at list positions >= split_begin are 1/split-wide column slices
    int32_t split_log2;                 // log2(split)
    int32_t band_m;                     // raster: tiles are walked in bands of this many tile rows, column by column
    FastDiv div_per;                    // dense / conv: by tiles_m * tiles_n (tiles of one problem)
    FastDiv div_band_tiles;             // by band_m * tiles_n
    FastDiv div_band_m;                 // by band_m (rows of every band but a shorter last one)
    FastDiv div_pq, div_q;              // conv: by P * Q and by Q
    int32_t ksplit;                     // > 1: tail tiles are cut into this many K ranges instead (split is then 1)
    int32_t sk_arrivals;                // warp arrivals that complete one part's parked tile (epilogue warps x CTAs)
    float* sk_partials;                 // K-split scratch: [tail tile][part][CTA of the tile][128 rows][BN] fp32
    uint32_t* sk_flags;                 // K-split scratch: [tail tile] arrival counters, then [tail tile] done counters
    int32_t sk_consumed_off;            // index of the first consumed counter inside sk_flags
    int32_t sk_early;                   // > 0: "early donors" (see decode_tile); the number of donor items at the list's head
    int32_t sk_park_all;                // 1: two-pass K split: every part parks all its sums, a second kernel adds them up
    float alpha, beta;
    float epi_arg0, epi_arg1;           // activation parameters (leaky_relu / elu slope, clip bounds)
    int32_t epi, mode;
    int32_t in_f16;                     // 1: the bias (and 16-bit A, B) are fp16, else bf16
    int32_t in_fp8;                     // operand kind: 0 sixteen-bit A and B; 1 e4m3; 2 e5m2 (bias bf16 or fp16 as in_f16 says);
                                        // 3 fp32 storage read as tf32 (bias fp32); 4 signed int8 with int32 accumulators (bias bf16)
    int32_t bk_elems;                   // elements of K per 128-byte stage row: 64 (16-bit) or 128 (8-bit)
    int32_t a_mn_major, b_mn_major;     // 1: the operand is stored with M (resp. N) contiguous: column-major A, row-major B
    int32_t P, Q, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w, S, cblocks;   // conv
    int32_t num_taps;                   // conv: taps walked by the K loop
    // conv (data gradient): the filter tap B reads for A's tap (c_r, c_s) is row tapb_r0 + tapb_rs * c_r, column
    // tapb_s0 + tapb_ss * c_s of the full R x S filter (mirrored, and for a strided gradient a subset), filt_s = S
    int32_t tapb_r0, tapb_rs, tapb_s0, tapb_ss, filt_s;
    // conv (strided data gradient): row m = (n, i, j) of this launch's output is pixel (n, remap_h0 + remap_sh * i,
    // remap_w0 + remap_sw * j) of the remap_H x remap_W image that C and D address; 0 = rows are stored as they come
    int32_t d_remap, remap_h0, remap_sh, remap_w0, remap_sw, remap_H, remap_W;
    int32_t a_rows;                     // rows of A loaded per tile (128; 64 or 32 in the short-A variants)
    int32_t warm_kb;                    // k-blocks of a CTA's first tile prefetched into the L2 at kernel entry
    int32_t nphases;                    // > 1: the tile list is the concatenation of ph[0 .. nphases), A maps in tmPh
    ConvPhase ph[kMaxPhases];
    CUtensorMap tmPh[kMaxPhases];
    // extended epilogue chain (all optional; ex_any = 1 when any of them is in use; dense and conv modes only):
    //   t = alpha acc * row_scale[i] * col_scale[j] + beta C + bias[j] + row_bias[i];  aux_store[i][j] = t;
    //   D = post_scale * act(t) + aux_load[i][j]
    int32_t ex_any;
    float post_scale;
    const float* row_scale;             // fp32 [M]
    const float* col_scale;             // fp32 [N]
    const float* row_bias;              // fp32 [M]
    const void* aux_load;               // out dtype, row-major, leading dimension ld_aux_load
    void* aux_store;                    // out dtype, row-major, leading dimension ld_aux_store
    int64_t ld_aux_load, ld_aux_store;  // elements
    uint32_t* status;                   // device status words (8 x u32)
    uint64_t timeout_ns;                // bound of every device-side wait
};

// 16-bit storage types: two packed values -> two floats and back (bf16 is the upper half of an fp32; fp16 converts)
template <bool kF16>
__device__ __forceinline__ void unpack2(uint32_t w, float& lo, float& hi) {
    if constexpr (kF16) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w));
        lo = f.x;
        hi = f.y;
    } else {
        lo = __uint_as_float(w << 16);
        hi = __uint_as_float(w & 0xFFFF0000u);
    }
}
template <bool kF16>
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    if constexpr (kF16) {
        const __half2 h = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<const uint32_t*>(&h);
    } else {
        const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<const uint32_t*>(&h);
    }
}
// The same conversion with the ReLU folded in (negative values and -0 become +0): one instruction for both.
template <bool kF16>
__device__ __forceinline__ uint32_t pack2_relu(float lo, float hi) {
    uint32_t w;
    if constexpr (kF16) asm("cvt.rn.relu.f16x2.f32 %0, %1, %2;" : "=r"(w) : "f"(hi), "f"(lo));
    else asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(w) : "f"(hi), "f"(lo));
    return w;
}
// v0 += low half, v1 += high half of a packed pair of 16-bit values: the mixed-precision add widens the 16-bit operand
// exactly, so the sums are those of unpack2 followed by two fp32 adds, without the two unpacking instructions.
template <bool kF16>
__device__ __forceinline__ void add_pair(uint32_t w, float& v0, float& v1) {
    if constexpr (kF16)
        asm("{ .reg .b16 lo, hi; mov.b32 {lo, hi}, %2; add.rn.f32.f16 %0, lo, %0; add.rn.f32.f16 %1, hi, %1; }"
            : "+f"(v0), "+f"(v1) : "r"(w));
    else
        asm("{ .reg .b16 lo, hi; mov.b32 {lo, hi}, %2; add.rn.f32.bf16 %0, lo, %0; add.rn.f32.bf16 %1, hi, %1; }"
            : "+f"(v0), "+f"(v1) : "r"(w));
}
__device__ __forceinline__ float half_bits_to_float(uint16_t b, bool f16) {
    return f16 ? __half2float(__ushort_as_half(b)) : __uint_as_float(static_cast<uint32_t>(b) << 16);
}

// Diagnostic build (-DSG_DEBUG_STAMPS, off in the product library): one CTA -- its index is the 64-bit word 31 of the
// stamp area, written by sg_debug_select_cta() -- records %globaltimer values at a few points of its life (entry,
// set-up done, first load issued, first MMA, accumulator ready, last store, exit) into the words after the status
// words; sg_debug_stamps() reads them back.  This is how the per-role time lines of a launch's start and end were
// measured.
#ifdef SG_DEBUG_STAMPS
#define SG_STAMP(slot)                                                                           \
    do {                                                                                         \
        if (blockIdx.x == sg_stamp_cta) {                                                        \
            reinterpret_cast<volatile uint64_t*>(p.status + 8)[slot] = global_timer_ns();        \
        }                                                                                        \
    } while (0)
#else
#define SG_STAMP(slot) do {} while (0)
#endif

struct Tile {
    int m0, n0, b, rows, width;   // first row / column, problem index, valid rows of the problem, tile width in columns
    int kb0, kb1;                 // k-blocks [kb0, kb1) this work item contracts (the whole K unless the tile is K-split)
    int part, nparts, tail;       // K-split: this item is part `part` of `nparts` sharing the tile's K range; index of the tail tile
};

// The convolution geometry a tile works with: the launch's own, or its phase's.
struct ConvView {
    int P, Q, pad_h, pad_w, dil_h, dil_w, S, tapb_r0, tapb_rs, tapb_s0, tapb_ss, remap_h0, remap_w0;
    FastDiv div_pq, div_q;
};
__device__ __forceinline__ ConvView conv_view(const Params& p, int phase, bool phased) {
    ConvView v;
    if (phased) {
        const ConvPhase& f = p.ph[phase];
        v.P = f.P; v.Q = f.Q; v.pad_h = f.pad_h; v.pad_w = f.pad_w; v.dil_h = f.dil_h; v.dil_w = f.dil_w; v.S = f.S;
        v.tapb_r0 = f.tapb_r0; v.tapb_rs = f.tapb_rs; v.tapb_s0 = f.tapb_s0; v.tapb_ss = f.tapb_ss;
        v.remap_h0 = f.remap_h0; v.remap_w0 = f.remap_w0; v.div_pq = f.div_pq; v.div_q = f.div_q;
    } else {
        v.P = p.P; v.Q = p.Q; v.pad_h = p.pad_h; v.pad_w = p.pad_w; v.dil_h = p.dil_h; v.dil_w = p.dil_w; v.S = p.S;
        v.tapb_r0 = p.tapb_r0; v.tapb_rs = p.tapb_rs; v.tapb_s0 = p.tapb_s0; v.tapb_ss = p.tapb_ss;
        v.remap_h0 = p.remap_h0; v.remap_w0 = p.remap_w0; v.div_pq = p.div_pq; v.div_q = p.div_q;
    }
    return v;
}

// Tile r of one problem -> (tile row, tile column).  Tiles are walked in horizontal bands of band_m tile
// rows; inside a band the walk goes down a column of the band, then to the next column.  The tiles running
// at the same time then share few A and B panels, and a band's A rows stay in L2 while its columns stream by.
__device__ __forceinline__ void raster(const Params& p, int r, int tiles_m, int& tm, int& tn) {
    const int band_tiles = p.band_m * p.tiles_n;
    const int band = fast_div(r, p.div_band_tiles);
    const int in_band = r - band * band_tiles;
    const int band_rows = min(p.band_m, tiles_m - band * p.band_m);
    tn = band_rows == p.band_m ? fast_div(in_band, p.div_band_m) : in_band / band_rows;
    tm = band * p.band_m + (in_band - tn * band_rows);
}

// Position t of the tile list -> tile.  The list holds the full-width tiles of all complete waves first;
// the tiles of the last, partial wave follow as `split` column slices each, so that more SMs share them.
// kV: kernel variant (see contract_kernel).
//
// K ranges with early donors (p.sk_early > 0; problems with whole waves of tiles plus a partial last wave): each of the
// R tiles of the last wave has its K loop cut into ksplit ranges.  The first ksplit - 1 of them ("donor" parts) are the
// very FIRST items of R (ksplit - 1) CTAs (list positions 0 .. sk_early), which park their raw sums in the scratch and
// go on to their full tiles; the last range (the "owner" part) is the very LAST item of another R CTAs (positions
// split_begin ..).  Long before an owner part starts, the epilogue warps of its CTA -- idle between two epilogues -- add
// the donors' parked sums up and write them into the TMEM accumulator the part will use (tcgen05.st); its MMAs then
// accumulate on top of them and its epilogue is an ordinary one.  Nobody waits for a peer that runs at the same time,
// nothing is fetched after the last MMA, and every CTA gets the same amount of work to within one K range.
template <int TILE_M, int BN, int kV = 0, bool kSplitK = (kV == 0)>
__device__ __forceinline__ Tile decode_tile(const Params& p, int t, int& g_hint) {
    Tile ti;
    int sub = 0;
    ti.width = BN;
    ti.kb0 = 0;
    ti.kb1 = p.num_kb;
    ti.part = 0;
    ti.nparts = 1;
    ti.tail = 0;
    if (kSplitK && p.sk_early > 0) {
        const int first_tail = p.split_begin - p.sk_early;     // id of the first tile of the last wave
        if (t < p.sk_early || t >= p.split_begin) {
            ti.nparts = p.ksplit;
            if (t < p.sk_early) {
                ti.tail = t / (p.ksplit - 1);
                ti.part = t - ti.tail * (p.ksplit - 1);
            } else {
                ti.tail = t - p.split_begin;
                ti.part = p.ksplit - 1;
            }
            t = first_tail + ti.tail;
            const int base = p.num_kb / p.ksplit, extra = p.num_kb - base * p.ksplit;
            ti.kb0 = ti.part * base + min(ti.part, extra);
            ti.kb1 = ti.kb0 + base + (ti.part < extra ? 1 : 0);
        } else {
            t -= p.sk_early;
        }
    } else if (t >= p.split_begin) {
        const int u = t - p.split_begin;
        if (kSplitK && p.ksplit > 1) {
            // the tile's K range is shared by ksplit work items
            ti.nparts = p.ksplit;
            ti.tail = u / p.ksplit;
            ti.part = u - ti.tail * p.ksplit;
            t = p.split_begin + ti.tail;
            const int base = p.num_kb / p.ksplit, extra = p.num_kb - base * p.ksplit;
            ti.kb0 = ti.part * base + min(ti.part, extra);
            ti.kb1 = ti.kb0 + base + (ti.part < extra ? 1 : 0);
        } else {
            const int parent = u >> p.split_log2;      // split is 1, 2 or 4
            sub = u - (parent << p.split_log2);
            t = p.split_begin + parent;
            ti.width = BN >> p.split_log2;
        }
    }
    int tm, tn;
    if (kV == 3 || (kV == 0 && p.mode == MODE_GROUPED)) {
        int g = g_hint;
        while (t >= p.g_tile_start[g + 1]) ++g;      // tiles are visited in increasing order
        g_hint = g;
        const int rows = p.g_M[g];
        ti.b = g;
        ti.rows = rows;
        raster(p, t - p.g_tile_start[g], (rows + TILE_M - 1) / TILE_M, tm, tn);
    } else if ((kV == 0 || kV == 5) && p.nphases > 1) {
        int ph = 0;
        while (ph + 1 < p.nphases && t >= p.ph[ph + 1].tile_start) ++ph;
        const int local = t - p.ph[ph].tile_start;
        ti.b = ph;
        ti.rows = p.ph[ph].M;
        ti.kb1 = p.ph[ph].num_kb;
        const int tm_count = (ti.rows + TILE_M - 1) / TILE_M;
        tn = local / tm_count;                  // down a column of tiles, then the next column
        tm = local - tn * tm_count;
    } else {
        const int per = p.tiles_m * p.tiles_n;
        ti.b = fast_div(t, p.div_per);
        ti.rows = p.M;
        raster(p, t - ti.b * per, p.tiles_m, tm, tn);
    }
    ti.m0 = tm * TILE_M;
    ti.n0 = tn * BN + sub * ti.width;
    return ti;
}

// Bounded mbarrier wait.  Returns false when the wait expired or another role already gave up.
static __device__ __noinline__ bool wait_slow(uint32_t bar, uint32_t parity, const Params& p, uint32_t role, uint32_t tile,
                                       uint32_t which) {
    volatile uint32_t* st = p.status;
    const uint64_t t0 = global_timer_ns();
    uint32_t it = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++it & 63u) == 0) {
            if (st[0] != 0) return false;
            if (global_timer_ns() - t0 > p.timeout_ns) {
                if (atomicCAS(p.status, 0u, (role << 24) | (which & 0xFFFFFF)) == 0u) {
                    st[1] = tile;
                    st[2] = parity;
                    st[3] = blockIdx.x;
                }
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, const Params& p, uint32_t role, uint32_t tile,
                                         uint32_t which) {
    if (mbar_try_wait(bar, parity)) return true;
    return wait_slow(bar, parity, p, role, tile, which);
}


__device__ __forceinline__ float tanh_approx(float x) {
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Activation of the fused epilogue.
//   gelu(v) = 0.5 v (1 + tanh(u)) = v * sigmoid(2u),  u = sqrt(2/pi) (v + 0.044715 v^3)
//   silu(v) = v * sigmoid(v) = 0.5 v (1 + tanh(v / 2))
// kFast (bf16 output): the hardware tanh approximation (relative error about 2^-11, an eighth of a bf16
// rounding step), one special-function operation per element -- twice the throughput of the exact form in
// isolation.  Otherwise (fp32 output): one exp and one division, accurate to a few fp32 ulps.
#ifndef SG_FAST_ACT
#define SG_FAST_ACT 1
#endif
template <bool kFast, int kEpi>
__device__ __forceinline__ float act_one(float v, float a0, float a1) {
    constexpr bool fast = kFast && SG_FAST_ACT;
    if constexpr (kEpi == EPI_RELU) {
        return fmaxf(v, 0.0f);
    } else if constexpr (kEpi == EPI_GELU) {
        // u = sqrt(2/pi) (v + 0.044715 v^3) = v (c1 + c2 v^2)
        const float u = v * fmaf(v * v, 0.7978845608028654f * 0.044715f, 0.7978845608028654f);
        if constexpr (fast) {
            const float h = 0.5f * v;
            return fmaf(h, tanh_approx(u), h);
        } else {
            return __fdividef(v, 1.0f + __expf(-2.0f * u));
        }
    } else if constexpr (kEpi == EPI_SILU) {
        if constexpr (fast) {
            const float h = 0.5f * v;
            return fmaf(h, tanh_approx(h), h);
        } else {
            return __fdividef(v, 1.0f + __expf(-v));
        }
    } else if constexpr (kEpi == EPI_SIGMOID) {
        if constexpr (fast) return fmaf(0.5f, tanh_approx(0.5f * v), 0.5f);
        else return __fdividef(1.0f, 1.0f + __expf(-v));
    } else if constexpr (kEpi == EPI_TANH) {
        if constexpr (fast) return tanh_approx(v);
        else return tanhf(v);
    } else if constexpr (kEpi == EPI_MISH) {
        // x tanh(softplus(x)); softplus(x) = x beyond 20 (e^-20 is below fp32 resolution next to x)
        if constexpr (fast) return v * tanh_approx(v > 20.0f ? v : __logf(1.0f + __expf(v)));
        else return v * tanhf(v > 20.0f ? v : log1pf(expf(v)));
    } else if constexpr (kEpi == EPI_HARDSWISH) {
        return v * fminf(fmaxf(v + 3.0f, 0.0f), 6.0f) * (1.0f / 6.0f);
    } else if constexpr (kEpi == EPI_LEAKY_RELU) {
        return v > 0.0f ? v : a0 * v;
    } else if constexpr (kEpi == EPI_ELU) {
        if constexpr (fast) return v > 0.0f ? v : a0 * (__expf(v) - 1.0f);
        else return v > 0.0f ? v : a0 * expm1f(v);
    } else if constexpr (kEpi == EPI_CLIP) {
        return fminf(fmaxf(v, a0), a1);
    } else {
        return v;
    }
}

// Applies the activation to a whole chunk of values: the (runtime) choice of the activation is taken once per
// chunk, outside the element loop.
template <bool kFast, int kN>
__device__ __forceinline__ void apply_act_chunk(float (&v)[kN], int epi, float a0, float a1) {
#define SG_ACT_CASE(E)                                                        \
    case E:                                                                   \
        _Pragma("unroll") for (int i = 0; i < kN; ++i) v[i] = act_one<kFast, E>(v[i], a0, a1); \
        break;
    switch (epi) {
        SG_ACT_CASE(EPI_RELU)
        SG_ACT_CASE(EPI_GELU)
        SG_ACT_CASE(EPI_SILU)
        SG_ACT_CASE(EPI_SIGMOID)
        SG_ACT_CASE(EPI_TANH)
        SG_ACT_CASE(EPI_MISH)
        SG_ACT_CASE(EPI_HARDSWISH)
        SG_ACT_CASE(EPI_LEAKY_RELU)
        SG_ACT_CASE(EPI_ELU)
        SG_ACT_CASE(EPI_CLIP)
        default:
            break;
    }
#undef SG_ACT_CASE
}

// Bounded wait until a global arrival counter (written by another CTA of this launch with a release pattern)
// reaches `target`.  Returns false when the wait expired or another role already gave up.
static __device__ __noinline__ bool wait_counter(const uint32_t* counter, uint32_t target, const Params& p, uint32_t tile) {
    const volatile uint32_t* c = counter;
    volatile uint32_t* st = p.status;
    const uint64_t t0 = global_timer_ns();
    uint32_t it = 0;
    while (*c < target) {
        __nanosleep(64);
        if ((++it & 63u) == 0) {
            if (st[0] != 0) return false;
            if (global_timer_ns() - t0 > p.timeout_ns) {
                if (atomicCAS(p.status, 0u, (ROLE_EPILOGUE << 24) | 300u) == 0u) {
                    st[1] = tile;
                    st[2] = *c;
                    st[3] = blockIdx.x;
                }
                return false;
            }
        }
    }
    return true;
}

// A_ROWS: rows of the A tile that are loaded.  128 = the whole tile; 64 or 32 when the problem has no more rows than
// that (a few activations against a large weight matrix): the A share of a stage shrinks to those rows, so more
// stages fit and more of B is in flight.  The MMA still reads 128 rows from the stage's A address -- the rows past
// A_ROWS are whatever follows in shared memory (the stage's B tile, later stages, the staging area: always inside the
// CTA's allocation) and produce accumulator rows past M, which no store ever writes.
template <int BN, bool kPair, int kEpiWarps = 4, int A_ROWS = 128>
struct Config {
    static constexpr int kCtas = kPair ? 2 : 1;
    static constexpr int BM = 128;                 // rows per CTA (= TMEM lanes)
    static constexpr int TILE_M = BM * kCtas;      // rows per tile
    static constexpr int BK = 64;                  // 64 bf16 = one 128-byte swizzled row
    static constexpr int B_ROWS = BN / kCtas;      // rows of the B tile this CTA loads
    static constexpr int A_BYTES = A_ROWS * BK * 2;
    static constexpr int B_BYTES = B_ROWS * BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES_RAW = (192 * 1024) / STAGE_BYTES;
#ifdef SG_MAX_STAGES
    static constexpr int STAGES = STAGES_RAW > SG_MAX_STAGES ? SG_MAX_STAGES : STAGES_RAW;   // experiments only
#else
    static constexpr int STAGES = STAGES_RAW > (A_ROWS < 128 ? 16 : 8) ? (A_ROWS < 128 ? 16 : 8) : STAGES_RAW;
#endif
    static_assert(A_ROWS == 128 || !kPair, "short A tiles are for single-CTA tiles");
    static constexpr int TMEM_COLS = 2 * BN < 32 ? 32 : 2 * BN;   // BN in {64,128,256} -> power of two
    static constexpr int EPI_WARPS = kEpiWarps;                    // 4: one per TMEM lane quarter; 8: two, alternating chunks
    static constexpr int CHUNK_STEP = EPI_WARPS / 4;
    static constexpr int STAGING_BUFS = 8 / EPI_WARPS;             // 32-row x 128-byte staging blocks per warp
    static constexpr int STAGING_BYTES = 8 * 4096;
    static constexpr int OFF_STAGING = STAGES * STAGE_BYTES;
    static constexpr int OFF_BIAS = OFF_STAGING + STAGING_BYTES;
    static constexpr int BIAS_SLOTS = BN / CHUNK_STEP < 64 ? 64 : BN / CHUNK_STEP;   // per warp: bf16 bias of its chunks
    static constexpr int OFF_BAR = OFF_BIAS + EPI_WARPS * BIAS_SLOTS * 2;
    static constexpr int NUM_BARS = 2 * STAGES + 5 + EPI_WARPS;    // full, empty, tmem_full[2], tmem_empty[2], drain, K-split fetch per warp
    static constexpr int SMEM_BYTES = OFF_BAR + NUM_BARS * 8 + 16;
    static constexpr int THREADS = 64 + 32 * EPI_WARPS;
    static_assert(SMEM_BYTES <= 227 * 1024, "configuration exceeds the shared memory of one CTA");
};

// kOut: 0 = bf16 output, 1 = fp32, 2 = fp16 (C, when read, has the output's type)
// kV selects a variant of the same kernel.  0: every mode and option.  The others keep one path and compile the rest
// out (16-bit operands throughout): 1 dense, 2 convolution forward, 3 grouped -- K-contiguous operands, no K ranges, no
// extended epilogue chain; 4 dense with the extended chain; 5 convolution data gradient (filter read C-contiguous,
// phase table and pixel scatter).  (A weight-gradient variant measured no faster than variant 0.)  The instructions executed are the same; the code is a quarter smaller and needs fewer
// registers, which measurably shortens every launch (4096^3 GEMM 96.4 -> 93.4 us, the benchmark convolution
// 85.8 -> 81.8 us, 128 x (256 x 256 x 512) 19.6 -> 18.75 us, 256^3 6.3 -> 4.7 us, each pair timed in one GPU call).
template <int BN, bool kPair, int kOut, int kEpiWarps, int kV = 0>
__global__ void __launch_bounds__(Config<BN, kPair, kEpiWarps>::THREADS, 1) contract_kernel(const __grid_constant__ Params p) {
    // variants 6 and 7 are variant 1 with an A tile of 64 resp. 32 loaded rows
    constexpr int kARows = kV == 6 ? 64 : (kV == 7 ? 32 : 128);
    // variants 8 and 9 are variants 1 and 2 (dense, convolution forward) with the K-range code kept in
    constexpr int kVB = kV >= 8 ? kV - 7 : (kV >= 6 ? 1 : kV);
    constexpr bool kSplitK = (kV == 0 || kV >= 8);
    using Cfg = Config<BN, kPair, kEpiWarps, kARows>;
    // options the specialised variants fold away at compile time
    constexpr bool kLean = kVB != 0;
    const int32_t mode = (kVB == 1 || kVB == 4) ? MODE_DENSE : ((kVB == 2 || kVB == 5) ? MODE_CONV : (kVB == 3 ? MODE_GROUPED : p.mode));
    const bool a_mn = kLean ? false : p.a_mn_major != 0;
    const bool b_mn = kLean ? kVB == 5 : p.b_mn_major != 0;
    const bool d_remap = (kVB == 0 || kVB == 5) ? p.d_remap != 0 : false;
    const bool phased = (kVB == 0 || kVB == 5) ? p.nphases > 1 : false;
    constexpr int kCtas = Cfg::kCtas;
    constexpr int STAGES = Cfg::STAGES;
    constexpr bool kOutF32 = (kOut == 1);
    constexpr bool kOutF16 = (kOut == 2);
    constexpr int CH = kOutF32 ? 32 : 64;          // output columns per 128-byte staging row

    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t smem_base = smem_u32(smem);
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t cta_rank = kPair ? cluster_ctarank() : 0u;
    const bool leader = (cta_rank == 0);

    const uint32_t bar_base = smem_base + Cfg::OFF_BAR;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
    const uint32_t drain_bar = bar_base + 8u * (2 * STAGES + 4);
    auto fetch_bar = [&](int w) { return bar_base + 8u * (2 * STAGES + 5 + w); };
    const uint32_t tmem_slot = bar_base + 8u * Cfg::NUM_BARS;
    volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(smem + Cfg::OFF_BAR + 8 * Cfg::NUM_BARS);

#ifdef SG_DEBUG_STAMPS
    const uint32_t sg_stamp_cta = static_cast<uint32_t>(reinterpret_cast<volatile uint64_t*>(p.status + 8)[31]);
#endif
    if (threadIdx.x == 0) SG_STAMP(0);
    // The first operand tile cannot arrive before the TMA unit holds the tensor maps: fetch them at once, from a warp
    // that has nothing else to do yet, while thread 0 sets the barriers up.
    if (threadIdx.x == 64 && p.mode != MODE_GROUPED) {
        prefetch_tensormap(&p.tmA);
        prefetch_tensormap(&p.tmB);
    }
    // CTA 0 measures the SM clock this launch actually ran at (cycle counter against the nanosecond timer);
    // the host reads it through sg_last_kernel_clock for clock-scaled Speed-of-Light figures.
    uint64_t clk0 = 0, ns0 = 0;
    if (blockIdx.x == 0 && threadIdx.x == 96) {
        clk0 = clock64();
        ns0 = global_timer_ns();
    }
#ifdef SG_DEBUG_STAMPS
    if (threadIdx.x == 32 && blockIdx.x == sg_stamp_cta) {
        reinterpret_cast<volatile uint64_t*>(p.status + 8)[11] = clock64();
        reinterpret_cast<volatile uint64_t*>(p.status + 8)[13] = global_timer_ns();
    }
#endif
    // A sticky failure recorded by an earlier launch, or a misaligned dynamic shared-memory base, makes this
    // launch a no-op.  The status word is fetched by one thread while the others set up, and the block-wide
    // OR below doubles as the set-up barrier.  (Both CTAs of a pair decide alike: the word can only have been
    // set by an earlier launch, and the base is the same in every CTA.)
    uint32_t bad = 0;
    if (threadIdx.x == 64) bad = *reinterpret_cast<volatile uint32_t*>(p.status);
    if ((smem_base & 1023u) != 0u) {
        if (threadIdx.x == 0) atomicCAS(p.status, 0u, (ROLE_SETUP << 24) | 1u);
        bad = 1;
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), Cfg::EPI_WARPS * kCtas);
        }
        mbar_init(drain_bar, 1);
        for (int w = 0; w < Cfg::EPI_WARPS; ++w) mbar_init(fetch_bar(w), 1);
        fence_barrier_init();
    }
    // Start of a launch.  Between kernel entry and the first operand bytes in shared memory lie the set-up (TMEM
    // allocation, barriers), the first execution of the producer's code and a DRAM round trip; under programmatic
    // dependent launch a CTA may also sit for a microsecond or two waiting for the previous kernel in the stream to
    // finish.  For plain K-contiguous dense problems two things shorten that:
    //  * L2 warm-up: an otherwise idle thread asks the TMA unit to PREFETCH the first k-blocks of the CTA's first
    //    tile into the L2 -- before the launch dependency is waited for (nothing reaches the SM, and the L2 is the
    //    point of coherence, so this is safe even if the previous kernel is still writing those very lines);
    //  * early start (single-CTA tiles): the thread that initialised the barriers issues the loads of the first
    //    tile's first stages itself, before the set-up barrier; the producer loop skips those k-blocks.
    int early_kb = 0;
    if (mode == MODE_DENSE && !a_mn && !b_mn && (smem_base & 1023u) == 0u && p.num_kb > 0 &&
        static_cast<int>(blockIdx.x) / kCtas < p.num_tiles) {
        int g_hint0 = 0;
        const Tile t0 = decode_tile<Cfg::TILE_M, BN, kVB, kSplitK>(p, static_cast<int>(blockIdx.x) / kCtas, g_hint0);
        if (t0.n0 < p.N) {
            const CUtensorMap* mapB0 = (t0.width != BN) ? &p.tmB2 : &p.tmB;
            const int b_rows0 = t0.width / kCtas;
            const int m00 = t0.m0 + static_cast<int>(cta_rank) * Cfg::BM;
            const int nb00 = t0.n0 + static_cast<int>(cta_rank) * b_rows0;
            if (threadIdx.x == 96) {
                const int npf = min(p.warm_kb, t0.kb1 - t0.kb0);
                for (int j = 0; j < npf; ++j) {
                    tma_prefetch_3d(&p.tmA, (t0.kb0 + j) * p.bk_elems, m00, t0.b);
                    tma_prefetch_3d(mapB0, (t0.kb0 + j) * p.bk_elems, nb00, t0.b);
                }
            }
            if constexpr (!kPair) {
                early_kb = min(STAGES, t0.kb1 - t0.kb0);
                if (threadIdx.x == 0) {
                    grid_dependency_wait();
                    SG_STAMP(2);
                    const uint32_t tx0 = static_cast<uint32_t>(Cfg::A_BYTES + t0.width * Cfg::BK * 2);
                    for (int j = 0; j < early_kb; ++j) {
                        const uint32_t a_dst = smem_base + j * Cfg::STAGE_BYTES;
                        mbar_arrive_expect_tx(full_bar(j), tx0);
                        tma_load_3d<false>(a_dst, &p.tmA, full_bar(j), (t0.kb0 + j) * p.bk_elems, t0.m0, t0.b);
                        tma_load_3d<false>(a_dst + Cfg::A_BYTES, mapB0, full_bar(j), (t0.kb0 + j) * p.bk_elems, t0.n0, t0.b);
                    }
                }
            }
        }
    }
    if (warp == 1) {
        tmem_alloc<kPair>(tmem_slot, Cfg::TMEM_COLS);
        tmem_relinquish<kPair>();
    }
    if (warp == 0 && lane == 0 && mode != MODE_GROUPED) prefetch_tensormap(&p.tmD);
    tc_fence_before_sync();
    const bool dead = __syncthreads_or(bad != 0u) != 0;
    if constexpr (kPair) {
        cluster_arrive();
        cluster_wait();
    }
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot_ptr;
    if (threadIdx.x == 0) SG_STAMP(1);
    // Everything above touched only this CTA's shared memory, TMEM and the kernel parameters, so under
    // programmatic dependent launch it may overlap the tail of the previous kernel in the stream.  From here
    // on global memory is read and written: wait for the previous kernel, then let the next one start setting up.
    grid_dependency_wait();
    grid_launch_dependents();

    const int num_kb = p.num_kb;
    const int first_tile = blockIdx.x / kCtas;
    const int tile_step = gridDim.x / kCtas;
    bool ok = !dead;

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (elect_one()) {
            int stage = 0;
            uint32_t phase = 0;
            int g_hint = 0, g_fenced = -1;
            for (int t = first_tile; t < p.num_tiles && ok && num_kb > 0; t += tile_step) {
                Tile ti = decode_tile<Cfg::TILE_M, BN, kVB, kSplitK>(p, t, g_hint);
                if (ti.n0 >= p.N) continue;                       // a column slice past the last column: no work
                const int m0 = ti.m0 + static_cast<int>(cta_rank) * Cfg::BM;
                const int b_rows = ti.width / kCtas;              // rows of B this CTA loads
                const int nb0 = ti.n0 + static_cast<int>(cta_rank) * b_rows;
                const uint32_t stage_tx = static_cast<uint32_t>(Cfg::A_BYTES + b_rows * Cfg::BK * 2) * kCtas;
                const bool narrow = ti.width != BN;
                const int bk_elems = p.bk_elems;
                const CUtensorMap* mapA = &p.tmA;
                const CUtensorMap* mapB = narrow ? &p.tmB2 : &p.tmB;
                int bz = ti.b;
                if (mode == MODE_GROUPED) {
                    mapA = p.gmaps + 4 * ti.b;
                    mapB = mapA + (narrow ? 3 : 1);
                    bz = 0;
                    if (g_fenced != ti.b) {
                        fence_tensormap_acquire(mapA);
                        fence_tensormap_acquire(mapA + 1);
                        fence_tensormap_acquire(mapA + 3);
                        g_fenced = ti.b;
                    }
                }
                int cw = 0, ch = 0, cn = 0;
                ConvView cv = {};
                if (mode == MODE_CONV) {
                    cv = conv_view(p, ti.b, phased);
                    if (phased) mapA = &p.tmPh[ti.b];
                    const int pq = cv.P * cv.Q;
                    cn = fast_div(m0, cv.div_pq);
                    const int rem = m0 - cn * pq;
                    const int op = fast_div(rem, cv.div_q);
                    const int oq = rem - op * cv.Q;
                    cw = oq * p.stride_w - cv.pad_w;
                    ch = op * p.stride_h - cv.pad_h;
                }
                // conv: filter tap (r, s) and channel block of the current k-block, advanced incrementally
                int c_tap = 0, c_cb = 0, c_r = 0, c_s = 0;
                if (mode == MODE_CONV) {
                    c_tap = ti.kb0 / p.cblocks;
                    c_cb = ti.kb0 - c_tap * p.cblocks;
                    c_r = c_tap / cv.S;
                    c_s = c_tap - c_r * cv.S;
                }
                // weight gradient: the problem index is the filter tap, the contraction runs over output pixels;
                // (w_n, w_p, w_q) is the first pixel of the current k-block
                int w_n = 0, w_p = 0, w_q = 0;
                if (mode == MODE_WGRAD) {
                    c_r = ti.b / p.S;
                    c_s = ti.b - c_r * p.S;
                    const int pix = ti.kb0 * Cfg::BK;
                    w_n = fast_div(pix, p.div_pq);
                    const int rem = pix - w_n * (p.P * p.Q);
                    w_p = fast_div(rem, p.div_q);
                    w_q = rem - w_p * p.Q;
                }
                for (int kb = ti.kb0; kb < ti.kb1; ++kb) {
                    if (t == first_tile && kb - ti.kb0 < early_kb) {
                        // issued before the set-up barrier (see "Early start"): this k-block sits in stage kb - kb0
                        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                        continue;
                    }
                    if (!wait_bar(empty_bar(stage), phase ^ 1u, p, ROLE_PRODUCER, t, stage)) { ok = false; break; }
                    const uint32_t a_dst = smem_base + stage * Cfg::STAGE_BYTES;
                    const uint32_t b_dst = a_dst + Cfg::A_BYTES;
                    uint32_t fb = full_bar(stage);
                    if constexpr (kPair) fb = map_to_cta(fb, 0);
                    if (leader) mbar_arrive_expect_tx(full_bar(stage), stage_tx);
                    if (mode == MODE_CONV) {
                        const int c0 = c_cb * bk_elems;
                        tma_load_im2col_4d<kPair>(a_dst, mapA, fb, c0, cw, ch, cn, static_cast<uint16_t>(c_s * cv.dil_w),
                                                  static_cast<uint16_t>(c_r * cv.dil_h));
                        if (b_mn) {
                            // data gradient: the filter [k][tap][c] is read with c contiguous, 64 k x 64 c per box
                            const int tap_b = (cv.tapb_r0 + cv.tapb_rs * c_r) * p.filt_s + cv.tapb_s0 + cv.tapb_ss * c_s;
                            for (int j = 0; j < b_rows / 64; ++j)
                                tma_load_3d<kPair>(b_dst + j * 8192, mapB, fb, nb0 + j * 64, tap_b, c0);
                        } else {
                            tma_load_3d<kPair>(b_dst, mapB, fb, c0, c_tap, nb0);
                        }
                        if (++c_cb == p.cblocks) {
                            c_cb = 0;
                            ++c_tap;
                            if (++c_s == cv.S) { c_s = 0; ++c_r; }
                        }
                    } else if (mode == MODE_WGRAD) {
                        // A = dY^T: [pixels][filters] read with the filter index contiguous; B = the 64 pixels of
                        // this k-block shifted by the tap, 64 channels per box (im2col addressing)
#pragma unroll
                        for (int j = 0; j < Cfg::BM / 64; ++j)
                            tma_load_3d<kPair>(a_dst + j * 8192, mapA, fb, m0 + j * 64, kb * Cfg::BK, 0);
                        for (int j = 0; j < b_rows / 64; ++j)
                            tma_load_im2col_4d<kPair>(b_dst + j * 8192, mapB, fb, nb0 + j * 64, w_q * p.stride_w - p.pad_w,
                                                      w_p * p.stride_h - p.pad_h, w_n, static_cast<uint16_t>(c_s * p.dil_w),
                                                      static_cast<uint16_t>(c_r * p.dil_h));
                        w_q += Cfg::BK;
                        while (w_q >= p.Q) {
                            w_q -= p.Q;
                            if (++w_p == p.P) { w_p = 0; ++w_n; }
                        }
                    } else {
                        if (a_mn) {
                            // column-major A: boxes of 64 rows of the tile (contiguous) x 64 k, one per 64 tile rows
#pragma unroll
                            for (int j = 0; j < Cfg::BM / 64; ++j)
                                tma_load_3d<kPair>(a_dst + j * 8192, mapA, fb, m0 + j * 64, kb * Cfg::BK, bz);   // 16-bit only
                        } else {
                            tma_load_3d<kPair>(a_dst, mapA, fb, kb * bk_elems, m0, bz);
                        }
                        if (b_mn) {
                            for (int j = 0; j < b_rows / 64; ++j)
                                tma_load_3d<kPair>(b_dst + j * 8192, mapB, fb, nb0 + j * 64, kb * Cfg::BK, bz);
                        } else {
                            tma_load_3d<kPair>(b_dst, mapB, fb, kb * bk_elems, nb0, bz);
                        }
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                    if (t == first_tile && kb == ti.kb0) SG_STAMP(2);
                }
            }
            SG_STAMP(3);
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (leader && elect_one()) {
            int stage = 0;
            uint32_t phase = 0;
            int iter = 0;
            int g_hint = 0;
            const uint64_t a_desc0 = a_mn ? smem_desc_mn_major_sw128(smem_base) : smem_desc_k_major_sw128(smem_base);
            const uint64_t b_desc0 = b_mn ? smem_desc_mn_major_sw128(smem_base + Cfg::A_BYTES)
                                                  : smem_desc_k_major_sw128(smem_base + Cfg::A_BYTES);
            for (int t = first_tile; t < p.num_tiles && ok && num_kb > 0; t += tile_step) {
                const Tile ti = decode_tile<Cfg::TILE_M, BN, kVB, kSplitK>(p, t, g_hint);
                if (ti.n0 >= p.N) continue;
                if (ti.kb1 <= ti.kb0) continue;                  // a phase no filter tap reaches: the epilogue writes beta C
                const int in_kind = kLean ? 0 : p.in_fp8;          // 0 sixteen-bit, 1 / 2 fp8, 3 tf32, 4 int8
                const uint32_t in_fmt = in_kind == 4 ? 1u
                                        : (in_kind == 3 ? 2u : (in_kind ? static_cast<uint32_t>(in_kind - 1) : (p.in_f16 ? 0u : 1u)));
                const uint32_t idesc = umma_idesc_f32acc(Cfg::TILE_M, ti.width, a_mn, b_mn, in_fmt, in_kind == 4);
                const uint32_t a_step = a_mn ? (2048u >> 4) : (32u >> 4);    // descriptor address units per K=16
                const uint32_t b_step = b_mn ? (2048u >> 4) : (32u >> 4);
                const int acc = iter & 1;
                const uint32_t acc_phase = (iter >> 1) & 1u;
                ++iter;
                // an owner part of the early-donor scheme finds the donors' sums in its accumulator: add to them
                const bool preloaded = kSplitK ? (p.sk_early > 0 && ti.nparts > 1 && ti.part == ti.nparts - 1) : false;
                if (!wait_bar(tempty_bar(acc), acc_phase ^ 1u, p, ROLE_MMA, t, 100 + acc)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN);
                for (int kb = ti.kb0; kb < ti.kb1; ++kb) {
                    if (!wait_bar(full_bar(stage), phase, p, ROLE_MMA, t, stage)) { ok = false; break; }
                    if (t == first_tile && kb == ti.kb0) SG_STAMP(4);
                    tc_fence_after_sync();
                    // descriptors of this stage: those of stage 0 plus the stage offset in the 16-byte address field
                    const uint64_t a_desc = a_desc0 + static_cast<uint64_t>(stage * (Cfg::STAGE_BYTES >> 4));
                    const uint64_t b_desc = b_desc0 + static_cast<uint64_t>(stage * (Cfg::STAGE_BYTES >> 4));
                    // One instruction-K step is 32 bytes along a K-major row (16 two-byte or 32 one-byte elements), or two
                    // 1 KB k-groups of an MN-major tile; a 128-byte stage row holds four of them for either width.
                    if (in_kind == 4) {
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            umma_i8<kPair>(d_tmem, a_desc + a_step * kk, b_desc + b_step * kk, idesc,
                                           (kb != ti.kb0 || kk != 0 || preloaded) ? 1u : 0u);
                    } else if (in_kind == 3) {
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            umma_tf32<kPair>(d_tmem, a_desc + a_step * kk, b_desc + b_step * kk, idesc,
                                             (kb != ti.kb0 || kk != 0 || preloaded) ? 1u : 0u);
                    } else if (in_kind != 0) {
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            umma_fp8<kPair>(d_tmem, a_desc + a_step * kk, b_desc + b_step * kk, idesc,
                                            (kb != ti.kb0 || kk != 0 || preloaded) ? 1u : 0u);
                    } else {
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            umma_bf16<kPair>(d_tmem, a_desc + a_step * kk, b_desc + b_step * kk, idesc,
                                             (kb != ti.kb0 || kk != 0 || preloaded) ? 1u : 0u);
                    }
                    umma_commit<kPair>(empty_bar(stage));
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit<kPair>(tfull_bar(acc));
                if (t == first_tile) SG_STAMP(5);
#ifdef SG_DEBUG_STAMPS
                if (iter <= 8) SG_STAMP(21 + iter);      // last MMA of this CTA's iter-th item issued
#endif
            }
            SG_STAMP(6);
            if (!ok) {
                // let every MMA already issued finish before TMEM is freed
                umma_commit<kPair>(drain_bar);
                const uint64_t t0 = global_timer_ns();
                while (!mbar_try_wait(drain_bar, 0) && global_timer_ns() - t0 < 100000000ull) {}
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue warps 2..9
        // Two warps serve each TMEM lane quarter; the warp with half == 0 takes the even 128-byte column
        // chunks of a tile, its partner the odd ones.
        const int q = warp & 3;               // TMEM lane quarter this warp may read
        const int ew = warp - 2;              // staging slot
        const int half = ew >> 2;             // which chunks of a tile this warp takes (always 0 with four warps)
        constexpr int kStep = Cfg::CHUNK_STEP;
        uint32_t chunk_ctr = 0;
        uint32_t fetch_phase = 0;             // phase of this warp's K-split fetch barrier
        uint16_t* bias_w = reinterpret_cast<uint16_t*>(smem + Cfg::OFF_BIAS) + ew * Cfg::BIAS_SLOTS;   // bf16 bias of its chunks
        constexpr int kMyBiasSlots = ((BN / CH + kStep - 1) / kStep) * CH;     // columns of the chunks one warp handles
        const bool has_bias = (mode == MODE_GROUPED) ? (p.g_bias != nullptr) : (p.bias != nullptr);
        const bool bias_f32 = kLean ? false : p.in_fp8 == 3;       // tf32 operands come with an fp32 bias, read directly
        const bool acc_s32 = kLean ? false : p.in_fp8 == 4;        // int8 operands accumulate in 32-bit integers
        const bool has_c = (p.beta != 0.0f);
        const bool in_f16 = (p.in_f16 != 0);
        const float alpha = p.alpha, beta = p.beta;
        const int epi = p.epi;
        int iter = 0, g_hint = 0, g_fenced = -1;
        uint32_t tempty_remote[2];
#pragma unroll
        for (int a = 0; a < 2; ++a) tempty_remote[a] = kPair ? map_to_cta(tempty_bar(a), 0) : tempty_bar(a);

        for (int t = first_tile; t < p.num_tiles && ok; t += tile_step) {
            Tile ti = decode_tile<Cfg::TILE_M, BN, kVB, kSplitK>(p, t, g_hint);
            if (ti.n0 >= p.N) continue;
            const bool has_k = num_kb > 0 && ti.kb1 > ti.kb0;   // else the tile is the empty sum: no accumulator is involved
            const int acc = iter & 1;
            const uint32_t acc_phase = (iter >> 1) & 1u;
            if (has_k) ++iter;
            // K ranges with early donors: an owner part (list positions from split_begin on) finds the donors' sums in
            // its accumulator, so its epilogue is an ordinary one; and the item that used that accumulator buffer before
            // it -- two items earlier in this CTA's walk -- keeps the buffer until it has put them there.
            const bool early = kSplitK ? p.sk_early > 0 : false;
            const bool early_owner = early && ti.nparts > 1 && ti.part == ti.nparts - 1;
            const int t_next2 = t + 2 * tile_step;
            const bool preload_next = early && has_k && t_next2 >= p.split_begin && t_next2 < p.num_tiles;
            // The accumulator buffer is handed back to the MMA warp only if a later item of this CTA will use it: at most
            // the item after next can (the next one takes the other buffer).  On a CTA pair the hand-back is an arrival with
            // cluster-scope release on the leader's barrier, about a microsecond -- in the middle of the one epilogue of
            // the launch that nothing overlaps with.
            const bool handback = t_next2 < p.num_tiles;
            const int n0 = ti.n0;
            const int row0 = ti.m0 + static_cast<int>(cta_rank) * Cfg::BM + q * 32;
            const CUtensorMap* mapD = &p.tmD;
            const uint16_t* bias_g = reinterpret_cast<const uint16_t*>(p.bias);
            const uint8_t* c_g = reinterpret_cast<const uint8_t*>(p.C);
            uint8_t* d_g = reinterpret_cast<uint8_t*>(p.D);
            int bz = ti.b;
            if (mode == MODE_GROUPED) {
                mapD = p.gmaps + 4 * ti.b + 2;
                bz = 0;
                if (has_bias) bias_g = reinterpret_cast<const uint16_t*>(p.g_bias[ti.b]);
                if (has_c) c_g = reinterpret_cast<const uint8_t*>(p.g_C[ti.b]);
                d_g = reinterpret_cast<uint8_t*>(p.g_D[ti.b]);
                if (g_fenced != ti.b) {
                    fence_tensormap_acquire(mapD);
                    g_fenced = ti.b;
                }
            } else {
                if (has_bias) bias_g += static_cast<int64_t>(ti.b) * p.strideBias;
                if (has_c) c_g += static_cast<int64_t>(ti.b) * p.strideC * (kOutF32 ? 4 : 2);
                d_g += static_cast<int64_t>(ti.b) * p.strideD * (kOutF32 ? 4 : 2);
            }
            if (has_bias && !bias_f32) {
                // every warp keeps its own copy of the tile's bias values, so no barrier between warps is needed
                __syncwarp();
                const uint16_t* bsrc = bias_g;
                for (int i = lane; i < kMyBiasSlots; i += 32) {
                    const int n = n0 + ((i / CH) * kStep + half) * CH + (i % CH);     // column of local slot i
                    bias_w[i] = (n < p.N) ? bsrc[n] : static_cast<uint16_t>(0);
                }
                __syncwarp();
            }
            if (has_k) {
                // one lane polls; the other 31 wait at the warp barrier without issuing instructions
                uint32_t done = 1;
                if (lane == 0) done = wait_bar(tfull_bar(acc), acc_phase, p, ROLE_EPILOGUE, t, 200 + acc) ? 1u : 0u;
                done = __shfl_sync(0xFFFFFFFFu, done, 0);
                if (!done) { ok = false; break; }
                tc_fence_after_sync();
                if (warp == 2 && lane == 0 && t == first_tile) SG_STAMP(7);
            }
            const int ncols = min(ti.width, p.N - n0);
            const int nchunks = (ncols + CH - 1) / CH;
            const bool rows_live = row0 < ti.rows;
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + static_cast<uint32_t>(acc * BN);
            const int row = row0 + lane;
            // row of C and D in memory: the row itself, or for a strided data gradient the pixel it stands for
            int64_t mem_row = row;
            if (d_remap && row < ti.rows) {
                const ConvView cv = conv_view(p, ti.b, phased);
                const int pq = cv.P * cv.Q;
                const int n_img = fast_div(row, cv.div_pq);
                const int rem = row - n_img * pq;
                const int pi = fast_div(rem, cv.div_q);
                const int pj = rem - pi * cv.Q;
                mem_row = (static_cast<int64_t>(n_img) * p.remap_H + cv.remap_h0 + p.remap_sh * pi) * p.remap_W + cv.remap_w0 +
                          p.remap_sw * pj;
            }

            // K-split tile: the tile's K range is shared by nparts work items.  Every part parks its raw fp32 sums of
            // the column chunks it does not finish in the scratch (pass 0), then finishes the chunks it owns
            // from its own accumulator plus the other parts' parked sums
            // (pass 1), so the exchange is spread over all parts instead of serialised in one.  The unit of ownership
            // is one warp's 32 rows x one column chunk of one CTA: unit u belongs to part u mod nparts.
            const bool ksplit_tile = kSplitK ? (ti.nparts > 1 && !early_owner) : false;
            // chunk index first: one warp's chunks then go to different parts, and so do one chunk's warps
            // (early donors, and the parts of a two-pass K split, park every unit: nothing is theirs to finish)
            const bool two_pass = kSplitK ? p.sk_park_all != 0 : false;
            auto owned_by = [&](int c, int qq) {
                return (early || two_pass) ? false : (c + (BN / CH) * (qq * kCtas + static_cast<int>(cta_rank))) % ti.nparts == ti.part;
            };
            auto owned = [&](int c) { return owned_by(c, q); };
            // how many epilogue warps of this CTA finish at least one unit, and this warp's rank among them: the
            // stage ring (idle by then) is divided between them as the landing zone of the other parts' sums
            int fetch_owners = 0, fetch_rank = 0;
            if (ksplit_tile) {
                for (int w = 0; w < Cfg::EPI_WARPS; ++w) {
                    const int qq = (w + 2) & 3;
                    bool o = false;
                    for (int c = w >> 2; c < nchunks; c += kStep) o = o || owned_by(c, qq);
                    o = o && (ti.m0 + static_cast<int>(cta_rank) * Cfg::BM + qq * 32 < ti.rows);
                    if (o) {
                        if (w < ew) ++fetch_rank;
                        ++fetch_owners;
                    }
                }
            }
            const int passes = (ksplit_tile && !two_pass) ? 2 : 1;      // (two-pass: the kernel's end publishes the sums)
            if (has_k && half >= nchunks && !ksplit_tile && !preload_next && handback) {
                // no chunk of this tile is this warp's: it still has to hand the accumulator back
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) {
                    if constexpr (kPair) mbar_arrive_cluster(tempty_remote[acc]);
                    else mbar_arrive(tempty_remote[acc]);
                }
            }
#pragma unroll 1
            for (int pass = 0; pass < passes && ok; ++pass) {
            if (ksplit_tile && pass == 1) {
                // this warp's share of the parked sums is complete: publish it, then wait for the other parts
                // (the readers fetch it with bulk copies, i.e. through the asynchronous proxy)
                __threadfence();
                fence_proxy_async_all();
                __syncwarp();
                uint32_t okw = 1;
                bool owns = false;
                for (int c = half; c < nchunks; c += kStep) owns = owns || owned(c);
                owns = owns && rows_live;
                if (lane == 0) {
                    uint32_t* arrived = p.sk_flags + ti.tail;       // one counter per tile: every warp of every part
                    atomicAdd(arrived, 1u);
                    if (owns) okw = wait_counter(arrived, static_cast<uint32_t>(p.sk_arrivals * ti.nparts), p, t) ? 1u : 0u;
                }
                okw = __shfl_sync(0xFFFFFFFFu, okw, 0);
                if (!okw) { ok = false; break; }
                if (owns) __threadfence();      // the other parts' sums are read after their flags
            }
#pragma unroll 1
            for (int c = half; c < nchunks; c += kStep) {
                if (ksplit_tile && owned(c) != (pass == 1)) continue;
                float v[CH];
#ifdef SG_DEBUG_STAMPS
                const bool stamp_chunk = warp == 2 && lane == 0 && t + tile_step >= p.num_tiles && c < 2;
                if (stamp_chunk) SG_STAMP(16 + 3 * c);
#endif
                if (has_k) {
                    uint32_t r0[32];
                    tmem_ld_32x32(t_row + c * CH, r0);
                    if constexpr (!kOutF32) {
                        uint32_t r1[32];
                        tmem_ld_32x32(t_row + c * CH + 32, r1);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            v[i] = acc_s32 ? static_cast<float>(static_cast<int32_t>(r0[i])) : __uint_as_float(r0[i]);
                            v[32 + i] = acc_s32 ? static_cast<float>(static_cast<int32_t>(r1[i])) : __uint_as_float(r1[i]);
                        }
                    } else {
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            v[i] = acc_s32 ? static_cast<float>(static_cast<int32_t>(r0[i])) : __uint_as_float(r0[i]);
                    }
                    if (c + kStep >= nchunks && !ksplit_tile && !preload_next && handback) {
                        // this warp has read its last columns of the accumulator: hand its share back to the MMA warp
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) {
                            if constexpr (kPair) mbar_arrive_cluster(tempty_remote[acc]);
                            else mbar_arrive(tempty_remote[acc]);
                        }
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < CH; ++i) v[i] = 0.0f;
                }
                if (!rows_live) continue;       // nothing of this warp's 32 rows exists (ragged last tile)

                if (ksplit_tile) {
                    // Scratch layout of one CTA's parked tile: [chunk][lane quarter][group of 4 columns][32 rows] float4:
                    // a unit (one warp's rows of one chunk) is one contiguous block of CH x 128 bytes, and the 32 lanes
                    // (= rows) of a warp touch 512 contiguous bytes per access.
                    constexpr uint32_t kUnitBytes = CH * 128u;
                    const size_t tile_elems = static_cast<size_t>(Cfg::BM) * BN;
                    const size_t unit_off = static_cast<size_t>(cta_rank) * tile_elems +
                                            static_cast<size_t>(c * 4 + q) * (kUnitBytes / 4);
                    float* tile_bufs = p.sk_partials + static_cast<size_t>(ti.tail) * p.ksplit * kCtas * tile_elems;
                    if (pass == 0) {
                        float* pb = tile_bufs + static_cast<size_t>(ti.part) * kCtas * tile_elems + unit_off + lane * 4;
#pragma unroll
                        for (int i = 0; i < CH; i += 4)
                            __stcg(reinterpret_cast<float4*>(pb + i * 32), make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]));
                        continue;
                    }
                    // Own sums first, then the other parts' in increasing order: reproducible for a given plan.
                    // The other parts' units are fetched with bulk copies, several at a time, into this warp's share
                    // of the stage ring (idle by now: a K-split item is the last work of its CTA, its MMAs are done),
                    // so the latency of the exchange is paid once per batch of parts rather than once per part.
                    const uint32_t fetch_bytes = static_cast<uint32_t>(STAGES * Cfg::STAGE_BYTES) /
                                                 static_cast<uint32_t>(fetch_owners > 0 ? fetch_owners : 1) / kUnitBytes * kUnitBytes;
                    const int kBatch = static_cast<int>(fetch_bytes / kUnitBytes);
                    const bool ring_idle = t + tile_step >= p.num_tiles;
                    if (kEpiWarps == 4 && kBatch >= 2 && ring_idle) {    // (8-warp kernels serve short K: registers are scarce there)
                        const uint32_t fetch_base = smem_base + static_cast<uint32_t>(fetch_rank) * fetch_bytes;
                        int h = 0;
                        while (h < ti.nparts && ok) {
                            int n = 0;
                            if (lane == 0) {
                                fence_proxy_async_all();
                                int hh = h;
                                for (; hh < ti.nparts && n < kBatch; ++hh)
                                    if (hh != ti.part) ++n;
                                if (n > 0) {
                                    mbar_arrive_expect_tx(fetch_bar(ew), static_cast<uint32_t>(n) * kUnitBytes);
                                    int k = 0;
                                    for (int g = h; g < hh; ++g) {
                                        if (g == ti.part) continue;
                                        bulk_load_1d(fetch_base + static_cast<uint32_t>(k) * kUnitBytes,
                                                     tile_bufs + static_cast<size_t>(g) * kCtas * tile_elems + unit_off, kUnitBytes,
                                                     fetch_bar(ew));
                                        ++k;
                                    }
                                }
                                h = hh;
                            }
                            n = __shfl_sync(0xFFFFFFFFu, n, 0);
                            h = __shfl_sync(0xFFFFFFFFu, h, 0);
                            if (n == 0) continue;
                            uint32_t got = 1;
                            if (lane == 0) got = wait_bar(fetch_bar(ew), fetch_phase, p, ROLE_EPILOGUE, t, 400 + ew) ? 1u : 0u;
                            got = __shfl_sync(0xFFFFFFFFu, got, 0);
                            if (!got) { ok = false; break; }
                            fetch_phase ^= 1u;
                            for (int k = 0; k < n; ++k) {
                                const uint32_t ub = fetch_base + static_cast<uint32_t>(k) * kUnitBytes + lane * 16u;
#pragma unroll
                                for (int i = 0; i < CH; i += 4) {
                                    float4 x;
                                    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                                 : "=f"(x.x), "=f"(x.y), "=f"(x.z), "=f"(x.w)
                                                 : "r"(ub + static_cast<uint32_t>(i) * 128u));
                                    v[i] += x.x; v[i + 1] += x.y; v[i + 2] += x.z; v[i + 3] += x.w;
                                }
                            }
                            __syncwarp();      // every lane has read the batch before lane 0 refills the buffer
                        }
                        if (!ok) break;
                    } else {
                        for (int h = 0; h < ti.nparts; ++h) {
                            if (h == ti.part) continue;
                            const float* pb = tile_bufs + static_cast<size_t>(h) * kCtas * tile_elems + unit_off + lane * 4;
#pragma unroll
                            for (int i = 0; i < CH; i += 4) {
                                const float4 x = __ldcg(reinterpret_cast<const float4*>(pb + i * 32));
                                v[i] += x.x; v[i + 1] += x.y; v[i + 2] += x.z; v[i + 3] += x.w;
                            }
                        }
                    }
                }

#ifdef SG_DEBUG_STAMPS
                if (stamp_chunk) SG_STAMP(17 + 3 * c);
#endif
                if (alpha != 1.0f) {
#pragma unroll
                    for (int i = 0; i < CH; ++i) v[i] *= alpha;
                }
                const bool ex_any = (kVB == 0 || kVB == 4) ? p.ex_any != 0 : false;
                if (ex_any) {
                    if (p.row_scale != nullptr) {
                        const float rs = row < ti.rows ? __ldg(p.row_scale + row) : 0.0f;
#pragma unroll
                        for (int i = 0; i < CH; ++i) v[i] *= rs;
                    }
                    if (p.col_scale != nullptr) {
                        // every lane reads the same addresses: one broadcast transaction per load
                        const float* cs = p.col_scale + n0 + c * CH;
                        if (n0 + (c + 1) * CH <= p.N) {
#pragma unroll
                            for (int i = 0; i < CH; i += 4) {
                                const float4 s4 = __ldg(reinterpret_cast<const float4*>(cs + i));
                                v[i] *= s4.x; v[i + 1] *= s4.y; v[i + 2] *= s4.z; v[i + 3] *= s4.w;
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < CH; ++i) v[i] *= (n0 + c * CH + i < p.N) ? __ldg(cs + i) : 0.0f;
                        }
                    }
                }
                if (has_c && row < ti.rows) {
                    const int col0 = n0 + c * CH;
                    if constexpr (kOutF32) {
                        const float* cp = reinterpret_cast<const float*>(c_g) + mem_row * p.ldc + col0;
                        if (col0 + CH <= p.N) {
#pragma unroll
                            for (int i = 0; i < CH; i += 4) {
                                const float4 cv = *reinterpret_cast<const float4*>(cp + i);
                                v[i] += beta * cv.x; v[i + 1] += beta * cv.y; v[i + 2] += beta * cv.z; v[i + 3] += beta * cv.w;
                            }
                        } else {
                            for (int i = 0; i < CH; ++i) if (col0 + i < p.N) v[i] += beta * cp[i];
                        }
                    } else {
                        const uint16_t* cp = reinterpret_cast<const uint16_t*>(c_g) + mem_row * p.ldc + col0;
                        if (col0 + CH <= p.N) {
#pragma unroll
                            for (int i = 0; i < CH; i += 8) {
                                const uint4 cv = *reinterpret_cast<const uint4*>(cp + i);
                                const uint32_t w[4] = {cv.x, cv.y, cv.z, cv.w};
#pragma unroll
                                for (int j = 0; j < 4; ++j) {
                                    float lo, hi;
                                    unpack2<kOutF16>(w[j], lo, hi);
                                    v[i + 2 * j] += beta * lo;
                                    v[i + 2 * j + 1] += beta * hi;
                                }
                            }
                        } else {
                            for (int i = 0; i < CH; ++i) if (col0 + i < p.N) v[i] += beta * half_bits_to_float(cp[i], kOutF16);
                        }
                    }
                }
                if (has_bias && bias_f32) {
                    // every lane reads the same addresses: broadcast loads
                    const float* bf = reinterpret_cast<const float*>(mode == MODE_GROUPED ? p.g_bias[ti.b] : p.bias) +
                                      (mode == MODE_GROUPED ? 0 : static_cast<int64_t>(ti.b) * p.strideBias) + n0 + c * CH;
#pragma unroll
                    for (int i = 0; i < CH; ++i) v[i] += (n0 + c * CH + i < p.N) ? __ldg(bf + i) : 0.0f;
                } else if (has_bias) {
#pragma unroll
                    for (int i = 0; i < CH; i += 4) {
                        const uint2 b2 = *reinterpret_cast<const uint2*>(bias_w + (c / kStep) * CH + i);   // 4 bf16, broadcast read
                        if constexpr (kEpiWarps == 4) {
                            // (the instantiations of long K loops; in the others the shorter code measured slower)
                            if (in_f16) { add_pair<true>(b2.x, v[i], v[i + 1]); add_pair<true>(b2.y, v[i + 2], v[i + 3]); }
                            else { add_pair<false>(b2.x, v[i], v[i + 1]); add_pair<false>(b2.y, v[i + 2], v[i + 3]); }
                        } else {
                            float b0, b1, b2f, b3;
                            if (in_f16) { unpack2<true>(b2.x, b0, b1); unpack2<true>(b2.y, b2f, b3); }
                            else { unpack2<false>(b2.x, b0, b1); unpack2<false>(b2.y, b2f, b3); }
                            v[i] += b0; v[i + 1] += b1; v[i + 2] += b2f; v[i + 3] += b3;
                        }
                    }
                }
                if (ex_any) {
                    if (p.row_bias != nullptr) {
                        const float rb = row < ti.rows ? __ldg(p.row_bias + row) : 0.0f;
#pragma unroll
                        for (int i = 0; i < CH; ++i) v[i] += rb;
                    }
                    if (p.aux_store != nullptr && row < ti.rows) {
                        // the value the activation is about to see, in the output's type; each lane owns one row
                        const int col0 = n0 + c * CH;
                        if constexpr (kOutF32) {
                            float* ap = reinterpret_cast<float*>(p.aux_store) + static_cast<int64_t>(row) * p.ld_aux_store + col0;
                            if (col0 + CH <= p.N) {
#pragma unroll
                                for (int i = 0; i < CH; i += 4)
                                    *reinterpret_cast<float4*>(ap + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                            } else {
                                for (int i = 0; i < CH; ++i) if (col0 + i < p.N) ap[i] = v[i];
                            }
                        } else {
                            uint16_t* ap = reinterpret_cast<uint16_t*>(p.aux_store) + static_cast<int64_t>(row) * p.ld_aux_store + col0;
                            if (col0 + CH <= p.N) {
#pragma unroll
                                for (int i = 0; i < CH; i += 8)
                                    *reinterpret_cast<uint4*>(ap + i) =
                                        make_uint4(pack2<kOutF16>(v[i], v[i + 1]), pack2<kOutF16>(v[i + 2], v[i + 3]),
                                                   pack2<kOutF16>(v[i + 4], v[i + 5]), pack2<kOutF16>(v[i + 6], v[i + 7]));
                            } else {
                                for (int i = 0; i < CH; ++i)
                                    if (col0 + i < p.N) ap[i] = static_cast<uint16_t>(pack2<kOutF16>(v[i], 0.0f) & 0xFFFFu);
                            }
                        }
                    }
                }
                // A plain ReLU in front of a 16-bit output that goes out through the staging block is folded into the
                // conversion below (one instruction per pair instead of two half-rate max operations and one).
                constexpr int kElemsPer16B = kOutF32 ? 4 : 8;
                const bool plain_store = d_remap || (n0 + (c + 1) * CH > p.N && (p.N % kElemsPer16B) != 0);
                // (Only in the four-epilogue-warp instantiations, the ones long K loops run in: the second copy of the
                // staging loop lengthens the code a short launch has to fetch once per SM -- 256^3 3.6 -> 3.8 us.)
                const bool relu_in_cvt = !kOutF32 && kEpiWarps == 4 && epi == EPI_RELU && !ex_any && !plain_store;
                if (epi >= EPI_RELU && !relu_in_cvt) apply_act_chunk<kOut == 0, CH>(v, epi, p.epi_arg0, p.epi_arg1);
                if (ex_any) {
                    if (p.post_scale != 1.0f) {
                        const float ps = p.post_scale;
#pragma unroll
                        for (int i = 0; i < CH; ++i) v[i] *= ps;
                    }
                    if (p.aux_load != nullptr && row < ti.rows) {
                        const int col0 = n0 + c * CH;
                        if constexpr (kOutF32) {
                            const float* rp = reinterpret_cast<const float*>(p.aux_load) + static_cast<int64_t>(row) * p.ld_aux_load + col0;
                            if (col0 + CH <= p.N) {
#pragma unroll
                                for (int i = 0; i < CH; i += 4) {
                                    const float4 rv = *reinterpret_cast<const float4*>(rp + i);
                                    v[i] += rv.x; v[i + 1] += rv.y; v[i + 2] += rv.z; v[i + 3] += rv.w;
                                }
                            } else {
                                for (int i = 0; i < CH; ++i) if (col0 + i < p.N) v[i] += rp[i];
                            }
                        } else {
                            const uint16_t* rp = reinterpret_cast<const uint16_t*>(p.aux_load) + static_cast<int64_t>(row) * p.ld_aux_load + col0;
                            if (col0 + CH <= p.N) {
#pragma unroll
                                for (int i = 0; i < CH; i += 8) {
                                    const uint4 rv = *reinterpret_cast<const uint4*>(rp + i);
                                    const uint32_t w[4] = {rv.x, rv.y, rv.z, rv.w};
#pragma unroll
                                    for (int j = 0; j < 4; ++j) {
                                        float lo, hi;
                                        unpack2<kOutF16>(w[j], lo, hi);
                                        v[i + 2 * j] += lo;
                                        v[i + 2 * j + 1] += hi;
                                    }
                                }
                            } else {
                                for (int i = 0; i < CH; ++i) if (col0 + i < p.N) v[i] += half_bits_to_float(rp[i], kOutF16);
                            }
                        }
                    }
                }

                // A TMA store clips at 16-byte granularity along the row.  When N is not a multiple of 16 bytes the
                // last, partial chunk is therefore written with plain stores so nothing beyond column N changes; a
                // strided data gradient, whose rows are scattered over the image, is always stored this way.
                if (plain_store) {
                    if (row < ti.rows) {
                        const int col0 = n0 + c * CH;
                        const int valid = min(CH, p.N - col0);
                        if constexpr (kOutF32) {
                            float* dp = reinterpret_cast<float*>(d_g) + mem_row * p.ldd + col0;
#pragma unroll
                            for (int i = 0; i < CH; i += 4) {
                                if (i + 4 <= valid) {
                                    *reinterpret_cast<float4*>(dp + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                                } else {
#pragma unroll
                                    for (int j = 0; j < 4; ++j) if (i + j < valid) dp[i + j] = v[i + j];
                                }
                            }
                        } else {
                            uint16_t* dp = reinterpret_cast<uint16_t*>(d_g) + mem_row * p.ldd + col0;
#pragma unroll
                            for (int i = 0; i < CH; i += 8) {
                                if (i + 8 <= valid) {
                                    *reinterpret_cast<uint4*>(dp + i) =
                                        make_uint4(pack2<kOutF16>(v[i], v[i + 1]), pack2<kOutF16>(v[i + 2], v[i + 3]),
                                                   pack2<kOutF16>(v[i + 4], v[i + 5]), pack2<kOutF16>(v[i + 6], v[i + 7]));
                                } else {
#pragma unroll
                                    for (int j = 0; j < 8; ++j)
                                        if (i + j < valid) dp[i + j] = static_cast<uint16_t>(pack2<kOutF16>(v[i + j], 0.0f) & 0xFFFFu);
                                }
                            }
                        }
                    }
                    __syncwarp();
                    continue;
                }

#ifdef SG_DEBUG_STAMPS
                if (stamp_chunk) SG_STAMP(18 + 3 * c);
#endif
                // stage the 32 x 128-byte block (row = lane) in the swizzled layout the store map expects
                const uint32_t sb = chunk_ctr % Cfg::STAGING_BUFS;
                ++chunk_ctr;
                if (lane == 0) tma_store_wait_read<Cfg::STAGING_BUFS - 1>();   // the store that last read this block is done
                __syncwarp();
                const uint32_t stg = smem_base + Cfg::OFF_STAGING + (ew * Cfg::STAGING_BUFS + sb) * 4096u;
                const uint32_t row_addr = stg + lane * 128u;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    uint32_t w0, w1, w2, w3;
                    if constexpr (kOutF32) {
                        w0 = __float_as_uint(v[4 * j]); w1 = __float_as_uint(v[4 * j + 1]);
                        w2 = __float_as_uint(v[4 * j + 2]); w3 = __float_as_uint(v[4 * j + 3]);
                    } else if (relu_in_cvt) {
                        w0 = pack2_relu<kOutF16>(v[8 * j], v[8 * j + 1]);
                        w1 = pack2_relu<kOutF16>(v[8 * j + 2], v[8 * j + 3]);
                        w2 = pack2_relu<kOutF16>(v[8 * j + 4], v[8 * j + 5]);
                        w3 = pack2_relu<kOutF16>(v[8 * j + 6], v[8 * j + 7]);
                    } else {
                        w0 = pack2<kOutF16>(v[8 * j], v[8 * j + 1]);
                        w1 = pack2<kOutF16>(v[8 * j + 2], v[8 * j + 3]);
                        w2 = pack2<kOutF16>(v[8 * j + 4], v[8 * j + 5]);
                        w3 = pack2<kOutF16>(v[8 * j + 6], v[8 * j + 7]);
                    }
                    const uint32_t addr = row_addr + ((static_cast<uint32_t>(j) ^ (lane & 7u)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(w0), "r"(w1), "r"(w2), "r"(w3) : "memory");
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_3d(mapD, stg, n0 + c * CH, row0, bz);
                    tma_store_commit();
                }
            }
            if (!ok) break;
            }   // passes
            if (!ok) break;
            if (ksplit_tile) {
                // the accumulator was read in both passes: hand it back now; then count this warp as done with the
                // tile's scratch -- the last warp of all parts leaves every counter at zero for the next launch
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) {
                    if constexpr (kPair) mbar_arrive_cluster(tempty_remote[acc]);
                    else mbar_arrive(tempty_remote[acc]);
                    if (!early && !two_pass) {       // (with early donors the owner's CTA resets the counters)
                        uint32_t* arrived = p.sk_flags + ti.tail;
                        uint32_t* consumed = p.sk_flags + p.sk_consumed_off + ti.tail;
                        if (atomicAdd(consumed, 1u) == static_cast<uint32_t>(p.sk_arrivals * ti.nparts) - 1u) {
                            *arrived = 0u;
                            *consumed = 0u;
                            __threadfence();
                        }
                    }
                }
            }
            if (kSplitK && preload_next) {
                // The item two further on is an owner part and will accumulate in the buffer this item just used: wait
                // for the donors of its tile (they ran at the very start of the launch), add their parked sums up, write
                // them into the buffer, and only then hand the buffer back to the MMA warp.
                int g_hint2 = 0;
                const Tile tn = decode_tile<Cfg::TILE_M, BN, kVB, kSplitK>(p, t_next2, g_hint2);
                uint32_t* arrived = p.sk_flags + tn.tail;
                uint32_t okw = 1;
                if (lane == 0) okw = wait_counter(arrived, static_cast<uint32_t>(p.sk_arrivals * (tn.nparts - 1)), p, t_next2) ? 1u : 0u;
                okw = __shfl_sync(0xFFFFFFFFu, okw, 0);
                if (!okw) { ok = false; break; }
                __threadfence();                // the donors' sums are read after their arrivals
                if (tn.m0 + static_cast<int>(cta_rank) * Cfg::BM + q * 32 < tn.rows) {
                    constexpr uint32_t kUnitBytes = CH * 128u;
                    const size_t tile_elems = static_cast<size_t>(Cfg::BM) * BN;
                    const float* bufs = p.sk_partials + static_cast<size_t>(tn.tail) * p.ksplit * kCtas * tile_elems +
                                        static_cast<size_t>(cta_rank) * tile_elems + lane * 4;
                    const int nchunks2 = (min(tn.width, p.N - tn.n0) + CH - 1) / CH;
#pragma unroll 1
                    for (int c = half; c < nchunks2; c += kStep) {
                        uint32_t w[CH];
#pragma unroll
                        for (int i = 0; i < CH; ++i) w[i] = 0u;
                        for (int g = 0; g < tn.nparts - 1; ++g) {
                            const float* pb = bufs + static_cast<size_t>(g) * kCtas * tile_elems + static_cast<size_t>(c * 4 + q) * (kUnitBytes / 4);
#pragma unroll
                            for (int i = 0; i < CH; i += 4) {
                                const float4 x = __ldcg(reinterpret_cast<const float4*>(pb + i * 32));
                                w[i] = __float_as_uint(__uint_as_float(w[i]) + x.x);
                                w[i + 1] = __float_as_uint(__uint_as_float(w[i + 1]) + x.y);
                                w[i + 2] = __float_as_uint(__uint_as_float(w[i + 2]) + x.z);
                                w[i + 3] = __float_as_uint(__uint_as_float(w[i + 3]) + x.w);
                            }
                        }
                        uint32_t lo[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) lo[i] = w[i];
                        tmem_st_32x32(t_row + c * CH, lo);
                        if constexpr (!kOutF32) {
                            uint32_t hi[32];
#pragma unroll
                            for (int i = 0; i < 32; ++i) hi[i] = w[32 + i];
                            tmem_st_32x32(t_row + c * CH + 32, hi);
                        }
                    }
                    tmem_st_wait();
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) {
                    if constexpr (kPair) mbar_arrive_cluster(tempty_remote[acc]);
                    else mbar_arrive(tempty_remote[acc]);
                    // this warp is done with the tile's scratch: the last warp of the owner's CTAs leaves the counters at zero
                    uint32_t* consumed = p.sk_flags + p.sk_consumed_off + tn.tail;
                    if (atomicAdd(consumed, 1u) == static_cast<uint32_t>(p.sk_arrivals) - 1u) {
                        *arrived = 0u;
                        *consumed = 0u;
                        __threadfence();
                    }
                }
            }
        }
        if (warp == 2 && lane == 0) SG_STAMP(8);
        // the staging blocks must have been read before the CTA's shared memory goes away; the writes themselves
        // complete with the grid
        if (lane == 0) tma_store_wait_read<0>();
        if (warp == 2 && lane == 0) SG_STAMP(9);
        __syncwarp();
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before_sync();
    if (__syncthreads_or(!ok && !dead)) {
        // a wait expired somewhere: give copies still in flight time to land before the CTA retires
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    if (dead && early_kb > 0 && threadIdx.x == 0) {
        // the launch is a no-op, but the early loads are in flight: let them land before the shared memory goes away
        const uint64_t t0 = global_timer_ns();
        for (int j = 0; j < early_kb; ++j)
            while (!mbar_try_wait(full_bar(j), 0) && global_timer_ns() - t0 < 1000000ull) {}
    }
    if constexpr (kPair) {
        cluster_arrive();
        cluster_wait();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc<kPair>(tmem_base, Cfg::TMEM_COLS);
    }
    if (blockIdx.x == 0 && threadIdx.x == 96) {
        volatile uint64_t* w = reinterpret_cast<volatile uint64_t*>(p.status + 4);
        w[0] = static_cast<uint64_t>(clock64()) - clk0;
        w[1] = global_timer_ns() - ns0;
    }
    if (threadIdx.x == 32) SG_STAMP(10);
#ifdef SG_DEBUG_STAMPS
    if (threadIdx.x == 32 && blockIdx.x == sg_stamp_cta) {
        reinterpret_cast<volatile uint64_t*>(p.status + 8)[12] = clock64();
        reinterpret_cast<volatile uint64_t*>(p.status + 8)[14] = global_timer_ns();
    }
#endif
}

}  // namespace sg
