// Host-side table of the contraction kernel's instantiations, one translation unit per kernel variant so that the
// variants compile in parallel.
#pragma once
#include "sg_kernel.cuh"

namespace sg {

using KernelFn = void (*)(const Params);

struct KernelEntry {
    KernelFn fn;
    int smem;
    int threads;
};

// tile width (64, 128, 256) x CTA pairing x output type (0 bf16, 1 fp32, 2 fp16) x epilogue warps (4 or 8), for
// variant 0 (every mode and option), 1 dense, 2 convolution forward, 3 grouped, 4 dense with the extended epilogue
// chain, 5 convolution data gradient, 6 / 7 dense with a short A tile
KernelEntry kernel_variant_0(int bn, bool pair, int out, int epi_warps);
KernelEntry kernel_variant_1(int bn, bool pair, int out, int epi_warps);
KernelEntry kernel_variant_2(int bn, bool pair, int out, int epi_warps);
KernelEntry kernel_variant_3(int bn, bool pair, int out, int epi_warps);
KernelEntry kernel_variant_4(int bn, bool pair, int out, int epi_warps);
KernelEntry kernel_variant_5(int bn, bool pair, int out, int epi_warps);
KernelEntry kernel_variant_6(int bn, bool pair, int out, int epi_warps);   // dense, 64 rows of A loaded (single-CTA tiles)
KernelEntry kernel_variant_7(int bn, bool pair, int out, int epi_warps);   // dense, 32 rows of A loaded
KernelEntry kernel_variant_8(int bn, bool pair, int out, int epi_warps);   // dense, K ranges kept in
KernelEntry kernel_variant_9(int bn, bool pair, int out, int epi_warps);   // convolution forward, K ranges kept in

}  // namespace sg
