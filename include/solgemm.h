/*
 * solgemm.h -- C ABI of libsolgemm: fused dense tensor-core contractions for NVIDIA B200 (sm_100a)
 *
 *     D = act(alpha * A.B + beta * C + bias)
 *
 * for one GEMM, a strided batch of GEMMs, a ragged group of GEMMs and a 2-D forward
 * convolution evaluated as an implicit GEMM, plus the Speed-of-Light bound
 * t_SOL = max(FLOPs / peak, bytes / bandwidth) used to judge their headroom.
 *
 * These are the operations the muCUTLASS DSL of arXiv 2603.29010 names gemm(),
 * batched_gemm(), grouped_gemm(expert_count=E) and conv2d_fprop(kernel_h, kernel_w),
 * with its .with_dtype / .with_layout / .with_scaling clauses and its `>>` epilogue chain
 * (Section 3, Table 1, Appendix A.1), and the SOL analysis of Section 4.1 / Appendix A.2.
 *
 * General rules (they hold for every entry point unless it says otherwise)
 *  - Pointers named *_host are host memory; every other data pointer is DEVICE memory on the
 *    current CUDA device.  The caller owns all buffers; the library allocates no device memory.
 *  - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls
 *    enqueue work on that stream and return; they never synchronise.
 *  - Inputs A, B, bias (and conv X, Wf) are bf16 or fp16 (`in_dtype`, the same for all of them).  The
 *    output D is bf16, fp16 or fp32 (`out_dtype`); C, when read, has the output's dtype and shape.
 *    Accumulation and the epilogue run in fp32; the result is rounded to nearest-even.
 *    (The DSL's .with_dtype(input, acc, output); its running example is input=fp16, acc=fp32, output=fp16.)
 *    A and B (conv: X and Wf) may also be 8-bit floating point, SG_FP8_E4M3 or SG_FP8_E5M2 (both the same;
 *    the DSL's fp8_e4m3 / fp8_e5m2 input types): K-contiguous layouts only, leading dimensions multiples of 16
 *    elements; the bias then is bf16, the output bf16, fp16 or fp32.  Scale factors go through alpha.
 *    in_dtype SG_F32: A and B are fp32 in memory and are contracted on the TF32 tensor-core path (the paper's FP32
 *    problems with TF32 throughput, Appendix A.2): of every operand element the sign, the exponent and the upper 10
 *    fraction bits take part, the lower 13 fraction bits are ignored; accumulation is fp32.  K-contiguous layouts
 *    only, leading dimensions multiples of 4 elements; the bias then is fp32 (4-byte aligned).
 *    in_dtype SG_INT8 (the DSL's int8 / s8): signed 8-bit A and B, exact 32-bit integer accumulation; the accumulator
 *    is converted to fp32 (exact below 2^24) and goes through the same floating-point epilogue (alpha and the scale
 *    vectors of the extended chain dequantise); rules as for the 8-bit floats (K-contiguous, bf16 bias).
 *  - Epilogue: v = alpha*acc (+ beta*C if beta != 0) (+ bias[j] if bias != NULL); D = act(v).
 *    bias holds one value per output column j (GEMM) or output channel (conv); it is NOT scaled
 *    by alpha.  SG_EPI_BIAS is the identity activation and requires bias != NULL; every other
 *    activation accepts an optional bias.  SG_EPI_GELU is the tanh form
 *    0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3))).  beta == 0 means C is never read.
 *    With bf16 output the transcendental activations use hardware approximations (error well below one
 *    bf16 rounding step); with fp32 output they are evaluated to a few fp32 ulps.
 *  - Alignment (the TMA rule of the paper's Appendix A.1, constraint 3): every base pointer must
 *    be 16-byte aligned and every leading dimension / batch stride a multiple of 16 bytes
 *    (8 bf16 or 4 fp32 elements), else SG_ERR_ALIGNMENT.
 *  - Errors that can be detected from the arguments return before anything is launched and
 *    leave D untouched.  Exceptions never cross this boundary.  sg_last_error() gives a
 *    thread-local, human readable reason for the last non-OK status.
 *  - A device-side wait that runs out (it should never) makes the kernel stop early and record a
 *    code; sg_poll_status() reports it after the caller has synchronised the stream.
 */
#ifndef SOLGEMM_H_
#define SOLGEMM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SG_OK = 0,
    SG_ERR_INVALID_ARG = 1,   /* negative size, ld smaller than the extent, unknown enum value */
    SG_ERR_NULL_POINTER = 2,  /* a required pointer is NULL */
    SG_ERR_ALIGNMENT = 3,     /* base pointer or stride breaks the 16-byte rule */
    SG_ERR_UNSUPPORTED = 4,   /* valid request this build does not implement */
    SG_ERR_ARCH = 5,          /* current device is not compute capability 10.0 */
    SG_ERR_WORKSPACE = 6,     /* workspace NULL, misaligned or too small */
    SG_ERR_CUDA = 7,          /* a CUDA runtime/driver call failed */
    SG_ERR_TIMEOUT = 8        /* a bounded device-side wait expired (see sg_poll_status) */
} sg_status_t;

typedef enum { SG_BF16 = 0, SG_F32 = 1, SG_F16 = 2, SG_FP8_E4M3 = 3, SG_FP8_E5M2 = 4, SG_INT8 = 5 } sg_dtype_t;
typedef enum { SG_ROW_MAJOR = 0, SG_COL_MAJOR = 1 } sg_layout_t;
typedef enum {
    SG_EPI_NONE = 0, SG_EPI_BIAS = 1, SG_EPI_RELU = 2, SG_EPI_GELU = 3, SG_EPI_SILU = 4,
    /* (SG_EPI_RELU is max(x, 0); where x is NaN the result is NaN or +0, depending on the kernel variant that runs) */
    /* further built-ins of the paper's Table 1c; epi_arg0 / epi_arg1 carry their parameters */
    SG_EPI_SIGMOID = 5,     /* 1 / (1 + e^-x) */
    SG_EPI_TANH = 6,
    SG_EPI_MISH = 7,        /* x tanh(ln(1 + e^x)) */
    SG_EPI_HARDSWISH = 8,   /* x min(max(x + 3, 0), 6) / 6 */
    SG_EPI_LEAKY_RELU = 9,  /* x > 0 ? x : epi_arg0 * x */
    SG_EPI_ELU = 10,        /* x > 0 ? x : epi_arg0 * (e^x - 1) */
    SG_EPI_CLIP = 11        /* min(max(x, epi_arg0), epi_arg1), epi_arg0 <= epi_arg1 (the DSL's clip / clamp) */
} sg_epilogue_t;

/*
 * One GEMM problem (DSL: gemm().with_dtype(...).with_layout(A,B,C).with_scaling(alpha,beta) >> ...).
 *   a(i,k) = A[i*lda + k] (row-major) or A[k*lda + i] (column-major)
 *   b(k,j) = B[k*ldb + j] (row-major) or B[j*ldb + k] (column-major)
 *   C and D are row-major with leading dimensions ldc, ldd.  All ld* are in ELEMENTS.
 *   All four A/B layout pairs are implemented; the K-contiguous pair (A row-major, B column-major) is the
 *   tuned one.  (sg_grouped_gemm with a column-major A: every A_g is stored [K][M_g] with the one leading dimension
 *   lda >= max M_g.)
 *   Performance note: operand rows that start on 64-byte boundaries (lda, ldb multiples of 64 bytes) run at full
 *   speed; rows that do not (the 16-byte rule alone) cost a large product 16-19 % (measured), so pad where you can.
 * Enum-valued fields are int32_t so that the layout is the same from C, C++ and ctypes.
 */
typedef struct sg_gemm_desc {
    int64_t M, N, K;
    int32_t layout_a, layout_b;   /* sg_layout_t */
    int64_t lda, ldb, ldc, ldd;
    int32_t in_dtype, out_dtype;  /* sg_dtype_t; in_dtype SG_BF16, SG_F16, SG_F32 (tf32), SG_FP8_E4M3 or SG_FP8_E5M2 */
    float alpha, beta;
    int32_t epi;                  /* sg_epilogue_t */
    float epi_arg0, epi_arg1;     /* activation parameters (leaky_relu / elu slope, clip bounds); else ignored */
    int32_t reserved;             /* must be 0 */
} sg_gemm_desc_t;

/*
 * sg_gemm: D[M,N] = act(alpha * A.B + beta * C + bias).      (paper: gemm(), Table 1a, Appendix A.1)
 *   A, B   device, in_dtype, laid out as layout_a / layout_b and lda / ldb say.
 *   C      device, out_dtype, [M,N] row-major; may be NULL when beta == 0.
 *   bias   device, in_dtype, [N]; may be NULL unless epi == SG_EPI_BIAS.
 *   D      device, out_dtype, [M,N] row-major; written in full (all M x N elements).
 * M == 0 or N == 0: SG_OK, nothing is launched.  K == 0: D = act(beta*C + bias).
 * Matrix-vector form (the workload list's single-token decode product): when N <= 8 (or M <= 8; 4 for SG_F32 inputs or
 *   when K is no multiple of 8; also 9..32 for 16-bit inputs against a matrix of at most 48 MB and few enough rows that
 *   the groups of eight vectors are all resident at once), the matrix operand is
 *   K-contiguous (A row-major, resp. B column-major) and 16-byte aligned with a leading dimension that is a multiple
 *   of 16 bytes, the vectors are K-contiguous, 16-byte aligned and a multiple of 16 bytes apart (a single vector may
 *   also be stored as K x 1 with a leading dimension of 1), and in_dtype is SG_BF16, SG_F16 or SG_F32, the product
 *   runs as one pass over the matrix at HBM speed instead of through tensor-core tiles.  In that form ldc and ldd may
 *   be any value >= N (no 16-byte rule) and C, D and bias need only their element alignment; results are reproducible
 *   from run to run.  A small product of 16-bit K-contiguous operands (at most 160 M multiply-adds, and few enough
 *   outputs that one CTA per 16 x 8, 16 x 16 or 16 x 32 of them fits on the GPU at once) runs on the same kernels, in
 *   groups of vectors, for their shorter start and end; a tile shape forced through sg_set_tuning keeps it on the tiles.
 */
sg_status_t sg_gemm(const sg_gemm_desc_t* desc, const void* A, const void* B, const void* C,
                    const void* bias, void* D, void* cuda_stream);

/*
 * sg_gemm_host: sg_gemm for callers whose operands and result live in HOST memory (the end-to-end form the paper's
 * generated wrappers have around a kernel: move the operands in, launch, hand the result back; Section 3, PyTorch wrapper).
 *   A_host, B_host, C_host, bias_host, D_host   host pointers laid out exactly as `desc` says (same leading dimensions);
 *                    pinned memory lets the copies overlap the kernel, pageable memory works but serialises them.
 *                    Element alignment is enough.  C_host may be NULL when beta == 0, bias_host unless SG_EPI_BIAS.
 *   staging_dev      device buffer lent by the caller, 256-byte aligned, at least sg_gemm_host_staging_size(desc)
 *                    bytes: device copies of A, B, bias, C and D with the host's geometry.  The library allocates none.
 *   chunks           the rows of A, C and D are cut into this many blocks (multiples of 256 rows; 0 = 4, at most 16):
 *                    while one copy engine brings in block i+1 the kernel works on block i and the other copy engine
 *                    takes block i-1 of D back, so the call costs about the larger of the two transfers, not their sum.
 * Everything is ordered against `cuda_stream`: the call's work starts after what is already on it, and the stream
 * continues only when D_host is complete; the call itself returns without synchronising.  The first call on a device
 * creates two internal streams and a few events (not inside a stream capture).  Calls on one device share them: two
 * calls may be in flight at once only on the same stream.
 * Errors as for sg_gemm, SG_ERR_WORKSPACE for the staging buffer.  M == 0 or N == 0: SG_OK, nothing is enqueued.
 */
sg_status_t sg_gemm_host_staging_size(const sg_gemm_desc_t* desc, size_t* bytes);
sg_status_t sg_gemm_host(const sg_gemm_desc_t* desc, const void* A_host, const void* B_host, const void* C_host,
                         const void* bias_host, void* D_host, void* staging_dev, size_t staging_bytes, int32_t chunks,
                         void* cuda_stream);

/*
 * sg_batched_gemm: the same product for b = 0 .. batch-1, operand X of problem b starting at
 * X + b*strideX elements.                                      (paper: batched_gemm(), Appendix A.1)
 *   strideBias == 0 shares one bias vector between all problems.
 * batch == 0: SG_OK, nothing is launched.
 */
sg_status_t sg_batched_gemm(const sg_gemm_desc_t* desc, int64_t batch,
                            int64_t strideA, int64_t strideB, int64_t strideC, int64_t strideD,
                            int64_t strideBias,
                            const void* A, const void* B, const void* C, const void* bias, void* D,
                            void* cuda_stream);

/*
 * sg_grouped_gemm: `groups` independent products D_g[M_g,N] = act(alpha*A_g.B_g + beta*C_g + bias_g)
 * in one launch; N, K, layouts, leading dimensions, dtypes, alpha, beta and epi come from `common`
 * (its M is ignored), M_g from M_host.              (paper: grouped_gemm(expert_count=E), Table 1a)
 *   M_host           host, [groups], M_g >= 0 (a group with M_g == 0 is skipped).
 *   *_ptrs_host      host arrays of `groups` DEVICE pointers.  C_ptrs_host may be NULL when
 *                    beta == 0; bias_ptrs_host may be NULL (no bias) unless epi == SG_EPI_BIAS.
 *   workspace_dev    device scratch of at least sg_grouped_gemm_workspace_size(groups) bytes,
 *                    128-byte aligned; the call writes per-group tensor maps and the tile table
 *                    into it with a stream-ordered copy.  It must stay untouched until the work
 *                    enqueued by this call has finished.  The host arrays may be freed on return.
 */
sg_status_t sg_grouped_gemm_workspace_size(int32_t groups, size_t* bytes);
sg_status_t sg_grouped_gemm(const sg_gemm_desc_t* common, int32_t groups, const int64_t* M_host,
                            const void* const* A_ptrs_host, const void* const* B_ptrs_host,
                            const void* const* C_ptrs_host, const void* const* bias_ptrs_host,
                            void* const* D_ptrs_host,
                            void* workspace_dev, size_t workspace_bytes, void* cuda_stream);

/*
 * sg_grouped_gemm_static: sg_grouped_gemm for callers that cannot provide a workspace because they cannot
 * allocate device memory at all -- for example code that runs after its process has handed the whole GPU to
 * a memory pool it may not draw from, or a latency-critical path where cudaMalloc (which may synchronise the
 * device) is forbidden.  (The paper has no counterpart: its generated wrappers allocate their workspace.)
 *   The per-group tensor maps and the tile table go into a fixed scratch array that is part of the library
 *   image (about 36 KB of device memory on every GPU that loads the library, held until the process exits),
 *   so the call takes no workspace arguments and (after the first call on a device, see below) allocates nothing.  Inputs and
 *   outputs are still the caller's buffers; all other arguments and the result are those of sg_grouped_gemm.
 *   groups > SG_STATIC_MAX_GROUPS           -> SG_ERR_WORKSPACE, nothing is launched.
 *   The first call on a device looks up the array's device address (once per device, with that device
 *   current).  That look-up, like the first use of any kernel of the library, makes the CUDA runtime load the
 *   library's device code, which itself takes device memory and may synchronise: make the first call on each
 *   device early -- before the GPU's memory is handed to the pool -- and outside any stream capture.  From the
 *   second call on nothing is allocated or loaded.
 *   All calls on a device share the one array and it keeps the previous call's tables until they are
 *   overwritten: every call rewrites all entries it uses before its kernel reads them, but two calls whose
 *   work overlaps on the GPU (different streams, or the same stream from two threads) race on it.  Serialise
 *   such calls or use sg_grouped_gemm with separate workspaces.
 */
#define SG_STATIC_MAX_GROUPS 64
sg_status_t sg_grouped_gemm_static(const sg_gemm_desc_t* common, int32_t groups, const int64_t* M_host,
                                   const void* const* A_ptrs_host, const void* const* B_ptrs_host,
                                   const void* const* C_ptrs_host, const void* const* bias_ptrs_host,
                                   void* const* D_ptrs_host, void* cuda_stream);

/*
 * One forward convolution (cross-correlation, groups = 1), tensors in the paper's TensorNHWC
 * layout (Table 1a "Conv2d ... NHWC"; Appendix A.1 conv2d_fprop(kernel_h=R, kernel_w=S)):
 *   X [N,H,W,C], Wf [K,R,S,C], Y and Cin [N,P,Q,K], bias [K], all contiguous;
 *   P = floor((H + 2 pad_h - dil_h (R-1) - 1) / stride_h) + 1, Q likewise;
 *   Y[n,p,q,k] = act( alpha * sum_{r,s,c} X[n, p stride_h - pad_h + r dil_h, q stride_w - pad_w + s dil_w, c]
 *                                         * Wf[k,r,s,c]  + beta * Cin[n,p,q,k] + bias[k] ),
 *   taps outside the image contribute zero.  The im2col matrix is never materialised.
 * Requires C * (input element size) and K * (output element size) to be multiples of 16 bytes (C % 8 == 0 and
 * K % 8 == 0 for bf16; C % 16 == 0 for 8-bit inputs) and pads / filter extents within the TMA
 * im2col limits (pad <= 127, (R-1) dil_h <= 255, (S-1) dil_w <= 255), else SG_ERR_ALIGNMENT /
 * SG_ERR_UNSUPPORTED.
 */
typedef struct sg_conv2d_desc {
    int64_t N, H, W, C, K, R, S;
    int32_t pad_h, pad_w, stride_h, stride_w, dil_h, dil_w;
    int32_t in_dtype, out_dtype;  /* sg_dtype_t */
    float alpha, beta;
    int32_t epi;                  /* sg_epilogue_t */
    float epi_arg0, epi_arg1;     /* activation parameters, as in sg_gemm_desc_t */
    int32_t reserved;             /* must be 0 */
} sg_conv2d_desc_t;

sg_status_t sg_conv2d_fprop(const sg_conv2d_desc_t* desc, const void* X, const void* Wf,
                            const void* Cin, const void* bias, void* Y, void* cuda_stream);

/*
 * sg_conv2d_dgrad / sg_conv2d_wgrad: the gradients of sg_conv2d_fprop with respect to its input and its filter
 * (paper: conv2d_dgrad(...), conv2d_wgrad(...), Appendix A.1 operator list).  `desc` describes the FORWARD problem
 * (N,H,W,C input, K filters of R x S, pads, strides, dilations); P, Q are its output extents.
 *   dgrad:  dX[n,h,w,c] = alpha * sum_{k,r,s} dY[n,p,q,k] * Wf[k,r,s,c]   over the (p,r), (q,s) with
 *           p*stride_h - pad_h + r*dil_h == h and q*stride_w - pad_w + s*dil_w == w,       + beta * Cin[n,h,w,c]
 *   wgrad:  dW[k,r,s,c] = alpha * sum_{n,p,q} dY[n,p,q,k] * X[n, p*stride_h - pad_h + r*dil_h, q*stride_w - pad_w + s*dil_w, c]
 *           (taps outside the image contribute 0)                                         + beta * Cin[k,r,s,c]
 *   dY   device, in_dtype (bf16 or fp16), [N,P,Q,K]        Wf  device, in_dtype, [K,R,S,C]       X  device, in_dtype, [N,H,W,C]
 *   Cin  device, out_dtype, the output's shape; may be NULL when beta == 0
 *   dX   device, out_dtype, [N,H,W,C], written in full     dW  device, out_dtype, [K,R,S,C], written in full
 * Both run as implicit GEMMs in the forward kernel: dgrad contracts over (tap, k) with the filter read C-contiguous
 * and its taps mirrored -- with a stride, one launch per output phase (h mod stride_h, w mod stride_w), each a
 * stride-1 problem over the taps that reach that phase, its rows scattered to their pixels of dX; wgrad is one
 * product per tap, dY^T (K x NPQ) times the tap-shifted X (NPQ x C), whose long contraction is cut into K ranges
 * through the scratch of sg_set_scratch when one is lent (few output tiles).
 * desc->epi must be SG_EPI_NONE.  K and C must span multiples of 16 bytes in both types.
 * SG_ERR_UNSUPPORTED: 8-bit inputs; strides above 8 or filter extents beyond the im2col TMA limits.
 * Empty outputs return SG_OK without a launch; an empty sum (no output pixels) gives beta * Cin.
 */
sg_status_t sg_conv2d_dgrad(const sg_conv2d_desc_t* desc, const void* dY, const void* Wf, const void* Cin,
                            void* dX, void* cuda_stream);
sg_status_t sg_conv2d_wgrad(const sg_conv2d_desc_t* desc, const void* dY, const void* X, const void* Cin,
                            void* dW, void* cuda_stream);

/*
 * Extended epilogue chain: the remaining built-ins of the DSL's `>>` chain (Table 1c; Appendix A.1
 * broadcast_op and fusion_op: per_row_scale, per_col_scale / per_channel_scale, column_broadcast,
 * scale(alpha=), aux_store, aux_load).  The DSL lets these follow one another in any order; this library
 * evaluates one fixed order (the order a dequantise - bias - activation - residual chain uses):
 *
 *   t          = alpha * acc[i][j] * row_scale[i] * col_scale[j] + beta * C[i][j] + bias[j] + row_bias[i]
 *   aux_store[i][j] = t                        (cast to out_dtype; the value the activation sees)
 *   D[i][j]    = post_scale * act(t) + aux_load[i][j]
 *
 * Every member is optional (NULL pointer / post_scale == 1 leaves its term out).
 *   row_scale, row_bias   device, fp32, [M]   (conv: one per output pixel, [N*P*Q]); 4-byte aligned
 *   col_scale             device, fp32, [N]   (conv: one per output channel, [K]);   16-byte aligned
 *   aux_load, aux_store   device, out_dtype, row-major [M][ld] with ld >= N; base and ld multiples of 16 bytes;
 *                         aux_store must not overlap D or any input; nothing beyond column N is read or written
 * Errors as for sg_gemm / sg_conv2d_fprop, plus SG_ERR_ALIGNMENT / SG_ERR_INVALID_ARG for the rules above.
 * ex == NULL makes the calls identical to sg_gemm / sg_conv2d_fprop.
 */
typedef struct sg_epilogue_ex {
    const void* row_scale;
    const void* col_scale;
    const void* row_bias;
    float post_scale;
    int32_t reserved0;            /* must be 0 */
    const void* aux_load;
    int64_t ld_aux_load;          /* elements */
    void* aux_store;
    int64_t ld_aux_store;         /* elements */
} sg_epilogue_ex_t;

sg_status_t sg_gemm_ex(const sg_gemm_desc_t* desc, const sg_epilogue_ex_t* ex, const void* A, const void* B,
                       const void* C, const void* bias, void* D, void* cuda_stream);
sg_status_t sg_conv2d_fprop_ex(const sg_conv2d_desc_t* desc, const sg_epilogue_ex_t* ex, const void* X,
                               const void* Wf, const void* Cin, const void* bias, void* Y, void* cuda_stream);

/*
 * sg_transpose: out[b][c][r] = convert(in[b][r][c]) for b < batch, r < rows, c < cols -- the layout-transpose
 * stage with fused dtype conversion that the DSL's pipeline(transpose(...), kernel, transpose(...)) places
 * around a kernel (Section 3 "Multi-stage pipelines"; Appendix A.1 transpose_op: NCL <-> NLC, and
 * NCHW <-> NHWC "implemented by flattening HW": batch = N, rows = C, cols = H*W or the reverse).
 *   in   device, in_dtype (bf16, fp16 or fp32), [batch][rows][cols], row stride ld_in, batch stride stride_in (elements)
 *   out  device, out_dtype (bf16, fp16 or fp32), [batch][cols][rows], row stride ld_out, batch stride stride_out
 *   A conversion to a narrower significand (fp32 -> bf16 / fp16, bf16 <-> fp16) rounds to nearest even; widening is
 *   exact.  in and out must not overlap.
 * Base pointers 16-byte aligned, ld and strides multiples of 16 bytes, ld_in >= cols, ld_out >= rows.
 * When rows and cols both span multiples of 16 bytes (in the output resp. input type) the stage runs as a persistent
 * kernel that streams tiles through shared memory with TMA loads and stores; other extents take a plain-store kernel
 * with element-wise edges.  Either way nothing outside out[b][c][0 .. rows) is written.
 * An empty extent returns SG_OK without a launch.  A memory-bound kernel: its Speed-of-Light time is
 * batch*rows*cols*(input + output element bytes) / bandwidth (sg_sol_bound, SG_OP_TRANSPOSE).
 */
typedef struct sg_transpose_desc {
    int64_t batch, rows, cols;
    int64_t ld_in, ld_out, stride_in, stride_out;
    int32_t in_dtype, out_dtype;  /* sg_dtype_t */
    int32_t reserved, reserved2;  /* must be 0 */
} sg_transpose_desc_t;

sg_status_t sg_transpose(const sg_transpose_desc_t* desc, const void* in, void* out, void* cuda_stream);

/*
 * Speed-of-Light bound (paper: Section 4.1 steps 1-4; worked example in Appendix A.2).
 * Host-only, pure function of its arguments.
 *   flops = 2 per multiply-accumulate of the contraction (halo taps of a padded conv included;
 *           epilogue arithmetic excluded);
 *   bytes = every unique input element read once + every output element written once
 *           (C only if beta != 0, bias only if has_bias);
 *   peaks scaled linearly by current/max clock (a zero clock means ratio 1);
 *   t_compute = flops / eff_peak, t_mem = bytes / eff_bandwidth, t_sol = max of the two;
 *   ai = flops / bytes, ridge = eff_peak / eff_bandwidth, compute_bound = ai > ridge.
 *   op                SG_OP_GEMM / SG_OP_BATCHED / SG_OP_GROUPED: desc is sg_gemm_desc_t;
 *                     SG_OP_CONV2D, SG_OP_CONV2D_DGRAD, SG_OP_CONV2D_WGRAD: desc is sg_conv2d_desc_t (the forward
 *                     problem; the gradients execute the same 2*NPQ*K*CRS FLOPs and move dY + Wf + dX, resp. dY + X + dW);
 *                     SG_OP_TRANSPOSE: desc is sg_transpose_desc_t
 *                     (flops = 0; element sizes come from its dtypes, elem_bytes_* are ignored).
 *   batch_or_groups   batch count (BATCHED), group count (GROUPED), ignored otherwise.
 *   M_host            [groups] for GROUPED (desc->M ignored), else may be NULL.
 *   has_bias          0 none; 1 one bias vector per problem; for BATCHED, 2 = one shared vector.
 */
typedef struct sg_hw {
    double peak_flops, peak_bytes_per_s;                 /* at maximum clocks */
    double sm_clock_mhz, sm_clock_max_mhz, mem_clock_mhz, mem_clock_max_mhz;
} sg_hw_t;

typedef struct sg_sol {
    int64_t flops, bytes;
    double ai, t_compute_s, t_mem_s, t_sol_s, ridge, eff_peak_flops, eff_bytes_per_s;
    int32_t compute_bound;
    int32_t reserved;
} sg_sol_t;

typedef enum { SG_OP_GEMM = 0, SG_OP_BATCHED = 1, SG_OP_GROUPED = 2, SG_OP_CONV2D = 3, SG_OP_TRANSPOSE = 4,
               SG_OP_CONV2D_DGRAD = 5, SG_OP_CONV2D_WGRAD = 6 } sg_op_t;

sg_status_t sg_sol_bound(int32_t op, const void* desc, int64_t batch_or_groups, const int64_t* M_host,
                         int32_t elem_bytes_in, int32_t elem_bytes_out, int32_t has_bias,
                         const sg_hw_t* hw, sg_sol_t* out);

/* Status helpers.  sg_status_string / sg_last_error return pointers to static / thread-local text. */
const char* sg_status_string(sg_status_t status);
const char* sg_last_error(void);

/*
 * sg_poll_status: reads (and clears) the device-side status word of the current device.  Call it
 * after synchronising the stream(s) the work was enqueued on; `cuda_stream` is used for the read.
 * SG_OK, or SG_ERR_TIMEOUT with the role / tile / barrier that gave up in sg_last_error().  While
 * the word is set, later launches of the tensor-core contraction kernel return at once without computing, and the
 * kernels of the matrix-vector / small-product form of sg_gemm store nothing: their outputs stay untouched
 * (sg_transpose, whose kernel waits on nothing outside its own CTA, does not read the word); the poll that reports the word also clears it and
 * the K-range counters of a lent scratch, after which calls compute again.
 */
sg_status_t sg_poll_status(void* cuda_stream);

/*
 * Tuning knobs for experiments (not needed for correct use): a non-negative value overrides the
 * shape heuristic for later calls from any thread; -1 restores the heuristic.
 *   tile_n    64, 128 or 256            cta_pair   0 = one CTA per tile, 1 = two-CTA tiles
 */
sg_status_t sg_set_tuning(int32_t tile_n, int32_t cta_pair);

/*
 * sg_last_kernel_clock: the SM clock (MHz) at which the most recent contraction kernel on the current device
 * actually ran, measured inside the kernel (cycle counter over nanosecond timer of its first CTA).  Under a
 * board power cap this is what the paper's clock-aware Speed-of-Light rule should scale the peak by (Section 4.1,
 * hardware-limits step); management libraries may report the requested clock instead.
 * Synchronises `cuda_stream`.  0 if no kernel has run yet.
 */
sg_status_t sg_last_kernel_clock(double* sm_mhz, void* cuda_stream);

/*
 * sg_set_tail_mode: how the tiles of the last, partial wave are shared between SMs (tuning / tests):
 *   -1 let the planner decide (default), 0 leave them whole, 1 cut them into column slices,
 *    2 cut their K loop into ranges exchanged through the scratch (needs sg_set_scratch; else as 1).
 */
sg_status_t sg_set_tail_mode(int32_t mode);

/*
 * sg_set_scratch: lends the library a device buffer (current device) through which several SM groups can share
 * one output tile's K loop: every group parks its fp32 partial sums in the buffer and finishes a share of the tile
 * from all groups' sums (the DSL's split-K / tile=stream_k knobs, Appendix A.1).  With a scratch lent the planner
 * uses K ranges for problems with few output tiles and a long K -- skinny GEMMs, the convolution weight gradient --
 * where they are several times faster than whole tiles on a few SMs; for the last partial wave of large problems it
 * keeps column slices (as measured the exchange costs what it saves there; sg_set_tail_mode(2) forces K ranges).
 * Optional: without a scratch every tile runs its whole K loop; results agree up to fp32 summation order, and are
 * reproducible for a given shape and scratch.  256-byte aligned, at least 1 MB + 8 KB; SG_SCRATCH_BYTES_RECOMMENDED
 * covers every shape; the first 8 KB (counters) are cleared synchronously by this call and left at zero by every
 * launch.  The caller keeps ownership and must keep the buffer alive and untouched until it calls
 * sg_set_scratch(NULL, 0).  All calls on the device share it: work that overlaps on the GPU (several streams) must
 * not use it concurrently -- unregister it, or serialise such calls.
 */
#define SG_SCRATCH_BYTES_RECOMMENDED (32u << 20)
sg_status_t sg_set_scratch(void* scratch_dev, size_t bytes);

/*
 * sg_set_option: planner and launch overrides for measurements and tests (never needed for correct use; they apply to
 * later calls from any thread).  value -1 restores the default.  (The paper's DSL exposes such choices as explicit
 * clauses -- .with_tile, .with_stages, .with_scheduler, splits=, Table 1b; here a host heuristic takes them and these
 * knobs pin it.)
 */
typedef enum {
    SG_OPT_EPI_WARPS = 0,       /* 4 or 8 epilogue warps per CTA (default: 8 when K <= 1024) */
    SG_OPT_TAIL_SPLIT = 1,      /* 1, 2 or 4: column slices per tile of the last partial wave */
    SG_OPT_TAIL_KSPLIT = 2,     /* 0: never cut a K loop into ranges; k >= 2: k ranges where ranges are possible */
    SG_OPT_BAND_M = 3,          /* tile rows per raster band */
    SG_OPT_GENERAL_KERNEL = 4,  /* 1: always run the all-options kernel variant instead of the specialised ones */
    SG_OPT_NO_PDL = 5,          /* 1: launch without programmatic dependent launch */
    SG_OPT_NO_SHORT_A = 6,      /* 1: no short-A tiles for M <= 64 */
    SG_OPT_NO_GEMV = 7,         /* 1: matrix-vector shaped calls go through the tensor-core tiles */
    SG_OPT_GEMV_NO_MMA = 8,     /* 1: several vectors on the FMA matrix-vector kernel (<= 4 vectors) */
    SG_OPT_GEMV_NO_WIDE = 9,    /* 1: 16-byte loads only in the multi-vector kernel */
    SG_OPT_GEMV_ROWS = 10,      /* 1, 2 or 4 matrix rows per CTA in the single-vector kernel */
    SG_OPT_WAIT_LIMIT_NS = 11,  /* bound of every device-side wait in nanoseconds (default 2 s); tests shorten it to
                                   see the kernel give up, record where, and return */
    SG_OPT_L2_WARM_KBLOCKS = 12, /* k-blocks of every CTA's first tile prefetched into the L2 at kernel entry, before the
                                   launch dependency is waited for (default: 4 when the K loop has at most 16 k-blocks, else 0) */
    SG_OPT_TRANSPOSE_PLAIN = 13, /* 1: sg_transpose always runs its plain-store kernel (the one ragged extents take) */
    SG_OPT_EARLY_DONORS = 14,   /* K ranges for the last partial wave with the donor ranges run first (needs a scratch):
                                   0 never, k = 2..4 that many ranges per tile (default: the planner's estimate) */
    SG_OPT_TWO_PASS_SPLIT_K = 15, /* problems with fewer tiles than half the SMs and a long K loop: 0 = never cut the K loop
                                   into ranges summed by a second kernel, k >= 2 = at most k ranges (default: as many as
                                   there are SMs to go round) */
    SG_OPT_SPLIT_K_REDUCE_WARPS = 16, /* second pass of a two-pass K split: 1, 2, 4 or 8 warps share the parts of a column slice */
    SG_OPT_GEMV_MAX_VECTORS = 17, /* > 0: the matrix-vector kernels take at most this many vectors (4..32), all of them in one
                                   CTA, and the grouped form below is off (default: 8 in one CTA, more in groups) */
    SG_OPT_GEMV_SMALL_LOG2 = 18,  /* products of at most 2^value multiply-adds (16-bit operands) run on the warp-level MMA
                                   kernel in groups of vectors, whether or not their CTAs are all resident; 0 = none
                                   (default: 160 M multiply-adds, resident CTAs only) */
    SG_OPT_GEMV_VECTOR_BLOCKS = 19, /* blocks of eight vectors a CTA of the warp-level MMA kernel takes: 1, 2 or 4 */
    SG_OPT_COUNT_ = 20
} sg_option_t;
sg_status_t sg_set_option(int32_t option, int64_t value);

/*
 * sg_test_set_status_word: TEST HOOK.  Writes `value` into the device-side status word of the current device (what a
 * kernel whose wait ran out would do) and synchronises `cuda_stream`, so that the containment path -- later launches
 * are no-ops, sg_poll_status reports and clears -- can be exercised without any kernel waiting on anything.
 */
sg_status_t sg_test_set_status_word(uint32_t value, void* cuda_stream);

/* Number of kernel launches this library has enqueued from this process (monotonic). */
int64_t sg_launch_count(void);

/*
 * sg_last_kernel_name: the device function the calling thread's most recent compute launch ran, as the library's
 * own record (e.g. "sg::contract_kernel<256, true, 0, 4, 1>": tile width, two-CTA tiles, output type, epilogue
 * warps, variant).  Benchmarks list it next to their timings so that a reader can see that no vendor-library kernel
 * stands behind a number -- the check the paper's integrity pipeline makes on profiler kernel names (Section 4.4,
 * PyTorch-only detector).  Thread-local text, valid until the thread's next launch; "" before the first.
 */
const char* sg_last_kernel_name(void);

/*
 * How the calling thread's most recent contraction launch was tiled, for tests and benchmark records:
 *   plan6[0] tile width in columns, [1] 1 for two-CTA tiles, [2] tail split (the tiles of the last,
 *   partial wave are cut into this many column slices; 1 = none; a negative value -k means they are
 *   cut into k ranges of the K loop through the scratch instead), [3] length of the tile list,
 *   [4] list position of the first slice, [5] grid size in CTAs.
 */
sg_status_t sg_last_launch_plan(int32_t* plan6);

#ifdef __cplusplus
}
#endif
#endif /* SOLGEMM_H_ */
