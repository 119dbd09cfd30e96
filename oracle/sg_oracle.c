/*
 * sg_oracle.c -- CPU oracle for the fused dense contraction
 *
 *     D = act(alpha * A.B + beta * C + bias)
 *
 * THIS IS TEST INFRASTRUCTURE, NOT PART OF THE PRODUCT.  It exists so that the CUDA
 * library can be compared element by element with a plain, slow, obviously
 * correct definition.  Only the tests, the smoke check and the benchmark's
 * cpu-baseline / reference arm may load it.  It shares no code, header, table or
 * helper with the CUDA path and is never tuned for speed.
 *
 * Everything is evaluated in fp64.  bf16 / fp16 inputs are widened exactly; a product
 * of two such values (8- or 11-bit significands) is exact in fp64, so the only error
 * is the summation's (<= K * 2^-53 relative to sum |a||b|).
 *
 * What each function follows in the paper (arXiv 2603.29010):
 *   gemm / batched / grouped  -- the DSL operations gemm(), batched_gemm(),
 *       grouped_gemm(expert_count=E) with .with_dtype(input, acc, output),
 *       .with_layout(A, B, C) and .with_scaling(alpha, beta)  (Appendix A.1,
 *       grammar: OPERATIONS and CONFIGURATION); "each output element is a dot
 *       product" (Appendix A.2, section 1 of the SOL report).
 *   conv2d_fprop -- conv2d_fprop(kernel_h, kernel_w) on TensorNHWC input /
 *       filter / output (Appendix A.1; Table 1a "Conv2d ... NHWC").
 *   epilogue -- the `>>` chain bias() followed by one of relu(), gelu(), silu(), sigmoid(), tanh(),
 *       mish(), hardswish(), leaky_relu(alpha), elu(alpha), clip(min, max), compiled into one
 *       fused epilogue (Section 3, "Epilogue fusion"; Table 1c; Appendix A.1 EPILOGUE).
 *   sol -- the four-step Speed-of-Light analysis of Section 4.1 and its worked
 *       report in Appendix A.2.
 *
 * Readings taken where the paper is silent (listed in full in the design notes):
 *   bias is added after alpha/beta scaling and is not scaled by alpha; it holds
 *   one value per output column (GEMM) / output channel (conv); gelu is the tanh
 *   form; conv is cross-correlation with zero padding; the conv FLOP count
 *   includes the taps that fall in the padding halo; the result is NOT rounded
 *   to the output type here (the comparison tolerance absorbs that rounding).
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC sg_oracle.c -o libsg_oracle.so -lm
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_ROW_MAJOR = 0, ORC_COL_MAJOR = 1 };
enum { ORC_BF16 = 0, ORC_F32 = 1, ORC_F16 = 2, ORC_FP8_E4M3 = 3, ORC_FP8_E5M2 = 4, ORC_TF32 = 5, ORC_INT8 = 6 };
enum { ORC_EPI_NONE = 0, ORC_EPI_BIAS = 1, ORC_EPI_RELU = 2, ORC_EPI_GELU = 3, ORC_EPI_SILU = 4,
       ORC_EPI_SIGMOID = 5, ORC_EPI_TANH = 6, ORC_EPI_MISH = 7, ORC_EPI_HARDSWISH = 8, ORC_EPI_LEAKY_RELU = 9,
       ORC_EPI_ELU = 10, ORC_EPI_CLIP = 11 };

/* Number of host threads the parallel loops use. */
int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* bf16 -> fp64, exact: a bf16 is the upper half of an IEEE binary32. */
static double bf16_to_f64(uint16_t bits) {
    uint32_t u = (uint32_t)bits << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* IEEE binary16 -> fp64, exact: 1 sign, 5 exponent (bias 15), 10 fraction bits. */
static double f16_to_f64(uint16_t bits) {
    int sign = bits >> 15, e = (bits >> 10) & 0x1F, f = bits & 0x3FF;
    double v;
    if (e == 0) v = ldexp((double)f, -24);                       /* zero and subnormals: f * 2^-24 */
    else if (e == 31) v = f ? NAN : INFINITY;
    else v = ldexp(1.0 + (double)f / 1024.0, e - 15);
    return sign ? -v : v;
}

/* 8-bit floats (the DSL's fp8_e4m3 / fp8_e5m2).  e4m3 ("fn" flavour): 1 sign, 4 exponent (bias 7), 3 fraction
 * bits, no infinities, only S.1111.111 is NaN, largest value 448.  e5m2: 1, 5 (bias 15), 2, IEEE-like with
 * infinities and NaNs. */
static double fp8_e4m3_to_f64(uint8_t bits) {
    int sign = bits >> 7, e = (bits >> 3) & 0xF, f = bits & 0x7;
    double v;
    if (e == 15 && f == 7) v = NAN;
    else if (e == 0) v = ldexp((double)f, -9);                    /* subnormals: f/8 * 2^-6 */
    else v = ldexp(1.0 + (double)f / 8.0, e - 7);
    return sign ? -v : v;
}
static double fp8_e5m2_to_f64(uint8_t bits) {
    int sign = bits >> 7, e = (bits >> 2) & 0x1F, f = bits & 0x3;
    double v;
    if (e == 31) v = f ? NAN : INFINITY;
    else if (e == 0) v = ldexp((double)f, -16);                   /* subnormals: f/4 * 2^-14 */
    else v = ldexp(1.0 + (double)f / 4.0, e - 15);
    return sign ? -v : v;
}

/* fp32 storage used as a tf32 operand (the DSL's input=fp32 problems run on TF32 tensor cores, Appendix A.2 "TF32
 * note"): 1 sign, 8 exponent and the upper 10 fraction bits take part, the lower 13 fraction bits are ignored. */
static double tf32_to_f64(float f) {
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    u &= 0xFFFFE000u;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Element idx of an input operand (.with_dtype(input=bf16 | fp16 | fp8_e4m3 | fp8_e5m2 | fp32-as-tf32, ...)), widened
 * exactly (for tf32: after dropping the bits the tensor core does not read). */
static double in_to_f64(const void* p, int dtype, int64_t idx) {
    switch (dtype) {
        case ORC_TF32: return tf32_to_f64(((const float*)p)[idx]);
        case ORC_INT8: return (double)((const int8_t*)p)[idx];       /* the DSL's int8 / s8 input type */
        case ORC_F32: return (double)((const float*)p)[idx];
        case ORC_F16: return f16_to_f64(((const uint16_t*)p)[idx]);
        case ORC_FP8_E4M3: return fp8_e4m3_to_f64(((const uint8_t*)p)[idx]);
        case ORC_FP8_E5M2: return fp8_e5m2_to_f64(((const uint8_t*)p)[idx]);
        default: return bf16_to_f64(((const uint16_t*)p)[idx]);
    }
}

static double load_as_f64(const void* p, int dtype, int64_t idx) {
    if (dtype == ORC_BF16) return bf16_to_f64(((const uint16_t*)p)[idx]);
    if (dtype == ORC_F16) return f16_to_f64(((const uint16_t*)p)[idx]);
    return (double)((const float*)p)[idx];
}

/*
 * Activations of the fused epilogue (Table 1c built-ins): relu, gelu (tanh form), silu, sigmoid, tanh,
 * mish(x) = x tanh(ln(1 + e^x)), hardswish(x) = x min(max(x + 3, 0), 6) / 6, leaky_relu(x; a0) = x or a0 x,
 * elu(x; a0) = x or a0 (e^x - 1), clip(x; a0, a1) = min(max(x, a0), a1).
 * BIAS and NONE are the identity: the bias itself is added by the caller.
 */
double orc_act2(int epi, double x, double a0, double a1) {
    switch (epi) {
        case ORC_EPI_RELU:
            return x > 0.0 ? x : 0.0;
        case ORC_EPI_GELU: {
            const double c = 0.79788456080286535588; /* sqrt(2/pi) */
            return 0.5 * x * (1.0 + tanh(c * (x + 0.044715 * x * x * x)));
        }
        case ORC_EPI_SILU:
            return x / (1.0 + exp(-x));
        case ORC_EPI_SIGMOID:
            return 1.0 / (1.0 + exp(-x));
        case ORC_EPI_TANH:
            return tanh(x);
        case ORC_EPI_MISH:
            return x * tanh(x > 30.0 ? x : log1p(exp(x)));
        case ORC_EPI_HARDSWISH: {
            double r = x + 3.0;
            r = r < 0.0 ? 0.0 : (r > 6.0 ? 6.0 : r);
            return x * r / 6.0;
        }
        case ORC_EPI_LEAKY_RELU:
            return x > 0.0 ? x : a0 * x;
        case ORC_EPI_ELU:
            return x > 0.0 ? x : a0 * expm1(x);
        case ORC_EPI_CLIP:
            return x < a0 ? a0 : (x > a1 ? a1 : x);
        default:
            return x;
    }
}

double orc_act(int epi, double x) { return orc_act2(epi, x, 0.0, 0.0); }

/* The activation applied to n values (used by the extended epilogue chain of oracle.py). */
void orc_act_array(int epi, double a0, double a1, int64_t n, const double* in, double* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = orc_act2(epi, in[i], a0, a1);
}

/* -------------------------------------------------------------------------------------------
 * GEMM.   a(i,k) = A[i*lda + k] (row-major) or A[k*lda + i] (column-major)
 *         b(k,j) = B[k*ldb + j] (row-major) or B[j*ldb + k] (column-major)
 *         C and the result are row-major.
 * ----------------------------------------------------------------------------------------- */
typedef struct {
    int64_t M, N, K;
    int layout_a, layout_b;
    const void* A; int64_t lda;
    const void* B; int64_t ldb;
    const void* C; int c_dtype; int64_t ldc;     /* read only when beta != 0 */
    const void* bias; int bias_dtype;            /* [N] or NULL */
    double alpha, beta;
    int epi;
    double a0, a1;                               /* activation parameters */
    int in_dtype;                                /* type of A and B */
} gemm_problem;

/* One output element and, optionally, the magnitude sum used to scale fp32 tolerances. */
static double gemm_element(const gemm_problem* g, int64_t i, int64_t j, double* absacc) {
    double sum = 0.0, asum = 0.0;
    for (int64_t k = 0; k < g->K; ++k) {
        double a = in_to_f64(g->A, g->in_dtype, g->layout_a == ORC_ROW_MAJOR ? i * g->lda + k : k * g->lda + i);
        double b = in_to_f64(g->B, g->in_dtype, g->layout_b == ORC_ROW_MAJOR ? k * g->ldb + j : j * g->ldb + k);
        sum += a * b;
        asum += fabs(a * b);
    }
    double v = g->alpha * sum;
    double av = fabs(g->alpha) * asum;
    if (g->beta != 0.0) {                       /* beta == 0: C is never read */
        double c = load_as_f64(g->C, g->c_dtype, i * g->ldc + j);
        v += g->beta * c;
        av += fabs(g->beta * c);
    }
    if (g->bias) {
        double bj = in_to_f64(g->bias, g->bias_dtype, j);
        v += bj;
        av += fabs(bj);
    }
    if (absacc) *absacc = av;
    return orc_act2(g->epi, v, g->a0, g->a1);
}

/*
 * Rows [row_begin, row_end) of the result.  ref (and absacc, if not NULL) hold
 * (row_end-row_begin) x N values, row stride ldr, row 0 = row_begin.
 */
int orc_gemm(int64_t M, int64_t N, int64_t K, int layout_a, int layout_b,
             const void* A, int64_t lda, const void* B, int64_t ldb,
             const void* C, int c_dtype, int64_t ldc, const void* bias, int bias_dtype,
             double alpha, double beta, int epi, double a0, double a1, int in_dtype,
             int64_t row_begin, int64_t row_end, double* ref, double* absacc, int64_t ldr) {
    if (M < 0 || N < 0 || K < 0 || row_begin < 0 || row_end > M || row_begin > row_end) return 1;
    if (beta != 0.0 && !C) return 2;
    gemm_problem g = {M, N, K, layout_a, layout_b, A, lda, B, ldb, C, c_dtype, ldc, bias, bias_dtype, alpha, beta, epi, a0, a1, in_dtype};
#pragma omp parallel for schedule(static)
    for (int64_t i = row_begin; i < row_end; ++i) {
        for (int64_t j = 0; j < N; ++j) {
            double av;
            double v = gemm_element(&g, i, j, &av);
            ref[(i - row_begin) * ldr + j] = v;
            if (absacc) absacc[(i - row_begin) * ldr + j] = av;
        }
    }
    return 0;
}

/* The listed elements (pi[t], pj[t]) only: used to spot-check full-size problems. */
int orc_gemm_points(int64_t M, int64_t N, int64_t K, int layout_a, int layout_b,
                    const void* A, int64_t lda, const void* B, int64_t ldb,
                    const void* C, int c_dtype, int64_t ldc, const void* bias, int bias_dtype,
                    double alpha, double beta, int epi, double a0, double a1, int in_dtype,
                    int64_t npts, const int64_t* pi, const int64_t* pj, double* ref, double* absacc) {
    if (beta != 0.0 && !C) return 2;
    gemm_problem g = {M, N, K, layout_a, layout_b, A, lda, B, ldb, C, c_dtype, ldc, bias, bias_dtype, alpha, beta, epi, a0, a1, in_dtype};
    for (int64_t t = 0; t < npts; ++t)
        if (pi[t] < 0 || pi[t] >= M || pj[t] < 0 || pj[t] >= N) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < npts; ++t) {
        double av;
        ref[t] = gemm_element(&g, pi[t], pj[t], &av);
        if (absacc) absacc[t] = av;
    }
    return 0;
}

/* -------------------------------------------------------------------------------------------
 * conv2d forward (cross-correlation), X in NHWC, filter in KRSC, output in NPQK:
 *   P = floor((H + 2 pad_h - dil_h (R-1) - 1) / stride_h) + 1, Q likewise,
 *   y[n,p,q,k] = act( alpha * sum_{r,s,c} X[n, p stride_h - pad_h + r dil_h,
 *                                            q stride_w - pad_w + s dil_w, c] * Wf[k,r,s,c]
 *                     + beta * Cin[n,p,q,k] + bias[k] ),  taps outside the image contribute 0.
 * ----------------------------------------------------------------------------------------- */
typedef struct {
    int64_t N, H, W, C, K, R, S;
    int64_t pad_h, pad_w, stride_h, stride_w, dil_h, dil_w;
    int64_t P, Q;
    const void* X; const void* Wf;
    const void* Cin; int c_dtype;
    const void* bias; int bias_dtype;
    double alpha, beta;
    int epi;
    double a0, a1;
    int in_dtype;
} conv_problem;

int64_t orc_conv_out_extent(int64_t in, int64_t pad, int64_t dil, int64_t filt, int64_t stride) {
    int64_t span = in + 2 * pad - dil * (filt - 1) - 1;
    if (span < 0) return 0;
    return span / stride + 1;
}

static double conv_element(const conv_problem* cv, int64_t n, int64_t p, int64_t q, int64_t k, double* absacc) {
    double sum = 0.0, asum = 0.0;
    for (int64_t r = 0; r < cv->R; ++r) {
        int64_t h = p * cv->stride_h - cv->pad_h + r * cv->dil_h;
        if (h < 0 || h >= cv->H) continue;
        for (int64_t s = 0; s < cv->S; ++s) {
            int64_t w = q * cv->stride_w - cv->pad_w + s * cv->dil_w;
            if (w < 0 || w >= cv->W) continue;
            const int64_t xo = ((n * cv->H + h) * cv->W + w) * cv->C;
            const int64_t wo = ((k * cv->R + r) * cv->S + s) * cv->C;
            for (int64_t c = 0; c < cv->C; ++c) {
                double t = in_to_f64(cv->X, cv->in_dtype, xo + c) * in_to_f64(cv->Wf, cv->in_dtype, wo + c);
                sum += t;
                asum += fabs(t);
            }
        }
    }
    double v = cv->alpha * sum;
    double av = fabs(cv->alpha) * asum;
    if (cv->beta != 0.0) {
        double c = load_as_f64(cv->Cin, cv->c_dtype, ((n * cv->P + p) * cv->Q + q) * cv->K + k);
        v += cv->beta * c;
        av += fabs(cv->beta * c);
    }
    if (cv->bias) {
        double bk = in_to_f64(cv->bias, cv->bias_dtype, k);
        v += bk;
        av += fabs(bk);
    }
    if (absacc) *absacc = av;
    return orc_act2(cv->epi, v, cv->a0, cv->a1);
}

static int conv_setup(conv_problem* cv, const int64_t* d, const void* X, const void* Wf,
                      const void* Cin, int c_dtype, const void* bias, int bias_dtype, double alpha, double beta, int epi,
                      double a0, double a1, int in_dtype) {
    cv->N = d[0]; cv->H = d[1]; cv->W = d[2]; cv->C = d[3]; cv->K = d[4]; cv->R = d[5]; cv->S = d[6];
    cv->pad_h = d[7]; cv->pad_w = d[8]; cv->stride_h = d[9]; cv->stride_w = d[10];
    cv->dil_h = d[11]; cv->dil_w = d[12];
    if (cv->N < 0 || cv->H < 0 || cv->W < 0 || cv->C < 0 || cv->K < 0 || cv->R < 1 || cv->S < 1) return 1;
    if (cv->stride_h < 1 || cv->stride_w < 1 || cv->dil_h < 1 || cv->dil_w < 1 || cv->pad_h < 0 || cv->pad_w < 0) return 1;
    if (beta != 0.0 && !Cin) return 2;
    cv->P = orc_conv_out_extent(cv->H, cv->pad_h, cv->dil_h, cv->R, cv->stride_h);
    cv->Q = orc_conv_out_extent(cv->W, cv->pad_w, cv->dil_w, cv->S, cv->stride_w);
    cv->X = X; cv->Wf = Wf; cv->Cin = Cin; cv->c_dtype = c_dtype; cv->bias = bias; cv->bias_dtype = bias_dtype;
    cv->alpha = alpha; cv->beta = beta; cv->epi = epi; cv->a0 = a0; cv->a1 = a1; cv->in_dtype = in_dtype;
    return 0;
}

/*
 * dims = {N,H,W,C,K,R,S,pad_h,pad_w,stride_h,stride_w,dil_h,dil_w}.
 * Output pixels [pix_begin, pix_end) in flattened (n,p,q) order; ref holds
 * (pix_end-pix_begin) x K values.
 */
int orc_conv2d_fprop(const int64_t* dims, const void* X, const void* Wf,
                     const void* Cin, int c_dtype, const void* bias, int bias_dtype,
                     double alpha, double beta, int epi, double a0, double a1, int in_dtype,
                     int64_t pix_begin, int64_t pix_end, double* ref, double* absacc) {
    conv_problem cv;
    int rc = conv_setup(&cv, dims, X, Wf, Cin, c_dtype, bias, bias_dtype, alpha, beta, epi, a0, a1, in_dtype);
    if (rc) return rc;
    if (pix_begin < 0 || pix_end > cv.N * cv.P * cv.Q || pix_begin > pix_end) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t pix = pix_begin; pix < pix_end; ++pix) {
        int64_t n = pix / (cv.P * cv.Q);
        int64_t p = (pix / cv.Q) % cv.P;
        int64_t q = pix % cv.Q;
        for (int64_t k = 0; k < cv.K; ++k) {
            double av;
            double v = conv_element(&cv, n, p, q, k, &av);
            ref[(pix - pix_begin) * cv.K + k] = v;
            if (absacc) absacc[(pix - pix_begin) * cv.K + k] = av;
        }
    }
    return 0;
}

/* The listed (flattened pixel, output channel) pairs only. */
int orc_conv2d_points(const int64_t* dims, const void* X, const void* Wf,
                      const void* Cin, int c_dtype, const void* bias, int bias_dtype,
                      double alpha, double beta, int epi, double a0, double a1, int in_dtype,
                      int64_t npts, const int64_t* ppix, const int64_t* pk, double* ref, double* absacc) {
    conv_problem cv;
    int rc = conv_setup(&cv, dims, X, Wf, Cin, c_dtype, bias, bias_dtype, alpha, beta, epi, a0, a1, in_dtype);
    if (rc) return rc;
    for (int64_t t = 0; t < npts; ++t)
        if (ppix[t] < 0 || ppix[t] >= cv.N * cv.P * cv.Q || pk[t] < 0 || pk[t] >= cv.K) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < npts; ++t) {
        int64_t pix = ppix[t];
        double av;
        ref[t] = conv_element(&cv, pix / (cv.P * cv.Q), (pix / cv.Q) % cv.P, pix % cv.Q, pk[t], &av);
        if (absacc) absacc[t] = av;
    }
    return 0;
}

/* -------------------------------------------------------------------------------------------
 * conv2d data and weight gradients (the DSL's conv2d_dgrad / conv2d_wgrad operators, Appendix A.1): the two
 * adjoints of the forward map  y[n,p,q,k] = sum_{r,s,c} x[n, p sh - ph + r dh, q sw - pw + s dw, c] w[k,r,s,c].
 *   dgrad:  dx[n,h,w,c]  = alpha * sum over all (p,r), (q,s), k with  p sh - ph + r dh = h  and  q sw - pw + s dw = w
 *                          of dy[n,p,q,k] w[k,r,s,c]                     + beta * Cin[n,h,w,c]
 *   wgrad:  dw[k,r,s,c]  = alpha * sum_{n,p,q} dy[n,p,q,k] x[n, p sh - ph + r dh, q sw - pw + s dw, c]
 *                          (taps outside the image contribute 0)        + beta * Cin[k,r,s,c]
 * dims as for the forward convolution (N,H,W,C describe x / dx; K,R,S the filter); dy is [N,P,Q,K].
 * ----------------------------------------------------------------------------------------- */
int orc_conv2d_dgrad(const int64_t* dims, const void* dY, const void* Wf, const void* Cin, int c_dtype,
                     double alpha, double beta, int in_dtype, int64_t pix_begin, int64_t pix_end,
                     double* ref, double* absacc) {
    conv_problem cv;
    int rc = conv_setup(&cv, dims, NULL, Wf, Cin, c_dtype, NULL, 0, alpha, beta, 0, 0.0, 0.0, in_dtype);
    if (rc) return rc;
    if (pix_begin < 0 || pix_end > cv.N * cv.H * cv.W || pix_begin > pix_end) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t pix = pix_begin; pix < pix_end; ++pix) {
        const int64_t n = pix / (cv.H * cv.W), h = (pix / cv.W) % cv.H, w = pix % cv.W;
        for (int64_t c = 0; c < cv.C; ++c) {
            double sum = 0.0, asum = 0.0;
            for (int64_t p = 0; p < cv.P; ++p)
                for (int64_t r = 0; r < cv.R; ++r) {
                    if (p * cv.stride_h - cv.pad_h + r * cv.dil_h != h) continue;
                    for (int64_t q = 0; q < cv.Q; ++q)
                        for (int64_t s2 = 0; s2 < cv.S; ++s2) {
                            if (q * cv.stride_w - cv.pad_w + s2 * cv.dil_w != w) continue;
                            for (int64_t k = 0; k < cv.K; ++k) {
                                double t = in_to_f64(dY, in_dtype, ((n * cv.P + p) * cv.Q + q) * cv.K + k) *
                                           in_to_f64(Wf, in_dtype, ((k * cv.R + r) * cv.S + s2) * cv.C + c);
                                sum += t;
                                asum += fabs(t);
                            }
                        }
                }
            double v = alpha * sum, av = fabs(alpha) * asum;
            if (beta != 0.0) {
                double cc = load_as_f64(Cin, c_dtype, pix * cv.C + c);
                v += beta * cc;
                av += fabs(beta * cc);
            }
            ref[(pix - pix_begin) * cv.C + c] = v;
            if (absacc) absacc[(pix - pix_begin) * cv.C + c] = av;
        }
    }
    return 0;
}

/* Filters [k_begin, k_end): ref holds (k_end-k_begin) x R x S x C values. */
int orc_conv2d_wgrad(const int64_t* dims, const void* dY, const void* X, const void* Cin, int c_dtype,
                     double alpha, double beta, int in_dtype, int64_t k_begin, int64_t k_end,
                     double* ref, double* absacc) {
    conv_problem cv;
    int rc = conv_setup(&cv, dims, X, NULL, Cin, c_dtype, NULL, 0, alpha, beta, 0, 0.0, 0.0, in_dtype);
    if (rc) return rc;
    if (k_begin < 0 || k_end > cv.K || k_begin > k_end) return 1;
    const int64_t rsc = cv.R * cv.S * cv.C;
#pragma omp parallel for schedule(static)
    for (int64_t e = k_begin * rsc; e < k_end * rsc; ++e) {
        const int64_t k = e / rsc, r = (e / (cv.S * cv.C)) % cv.R, s2 = (e / cv.C) % cv.S, c = e % cv.C;
        double sum = 0.0, asum = 0.0;
        for (int64_t n = 0; n < cv.N; ++n)
            for (int64_t p = 0; p < cv.P; ++p) {
                const int64_t h = p * cv.stride_h - cv.pad_h + r * cv.dil_h;
                if (h < 0 || h >= cv.H) continue;
                for (int64_t q = 0; q < cv.Q; ++q) {
                    const int64_t w = q * cv.stride_w - cv.pad_w + s2 * cv.dil_w;
                    if (w < 0 || w >= cv.W) continue;
                    double t = in_to_f64(dY, in_dtype, ((n * cv.P + p) * cv.Q + q) * cv.K + k) *
                               in_to_f64(X, in_dtype, ((n * cv.H + h) * cv.W + w) * cv.C + c);
                    sum += t;
                    asum += fabs(t);
                }
            }
        double v = alpha * sum, av = fabs(alpha) * asum;
        if (beta != 0.0) {
            double cc = load_as_f64(Cin, c_dtype, e);
            v += beta * cc;
            av += fabs(beta * cc);
        }
        ref[e - k_begin * rsc] = v;
        if (absacc) absacc[e - k_begin * rsc] = av;
    }
    return 0;
}

/* -------------------------------------------------------------------------------------------
 * Layout transpose with dtype conversion (the DSL's transpose(ref, L1, L2[, dt1, dt2]) stage, Appendix A.1):
 *   out[b][c][r] = convert(in[b][r][c]).  bf16 / fp16 -> fp32 is exact; a conversion to bf16 or fp16 rounds the (exactly
 *   widened) value to nearest, ties to even; a NaN stays a NaN.  The result is returned as fp64 holding the converted value.
 * ----------------------------------------------------------------------------------------- */
static double round_f32_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu) != 0) {
        u |= 0x00400000u;                       /* quiet NaN, keep it a NaN after truncation */
    } else {
        uint32_t lower = u & 0xFFFFu, odd = (u >> 16) & 1u;
        if (lower > 0x8000u || (lower == 0x8000u && odd)) u += 0x10000u;   /* may carry into the exponent: correct */
    }
    u &= 0xFFFF0000u;
    float r;
    memcpy(&r, &u, sizeof r);
    return (double)r;
}

/* fp32 -> fp16 (IEEE binary16: 5 exponent bits, 10 fraction bits), round to nearest, ties to even, written out
 * from the definition: values of 65520 and above go to infinity, values below 2^-14 land on the subnormal grid of
 * spacing 2^-24, a NaN stays a NaN.  Every bf16 and every fp32 input is a binary32 value, so this one rounding
 * covers bf16 -> fp16 as well. */
static double round_f32_to_f16(float f) {
    if (f != f) return (double)f;                               /* NaN */
    double x = (double)f, a = fabs(x), sign = (x < 0.0 || (x == 0.0 && 1.0 / x < 0.0)) ? -1.0 : 1.0;
    if (a == 0.0) return x;
    if (a >= 65520.0) return sign * INFINITY;                   /* the midpoint between 65504 and 2^16 rounds up (to even) */
    int e;
    (void)frexp(a, &e);                                         /* a = m 2^e, 0.5 <= m < 1: the leading bit has weight 2^(e-1) */
    int ulp_exp = (e - 1 < -14 ? -14 : e - 1) - 10;             /* spacing of fp16 values around a */
    double q = ldexp(a, -ulp_exp);                              /* a in units of that spacing: below 2^11, exact in fp64 */
    double fl = floor(q), frac = q - fl;
    if (frac > 0.5 || (frac == 0.5 && fmod(fl, 2.0) == 1.0)) fl += 1.0;
    return sign * ldexp(fl, ulp_exp);
}

int orc_transpose(int64_t batch, int64_t rows, int64_t cols, const void* in, int in_dtype, int64_t ld_in,
                  int64_t stride_in, int out_dtype, double* out) {
    if (batch < 0 || rows < 0 || cols < 0) return 1;
    for (int64_t b = 0; b < batch; ++b)
        for (int64_t r = 0; r < rows; ++r)
            for (int64_t c = 0; c < cols; ++c) {
                double v = load_as_f64(in, in_dtype, b * stride_in + r * ld_in + c);
                /* every 16-bit input value is exact in fp32; only a conversion to a narrower significand rounds */
                if (out_dtype == ORC_BF16 && in_dtype != ORC_BF16) v = round_f32_to_bf16((float)v);
                if (out_dtype == ORC_F16 && in_dtype != ORC_F16) v = round_f32_to_f16((float)v);
                out[(b * cols + c) * rows + r] = v;
            }
    return 0;
}

int64_t orc_transpose_bytes(int64_t batch, int64_t rows, int64_t cols, int64_t eb_in, int64_t eb_out) {
    return batch * rows * cols * (eb_in + eb_out);
}

/* -------------------------------------------------------------------------------------------
 * Speed-of-Light bound (Section 4.1; worked example in Appendix A.2).
 *   step 1  FLOPs (2 per multiply-accumulate) and best-case DRAM bytes: every
 *           unique input element read once, every output written once.
 *   step 2  peaks from the specification, scaled linearly by current/max clock.
 *   step 3  T_compute = FLOPs/peak, T_mem = bytes/bandwidth, t_SOL = max of them.
 *   step 4  arithmetic intensity against the ridge point peak/bandwidth.
 * ----------------------------------------------------------------------------------------- */
int64_t orc_gemm_flops(int64_t M, int64_t N, int64_t K) { return 2 * M * N * K; }

/* has_c: C is read (beta != 0); has_bias: a bias vector of N input-type elements is read. */
int64_t orc_gemm_bytes(int64_t M, int64_t N, int64_t K, int64_t eb_in, int64_t eb_out, int has_c, int has_bias) {
    int64_t bytes = (M * K + K * N) * eb_in + M * N * eb_out;
    if (has_c) bytes += M * N * eb_out;
    if (has_bias) bytes += N * eb_in;
    return bytes;
}

int64_t orc_conv_flops(const int64_t* dims) {
    int64_t P = orc_conv_out_extent(dims[1], dims[7], dims[11], dims[5], dims[9]);
    int64_t Q = orc_conv_out_extent(dims[2], dims[8], dims[12], dims[6], dims[10]);
    return 2 * (dims[0] * P * Q) * dims[4] * (dims[3] * dims[5] * dims[6]);
}

int64_t orc_conv_bytes(const int64_t* dims, int64_t eb_in, int64_t eb_out, int has_c, int has_bias) {
    int64_t P = orc_conv_out_extent(dims[1], dims[7], dims[11], dims[5], dims[9]);
    int64_t Q = orc_conv_out_extent(dims[2], dims[8], dims[12], dims[6], dims[10]);
    int64_t x = dims[0] * dims[1] * dims[2] * dims[3];
    int64_t w = dims[4] * dims[5] * dims[6] * dims[3];
    int64_t y = dims[0] * P * Q * dims[4];
    int64_t bytes = (x + w) * eb_in + y * eb_out;
    if (has_c) bytes += y * eb_out;
    if (has_bias) bytes += dims[4] * eb_in;
    return bytes;
}

/* Best-case bytes of the two gradients: which = 0 data gradient (reads dy and w, writes dx),
 * which = 1 weight gradient (reads dy and x, writes dw); has_c adds one read of the written tensor. */
int64_t orc_conv_grad_bytes(const int64_t* dims, int which, int64_t eb_in, int64_t eb_out, int has_c) {
    int64_t P = orc_conv_out_extent(dims[1], dims[7], dims[11], dims[5], dims[9]);
    int64_t Q = orc_conv_out_extent(dims[2], dims[8], dims[12], dims[6], dims[10]);
    int64_t x = dims[0] * dims[1] * dims[2] * dims[3];
    int64_t w = dims[4] * dims[5] * dims[6] * dims[3];
    int64_t y = dims[0] * P * Q * dims[4];
    int64_t rd = which == 0 ? y + w : y + x;
    int64_t wr = which == 0 ? x : w;
    return rd * eb_in + wr * eb_out * (has_c ? 2 : 1);
}

/*
 * hw = {peak_flops, peak_bytes_per_s, sm_clock, sm_clock_max, mem_clock, mem_clock_max}
 *      (a zero clock or zero max clock means "do not scale": ratio 1).
 * out = {ai, t_compute_s, t_mem_s, t_sol_s, ridge, eff_peak_flops, eff_bytes_per_s, compute_bound}
 */
int orc_sol_bound(int64_t flops, int64_t bytes, const double* hw, double* out) {
    if (flops < 0 || bytes < 0 || hw[0] <= 0.0 || hw[1] <= 0.0) return 1;
    double sm_ratio = (hw[2] > 0.0 && hw[3] > 0.0) ? hw[2] / hw[3] : 1.0;
    double mem_ratio = (hw[4] > 0.0 && hw[5] > 0.0) ? hw[4] / hw[5] : 1.0;
    double eff_peak = hw[0] * sm_ratio;
    double eff_bw = hw[1] * mem_ratio;
    double t_c = (double)flops / eff_peak;
    double t_m = (double)bytes / eff_bw;
    double ai = bytes > 0 ? (double)flops / (double)bytes : INFINITY;
    double ridge = eff_peak / eff_bw;
    out[0] = ai;
    out[1] = t_c;
    out[2] = t_m;
    out[3] = t_c > t_m ? t_c : t_m;
    out[4] = ridge;
    out[5] = eff_peak;
    out[6] = eff_bw;
    out[7] = ai > ridge ? 1.0 : 0.0;
    return 0;
}
