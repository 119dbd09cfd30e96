"""ctypes front end of the CPU oracle (``sg_oracle.c``).

TEST INFRASTRUCTURE, NOT PART OF THE PRODUCT.  Only the tests, the smoke check and
the benchmark's cpu-baseline / reference arm import this module.  It never
imports the CUDA package and the CUDA package never imports it.

Tensors are plain CPU torch tensors; torch is used here only as a typed buffer
(bf16 has no numpy dtype).  Operand conventions, shared with the C file:

* ``A`` is passed as it is stored: ``[M, K]`` for row-major, ``[K, M]`` for
  column-major; ``B`` is ``[K, N]`` for row-major, ``[N, K]`` for column-major.
  The inner stride must be 1, the outer stride is the leading dimension.
* ``C`` (read only when ``beta != 0``) and the result are row-major ``[M, N]``.
* ``bias`` holds one bf16 value per output column (GEMM) / output channel (conv).

Every function returns ``(ref, absacc)`` as fp64 tensors: the unrounded result
and ``|alpha| sum|a||b| + |beta c| + |bias|``, the scale of the fp32 tolerance.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sg_oracle.c")
_LIB = os.path.join(_HERE, "libsg_oracle.so")

LAYOUTS = {"row": 0, "col": 1}
EPILOGUES = {"none": 0, "bias": 1, "relu": 2, "gelu": 3, "silu": 4, "sigmoid": 5, "tanh": 6, "mish": 7,
             "hardswish": 8, "leaky_relu": 9, "elu": 10, "clip": 11}
_DTYPES = {torch.bfloat16: 0, torch.float32: 1, torch.float16: 2, torch.float8_e4m3fn: 3, torch.float8_e5m2: 4}
_IN_DTYPES = (torch.bfloat16, torch.float16, torch.float8_e4m3fn, torch.float8_e5m2, torch.float32, torch.int8)
_FP8 = (torch.float8_e4m3fn, torch.float8_e5m2)


def bias_dtype_for(in_dtype: torch.dtype) -> torch.dtype:
    """The bias has the inputs' type, except that 8-bit inputs (fp8, int8) come with a bf16 bias."""
    return torch.bfloat16 if in_dtype in _FP8 or in_dtype == torch.int8 else in_dtype


def _in_code(dtype: torch.dtype) -> int:
    """Type code of A / B (X / Wf): fp32 operands are read as tf32 (their low 13 fraction bits do not take part)."""
    if dtype == torch.int8:
        return 6
    return 5 if dtype == torch.float32 else _DTYPES[dtype]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over output rows only). Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c99", _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i64, dbl, vp, ci = ctypes.c_int64, ctypes.c_double, ctypes.c_void_p, ctypes.c_int
        L.orc_num_threads.restype = ci
        L.orc_act.restype = dbl
        L.orc_act.argtypes = [ci, dbl]
        L.orc_act2.restype = dbl
        L.orc_act2.argtypes = [ci, dbl, dbl, dbl]
        L.orc_act_array.restype = None
        L.orc_act_array.argtypes = [ci, dbl, dbl, i64, vp, vp]
        L.orc_gemm.restype = ci
        L.orc_gemm.argtypes = [i64, i64, i64, ci, ci, vp, i64, vp, i64, vp, ci, i64, vp, ci, dbl, dbl, ci, dbl, dbl, ci,
                               i64, i64, vp, vp, i64]
        L.orc_gemm_points.restype = ci
        L.orc_gemm_points.argtypes = [i64, i64, i64, ci, ci, vp, i64, vp, i64, vp, ci, i64, vp, ci, dbl, dbl, ci, dbl, dbl, ci,
                                      i64, vp, vp, vp, vp]
        L.orc_conv_out_extent.restype = i64
        L.orc_conv_out_extent.argtypes = [i64] * 5
        L.orc_conv2d_fprop.restype = ci
        L.orc_conv2d_fprop.argtypes = [vp, vp, vp, vp, ci, vp, ci, dbl, dbl, ci, dbl, dbl, ci, i64, i64, vp, vp]
        L.orc_conv2d_dgrad.restype = ci
        L.orc_conv2d_dgrad.argtypes = [vp, vp, vp, vp, ci, dbl, dbl, ci, i64, i64, vp, vp]
        L.orc_conv2d_wgrad.restype = ci
        L.orc_conv2d_wgrad.argtypes = [vp, vp, vp, vp, ci, dbl, dbl, ci, i64, i64, vp, vp]
        L.orc_conv2d_points.restype = ci
        L.orc_conv2d_points.argtypes = [vp, vp, vp, vp, ci, vp, ci, dbl, dbl, ci, dbl, dbl, ci, i64, vp, vp, vp, vp]
        L.orc_transpose.restype = ci
        L.orc_transpose.argtypes = [i64, i64, i64, vp, ci, i64, i64, ci, vp]
        L.orc_transpose_bytes.restype = i64
        L.orc_transpose_bytes.argtypes = [i64] * 5
        L.orc_gemm_flops.restype = i64
        L.orc_gemm_flops.argtypes = [i64, i64, i64]
        L.orc_gemm_bytes.restype = i64
        L.orc_gemm_bytes.argtypes = [i64, i64, i64, i64, i64, ci, ci]
        L.orc_conv_flops.restype = i64
        L.orc_conv_flops.argtypes = [vp]
        L.orc_conv_bytes.restype = i64
        L.orc_conv_bytes.argtypes = [vp, i64, i64, ci, ci]
        L.orc_conv_grad_bytes.restype = i64
        L.orc_conv_grad_bytes.argtypes = [vp, ci, i64, i64, ci]
        L.orc_sol_bound.restype = ci
        L.orc_sol_bound.argtypes = [i64, i64, vp, vp]
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def act(epi: str, x: float, args=(0.0, 0.0)) -> float:
    return float(lib().orc_act2(EPILOGUES[epi], float(x), float(args[0]), float(args[1])))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _check2d(t: torch.Tensor, name: str):
    if t.device.type != "cpu" or t.dim() != 2 or t.dtype not in _IN_DTYPES:
        raise ValueError(f"{name}: want a 2-D CPU bf16, fp16 or fp8 tensor")
    if t.shape[1] > 1 and t.stride(1) != 1:
        raise ValueError(f"{name}: inner stride must be 1")


def _gemm_shapes(A, B, layout_a, layout_b):
    _check2d(A, "A")
    _check2d(B, "B")
    if A.dtype != B.dtype:
        raise ValueError("A and B must have the same dtype")
    M, K = (A.shape if layout_a == "row" else (A.shape[1], A.shape[0]))
    Kb, N = (B.shape if layout_b == "row" else (B.shape[1], B.shape[0]))
    if K != Kb:
        raise ValueError("A and B disagree on K")
    lda = A.stride(0) if A.shape[0] > 1 else max(A.shape[1], 1)
    ldb = B.stride(0) if B.shape[0] > 1 else max(B.shape[1], 1)
    return M, N, K, lda, ldb


def _c_args(C, M, N):
    if C is None:
        return None, 0, max(N, 1)
    if C.device.type != "cpu" or C.dim() != 2 or tuple(C.shape) != (M, N) or C.dtype not in _DTYPES:
        raise ValueError("C: want a CPU [M, N] bf16, fp16 or fp32 tensor")
    if N > 1 and C.stride(1) != 1:
        raise ValueError("C: inner stride must be 1")
    return C, _DTYPES[C.dtype], (C.stride(0) if M > 1 else max(N, 1))


def _check_bias(bias, n, dtype=torch.bfloat16):
    if bias is not None and (bias.device.type != "cpu" or bias.dtype != dtype or bias.numel() != n
                             or not bias.is_contiguous()):
        raise ValueError("bias: want a contiguous CPU vector of the inputs' dtype with one value per output column")


def gemm(A: torch.Tensor, B: torch.Tensor, *, layout_a: str = "row", layout_b: str = "col",
         C: Optional[torch.Tensor] = None, bias: Optional[torch.Tensor] = None,
         alpha: float = 1.0, beta: float = 0.0, epi: str = "none", epi_args=(0.0, 0.0),
         rows: Optional[Tuple[int, int]] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """act(alpha A.B + beta C + bias) for rows ``rows=(begin, end)`` (default: all)."""
    M, N, K, lda, ldb = _gemm_shapes(A, B, layout_a, layout_b)
    _check_bias(bias, N, bias_dtype_for(A.dtype))
    C, c_dtype, ldc = _c_args(C, M, N)
    r0, r1 = rows if rows is not None else (0, M)
    ref = torch.empty((r1 - r0, N), dtype=torch.float64)
    absacc = torch.empty_like(ref)
    rc = lib().orc_gemm(M, N, K, LAYOUTS[layout_a], LAYOUTS[layout_b], _ptr(A), lda, _ptr(B), ldb,
                        _ptr(C), c_dtype, ldc, _ptr(bias), _DTYPES[bias_dtype_for(A.dtype)], float(alpha), float(beta),
                        EPILOGUES[epi], float(epi_args[0]), float(epi_args[1]), _in_code(A.dtype), r0, r1, _ptr(ref), _ptr(absacc),
                        max(N, 1))
    if rc:
        raise ValueError(f"orc_gemm rejected its arguments (code {rc})")
    return ref, absacc


def gemm_points(A, B, pi: Sequence[int], pj: Sequence[int], *, layout_a="row", layout_b="col", C=None, bias=None,
                alpha=1.0, beta=0.0, epi="none", epi_args=(0.0, 0.0)) -> Tuple[torch.Tensor, torch.Tensor]:
    """The elements (pi[t], pj[t]) of the result only."""
    M, N, K, lda, ldb = _gemm_shapes(A, B, layout_a, layout_b)
    _check_bias(bias, N, bias_dtype_for(A.dtype))
    C, c_dtype, ldc = _c_args(C, M, N)
    pi = torch.as_tensor(pi, dtype=torch.int64).contiguous()
    pj = torch.as_tensor(pj, dtype=torch.int64).contiguous()
    ref = torch.empty(pi.numel(), dtype=torch.float64)
    absacc = torch.empty_like(ref)
    rc = lib().orc_gemm_points(M, N, K, LAYOUTS[layout_a], LAYOUTS[layout_b], _ptr(A), lda, _ptr(B), ldb,
                               _ptr(C), c_dtype, ldc, _ptr(bias), _DTYPES[bias_dtype_for(A.dtype)], float(alpha),
                               float(beta), EPILOGUES[epi], float(epi_args[0]), float(epi_args[1]), _in_code(A.dtype), pi.numel(), _ptr(pi), _ptr(pj),
                               _ptr(ref), _ptr(absacc))
    if rc:
        raise ValueError(f"orc_gemm_points rejected its arguments (code {rc})")
    return ref, absacc


def batched_gemm(A: torch.Tensor, B: torch.Tensor, *, layout_a="row", layout_b="col", C=None, bias=None,
                 alpha=1.0, beta=0.0, epi="none", epi_args=(0.0, 0.0)):
    """The same product for every leading index b; ``bias`` is ``[N]`` (shared) or ``[batch, N]``."""
    refs, accs = [], []
    for b in range(A.shape[0]):
        bb = None if bias is None else (bias if bias.dim() == 1 else bias[b])
        r, a = gemm(A[b], B[b], layout_a=layout_a, layout_b=layout_b, C=None if C is None else C[b],
                    bias=bb, alpha=alpha, beta=beta, epi=epi, epi_args=epi_args)
        refs.append(r)
        accs.append(a)
    return torch.stack(refs), torch.stack(accs)


def grouped_gemm(As, Bs, *, layout_a="row", layout_b="col", Cs=None, biases=None, alpha=1.0, beta=0.0, epi="none",
                 epi_args=(0.0, 0.0)):
    """One independent product per group g with its own (M_g, A_g, B_g, C_g, bias_g)."""
    out = []
    for g in range(len(As)):
        out.append(gemm(As[g], Bs[g], layout_a=layout_a, layout_b=layout_b,
                        C=None if Cs is None else Cs[g], bias=None if biases is None else biases[g],
                        alpha=alpha, beta=beta, epi=epi, epi_args=epi_args))
    return [o[0] for o in out], [o[1] for o in out]


def act_array(epi: str, x: torch.Tensor, args=(0.0, 0.0)) -> torch.Tensor:
    """The activation applied to every element of an fp64 tensor."""
    x = x.to(torch.float64).contiguous()
    out = torch.empty_like(x)
    lib().orc_act_array(EPILOGUES[epi], float(args[0]), float(args[1]), x.numel(), _ptr(x), _ptr(out))
    return out


def epilogue_chain(acc: torch.Tensor, absacc: torch.Tensor, *, alpha=1.0, beta=0.0, C=None, bias=None, epi="none",
                   epi_args=(0.0, 0.0), row_scale=None, col_scale=None, row_bias=None, post_scale=1.0, aux_load=None):
    """The extended epilogue chain (Table 1c built-ins per_row_scale, per_col_scale / per_channel_scale,
    column_broadcast, scale, aux_store, aux_load) on a matrix of plain dot products, in the order the library fixes:

        t   = alpha acc[i,j] row_scale[i] col_scale[j] + beta C[i,j] + bias[j] + row_bias[i]
        aux = t                                   (what aux_store receives)
        D   = post_scale act(t) + aux_load[i,j]

    ``acc`` / ``absacc`` are sum a b and sum |a b| as fp64 [M, N]; every other tensor is widened to fp64 exactly.
    Returns (D, aux, absacc_D, absacc_aux): the last two are the sums of the magnitudes of all terms that enter D
    and aux (the scale of the fp32 tolerance)."""
    f = lambda x: None if x is None else x.to(torch.float64)
    M, N = acc.shape
    t = float(alpha) * acc.to(torch.float64)
    mag = abs(float(alpha)) * absacc.to(torch.float64)
    if row_scale is not None:
        t = t * f(row_scale).reshape(M, 1)
        mag = mag * f(row_scale).abs().reshape(M, 1)
    if col_scale is not None:
        t = t * f(col_scale).reshape(1, N)
        mag = mag * f(col_scale).abs().reshape(1, N)
    if beta != 0.0:
        t = t + float(beta) * f(C).reshape(M, N)
        mag = mag + (float(beta) * f(C).reshape(M, N)).abs()
    if bias is not None:
        t = t + f(bias).reshape(1, N)
        mag = mag + f(bias).abs().reshape(1, N)
    if row_bias is not None:
        t = t + f(row_bias).reshape(M, 1)
        mag = mag + f(row_bias).abs().reshape(M, 1)
    aux = t.clone()
    d = float(post_scale) * act_array(epi, t, epi_args)
    # the activations are 1-Lipschitz up to a small factor, so the magnitudes carry through scaled by post_scale
    mag_d = abs(float(post_scale)) * mag
    if aux_load is not None:
        d = d + f(aux_load).reshape(M, N)
        mag_d = mag_d + f(aux_load).abs().reshape(M, N)
    return d, aux, mag_d, mag


def gemm_ex(A, B, *, layout_a="row", layout_b="col", **chain):
    """``epilogue_chain`` on the plain products of ``gemm`` (alpha = 1, no C, bias or activation there)."""
    acc, absacc = gemm(A, B, layout_a=layout_a, layout_b=layout_b)
    return epilogue_chain(acc, absacc, **chain)


def conv2d_fprop_ex(X, Wf, *, pad=(0, 0), stride=(1, 1), dil=(1, 1), **chain):
    """``epilogue_chain`` on the plain sums of ``conv2d_fprop``, rows = output pixels (n, p, q), columns = channels."""
    acc, absacc = conv2d_fprop(X, Wf, pad=pad, stride=stride, dil=dil)
    K = acc.shape[-1]
    return epilogue_chain(acc.reshape(-1, K), absacc.reshape(-1, K), **chain)


def conv_out_extent(size: int, pad: int, dil: int, filt: int, stride: int) -> int:
    return int(lib().orc_conv_out_extent(size, pad, dil, filt, stride))


def _conv_dims(X, Wf, pad, stride, dil):
    if X.device.type != "cpu" or X.dim() != 4 or X.dtype not in _IN_DTYPES or not X.is_contiguous():
        raise ValueError("X: want a contiguous CPU bf16, fp16 or fp8 NHWC tensor")
    if Wf.device.type != "cpu" or Wf.dim() != 4 or Wf.dtype != X.dtype or not Wf.is_contiguous():
        raise ValueError("Wf: want a contiguous CPU KRSC tensor of X's dtype")
    N, H, W, C = X.shape
    K, R, S, Cw = Wf.shape
    if C != Cw:
        raise ValueError("X and Wf disagree on C")
    d = torch.tensor([N, H, W, C, K, R, S, pad[0], pad[1], stride[0], stride[1], dil[0], dil[1]], dtype=torch.int64)
    P = conv_out_extent(H, pad[0], dil[0], R, stride[0])
    Q = conv_out_extent(W, pad[1], dil[1], S, stride[1])
    return d, N, P, Q, K


def _conv_c(Cin, N, P, Q, K):
    if Cin is None:
        return None, 0
    if Cin.device.type != "cpu" or tuple(Cin.shape) != (N, P, Q, K) or Cin.dtype not in _DTYPES \
            or not Cin.is_contiguous():
        raise ValueError("Cin: want a contiguous CPU [N,P,Q,K] bf16 or fp32 tensor")
    return Cin, _DTYPES[Cin.dtype]


def conv2d_fprop(X: torch.Tensor, Wf: torch.Tensor, *, pad=(0, 0), stride=(1, 1), dil=(1, 1),
                 Cin=None, bias=None, alpha=1.0, beta=0.0, epi="none", epi_args=(0.0, 0.0),
                 pixels: Optional[Tuple[int, int]] = None):
    """Direct convolution; returns ``[N,P,Q,K]`` tensors, or ``[pixels, K]`` for a flattened pixel range."""
    d, N, P, Q, K = _conv_dims(X, Wf, pad, stride, dil)
    _check_bias(bias, K, bias_dtype_for(X.dtype))
    Cin, c_dtype = _conv_c(Cin, N, P, Q, K)
    p0, p1 = pixels if pixels is not None else (0, N * P * Q)
    ref = torch.empty((p1 - p0, K), dtype=torch.float64)
    absacc = torch.empty_like(ref)
    rc = lib().orc_conv2d_fprop(_ptr(d), _ptr(X), _ptr(Wf), _ptr(Cin), c_dtype, _ptr(bias), _DTYPES[bias_dtype_for(X.dtype)],
                                float(alpha), float(beta), EPILOGUES[epi], float(epi_args[0]), float(epi_args[1]),
                                _in_code(X.dtype), p0, p1, _ptr(ref), _ptr(absacc))
    if rc:
        raise ValueError(f"orc_conv2d_fprop rejected its arguments (code {rc})")
    if pixels is None:
        return ref.view(N, P, Q, K), absacc.view(N, P, Q, K)
    return ref, absacc


def _grad_dims(N, H, W, C, K, R, S, pad, stride, dil):
    d = torch.tensor([N, H, W, C, K, R, S, pad[0], pad[1], stride[0], stride[1], dil[0], dil[1]], dtype=torch.int64)
    P = conv_out_extent(H, pad[0], dil[0], R, stride[0])
    Q = conv_out_extent(W, pad[1], dil[1], S, stride[1])
    return d, P, Q


def _check_grad_operand(t, shape, name, dtype=None):
    if t.device.type != "cpu" or tuple(t.shape) != tuple(shape) or not t.is_contiguous() \
            or (dtype is not None and t.dtype != dtype) or (dtype is None and t.dtype not in (torch.bfloat16, torch.float16)):
        raise ValueError(f"{name}: want a contiguous CPU tensor of shape {tuple(shape)} (bf16 or fp16)")


def conv2d_dgrad(dY: torch.Tensor, Wf: torch.Tensor, hw: Tuple[int, int], *, pad=(0, 0), stride=(1, 1), dil=(1, 1),
                 Cin=None, alpha=1.0, beta=0.0, pixels: Optional[Tuple[int, int]] = None):
    """Gradient of the forward convolution with respect to its input: ``dY`` [N,P,Q,K], ``Wf`` [K,R,S,C] ->
    [N,H,W,C] with ``hw = (H, W)`` (or ``[pixels, C]`` for a flattened range of (n,h,w))."""
    K, R, S, C = Wf.shape
    N = dY.shape[0]
    H, W = hw
    d, P, Q = _grad_dims(N, H, W, C, K, R, S, pad, stride, dil)
    _check_grad_operand(dY, (N, P, Q, K), "dY")
    _check_grad_operand(Wf, (K, R, S, C), "Wf", dY.dtype)
    Cin, c_dtype = _conv_c(Cin, N, H, W, C)
    p0, p1 = pixels if pixels is not None else (0, N * H * W)
    ref = torch.empty((p1 - p0, C), dtype=torch.float64)
    absacc = torch.empty_like(ref)
    rc = lib().orc_conv2d_dgrad(_ptr(d), _ptr(dY), _ptr(Wf), _ptr(Cin), c_dtype, float(alpha), float(beta),
                                _DTYPES[dY.dtype], p0, p1, _ptr(ref), _ptr(absacc))
    if rc:
        raise ValueError(f"orc_conv2d_dgrad rejected its arguments (code {rc})")
    if pixels is None:
        return ref.view(N, H, W, C), absacc.view(N, H, W, C)
    return ref, absacc


def conv2d_wgrad(dY: torch.Tensor, X: torch.Tensor, rs: Tuple[int, int], *, pad=(0, 0), stride=(1, 1), dil=(1, 1),
                 Cin=None, alpha=1.0, beta=0.0, filters: Optional[Tuple[int, int]] = None):
    """Gradient with respect to the filter: ``dY`` [N,P,Q,K], ``X`` [N,H,W,C] -> [K,R,S,C] with ``rs = (R, S)``
    (or filters ``[k0, k1)`` only)."""
    N, H, W, C = X.shape
    K = dY.shape[3]
    R, S = rs
    d, P, Q = _grad_dims(N, H, W, C, K, R, S, pad, stride, dil)
    _check_grad_operand(dY, (N, P, Q, K), "dY")
    _check_grad_operand(X, (N, H, W, C), "X", dY.dtype)
    Cin, c_dtype = _conv_c(Cin, K, R, S, C)
    k0, k1 = filters if filters is not None else (0, K)
    ref = torch.empty((k1 - k0, R, S, C), dtype=torch.float64)
    absacc = torch.empty_like(ref)
    rc = lib().orc_conv2d_wgrad(_ptr(d), _ptr(dY), _ptr(X), _ptr(Cin), c_dtype, float(alpha), float(beta),
                                _DTYPES[dY.dtype], k0, k1, _ptr(ref), _ptr(absacc))
    if rc:
        raise ValueError(f"orc_conv2d_wgrad rejected its arguments (code {rc})")
    return ref, absacc


def conv2d_points(X, Wf, ppix: Sequence[int], pk: Sequence[int], *, pad=(0, 0), stride=(1, 1), dil=(1, 1),
                  Cin=None, bias=None, alpha=1.0, beta=0.0, epi="none", epi_args=(0.0, 0.0)):
    """The outputs (flattened pixel ppix[t], channel pk[t]) only."""
    d, N, P, Q, K = _conv_dims(X, Wf, pad, stride, dil)
    _check_bias(bias, K, bias_dtype_for(X.dtype))
    Cin, c_dtype = _conv_c(Cin, N, P, Q, K)
    ppix = torch.as_tensor(ppix, dtype=torch.int64).contiguous()
    pk = torch.as_tensor(pk, dtype=torch.int64).contiguous()
    ref = torch.empty(ppix.numel(), dtype=torch.float64)
    absacc = torch.empty_like(ref)
    rc = lib().orc_conv2d_points(_ptr(d), _ptr(X), _ptr(Wf), _ptr(Cin), c_dtype, _ptr(bias),
                                 _DTYPES[bias_dtype_for(X.dtype)], float(alpha), float(beta), EPILOGUES[epi], float(epi_args[0]), float(epi_args[1]),
                                 _in_code(X.dtype), ppix.numel(), _ptr(ppix), _ptr(pk), _ptr(ref), _ptr(absacc))
    if rc:
        raise ValueError(f"orc_conv2d_points rejected its arguments (code {rc})")
    return ref, absacc


def transpose(x: torch.Tensor, out_dtype: torch.dtype) -> torch.Tensor:
    """out[b, c, r] = convert(x[b, r, c]) as fp64 values of the converted result; x is [batch, rows, cols]."""
    if x.device.type != "cpu" or x.dim() != 3 or x.dtype not in _DTYPES or (x.shape[2] > 1 and x.stride(2) != 1):
        raise ValueError("x: want a CPU [batch, rows, cols] bf16, fp16 or fp32 tensor with inner stride 1")
    batch, rows, cols = x.shape
    out = torch.empty((batch, cols, rows), dtype=torch.float64)
    rc = lib().orc_transpose(batch, rows, cols, _ptr(x), _DTYPES[x.dtype], x.stride(1) if rows > 1 else max(cols, 1),
                             x.stride(0), _DTYPES[out_dtype], _ptr(out))
    if rc:
        raise ValueError(f"orc_transpose rejected its arguments (code {rc})")
    return out


def transpose_bytes(batch: int, rows: int, cols: int, eb_in: int, eb_out: int) -> int:
    return int(lib().orc_transpose_bytes(batch, rows, cols, eb_in, eb_out))


# ---- Speed-of-Light bound -------------------------------------------------------------------

def gemm_flops(M: int, N: int, K: int) -> int:
    return int(lib().orc_gemm_flops(M, N, K))


def gemm_bytes(M: int, N: int, K: int, eb_in: int = 2, eb_out: int = 2, has_c: bool = False,
               has_bias: bool = False) -> int:
    return int(lib().orc_gemm_bytes(M, N, K, eb_in, eb_out, int(has_c), int(has_bias)))


def _dims13(N, H, W, C, K, R, S, pad, stride, dil):
    return torch.tensor([N, H, W, C, K, R, S, pad[0], pad[1], stride[0], stride[1], dil[0], dil[1]],
                        dtype=torch.int64)


def conv_flops(N, H, W, C, K, R, S, pad=(0, 0), stride=(1, 1), dil=(1, 1)) -> int:
    d = _dims13(N, H, W, C, K, R, S, pad, stride, dil)       # keep the buffer alive across the call
    return int(lib().orc_conv_flops(_ptr(d)))


def conv_bytes(N, H, W, C, K, R, S, pad=(0, 0), stride=(1, 1), dil=(1, 1), eb_in=2, eb_out=2,
               has_c=False, has_bias=False) -> int:
    d = _dims13(N, H, W, C, K, R, S, pad, stride, dil)
    return int(lib().orc_conv_bytes(_ptr(d), eb_in, eb_out, int(has_c), int(has_bias)))


def conv_grad_bytes(which: str, N, H, W, C, K, R, S, pad=(0, 0), stride=(1, 1), dil=(1, 1), eb_in=2, eb_out=2,
                    has_c: bool = False) -> int:
    """Best-case bytes of ``which`` = "dgrad" (dY + Wf read, dX written) or "wgrad" (dY + X read, dW written)."""
    d = _dims13(N, H, W, C, K, R, S, pad, stride, dil)
    return int(lib().orc_conv_grad_bytes(_ptr(d), {"dgrad": 0, "wgrad": 1}[which], eb_in, eb_out, int(has_c)))


def sol_bound(flops: int, bytes_: int, peak_flops: float, peak_bytes_per_s: float,
              sm_clock: float = 0.0, sm_clock_max: float = 0.0,
              mem_clock: float = 0.0, mem_clock_max: float = 0.0) -> dict:
    hw = torch.tensor([peak_flops, peak_bytes_per_s, sm_clock, sm_clock_max, mem_clock, mem_clock_max],
                      dtype=torch.float64)
    out = torch.zeros(8, dtype=torch.float64)
    rc = lib().orc_sol_bound(int(flops), int(bytes_), _ptr(hw), _ptr(out))
    if rc:
        raise ValueError(f"orc_sol_bound rejected its arguments (code {rc})")
    keys = ["ai", "t_compute_s", "t_mem_s", "t_sol_s", "ridge", "eff_peak_flops", "eff_bytes_per_s"]
    res = {k: float(out[i]) for i, k in enumerate(keys)}
    res.update(flops=int(flops), bytes=int(bytes_), compute_bound=bool(out[7] != 0.0))
    return res
