"""Thin ctypes binding of libsolgemm (``include/solgemm.h``): argument marshalling only.

Every function takes CUDA torch tensors (torch supplies device memory and the
stream, nothing else), fills the C descriptor, and calls the entry point of the
same name.  There is no CPU path and no fallback: importing this module raises
if ``libsolgemm.so`` has not been built, and every call raises ``SolgemmError``
on a non-OK status.

Operand conventions (the library's): ``A`` is passed as stored, ``[M, K]`` for
row-major / ``[K, M]`` for column-major; ``B`` is ``[K, N]`` row-major /
``[N, K]`` column-major; inner stride 1, outer stride = leading dimension.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import torch

from .build import LIB_PATH

_LIB_FILE = os.environ.get("SOLGEMM_LIB", LIB_PATH)     # an experimental build may be selected explicitly
if not os.path.exists(_LIB_FILE):
    raise ImportError(f"{_LIB_FILE} is missing: build it with `python -m paper_2603_29010_b200.build` "
                      "(there is no CPU fallback)")
_lib = ctypes.CDLL(_LIB_FILE)

SG_OK = 0
STATUS_NAMES = ["SG_OK", "SG_ERR_INVALID_ARG", "SG_ERR_NULL_POINTER", "SG_ERR_ALIGNMENT", "SG_ERR_UNSUPPORTED",
                "SG_ERR_ARCH", "SG_ERR_WORKSPACE", "SG_ERR_CUDA", "SG_ERR_TIMEOUT"]
LAYOUTS = {"row": 0, "col": 1}
EPILOGUES = {"none": 0, "bias": 1, "relu": 2, "gelu": 3, "silu": 4, "sigmoid": 5, "tanh": 6, "mish": 7,
             "hardswish": 8, "leaky_relu": 9, "elu": 10, "clip": 11}
DTYPES = {torch.bfloat16: 0, torch.float32: 1, torch.float16: 2, torch.float8_e4m3fn: 3, torch.float8_e5m2: 4, torch.int8: 5}
OPS = {"gemm": 0, "batched": 1, "grouped": 2, "conv2d": 3, "transpose": 4, "conv2d_dgrad": 5, "conv2d_wgrad": 6}
EXPORTED = ["sg_gemm", "sg_batched_gemm", "sg_grouped_gemm_workspace_size", "sg_grouped_gemm",
            "sg_grouped_gemm_static", "sg_conv2d_fprop", "sg_gemm_ex", "sg_conv2d_fprop_ex",
            "sg_conv2d_dgrad", "sg_conv2d_wgrad",
            "sg_sol_bound", "sg_status_string", "sg_last_error", "sg_poll_status", "sg_set_tuning", "sg_launch_count",
            "sg_last_launch_plan", "sg_set_scratch", "sg_set_tail_mode",
            "sg_last_kernel_clock", "sg_transpose", "sg_set_option", "sg_test_set_status_word",
            "sg_last_kernel_name", "sg_gemm_host", "sg_gemm_host_staging_size"]
OPTIONS = {"epi_warps": 0, "tail_split": 1, "tail_ksplit": 2, "band_m": 3, "general_kernel": 4, "no_pdl": 5, "no_short_a": 6,
           "no_gemv": 7, "gemv_no_mma": 8, "gemv_no_wide": 9, "gemv_rows": 10, "wait_limit_ns": 11, "l2_warm_kblocks": 12, "transpose_plain": 13, "early_donors": 14,
           "two_pass_split_k": 15, "split_k_reduce_warps": 16,
           "gemv_max_vectors": 17, "gemv_small_log2": 18, "gemv_vector_blocks": 19}


class SolgemmError(RuntimeError):
    def __init__(self, status: int, detail: str):
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{name}: {detail}")
        self.status = status
        self.status_name = name


class GemmDesc(ctypes.Structure):
    _fields_ = [("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                ("layout_a", ctypes.c_int32), ("layout_b", ctypes.c_int32),
                ("lda", ctypes.c_int64), ("ldb", ctypes.c_int64), ("ldc", ctypes.c_int64), ("ldd", ctypes.c_int64),
                ("in_dtype", ctypes.c_int32), ("out_dtype", ctypes.c_int32),
                ("alpha", ctypes.c_float), ("beta", ctypes.c_float),
                ("epi", ctypes.c_int32), ("epi_arg0", ctypes.c_float), ("epi_arg1", ctypes.c_float),
                ("reserved", ctypes.c_int32)]


class Conv2dDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in ("N", "H", "W", "C", "K", "R", "S")] + \
               [(n, ctypes.c_int32) for n in ("pad_h", "pad_w", "stride_h", "stride_w", "dil_h", "dil_w",
                                              "in_dtype", "out_dtype")] + \
               [("alpha", ctypes.c_float), ("beta", ctypes.c_float), ("epi", ctypes.c_int32),
                ("epi_arg0", ctypes.c_float), ("epi_arg1", ctypes.c_float), ("reserved", ctypes.c_int32)]


class EpilogueEx(ctypes.Structure):
    _fields_ = [("row_scale", ctypes.c_void_p), ("col_scale", ctypes.c_void_p), ("row_bias", ctypes.c_void_p),
                ("post_scale", ctypes.c_float), ("reserved0", ctypes.c_int32),
                ("aux_load", ctypes.c_void_p), ("ld_aux_load", ctypes.c_int64),
                ("aux_store", ctypes.c_void_p), ("ld_aux_store", ctypes.c_int64)]


class TransposeDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in ("batch", "rows", "cols", "ld_in", "ld_out", "stride_in", "stride_out")] + \
               [(n, ctypes.c_int32) for n in ("in_dtype", "out_dtype", "reserved", "reserved2")]


class Hw(ctypes.Structure):
    _fields_ = [(n, ctypes.c_double) for n in ("peak_flops", "peak_bytes_per_s", "sm_clock_mhz", "sm_clock_max_mhz",
                                               "mem_clock_mhz", "mem_clock_max_mhz")]


class Sol(ctypes.Structure):
    _fields_ = [("flops", ctypes.c_int64), ("bytes", ctypes.c_int64)] + \
               [(n, ctypes.c_double) for n in ("ai", "t_compute_s", "t_mem_s", "t_sol_s", "ridge", "eff_peak_flops",
                                               "eff_bytes_per_s")] + \
               [("compute_bound", ctypes.c_int32), ("reserved", ctypes.c_int32)]


_vp, _i64, _i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32
_lib.sg_gemm.restype = ctypes.c_int
_lib.sg_gemm.argtypes = [ctypes.POINTER(GemmDesc), _vp, _vp, _vp, _vp, _vp, _vp]
_lib.sg_gemm_ex.restype = ctypes.c_int
_lib.sg_gemm_ex.argtypes = [ctypes.POINTER(GemmDesc), ctypes.POINTER(EpilogueEx), _vp, _vp, _vp, _vp, _vp, _vp]
_lib.sg_conv2d_fprop_ex.restype = ctypes.c_int
_lib.sg_conv2d_fprop_ex.argtypes = [ctypes.POINTER(Conv2dDesc), ctypes.POINTER(EpilogueEx), _vp, _vp, _vp, _vp, _vp, _vp]
_lib.sg_conv2d_dgrad.restype = ctypes.c_int
_lib.sg_conv2d_dgrad.argtypes = [ctypes.POINTER(Conv2dDesc), _vp, _vp, _vp, _vp, _vp]
_lib.sg_conv2d_wgrad.restype = ctypes.c_int
_lib.sg_conv2d_wgrad.argtypes = [ctypes.POINTER(Conv2dDesc), _vp, _vp, _vp, _vp, _vp]
_lib.sg_batched_gemm.restype = ctypes.c_int
_lib.sg_batched_gemm.argtypes = [ctypes.POINTER(GemmDesc), _i64, _i64, _i64, _i64, _i64, _i64, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.sg_grouped_gemm_workspace_size.restype = ctypes.c_int
_lib.sg_grouped_gemm_workspace_size.argtypes = [_i32, ctypes.POINTER(ctypes.c_size_t)]
_lib.sg_grouped_gemm.restype = ctypes.c_int
_lib.sg_grouped_gemm.argtypes = [ctypes.POINTER(GemmDesc), _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, ctypes.c_size_t, _vp]
_lib.sg_grouped_gemm_static.restype = ctypes.c_int
_lib.sg_grouped_gemm_static.argtypes = [ctypes.POINTER(GemmDesc), _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.sg_conv2d_fprop.restype = ctypes.c_int
_lib.sg_conv2d_fprop.argtypes = [ctypes.POINTER(Conv2dDesc), _vp, _vp, _vp, _vp, _vp, _vp]
_lib.sg_transpose.restype = ctypes.c_int
_lib.sg_transpose.argtypes = [ctypes.POINTER(TransposeDesc), _vp, _vp, _vp]
_lib.sg_sol_bound.restype = ctypes.c_int
_lib.sg_sol_bound.argtypes = [_i32, _vp, _i64, _vp, _i32, _i32, _i32, ctypes.POINTER(Hw), ctypes.POINTER(Sol)]
_lib.sg_status_string.restype = ctypes.c_char_p
_lib.sg_status_string.argtypes = [ctypes.c_int]
_lib.sg_last_error.restype = ctypes.c_char_p
_lib.sg_poll_status.restype = ctypes.c_int
_lib.sg_poll_status.argtypes = [_vp]
_lib.sg_set_tuning.restype = ctypes.c_int
_lib.sg_set_tuning.argtypes = [_i32, _i32]
_lib.sg_launch_count.restype = _i64
_lib.sg_last_kernel_clock.restype = ctypes.c_int
_lib.sg_last_kernel_clock.argtypes = [ctypes.POINTER(ctypes.c_double), _vp]
_lib.sg_set_tail_mode.restype = ctypes.c_int
_lib.sg_set_tail_mode.argtypes = [_i32]
_lib.sg_set_scratch.restype = ctypes.c_int
_lib.sg_set_scratch.argtypes = [_vp, ctypes.c_size_t]
_lib.sg_last_launch_plan.restype = ctypes.c_int
_lib.sg_last_launch_plan.argtypes = [ctypes.POINTER(ctypes.c_int32)]
_lib.sg_last_kernel_name.restype = ctypes.c_char_p
_lib.sg_gemm_host_staging_size.restype = ctypes.c_int
_lib.sg_gemm_host_staging_size.argtypes = [ctypes.POINTER(GemmDesc), ctypes.POINTER(ctypes.c_size_t)]
_lib.sg_gemm_host.restype = ctypes.c_int
_lib.sg_gemm_host.argtypes = [ctypes.POINTER(GemmDesc), _vp, _vp, _vp, _vp, _vp, _vp, ctypes.c_size_t, _i32, _vp]
_lib.sg_set_option.restype = ctypes.c_int
_lib.sg_set_option.argtypes = [_i32, _i64]
_lib.sg_test_set_status_word.restype = ctypes.c_int
_lib.sg_test_set_status_word.argtypes = [ctypes.c_uint32, _vp]


SCRATCH_BYTES = 32 << 20
_scratch = {}      # device index -> the torch buffer lent to the library (kept alive here)
_scratch_enabled = os.environ.get("SOLGEMM_NO_SCRATCH", "0") != "1"


def enable_scratch(on: bool = True) -> None:
    """Turn the automatic lending of a scratch buffer on or off (off also takes back the current device's)."""
    global _scratch_enabled
    _scratch_enabled = bool(on)
    if not on and torch.cuda.is_available() and torch.cuda.current_device() in _scratch:
        torch.cuda.synchronize()
        set_scratch(None)


def set_scratch(buf: Optional[torch.Tensor]) -> None:
    """``sg_set_scratch``: lend (or, with None, take back) the tail-balancing scratch of the current device."""
    dev = torch.cuda.current_device()
    if buf is None:
        _check(_lib.sg_set_scratch(None, 0))
        _scratch.pop(dev, None)
    else:
        _check(_lib.sg_set_scratch(_ptr(buf), buf.numel() * buf.element_size()))
        _scratch[dev] = buf


def ensure_scratch() -> None:
    """Lend the library a scratch buffer on the current device once (torch owns the memory).
    ``SOLGEMM_NO_SCRATCH=1`` keeps the library on its scratch-free tail strategy."""
    dev = torch.cuda.current_device()
    if dev not in _scratch and _scratch_enabled:
        set_scratch(torch.empty(SCRATCH_BYTES, dtype=torch.uint8, device=f"cuda:{dev}"))


def raw_lib() -> ctypes.CDLL:
    """The loaded shared library, for callers that want to drive the C ABI directly."""
    return _lib


def _check(status: int) -> None:
    if status != SG_OK:
        raise SolgemmError(status, _lib.sg_last_error().decode())


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _ld(t: torch.Tensor) -> int:
    """Leading dimension of a 2-D operand as stored (outer stride; the row length if there is one row)."""
    if t.dim() != 2 or (t.shape[1] > 1 and t.stride(1) != 1):
        raise ValueError("operands must be 2-D with inner stride 1")
    if t.shape[0] > 1 or t.stride(0) >= max(t.shape[1], 1):
        return t.stride(0)            # (a one-row view of a padded buffer keeps the buffer's row pitch)
    return max(t.shape[1], 1)


def _gemm_desc(M, N, K, lda, ldb, ldc, ldd, layout_a, layout_b, out_dtype, alpha, beta, epi,
               epi_args=(0.0, 0.0), in_dtype=torch.bfloat16) -> GemmDesc:
    return GemmDesc(M, N, K, LAYOUTS[layout_a], LAYOUTS[layout_b], lda, ldb, ldc, ldd, DTYPES[in_dtype], DTYPES[out_dtype],
                    float(alpha), float(beta), EPILOGUES[epi], float(epi_args[0]), float(epi_args[1]), 0)


def _mnk(A, B, layout_a, layout_b):
    M, K = (A.shape[-2], A.shape[-1]) if layout_a == "row" else (A.shape[-1], A.shape[-2])
    Kb, N = (B.shape[-2], B.shape[-1]) if layout_b == "row" else (B.shape[-1], B.shape[-2])
    if K != Kb:
        raise ValueError("A and B disagree on K")
    return M, N, K


def _addr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _ex_struct(ex: Optional[dict]) -> Optional[EpilogueEx]:
    """``ex``: dict with any of row_scale, col_scale, row_bias (fp32 vectors), post_scale (float), aux_load,
    aux_store (2-D tensors of the output's type, inner stride 1) -> the C structure (None when ``ex`` is None)."""
    if ex is None:
        return None
    unknown = set(ex) - {"row_scale", "col_scale", "row_bias", "post_scale", "aux_load", "aux_store"}
    if unknown:
        raise ValueError(f"unknown extended-epilogue members: {sorted(unknown)}")
    for name in ("row_scale", "col_scale", "row_bias"):
        t = ex.get(name)
        if t is not None and (t.dtype != torch.float32 or not t.is_contiguous()):
            raise ValueError(f"{name} must be a contiguous fp32 vector")
    al, ast = ex.get("aux_load"), ex.get("aux_store")
    def as2d(t, name):                      # conv: a contiguous [N, P, Q, K] tensor is the [NPQ, K] matrix
        if t is None or t.dim() == 2:
            return t
        if not t.is_contiguous():
            raise ValueError(f"{name} with more than two dimensions must be contiguous")
        return t.view(-1, t.shape[-1])
    al2, ast2 = as2d(al, "aux_load"), as2d(ast, "aux_store")
    return EpilogueEx(_addr(ex.get("row_scale")), _addr(ex.get("col_scale")), _addr(ex.get("row_bias")),
                      float(ex.get("post_scale", 1.0)), 0,
                      _addr(al2), _ld(al2) if al2 is not None else 0, _addr(ast2), _ld(ast2) if ast2 is not None else 0)


def gemm(A: torch.Tensor, B: torch.Tensor, *, C: Optional[torch.Tensor] = None, bias: Optional[torch.Tensor] = None,
         out: Optional[torch.Tensor] = None, out_dtype: torch.dtype = torch.bfloat16, alpha: float = 1.0,
         beta: float = 0.0, epi: str = "none", epi_args=(0.0, 0.0), layout_a: str = "row", layout_b: str = "col",
         stream=None, ex: Optional[dict] = None) -> torch.Tensor:
    """D = act(alpha A.B + beta C + bias) through ``sg_gemm``.  Returns D (``out`` if given).

    ``ex`` (see ``_ex_struct``) routes the call through ``sg_gemm_ex`` with the extended epilogue chain."""
    M, N, K = _mnk(A, B, layout_a, layout_b)
    ensure_scratch()
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=A.device)
    desc = _gemm_desc(M, N, K, _ld(A), _ld(B), _ld(C) if C is not None else max(N, 1), _ld(out), layout_a, layout_b,
                      out.dtype, alpha, beta, epi, epi_args, A.dtype)
    if ex is not None:
        exs = _ex_struct(ex)
        _check(_lib.sg_gemm_ex(ctypes.byref(desc), ctypes.byref(exs), _ptr(A), _ptr(B), _ptr(C), _ptr(bias), _ptr(out),
                               _stream(stream)))
        return out
    _check(_lib.sg_gemm(ctypes.byref(desc), _ptr(A), _ptr(B), _ptr(C), _ptr(bias), _ptr(out), _stream(stream)))
    return out


def batched_gemm(A: torch.Tensor, B: torch.Tensor, *, C=None, bias=None, out=None, out_dtype=torch.bfloat16,
                 alpha=1.0, beta=0.0, epi="none", epi_args=(0.0, 0.0), layout_a="row", layout_b="col",
                 stream=None) -> torch.Tensor:
    """The same product for every leading index through ``sg_batched_gemm``; ``bias`` is [N] or [batch, N]."""
    batch = A.shape[0]
    M, N, K = _mnk(A, B, layout_a, layout_b)
    ensure_scratch()
    if out is None:
        out = torch.empty((batch, M, N), dtype=out_dtype, device=A.device)
    for t in (A, B, out) + ((C,) if C is not None else ()):
        if t.dim() != 3 or (t.shape[2] > 1 and t.stride(2) != 1):
            raise ValueError("batched operands must be 3-D with inner stride 1")
    sbias = 0 if bias is None or bias.dim() == 1 else bias.stride(0)
    desc = _gemm_desc(M, N, K, A.stride(1), B.stride(1), C.stride(1) if C is not None else max(N, 1), out.stride(1),
                      layout_a, layout_b, out.dtype, alpha, beta, epi, epi_args, A.dtype)
    _check(_lib.sg_batched_gemm(ctypes.byref(desc), batch, A.stride(0), B.stride(0),
                                C.stride(0) if C is not None else 0, out.stride(0), sbias,
                                _ptr(A), _ptr(B), _ptr(C), _ptr(bias), _ptr(out), _stream(stream)))
    return out


def grouped_workspace_size(groups: int) -> int:
    n = ctypes.c_size_t(0)
    _check(_lib.sg_grouped_gemm_workspace_size(groups, ctypes.byref(n)))
    return int(n.value)


def _ptr_array(tensors: Optional[Sequence[Optional[torch.Tensor]]]):
    if tensors is None:
        return None
    arr = (ctypes.c_void_p * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = None if t is None else t.data_ptr()
    return arr


def grouped_gemm(As: Sequence[torch.Tensor], Bs: Sequence[torch.Tensor], *, Cs=None, biases=None,
                 outs: Optional[Sequence[torch.Tensor]] = None, out_dtype=torch.bfloat16, alpha=1.0, beta=0.0,
                 epi="none", epi_args=(0.0, 0.0), layout_a="row", layout_b="col",
                 workspace: Optional[torch.Tensor] = None, stream=None) -> List[torch.Tensor]:
    """One launch of ``sg_grouped_gemm`` over groups with their own M_g; N, K and leading dimensions are common."""
    groups = len(As)
    if groups == 0:
        return []
    ensure_scratch()
    _, N, K = _mnk(As[0], Bs[0], layout_a, layout_b)
    Ms = [(_mnk(a, b, layout_a, layout_b))[0] for a, b in zip(As, Bs)]
    if outs is None:
        outs = [torch.empty((m, N), dtype=out_dtype, device=As[0].device) for m in Ms]
    ld = lambda ts, default: next((_ld(t) for t in ts if t.shape[0] > 1), default)
    desc = _gemm_desc(0, N, K, ld(As, max(K, 1)), ld(Bs, max(K, 1)), ld(Cs, max(N, 1)) if Cs is not None else max(N, 1),
                      ld(outs, max(N, 1)), layout_a, layout_b, outs[0].dtype, alpha, beta, epi, epi_args, As[0].dtype)
    if workspace is None:
        workspace = torch.empty(grouped_workspace_size(groups), dtype=torch.uint8, device=As[0].device)
    m_arr = (ctypes.c_int64 * groups)(*Ms)
    _check(_lib.sg_grouped_gemm(ctypes.byref(desc), groups, m_arr, _ptr_array(As), _ptr_array(Bs), _ptr_array(Cs),
                                _ptr_array(biases), _ptr_array(outs), _ptr(workspace), workspace.numel(),
                                _stream(stream)))
    return list(outs)


STATIC_MAX_GROUPS = 64


def grouped_gemm_static(As: Sequence[torch.Tensor], Bs: Sequence[torch.Tensor], *, Cs=None, biases=None,
                        outs: Sequence[torch.Tensor], alpha=1.0, beta=0.0, epi="none", epi_args=(0.0, 0.0),
                        layout_a="row", layout_b="col", stream=None) -> List[torch.Tensor]:
    """``sg_grouped_gemm_static``: the grouped product for callers that may not allocate device memory.

    Unlike :func:`grouped_gemm` this wrapper allocates nothing either: ``outs`` must be given, and the
    library keeps its tables in a scratch array built into its image (at most ``STATIC_MAX_GROUPS``
    groups).  Calls on one device share that array, so calls that overlap on the GPU must be serialised.
    """
    groups = len(As)
    if groups == 0:
        return []
    _, N, K = _mnk(As[0], Bs[0], layout_a, layout_b)
    Ms = [(_mnk(a, b, layout_a, layout_b))[0] for a, b in zip(As, Bs)]
    ld = lambda ts, default: next((_ld(t) for t in ts if t.shape[0] > 1), default)
    desc = _gemm_desc(0, N, K, ld(As, max(K, 1)), ld(Bs, max(K, 1)), ld(Cs, max(N, 1)) if Cs is not None else max(N, 1),
                      ld(outs, max(N, 1)), layout_a, layout_b, outs[0].dtype, alpha, beta, epi, epi_args, As[0].dtype)
    m_arr = (ctypes.c_int64 * groups)(*Ms)
    _check(_lib.sg_grouped_gemm_static(ctypes.byref(desc), groups, m_arr, _ptr_array(As), _ptr_array(Bs),
                                       _ptr_array(Cs), _ptr_array(biases), _ptr_array(outs), _stream(stream)))
    return list(outs)


def conv2d_fprop(X: torch.Tensor, Wf: torch.Tensor, *, pad=(0, 0), stride=(1, 1), dil=(1, 1), Cin=None, bias=None,
                 out=None, out_dtype=torch.bfloat16, alpha=1.0, beta=0.0, epi="none", epi_args=(0.0, 0.0),
                 stream=None, ex: Optional[dict] = None) -> torch.Tensor:
    """NHWC x KRSC -> NPQK forward convolution through ``sg_conv2d_fprop`` (implicit GEMM, nothing materialised).

    ``ex`` routes the call through ``sg_conv2d_fprop_ex`` (rows are output pixels, columns output channels)."""
    if X.dim() != 4 or Wf.dim() != 4 or not X.is_contiguous() or not Wf.is_contiguous():
        raise ValueError("X (NHWC) and Wf (KRSC) must be contiguous 4-D tensors")
    N, H, W, C = X.shape
    K, R, S, Cw = Wf.shape
    if C != Cw:
        raise ValueError("X and Wf disagree on C")
    ext = lambda size, p, d, f, s: max((size + 2 * p - d * (f - 1) - 1) // s + 1, 0) if size + 2 * p - d * (f - 1) - 1 >= 0 else 0
    P, Q = ext(H, pad[0], dil[0], R, stride[0]), ext(W, pad[1], dil[1], S, stride[1])
    ensure_scratch()
    if out is None:
        out = torch.empty((N, P, Q, K), dtype=out_dtype, device=X.device)
    desc = Conv2dDesc(N, H, W, C, K, R, S, pad[0], pad[1], stride[0], stride[1], dil[0], dil[1], DTYPES[X.dtype],
                      DTYPES[out.dtype],
                      float(alpha), float(beta), EPILOGUES[epi], float(epi_args[0]), float(epi_args[1]), 0)
    if ex is not None:
        exs = _ex_struct(ex)
        _check(_lib.sg_conv2d_fprop_ex(ctypes.byref(desc), ctypes.byref(exs), _ptr(X), _ptr(Wf), _ptr(Cin), _ptr(bias),
                                       _ptr(out), _stream(stream)))
        return out
    _check(_lib.sg_conv2d_fprop(ctypes.byref(desc), _ptr(X), _ptr(Wf), _ptr(Cin), _ptr(bias), _ptr(out), _stream(stream)))
    return out


def conv2d_dgrad(dY: torch.Tensor, Wf: torch.Tensor, hw, *, pad=(0, 0), stride=(1, 1), dil=(1, 1), Cin=None, out=None,
                 out_dtype=torch.bfloat16, alpha=1.0, beta=0.0, stream=None) -> torch.Tensor:
    """Gradient of ``conv2d_fprop`` with respect to its input through ``sg_conv2d_dgrad``: ``dY`` [N,P,Q,K],
    ``Wf`` [K,R,S,C] -> [N,H,W,C] with ``hw = (H, W)`` of the forward input."""
    if dY.dim() != 4 or Wf.dim() != 4 or not dY.is_contiguous() or not Wf.is_contiguous():
        raise ValueError("dY (NPQK) and Wf (KRSC) must be contiguous 4-D tensors")
    N, K = dY.shape[0], dY.shape[3]
    Kw, R, S, C = Wf.shape
    if K != Kw:
        raise ValueError("dY and Wf disagree on K")
    H, W = hw
    ensure_scratch()
    if out is None:
        out = torch.empty((N, H, W, C), dtype=out_dtype, device=dY.device)
    desc = Conv2dDesc(N, H, W, C, K, R, S, pad[0], pad[1], stride[0], stride[1], dil[0], dil[1], DTYPES[dY.dtype],
                      DTYPES[out.dtype], float(alpha), float(beta), EPILOGUES["none"], 0.0, 0.0, 0)
    _check(_lib.sg_conv2d_dgrad(ctypes.byref(desc), _ptr(dY), _ptr(Wf), _ptr(Cin), _ptr(out), _stream(stream)))
    return out


def conv2d_wgrad(dY: torch.Tensor, X: torch.Tensor, rs, *, pad=(0, 0), stride=(1, 1), dil=(1, 1), Cin=None, out=None,
                 out_dtype=torch.float32, alpha=1.0, beta=0.0, stream=None) -> torch.Tensor:
    """Gradient of ``conv2d_fprop`` with respect to its filter through ``sg_conv2d_wgrad``: ``dY`` [N,P,Q,K],
    ``X`` [N,H,W,C] -> [K,R,S,C] with ``rs = (R, S)``."""
    if dY.dim() != 4 or X.dim() != 4 or not dY.is_contiguous() or not X.is_contiguous():
        raise ValueError("dY (NPQK) and X (NHWC) must be contiguous 4-D tensors")
    N, H, W, C = X.shape
    K = dY.shape[3]
    R, S = rs
    ensure_scratch()
    if out is None:
        out = torch.empty((K, R, S, C), dtype=out_dtype, device=dY.device)
    desc = Conv2dDesc(N, H, W, C, K, R, S, pad[0], pad[1], stride[0], stride[1], dil[0], dil[1], DTYPES[dY.dtype],
                      DTYPES[out.dtype], float(alpha), float(beta), EPILOGUES["none"], 0.0, 0.0, 0)
    _check(_lib.sg_conv2d_wgrad(ctypes.byref(desc), _ptr(dY), _ptr(X), _ptr(Cin), _ptr(out), _stream(stream)))
    return out


def transpose(x: torch.Tensor, *, out: Optional[torch.Tensor] = None, out_dtype: Optional[torch.dtype] = None,
              stream=None) -> torch.Tensor:
    """``sg_transpose``: ``out[b, c, r] = convert(x[b, r, c])`` for a 3-D (or 2-D) tensor with inner stride 1."""
    squeeze = x.dim() == 2
    x3 = x.unsqueeze(0) if squeeze else x
    if x3.dim() != 3 or (x3.shape[2] > 1 and x3.stride(2) != 1):
        raise ValueError("transpose wants a [batch, rows, cols] tensor with inner stride 1")
    batch, rows, cols = x3.shape
    if out is None:
        out = torch.empty((batch, cols, rows), dtype=out_dtype or x.dtype, device=x.device)
        out3 = out
        if squeeze:
            out = out[0]
    else:
        out3 = out.unsqueeze(0) if squeeze else out
    desc = TransposeDesc(batch, rows, cols, x3.stride(1) if rows > 1 else max(cols, 1),
                         out3.stride(1) if cols > 1 else max(rows, 1), x3.stride(0), out3.stride(0),
                         DTYPES[x.dtype], DTYPES[out3.dtype], 0, 0)
    _check(_lib.sg_transpose(ctypes.byref(desc), _ptr(x3), _ptr(out3), _stream(stream)))
    return out


def nchw_to_nhwc(x: torch.Tensor, out_dtype: Optional[torch.dtype] = None) -> torch.Tensor:
    """[N, C, H, W] -> [N, H, W, C] (with optional dtype conversion) through ``sg_transpose``."""
    n, c, h, w = x.shape
    return transpose(x.reshape(n, c, h * w), out_dtype=out_dtype).view(n, h, w, c)


def nhwc_to_nchw(x: torch.Tensor, out_dtype: Optional[torch.dtype] = None) -> torch.Tensor:
    """[N, H, W, C] -> [N, C, H, W] (with optional dtype conversion) through ``sg_transpose``."""
    n, h, w, c = x.shape
    return transpose(x.reshape(n, h * w, c), out_dtype=out_dtype).view(n, c, h, w)


def conv2d_fprop_nchw(x: torch.Tensor, Wf: torch.Tensor, *, compute_dtype: torch.dtype = torch.bfloat16,
                      out_dtype: Optional[torch.dtype] = None, stream=None, **conv_kw) -> torch.Tensor:
    """The DSL's three-stage pipeline (Appendix A.1) for a framework that keeps NCHW tensors:
    ``pipeline(transpose(input, NCHW, NHWC, dtype, compute_dtype), conv2d_fprop(...), transpose(output, NHWC, NCHW,
    compute_dtype, out_dtype))`` -- three launches on one stream, no host work in between.  ``x`` is [N, C, H, W]
    (fp32 or bf16), ``Wf`` is [K, R, S, C] in the compute type; ``conv_kw`` goes to ``conv2d_fprop``."""
    n, c, h, w = x.shape
    x_nhwc = transpose(x.reshape(n, c, h * w), out_dtype=compute_dtype, stream=stream).view(n, h, w, c)
    y = conv2d_fprop(x_nhwc, Wf, stream=stream, **conv_kw)
    _, p, q, k = y.shape
    return transpose(y.reshape(n, p * q, k), out_dtype=out_dtype or x.dtype, stream=stream).view(n, k, p, q)


def conv1d_fprop(X: torch.Tensor, Wf: torch.Tensor, *, pad=0, stride=1, dil=1, **kw) -> torch.Tensor:
    """1-D convolution lowered to ``sg_conv2d_fprop`` with H = 1 (the paper's Table 1a note): X [N, L, C], Wf [K, S, C]."""
    n, l, c = X.shape
    k, s, _ = Wf.shape
    y = conv2d_fprop(X.view(n, 1, l, c), Wf.view(k, 1, s, c), pad=(0, pad), stride=(1, stride), dil=(1, dil), **kw)
    return y.view(n, y.shape[2], k)


def gemm_host(A_host: torch.Tensor, B_host: torch.Tensor, out_host: torch.Tensor, *, C_host=None, bias_host=None, epi="none",
              alpha=1.0, beta=0.0, device="cuda", scratch: Optional[dict] = None, stream=None, chunks: int = 4,
              layout_a: str = "row", layout_b: str = "col") -> torch.Tensor:
    """``sg_gemm_host``: GEMM for callers whose data lives in (pinned) host memory.

    The library copies A, B (C, bias) to a device staging buffer, runs ``sg_gemm`` and copies D back into ``out_host``,
    pipelined over ``chunks`` row blocks on its own copy streams; everything is ordered against ``stream`` (default: the
    current stream).  ``scratch`` may hold the staging tensor ("staging") between calls; torch owns that memory.
    """
    scratch = {} if scratch is None else scratch
    dev = torch.device(device)
    if dev.index is None:
        dev = torch.device("cuda", torch.cuda.current_device())
    M, N, K = _mnk(A_host, B_host, layout_a, layout_b)
    desc = _gemm_desc(M, N, K, _ld(A_host), _ld(B_host), _ld(C_host) if C_host is not None else max(N, 1), _ld(out_host),
                      layout_a, layout_b, out_host.dtype, alpha, beta, epi, in_dtype=A_host.dtype)
    need = ctypes.c_size_t(0)
    _check(_lib.sg_gemm_host_staging_size(ctypes.byref(desc), ctypes.byref(need)))
    st = scratch.get("staging")
    if st is None or st.numel() < need.value or st.device != dev:
        st = scratch["staging"] = torch.empty(max(need.value, 256), dtype=torch.uint8, device=dev)
    with torch.cuda.device(dev):
        ensure_scratch()
        s = torch.cuda.current_stream(dev) if stream is None else stream
        _check(_lib.sg_gemm_host(ctypes.byref(desc), _ptr(A_host), _ptr(B_host), _ptr(C_host), _ptr(bias_host), _ptr(out_host),
                                 _ptr(st), st.numel(), int(chunks), ctypes.c_void_p(s.cuda_stream)))
    return out_host


def sol_bound(op: str, *, M=0, N=0, K=0, batch_or_groups=1, Ms: Optional[Sequence[int]] = None, conv: Optional[dict] = None,
              transpose_shape: Optional[tuple] = None, transpose_dtypes=(torch.bfloat16, torch.bfloat16),
              beta=0.0, elem_bytes_in=2, elem_bytes_out=2, has_bias=0, peak_flops: float, peak_bytes_per_s: float,
              sm_clock_mhz=0.0, sm_clock_max_mhz=0.0, mem_clock_mhz=0.0, mem_clock_max_mhz=0.0) -> dict:
    """``sg_sol_bound``: FLOPs, best-case bytes and t_SOL = max(FLOPs/peak, bytes/bandwidth) (host only)."""
    if op == "transpose":
        b, r, c_ = transpose_shape
        desc = TransposeDesc(b, r, c_, c_, r, r * c_, r * c_, DTYPES[transpose_dtypes[0]], DTYPES[transpose_dtypes[1]], 0, 0)
    elif op in ("conv2d", "conv2d_dgrad", "conv2d_wgrad"):
        c = conv
        desc = Conv2dDesc(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], *c.get("pad", (0, 0)),
                          *c.get("stride", (1, 1)), *c.get("dil", (1, 1)), 0, 0, 1.0, float(beta), 0, 0.0, 0.0, 0)
    else:
        desc = GemmDesc(M, N, K, 0, 1, max(K, 1), max(K, 1), max(N, 1), max(N, 1), 0, 0, 1.0, float(beta), 0, 0.0, 0.0, 0)
    m_arr = (ctypes.c_int64 * len(Ms))(*Ms) if Ms is not None else None
    hw = Hw(peak_flops, peak_bytes_per_s, sm_clock_mhz, sm_clock_max_mhz, mem_clock_mhz, mem_clock_max_mhz)
    out = Sol()
    _check(_lib.sg_sol_bound(OPS[op], ctypes.byref(desc), batch_or_groups, m_arr, elem_bytes_in, elem_bytes_out,
                             int(has_bias), ctypes.byref(hw), ctypes.byref(out)))
    res = {n: getattr(out, n) for n, _ in Sol._fields_ if n != "reserved"}
    res["compute_bound"] = bool(res["compute_bound"])
    return res


def poll_status(stream=None) -> None:
    """Raise ``SolgemmError`` if a kernel recorded an expired device-side wait (after the caller has synchronised)."""
    _check(_lib.sg_poll_status(_stream(stream)))


def set_tuning(tile_n: int = -1, cta_pair: int = -1) -> None:
    _check(_lib.sg_set_tuning(tile_n, cta_pair))


def last_kernel_clock_mhz(stream=None) -> float:
    """SM clock the most recent contraction kernel really ran at (measured in the kernel); synchronises the stream."""
    mhz = ctypes.c_double(0.0)
    _check(_lib.sg_last_kernel_clock(ctypes.byref(mhz), _stream(stream)))
    return float(mhz.value)


def set_tail_mode(mode: int = -1) -> None:
    """-1 planner's choice, 0 whole tail tiles, 1 column slices, 2 K ranges through the scratch."""
    _check(_lib.sg_set_tail_mode(mode))


def set_option(name: str, value: int = -1) -> None:
    """``sg_set_option``: pin one of the planner's choices (see ``OPTIONS``); -1 restores the default."""
    _check(_lib.sg_set_option(OPTIONS[name], int(value)))


def test_set_status_word(value: int, stream=None) -> None:
    """``sg_test_set_status_word`` (test hook): write the device status word as an expired wait would."""
    _check(_lib.sg_test_set_status_word(int(value), _stream(stream)))


test_set_status_word.__test__ = False      # not a pytest test, whatever module imports it


def launch_count() -> int:
    return int(_lib.sg_launch_count())


def last_kernel_name() -> str:
    """``sg_last_kernel_name``: the device function this thread's most recent launch ran (the library's own record)."""
    return _lib.sg_last_kernel_name().decode()


def last_launch_plan() -> dict:
    """Tiling of this thread's most recent contraction launch (``sg_last_launch_plan``)."""
    a = (ctypes.c_int32 * 6)()
    _check(_lib.sg_last_launch_plan(a))
    return dict(zip(("tile_n", "cta_pair", "tail_split", "tiles", "split_begin", "grid"), (int(x) for x in a)))
