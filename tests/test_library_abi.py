"""CPU-side checks of the C-ABI library: it loads, exports what the header declares, validates
arguments before touching a device, and its Speed-of-Light calculator matches the oracle's."""
import ctypes
import os
import re

import pytest

from oracle import oracle as orc
from tests.test_sol_oracle import load_golden

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def sg():
    from paper_2603_29010_b200 import build
    build.build()                      # nvcc cross-compiles for sm_100a without a GPU
    from paper_2603_29010_b200 import solgemm
    return solgemm


def test_library_exports_every_declared_symbol(sg):
    header = open(os.path.join(ROOT, "include", "solgemm.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(sg_[a-z0-9_]+)\s*\(", header))
    assert declared == set(sg.EXPORTED)
    lib = sg.raw_lib()
    for name in declared:
        assert hasattr(lib, name), name


def test_struct_layouts_match_the_header(sg):
    assert ctypes.sizeof(sg.GemmDesc) == 96 and ctypes.sizeof(sg.Conv2dDesc) == 112
    assert ctypes.sizeof(sg.Hw) == 48 and ctypes.sizeof(sg.Sol) == 80
    assert ctypes.sizeof(sg.EpilogueEx) == 64


def test_status_strings(sg):
    lib = sg.raw_lib()
    for i, name in enumerate(sg.STATUS_NAMES):
        assert lib.sg_status_string(i).decode() == name


def _desc(sg, **kw):
    base = dict(M=128, N=128, K=128, layout_a=0, layout_b=1, lda=128, ldb=128, ldc=128, ldd=128, in_dtype=0,
                out_dtype=0, alpha=1.0, beta=0.0, epi=0, epi_arg0=0.0, epi_arg1=0.0, reserved=0)
    base.update(kw)
    return sg.GemmDesc(*[base[n] for n, _ in sg.GemmDesc._fields_])


def _call_gemm(sg, desc, A=0x1000, B=0x2000, C=None, bias=None, D=0x3000):
    return sg.raw_lib().sg_gemm(ctypes.byref(desc), A, B, C, bias, D, None)


@pytest.mark.parametrize("kw,ptrs,want", [
    (dict(M=-1), {}, "SG_ERR_INVALID_ARG"),
    (dict(lda=64), {}, "SG_ERR_INVALID_ARG"),
    (dict(epi=12), {}, "SG_ERR_INVALID_ARG"),
    (dict(epi=11, epi_arg0=1.0, epi_arg1=0.0), {}, "SG_ERR_INVALID_ARG"),      # clip with min > max
    (dict(epi=9, epi_arg0=float("nan")), {}, "SG_ERR_INVALID_ARG"),
    (dict(out_dtype=9), {}, "SG_ERR_INVALID_ARG"),
    (dict(out_dtype=5), {}, "SG_ERR_UNSUPPORTED"),          # SG_INT8 is an input type only
    (dict(reserved=1), {}, "SG_ERR_INVALID_ARG"),
    (dict(lda=132), {}, "SG_ERR_ALIGNMENT"),             # 264 bytes: not a multiple of 16
    (dict(ldd=129), {}, "SG_ERR_ALIGNMENT"),
    (dict(), dict(A=0x1008), "SG_ERR_ALIGNMENT"),
    (dict(), dict(D=None), "SG_ERR_NULL_POINTER"),
    (dict(), dict(A=None), "SG_ERR_NULL_POINTER"),
    (dict(beta=1.0), {}, "SG_ERR_NULL_POINTER"),         # beta != 0 without C
    (dict(epi=1), {}, "SG_ERR_NULL_POINTER"),            # SG_EPI_BIAS without bias
    (dict(in_dtype=9), {}, "SG_ERR_UNSUPPORTED"),
    (dict(in_dtype=1, layout_a=1), {}, "SG_ERR_UNSUPPORTED"),      # fp32 (tf32) operands: K-contiguous only
    (dict(in_dtype=1, lda=130), {}, "SG_ERR_ALIGNMENT"),           # 130 fp32 elements = 520 bytes
    (dict(layout_a=1, lda=64), {}, "SG_ERR_INVALID_ARG"),       # column-major A: lda must cover M = 128
    (dict(layout_b=7), {}, "SG_ERR_INVALID_ARG"),
    # matrix-vector form (N <= 4 or M <= 4): its own, relaxed checks, still before any launch
    (dict(N=1, ldd=1), dict(D=None), "SG_ERR_NULL_POINTER"),
    (dict(N=1, ldd=1, ldc=1, beta=1.0), {}, "SG_ERR_NULL_POINTER"),
    (dict(M=1, epi=1), {}, "SG_ERR_NULL_POINTER"),
    (dict(N=3, ldd=3, out_dtype=5), {}, "SG_ERR_UNSUPPORTED"),
    (dict(N=2, ldd=1), {}, "SG_ERR_INVALID_ARG"),                       # ldd < N
    (dict(N=1, ldd=1), dict(D=0x3001), "SG_ERR_ALIGNMENT"),              # a bf16 output on an odd address
    (dict(N=1, ldd=1, lda=132), {}, "SG_ERR_ALIGNMENT"),                 # rows not 16-byte multiples: general path's rule
])
def test_gemm_rejects_bad_arguments_before_any_launch(sg, kw, ptrs, want):
    before = sg.launch_count()
    st = _call_gemm(sg, _desc(sg, **kw), **ptrs)
    assert sg.STATUS_NAMES[st] == want, sg.raw_lib().sg_last_error().decode()
    assert sg.raw_lib().sg_last_error().decode() != ""
    assert sg.launch_count() == before


def test_empty_problems_succeed_without_a_device(sg):
    assert _call_gemm(sg, _desc(sg, M=0)) == 0
    assert _call_gemm(sg, _desc(sg, N=0, ldd=8)) == 0
    lib = sg.raw_lib()
    assert lib.sg_batched_gemm(ctypes.byref(_desc(sg)), 0, 0, 0, 0, 0, 0, 0x1000, 0x2000, None, None, 0x3000, None) == 0
    st = lib.sg_batched_gemm(ctypes.byref(_desc(sg)), 2, 4, 0, 0, 128 * 128, 0, 0x1000, 0x2000, None, None, 0x3000, None)
    assert sg.STATUS_NAMES[st] == "SG_ERR_ALIGNMENT"


def test_grouped_and_conv_validation(sg):
    lib = sg.raw_lib()
    n = ctypes.c_size_t(0)
    assert lib.sg_grouped_gemm_workspace_size(16, ctypes.byref(n)) == 0
    assert n.value >= 16 * 3 * 128 and n.value % 128 == 0
    assert sg.grouped_workspace_size(32) > n.value
    Ms = (ctypes.c_int64 * 2)(128, 64)
    ptrs = (ctypes.c_void_p * 2)(0x1000, 0x2000)
    d = _desc(sg)
    st = lib.sg_grouped_gemm(ctypes.byref(d), 2, Ms, ptrs, ptrs, None, None, ptrs, None, 0, None)
    assert sg.STATUS_NAMES[st] == "SG_ERR_WORKSPACE"
    st = lib.sg_grouped_gemm(ctypes.byref(d), 2, Ms, ptrs, ptrs, None, None, ptrs, 0x4010, 1 << 20, None)
    assert sg.STATUS_NAMES[st] == "SG_ERR_WORKSPACE"           # not 128-byte aligned
    st = lib.sg_grouped_gemm(ctypes.byref(d), 2, Ms, ptrs, ptrs, None, None, ptrs, 0x4000, 64, None)
    assert sg.STATUS_NAMES[st] == "SG_ERR_WORKSPACE"           # too small
    Mneg = (ctypes.c_int64 * 2)(128, -1)
    st = lib.sg_grouped_gemm(ctypes.byref(d), 2, Mneg, ptrs, ptrs, None, None, ptrs, 0x4000, 1 << 20, None)
    assert sg.STATUS_NAMES[st] == "SG_ERR_INVALID_ARG"
    assert lib.sg_grouped_gemm(ctypes.byref(d), 0, None, None, None, None, None, None, None, 0, None) == 0

    def conv(**kw):
        base = dict(N=1, H=8, W=8, C=64, K=64, R=3, S=3, pad_h=1, pad_w=1, stride_h=1, stride_w=1, dil_h=1, dil_w=1,
                    in_dtype=0, out_dtype=0, alpha=1.0, beta=0.0, epi=0, epi_arg0=0.0, epi_arg1=0.0, reserved=0)
        base.update(kw)
        return sg.Conv2dDesc(*[base[k] for k, _ in sg.Conv2dDesc._fields_])

    call = lambda d, X=0x1000: lib.sg_conv2d_fprop(ctypes.byref(d), X, 0x2000, None, None, 0x3000, None)
    assert sg.STATUS_NAMES[call(conv(C=20))] == "SG_ERR_ALIGNMENT"
    assert sg.STATUS_NAMES[call(conv(K=12))] == "SG_ERR_ALIGNMENT"
    assert sg.STATUS_NAMES[call(conv(stride_h=0))] == "SG_ERR_INVALID_ARG"
    assert sg.STATUS_NAMES[call(conv(pad_h=200))] == "SG_ERR_UNSUPPORTED"
    assert sg.STATUS_NAMES[call(conv(), X=None)] == "SG_ERR_NULL_POINTER"
    assert call(conv(N=0)) == 0 and call(conv(H=1, W=1, pad_h=0, pad_w=0)) == 0      # empty output

    # gradients: checked before any device is touched
    dgrad = lambda d, dY=0x1000: lib.sg_conv2d_dgrad(ctypes.byref(d), dY, 0x2000, None, 0x3000, None)
    wgrad = lambda d, dY=0x1000: lib.sg_conv2d_wgrad(ctypes.byref(d), dY, 0x2000, None, 0x3000, None)
    assert sg.STATUS_NAMES[dgrad(conv(stride_h=9))] == "SG_ERR_UNSUPPORTED"          # stride beyond the im2col limits
    assert sg.STATUS_NAMES[dgrad(conv(epi=2))] == "SG_ERR_INVALID_ARG"               # no activation on a gradient
    assert sg.STATUS_NAMES[wgrad(conv(in_dtype=3))] == "SG_ERR_UNSUPPORTED"          # fp8 inputs
    assert sg.STATUS_NAMES[wgrad(conv(C=20))] == "SG_ERR_ALIGNMENT"
    assert sg.STATUS_NAMES[dgrad(conv(K=12))] == "SG_ERR_ALIGNMENT"
    assert sg.STATUS_NAMES[wgrad(conv(dil_w=0))] == "SG_ERR_INVALID_ARG"
    assert sg.STATUS_NAMES[lib.sg_conv2d_wgrad(None, 0x1000, 0x2000, None, 0x3000, None)] == "SG_ERR_NULL_POINTER"
    assert dgrad(conv(N=0)) == 0 and wgrad(conv(K=0)) == 0                           # empty outputs

    # extended epilogue: the chain's own rules
    ex = sg.EpilogueEx(None, 0x5004, None, 1.0, 0, None, 0, None, 0)
    call_ex = lambda e: lib.sg_gemm_ex(ctypes.byref(_desc(sg)), ctypes.byref(e), 0x1000, 0x2000, None, None, 0x3000, None)
    assert sg.STATUS_NAMES[call_ex(ex)] == "SG_ERR_ALIGNMENT"                        # col_scale not 16-byte aligned
    assert sg.STATUS_NAMES[call_ex(sg.EpilogueEx(None, None, None, 1.0, 7, None, 0, None, 0))] == "SG_ERR_INVALID_ARG"
    assert sg.STATUS_NAMES[call_ex(sg.EpilogueEx(None, None, None, 1.0, 0, 0x6000, 64, None, 0))] == "SG_ERR_INVALID_ARG"  # ld < N


def test_sol_bound_matches_the_printed_report_and_the_oracle(sg, golden_dir):
    g = load_golden(os.path.join(golden_dir, "sol_report_gemm4096.txt"))
    n = int(g["n"])
    r = sg.sol_bound("gemm", M=n, N=n, K=n, elem_bytes_in=4, elem_bytes_out=4,
                     peak_flops=float(g["peak_tf32_flops"]), peak_bytes_per_s=float(g["peak_bytes_per_s"]),
                     sm_clock_mhz=float(g["sm_clock_mhz"]), sm_clock_max_mhz=float(g["sm_clock_max_mhz"]),
                     mem_clock_mhz=float(g["mem_clock_mhz"]), mem_clock_max_mhz=float(g["mem_clock_max_mhz"]))
    assert r["flops"] == int(g["total_flops"]) and r["bytes"] == int(g["total_bytes"])
    assert abs(r["t_sol_s"] * 1e3 - float(g["t_sol_tf32_ms"])) < 1e-3 and r["compute_bound"]
    o = orc.sol_bound(r["flops"], r["bytes"], float(g["peak_tf32_flops"]), float(g["peak_bytes_per_s"]),
                      float(g["sm_clock_mhz"]), float(g["sm_clock_max_mhz"]),
                      float(g["mem_clock_mhz"]), float(g["mem_clock_max_mhz"]))
    for k in ("ai", "t_compute_s", "t_mem_s", "t_sol_s", "ridge", "eff_peak_flops", "eff_bytes_per_s"):
        assert r[k] == pytest.approx(o[k], rel=1e-15), k


def test_sol_bound_counts_for_every_operation(sg):
    hw = dict(peak_flops=2250e12, peak_bytes_per_s=8e12)
    r = sg.sol_bound("gemm", M=4096, N=4096, K=4096, has_bias=1, **hw)
    assert (r["flops"], r["bytes"]) == (137_438_953_472, 100_671_488) and r["compute_bound"]
    assert r["t_sol_s"] == pytest.approx(137_438_953_472 / 2250e12)
    r = sg.sol_bound("batched", M=256, N=256, K=512, batch_or_groups=128, **hw)
    assert (r["flops"], r["bytes"]) == (8_589_934_592, 83_886_080) and not r["compute_bound"]
    assert r["t_sol_s"] == pytest.approx(83_886_080 / 8e12)
    conv = dict(N=32, H=56, W=56, C=256, K=256, R=3, S=3, pad=(1, 1))
    r = sg.sol_bound("conv2d", conv=conv, has_bias=1, **hw)
    assert (r["flops"], r["bytes"]) == (118_380_036_096, 103_940_608)
    assert r["flops"] == orc.conv_flops(**conv) and r["bytes"] == orc.conv_bytes(**conv, has_bias=True)
    # the gradients execute the forward problem's FLOPs; bytes: dY + Wf + dX and dY + X + dW (hand counts:
    # x = y = 25,690,112 elements, w = 589,824 elements; dW kept in fp32)
    r = sg.sol_bound("conv2d_dgrad", conv=conv, **hw)
    assert (r["flops"], r["bytes"]) == (118_380_036_096, 2 * (25_690_112 + 589_824) + 2 * 25_690_112)
    assert r["bytes"] == orc.conv_grad_bytes("dgrad", **conv)
    r = sg.sol_bound("conv2d_wgrad", conv=conv, elem_bytes_out=4, beta=1.0, **hw)
    assert (r["flops"], r["bytes"]) == (118_380_036_096, 2 * 2 * 25_690_112 + 2 * 4 * 589_824)
    assert r["bytes"] == orc.conv_grad_bytes("wgrad", **conv, eb_out=4, has_c=True)
    Ms = [128, 4096, 1000, 0]
    r = sg.sol_bound("grouped", N=4096, K=4096, batch_or_groups=4, Ms=Ms, **hw)
    assert r["flops"] == 33_554_432 * sum(Ms) and r["bytes"] == 16_384 * sum(Ms) + 4 * 33_554_432
    assert r["flops"] == sum(orc.gemm_flops(m, 4096, 4096) for m in Ms)
    assert r["bytes"] == sum(orc.gemm_bytes(m, 4096, 4096) for m in Ms)
    # beta != 0 reads C; a shared bias is counted once for a batch
    assert sg.sol_bound("gemm", M=8, N=8, K=8, beta=1.0, **hw)["bytes"] == 4 * 128
    assert sg.sol_bound("batched", M=8, N=8, K=8, batch_or_groups=3, has_bias=2, **hw)["bytes"] == 3 * 384 + 16
    assert sg.sol_bound("batched", M=8, N=8, K=8, batch_or_groups=3, has_bias=1, **hw)["bytes"] == 3 * 384 + 48
    with pytest.raises(sg.SolgemmError):
        sg.sol_bound("gemm", M=8, N=8, K=8, peak_flops=0.0, peak_bytes_per_s=1.0)


def test_gemm_host_rejects_a_missing_or_short_staging_buffer_before_touching_a_device(sg):
    lib = sg.raw_lib()
    desc = sg.GemmDesc(512, 64, 64, 0, 1, 64, 64, 64, 64, 0, 0, 1.0, 0.0, 0, 0.0, 0.0, 0)
    need = ctypes.c_size_t(0)
    assert lib.sg_gemm_host_staging_size(ctypes.byref(desc), ctypes.byref(need)) == 0
    assert need.value >= (512 * 64 + 64 * 64 + 512 * 64) * 2
    host = ctypes.c_void_p(0x1000)
    st = lib.sg_gemm_host(ctypes.byref(desc), host, host, None, None, host, None, 0, 4, None)
    assert sg.STATUS_NAMES[st] == "SG_ERR_WORKSPACE"
    st = lib.sg_gemm_host(ctypes.byref(desc), host, host, None, None, host, ctypes.c_void_p(0x10000), need.value - 1, 4, None)
    assert sg.STATUS_NAMES[st] == "SG_ERR_WORKSPACE" and str(need.value) in lib.sg_last_error().decode()
    st = lib.sg_gemm_host(ctypes.byref(desc), None, host, None, None, host, ctypes.c_void_p(0x10000), need.value, 4, None)
    assert sg.STATUS_NAMES[st] == "SG_ERR_NULL_POINTER"
