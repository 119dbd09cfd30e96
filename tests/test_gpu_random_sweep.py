"""Seeded random sweep over the entry points' argument space, every output element against the CPU oracle.

The parametrised parity tests pin chosen shapes; this module draws shapes, leading dimensions, layouts, element types,
scaling factors and epilogues from a seeded generator, so combinations nobody thought of are exercised too: odd extents
around the 64 / 128 / 256 tile edges, K = 0 and tiny K, padded leading dimensions, every A / B layout pair, bf16 and
fp16 inputs with all three output types, bias and residual on and off.  Outputs live inside NaN guard bands (rows before
and after, columns past N) that must stay NaN.  The draws are fixed by the seeds below; nothing depends on the clock.
"""
import random

import pytest
import torch

from paper_2603_29010_b200 import inputs
from tests import parity

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

from oracle import oracle as orc                      # noqa: E402
from paper_2603_29010_b200 import solgemm as sg       # noqa: E402

DEV = "cuda"
NAN = float("nan")
EPIS = ["none", "none", "relu", "gelu", "silu", "sigmoid", "tanh", "hardswish"]
EDGE = [1, 2, 7, 8, 31, 32, 33, 63, 64, 65, 127, 128, 129, 191, 255, 256, 257, 300, 383, 511, 513]


@pytest.fixture(autouse=True, params=["tiles", "own choice"])
def _clean_status(request):
    # every case twice: on the tensor-core tiles (the matrix-vector kernels kept to eight vectors, no small-product form),
    # and under the library's own choice of path
    sg.set_tuning(-1, -1)
    sg.set_tail_mode(-1)
    sg.enable_scratch(True)
    sg.set_option("gemv_small_log2", 0 if request.param == "tiles" else -1)
    sg.set_option("gemv_max_vectors", 8 if request.param == "tiles" else -1)
    yield
    torch.cuda.synchronize()
    sg.poll_status()
    sg.set_tuning(-1, -1)
    sg.set_tail_mode(-1)


def _extent(rng, hi):
    return rng.choice(EDGE) if rng.random() < 0.6 else rng.randint(1, hi)


def _pad8(n, rng):
    """A leading dimension >= n that keeps rows 16-byte aligned for 2-byte elements (and 4-byte ones)."""
    return (n + 7) // 8 * 8 + 8 * rng.choice([0, 0, 1, 3])


def _operand(rows, cols, ld, seed, tid, dtype):
    """[rows, cols] view with leading dimension ld; the padding columns hold NaN (they must never be read as data)."""
    whole = torch.full((rows, ld), NAN, dtype=dtype)
    if rows and cols:
        whole[:, :cols] = inputs.uniform([rows, cols], seed, tid).to(dtype)
    return whole[:, :cols]


def _dev(view):
    """The same view on the device, padding kept: the whole padded buffer is copied and sliced again (a plain .to() of a
    strided view would compact it)."""
    if view is None:
        return None
    base = view._base
    if base is None or base.dim() != view.dim() or view.is_contiguous():
        return view.to(DEV)
    return base.to(DEV)[tuple(slice(0, n) for n in view.shape)]


def _guarded_out(rows, cols, ld, dtype, pad_rows=4):
    whole = torch.full((rows + 2 * pad_rows, ld), NAN, dtype=dtype, device=DEV)
    return whole[pad_rows:pad_rows + rows, :cols], whole, pad_rows


def _guards_ok(whole, pad_rows, cols):
    ok = bool(torch.isnan(whole[:pad_rows]).all() and torch.isnan(whole[-pad_rows:]).all())
    if cols < whole.shape[1]:
        ok = ok and bool(torch.isnan(whole[:, cols:]).all())
    return ok


def _gemm_case(rng, seed):
    M, N = _extent(rng, 600), _extent(rng, 600)
    K = rng.choice([0, 1, 8, 63, 64, 65, 200, 520, 1031]) if rng.random() < 0.5 else rng.randint(1, 900)
    la, lb = rng.choice(["row", "col"]), rng.choice(["row", "col"])
    in_dtype = rng.choice([torch.bfloat16, torch.bfloat16, torch.float16])
    out_dtype = rng.choice([torch.bfloat16, torch.float32, torch.float16])
    a_shape = (M, K) if la == "row" else (K, M)
    b_shape = (N, K) if lb == "col" else (K, N)
    A = _operand(a_shape[0], a_shape[1], _pad8(max(a_shape[1], 1), rng), seed, 1, in_dtype)
    B = _operand(b_shape[0], b_shape[1], _pad8(max(b_shape[1], 1), rng), seed, 2, in_dtype)
    beta = rng.choice([0.0, 0.0, 1.0, -0.5])
    C = _operand(M, N, _pad8(N, rng), seed, 3, out_dtype) if beta != 0.0 else None
    bias = inputs.uniform([N], seed, 4).to(in_dtype) if rng.random() < 0.5 else None
    alpha = rng.choice([1.0, 1.0, 0.5, -1.25])
    epi = rng.choice(EPIS)
    return dict(M=M, N=N, K=K, la=la, lb=lb, A=A, B=B, C=C, bias=bias, alpha=alpha, beta=beta, epi=epi, out_dtype=out_dtype)


@pytest.mark.parametrize("case", range(160))
def test_random_gemm(case):
    rng = random.Random(7000 + case)
    c = _gemm_case(rng, 7000 + case)
    ref, absacc = orc.gemm(c["A"], c["B"], layout_a=c["la"], layout_b=c["lb"], C=c["C"], bias=c["bias"], alpha=c["alpha"],
                           beta=c["beta"], epi=c["epi"])
    out, whole, pr = _guarded_out(c["M"], c["N"], _pad8(c["N"], rng), c["out_dtype"])
    sg.gemm(_dev(c["A"]), _dev(c["B"]), C=_dev(c["C"]), bias=_dev(c["bias"]), out=out, alpha=c["alpha"], beta=c["beta"],
            epi=c["epi"], layout_a=c["la"], layout_b=c["lb"])
    what = f"gemm case {case}: {c['M']}x{c['N']}x{c['K']} {c['la']}/{c['lb']} {c['A'].dtype}->{c['out_dtype']} " \
           f"alpha={c['alpha']} beta={c['beta']} bias={c['bias'] is not None} epi={c['epi']}"
    parity.assert_matches(out, ref, absacc, what)
    assert _guards_ok(whole, pr, c["N"]), what


@pytest.mark.parametrize("case", range(32))
def test_random_batched_gemm(case):
    rng = random.Random(8000 + case)
    seed = 8000 + case
    batch = rng.randint(1, 6)
    M, N, K = _extent(rng, 300), _extent(rng, 300), rng.choice([8, 64, 72, 136, 512, 777])
    in_dtype = rng.choice([torch.bfloat16, torch.float16])
    out_dtype = rng.choice([torch.bfloat16, torch.float32])
    lda, ldb, ldd = _pad8(K, rng), _pad8(K, rng), _pad8(N, rng)
    gap = rng.choice([0, 1, 5])                           # extra rows between consecutive problems
    A = torch.full((batch, M + gap, lda), NAN, dtype=in_dtype)
    B = torch.full((batch, N + gap, ldb), NAN, dtype=in_dtype)
    A[:, :M, :K] = inputs.uniform([batch, M, K], seed, 1).to(in_dtype)
    B[:, :N, :K] = inputs.uniform([batch, N, K], seed, 2).to(in_dtype)
    A, B = A[:, :M, :K], B[:, :N, :K]
    per_batch_bias = rng.random() < 0.5
    bias = inputs.uniform([batch, N] if per_batch_bias else [N], seed, 4).to(in_dtype) if rng.random() < 0.7 else None
    epi = rng.choice(EPIS)
    alpha = rng.choice([1.0, 0.75])
    ref, absacc = orc.batched_gemm(A, B, bias=bias, alpha=alpha, epi=epi)
    whole = torch.full((batch, M + gap, ldd), NAN, dtype=out_dtype, device=DEV)
    out = whole[:, :M, :N]
    sg.batched_gemm(_dev(A), _dev(B), bias=_dev(bias), out=out, alpha=alpha, epi=epi)
    what = f"batched case {case}: {batch} x {M}x{N}x{K} gap {gap} {in_dtype}->{out_dtype} bias={bias is not None and tuple(bias.shape)} epi={epi}"
    parity.assert_matches(out, ref, absacc, what)
    assert bool(torch.isnan(whole[:, M:, :]).all()) and bool(torch.isnan(whole[:, :, N:]).all()), what


@pytest.mark.parametrize("case", range(24))
def test_random_grouped_gemm(case):
    rng = random.Random(9000 + case)
    seed = 9000 + case
    groups = rng.randint(1, 7)
    N, K = rng.choice([8, 64, 72, 200, 264]), rng.choice([8, 64, 136, 520])
    Ms = [rng.choice([0, 1, 5, 127, 128, 129, 255, 256, 257, 300]) for _ in range(groups)]
    out_dtype = rng.choice([torch.bfloat16, torch.float32])
    epi = rng.choice(EPIS)
    As = [inputs.uniform([m, K], seed + g, 1) for g, m in enumerate(Ms)]
    Bs = [inputs.uniform([N, K], seed + g, 2) for g in range(groups)]
    biases = [inputs.uniform([N], seed + g, 4) for g in range(groups)] if rng.random() < 0.5 else None
    refs, accs = orc.grouped_gemm(As, Bs, biases=biases, epi=epi)
    wholes = [torch.full((m + 8, N), NAN, dtype=out_dtype, device=DEV) for m in Ms]
    outs = [w[4:4 + m] for w, m in zip(wholes, Ms)]
    sg.grouped_gemm([a.to(DEV) for a in As], [b.to(DEV) for b in Bs],
                    biases=None if biases is None else [b.to(DEV) for b in biases], outs=outs, epi=epi)
    for g, m in enumerate(Ms):
        what = f"grouped case {case}: group {g} of {Ms} x{N}x{K} ->{out_dtype} epi={epi}"
        if m:
            parity.assert_matches(outs[g], refs[g], accs[g], what)
        assert bool(torch.isnan(wholes[g][:4]).all()) and bool(torch.isnan(wholes[g][4 + m:]).all()), what


@pytest.mark.parametrize("case", range(32))
def test_random_conv2d_fprop(case):
    rng = random.Random(10000 + case)
    seed = 10000 + case
    N, H, W = rng.randint(1, 3), rng.randint(3, 19), rng.randint(3, 19)
    C, K = rng.choice([8, 16, 24, 64, 72, 136]), rng.choice([8, 24, 64, 80, 264])
    R, S = rng.randint(1, 3), rng.randint(1, 3)
    pad = (rng.randint(0, 2), rng.randint(0, 2))
    stride = (rng.randint(1, 2), rng.randint(1, 2))
    dil = (rng.randint(1, 2), rng.randint(1, 2))
    if orc.conv_out_extent(H, pad[0], dil[0], R, stride[0]) < 1 or orc.conv_out_extent(W, pad[1], dil[1], S, stride[1]) < 1:
        pytest.skip("empty output for this draw")
    out_dtype = rng.choice([torch.bfloat16, torch.float32])
    X, Wf, bias = inputs.make_conv(N, H, W, C, K, R, S, "uniform", 1.0, bias=True, seed=seed)
    if rng.random() < 0.4:
        bias = None
    epi = rng.choice(EPIS)
    alpha = rng.choice([1.0, 0.5])
    ref, absacc = orc.conv2d_fprop(X, Wf, pad=pad, stride=stride, dil=dil, bias=bias, alpha=alpha, epi=epi)
    P, Q = ref.shape[1], ref.shape[2]
    whole = torch.full((N * P * Q + 8, K), NAN, dtype=out_dtype, device=DEV)
    out = whole[4:4 + N * P * Q].view(N, P, Q, K)
    sg.conv2d_fprop(X.to(DEV), Wf.to(DEV), pad=pad, stride=stride, dil=dil, bias=None if bias is None else bias.to(DEV),
                    alpha=alpha, epi=epi, out=out)
    what = f"conv case {case}: N{N} {H}x{W} C{C} K{K} {R}x{S} pad{pad} stride{stride} dil{dil} ->{out_dtype} epi={epi}"
    parity.assert_matches(out, ref, absacc, what)
    assert bool(torch.isnan(whole[:4]).all()) and bool(torch.isnan(whole[-4:]).all()), what


def _grad_geometry(rng):
    N, H, W = rng.randint(1, 3), rng.randint(4, 17), rng.randint(4, 17)
    C, K = rng.choice([8, 16, 64, 72, 136]), rng.choice([8, 24, 64, 80, 136])
    R, S = rng.randint(1, 3), rng.randint(1, 3)
    pad = (rng.randint(0, 1), rng.randint(0, 1))
    stride = (rng.randint(1, 2), rng.randint(1, 2))
    dil = (rng.randint(1, 2), rng.randint(1, 2))
    P = orc.conv_out_extent(H, pad[0], dil[0], R, stride[0])
    Q = orc.conv_out_extent(W, pad[1], dil[1], S, stride[1])
    return N, H, W, C, K, R, S, pad, stride, dil, P, Q


@pytest.mark.parametrize("case", range(24))
def test_random_conv2d_dgrad(case):
    rng = random.Random(11000 + case)
    seed = 11000 + case
    N, H, W, C, K, R, S, pad, stride, dil, P, Q = _grad_geometry(rng)
    if P < 1 or Q < 1:
        pytest.skip("empty output for this draw")
    out_dtype = rng.choice([torch.bfloat16, torch.float32])
    dY = inputs.uniform([N, P, Q, K], seed, 1)
    Wf = inputs.uniform([K, R, S, C], seed, 2)
    ref, absacc = orc.conv2d_dgrad(dY, Wf, (H, W), pad=pad, stride=stride, dil=dil)
    whole = torch.full((N * H * W + 8, C), NAN, dtype=out_dtype, device=DEV)
    out = whole[4:4 + N * H * W].view(N, H, W, C)
    sg.conv2d_dgrad(dY.to(DEV), Wf.to(DEV), (H, W), pad=pad, stride=stride, dil=dil, out=out)
    what = f"dgrad case {case}: N{N} {H}x{W} C{C} K{K} {R}x{S} pad{pad} stride{stride} dil{dil} ->{out_dtype}"
    parity.assert_matches(out, ref, absacc, what)
    assert bool(torch.isnan(whole[:4]).all()) and bool(torch.isnan(whole[-4:]).all()), what


@pytest.mark.parametrize("case", range(24))
def test_random_conv2d_wgrad(case):
    rng = random.Random(12000 + case)
    seed = 12000 + case
    N, H, W, C, K, R, S, pad, stride, dil, P, Q = _grad_geometry(rng)
    if P < 1 or Q < 1:
        pytest.skip("empty output for this draw")
    dY = inputs.uniform([N, P, Q, K], seed, 1)
    X = inputs.uniform([N, H, W, C], seed, 2)
    ref, absacc = orc.conv2d_wgrad(dY, X, (R, S), pad=pad, stride=stride, dil=dil)
    whole = torch.full((K * R * S + 8, C), NAN, dtype=torch.float32, device=DEV)
    out = whole[4:4 + K * R * S].view(K, R, S, C)
    sg.conv2d_wgrad(dY.to(DEV), X.to(DEV), (R, S), pad=pad, stride=stride, dil=dil, out=out)
    what = f"wgrad case {case}: N{N} {H}x{W} C{C} K{K} {R}x{S} pad{pad} stride{stride} dil{dil}"
    parity.assert_matches(out, ref, absacc, what)
    assert bool(torch.isnan(whole[:4]).all()) and bool(torch.isnan(whole[-4:]).all()), what


@pytest.mark.parametrize("case", range(40))
def test_random_skinny_long_k(case):
    # few output tiles and a long contraction: the planner's K-range forms (two-pass, early donors), the short-A
    # variants and the matrix-vector kernels (at most eight rows or columns) on extents nobody picked by hand
    rng = random.Random(13000 + case)
    seed = 13000 + case
    M = rng.choice([1, 2, 3, 5, 8, 9, 16, 31, 64, 100, 128, 129, 200, 256, 260])
    N = rng.choice([1, 2, 4, 7, 8, 9, 24, 64, 72, 128, 136, 256, 264])
    K = 8 * rng.randint(250, 4100)
    in_dtype = rng.choice([torch.bfloat16, torch.float16])
    out_dtype = rng.choice([torch.bfloat16, torch.float32])
    A = _operand(M, K, _pad8(K, rng), seed, 1, in_dtype)
    B = _operand(N, K, _pad8(K, rng), seed, 2, in_dtype)
    bias = inputs.uniform([N], seed, 4).to(in_dtype) if rng.random() < 0.5 else None
    epi = rng.choice(["none", "relu", "gelu"])
    alpha = rng.choice([1.0, 2.0 ** -5])
    ref, absacc = orc.gemm(A, B, bias=bias, alpha=alpha, epi=epi)
    out, whole, pr = _guarded_out(M, N, _pad8(N, rng), out_dtype)
    sg.gemm(_dev(A), _dev(B), bias=_dev(bias), out=out, alpha=alpha, epi=epi)
    plan = sg.last_launch_plan()
    what = f"skinny case {case}: {M}x{N}x{K} {in_dtype}->{out_dtype} alpha={alpha} bias={bias is not None} epi={epi} plan={plan}"
    parity.assert_matches(out, ref, absacc, what)
    assert _guards_ok(whole, pr, N), what


@pytest.mark.parametrize("case", range(24))
def test_random_multi_wave(case):
    # more tiles than SMs, under the planner's own choice or a forced tile shape and tail mode: the persistent tile walk,
    # the raster, tail slices and K ranges on ragged extents
    rng = random.Random(14000 + case)
    seed = 14000 + case
    M, N = rng.randint(700, 2000), rng.randint(700, 2000)
    K = 8 * rng.randint(8, 140)
    la, lb = rng.choice([("row", "col"), ("row", "col"), ("col", "col"), ("row", "row"), ("col", "row")])
    out_dtype = rng.choice([torch.bfloat16, torch.float32])
    a_shape = (M, K) if la == "row" else (K, M)
    b_shape = (N, K) if lb == "col" else (K, N)
    A = _operand(a_shape[0], a_shape[1], _pad8(a_shape[1], rng), seed, 1, torch.bfloat16)
    B = _operand(b_shape[0], b_shape[1], _pad8(b_shape[1], rng), seed, 2, torch.bfloat16)
    bias = inputs.uniform([N], seed, 4) if rng.random() < 0.5 else None
    beta = rng.choice([0.0, 1.0])
    C = _operand(M, N, _pad8(N, rng), seed, 3, out_dtype) if beta != 0.0 else None
    epi = rng.choice(["none", "relu", "silu"])
    tile_n, pair = rng.choice([(-1, -1), (-1, -1), (64, 0), (128, 0), (256, 0), (128, 1), (256, 1)])
    tail = rng.choice([-1, -1, 0, 1, 2])
    sg.set_tuning(tile_n, pair)
    sg.set_tail_mode(tail)
    ref, absacc = orc.gemm(A, B, layout_a=la, layout_b=lb, C=C, bias=bias, beta=beta, epi=epi)
    out, whole, pr = _guarded_out(M, N, _pad8(N, rng), out_dtype)
    sg.gemm(_dev(A), _dev(B), C=_dev(C), bias=_dev(bias), out=out, beta=beta, epi=epi, layout_a=la, layout_b=lb)
    what = f"multi-wave case {case}: {M}x{N}x{K} {la}/{lb} ->{out_dtype} beta={beta} bias={bias is not None} epi={epi} " \
           f"forced tile {tile_n}/{pair} tail {tail} plan={sg.last_launch_plan()}"
    parity.assert_matches(out, ref, absacc, what)
    assert _guards_ok(whole, pr, N), what
