"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same seeded inputs.

Integer-valued problems must match bit for bit (every partial sum is exact in
fp32 and the result is exact in the output type, so accumulation order cannot
matter); real-valued problems must match within the stated tolerance on every
element (small shapes) or on tile-edge rows plus seeded samples (full-size shapes).
"""
import math

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


@pytest.fixture(autouse=True)
def _clean_status():
    sg.set_tuning(-1, -1)
    sg.set_tail_mode(-1)
    sg.enable_scratch(True)
    yield
    torch.cuda.synchronize()
    sg.poll_status()          # raises if any kernel recorded an expired wait
    sg.set_tuning(-1, -1)
    sg.set_tail_mode(-1)
    sg.enable_scratch(True)


def guarded(shape, dtype, pad_rows=8):
    """An output buffer with NaN guard bands before and after; returns (view, whole)."""
    rows, cols = shape[-2], shape[-1]
    lead = int(math.prod(shape[:-2])) if len(shape) > 2 else 1
    if cols % 8 == 0:
        whole = torch.full((lead * rows + 2 * pad_rows, cols), float("nan"), dtype=dtype, device=DEV)
        view = whole[pad_rows:pad_rows + lead * rows].view(*shape)
        return view, whole
    assert len(shape) == 2                    # ragged width: pad the leading dimension to the 16-byte rule
    whole = torch.full((rows + 2 * pad_rows, (cols + 15) // 8 * 8), float("nan"), dtype=dtype, device=DEV)
    return whole[pad_rows:pad_rows + rows, :cols], whole


def guards_intact(whole, pad_rows=8, cols=None):
    ok = bool(torch.isnan(whole[:pad_rows]).all() and torch.isnan(whole[-pad_rows:]).all())
    if cols is not None and cols < whole.shape[1]:
        ok = ok and bool(torch.isnan(whole[:, cols:]).all())
    return ok


SHAPES_EXACT = [(128, 64, 64), (256, 256, 256), (300, 200, 136), (129, 72, 8), (1000, 520, 328), (17, 8, 200),
                (640, 768, 1024)]
TILINGS = [(64, 0), (128, 0), (256, 0), (64, 1), (128, 1), (256, 1)]


@pytest.mark.parametrize("tile_n,pair", TILINGS)
@pytest.mark.parametrize("M,N,K", SHAPES_EXACT)
def test_gemm_integer_inputs_bit_exact(M, N, K, tile_n, pair):
    sg.set_tuning(tile_n, pair)
    A = inputs.small_integers([M, K], 101, 1)
    B = inputs.small_integers([N, K], 101, 2)
    ref, _ = orc.gemm(A, B)
    assert float(ref.abs().max()) <= 256
    D, whole = guarded((M, N), torch.bfloat16)
    sg.gemm(A.to(DEV), B.to(DEV), out=D)
    parity.assert_bit_exact(D, ref, f"gemm {M}x{N}x{K} tile_n={tile_n} pair={pair}")
    assert guards_intact(whole)


LAYOUT_TILINGS = [(64, 0), (128, 0), (256, 0), (128, 1), (256, 1), (-1, -1)]


@pytest.mark.parametrize("tile_n,pair", LAYOUT_TILINGS)
@pytest.mark.parametrize("la,lb", [("row", "row"), ("col", "col"), ("col", "row")])
@pytest.mark.parametrize("M,N,K", [(256, 256, 256), (300, 200, 136), (129, 72, 8), (1000, 520, 328), (128 * 149, 136, 72)])
def test_gemm_other_operand_layouts_bit_exact(M, N, K, la, lb, tile_n, pair):
    # column-major A and/or row-major B: the M- or N-contiguous operand goes through the MN-major descriptor
    sg.set_tuning(tile_n, pair)
    Am = inputs.small_integers([M, K + 8], 111, 1)[:, :K]
    Bm = inputs.small_integers([K, N + 8], 111, 2)[:, :N]
    ref = Am.double() @ Bm.double()
    assert float(ref.abs().max()) <= 256
    def stored(mat, transposed):
        """The matrix as stored (transposed for a column-major A / B), leading dimension padded to 8 elements."""
        m = mat.t() if transposed else mat
        buf = torch.zeros(m.shape[0], (m.shape[1] + 7) // 8 * 8 + 8, dtype=torch.bfloat16)
        buf[:, :m.shape[1]] = m
        return buf, m.shape[1]
    Abuf, a_cols = stored(Am, la == "col")                               # stored [M,K] or [K,M]
    Bbuf, b_cols = stored(Bm, lb == "col")                               # stored [K,N] or [N,K]
    oref, _ = orc.gemm(Abuf[:, :a_cols], Bbuf[:, :b_cols], layout_a=la, layout_b=lb)
    assert torch.equal(oref, ref)
    D, whole = guarded((M, N), torch.bfloat16)
    sg.gemm(Abuf.to(DEV)[:, :a_cols], Bbuf.to(DEV)[:, :b_cols], out=D, layout_a=la, layout_b=lb)
    parity.assert_bit_exact(D, ref, f"layouts {la}/{lb} {M}x{N}x{K} tiling {sg.last_launch_plan()}")
    assert guards_intact(whole, cols=N)


def test_other_layouts_with_padded_leading_dimensions_batched_and_grouped():
    batch, M, N, K = 3, 200, 136, 72
    Ast = inputs.small_integers([batch, K, M + 24], 121, 1)             # column-major A: [K, M] with lda = M + 24
    Bst = inputs.small_integers([batch, K, N + 8], 121, 2)              # row-major B:    [K, N] with ldb = N + 8
    A, B = Ast[:, :, :M], Bst[:, :, :N]
    ref, absacc = orc.batched_gemm(A, B, layout_a="col", layout_b="row", epi="relu")
    D = sg.batched_gemm(Ast.to(DEV)[:, :, :M], Bst.to(DEV)[:, :, :N], layout_a="col", layout_b="row", epi="relu")
    parity.assert_bit_exact(D, ref, "batched col/row")
    # grouped: row-major A (ragged M), row-major B
    Ms = [130, 257, 64]
    As = [inputs.small_integers([m, K], 131 + g, 1) for g, m in enumerate(Ms)]
    Bs = [inputs.small_integers([K, N], 131 + g, 2) for g in range(len(Ms))]
    refs, _ = orc.grouped_gemm(As, Bs, layout_a="row", layout_b="row")
    outs = sg.grouped_gemm([a.to(DEV) for a in As], [b.to(DEV) for b in Bs], layout_a="row", layout_b="row")
    for g in range(len(Ms)):
        parity.assert_bit_exact(outs[g], refs[g], f"grouped row/row group {g}")
    # grouped: column-major A (every A_g stored [K, M_g] with one common leading dimension), both B layouts
    lda = 264
    Acs = [inputs.small_integers([K, lda], 141 + g, 1) for g in range(len(Ms))]
    for lb, Bg in (("row", Bs), ("col", [b.t().contiguous() for b in Bs])):
        refs, _ = orc.grouped_gemm([a[:, :m] for a, m in zip(Acs, Ms)], Bg, layout_a="col", layout_b=lb)
        outs = sg.grouped_gemm([a.to(DEV)[:, :m] for a, m in zip(Acs, Ms)], [b.to(DEV) for b in Bg], layout_a="col", layout_b=lb)
        for g in range(len(Ms)):
            parity.assert_bit_exact(outs[g], refs[g], f"grouped col/{lb} group {g}")


@pytest.mark.parametrize("pair", [0, 1])
@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("epi", ["none", "bias", "relu", "gelu", "silu"])
def test_gemm_epilogues_alpha_beta_bias(epi, out_dtype, pair):
    sg.set_tuning(128, pair)
    M, N, K = 200, 328, 264
    A, B, bias = inputs.make_gemm(M, N, K, "normal", K ** -0.25, bias=True, seed=202)
    C = inputs.normal([M, N], 202, 3).to(out_dtype)
    ref, absacc = orc.gemm(A, B, C=C, bias=bias, alpha=0.75, beta=-0.5, epi=epi)
    D = sg.gemm(A.to(DEV), B.to(DEV), C=C.to(DEV), bias=bias.to(DEV), out_dtype=out_dtype, alpha=0.75, beta=-0.5, epi=epi)
    parity.assert_matches(D, ref, absacc, f"gemm epi={epi} {out_dtype}")
    if epi != "bias":
        ref2, acc2 = orc.gemm(A, B, epi=epi)
        D2 = sg.gemm(A.to(DEV), B.to(DEV), out_dtype=out_dtype, epi=epi)
        parity.assert_matches(D2, ref2, acc2, f"gemm epi={epi} no bias {out_dtype}")


FURTHER_ACTS = [("sigmoid", (0.0, 0.0)), ("tanh", (0.0, 0.0)), ("mish", (0.0, 0.0)), ("hardswish", (0.0, 0.0)),
                ("leaky_relu", (0.125, 0.0)), ("elu", (1.5, 0.0)), ("clip", (-0.5, 2.0))]


@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("epi,args", FURTHER_ACTS)
def test_further_builtin_activations(epi, args, out_dtype):
    M, N, K = 200, 136, 264
    A, B, bias = inputs.make_gemm(M, N, K, "normal", K ** -0.25, bias=True, seed=515)
    ref, absacc = orc.gemm(A, B, bias=bias, alpha=1.5, epi=epi, epi_args=args)
    D = sg.gemm(A.to(DEV), B.to(DEV), bias=bias.to(DEV), alpha=1.5, epi=epi, epi_args=args, out_dtype=out_dtype)
    parity.assert_matches(D, ref, absacc, f"{epi} {out_dtype}")
    # K = 1 on the fp32 path: D = act(x) judged at 1e-4 |x|, over a range that reaches every branch
    x = torch.linspace(-9, 9, 512, dtype=torch.float64).to(torch.bfloat16).view(-1, 1)
    a = torch.zeros(512, 8, dtype=torch.bfloat16)
    a[:, :1] = x
    b = torch.zeros(8, 8, dtype=torch.bfloat16)
    b[:, 0] = 1
    ref1, acc1 = orc.gemm(a, b, epi=epi, epi_args=args)
    D1 = sg.gemm(a.to(DEV), b.to(DEV), out_dtype=torch.float32, epi=epi, epi_args=args)
    parity.assert_matches(D1, ref1, acc1, f"{epi} pointwise fp32")
    Dbf = sg.gemm(a.to(DEV), b.to(DEV), epi=epi, epi_args=args)
    parity.assert_matches(Dbf, ref1, acc1, f"{epi} pointwise bf16")


def test_further_activations_through_conv_batched_and_grouped():
    X, Wf, cb = inputs.make_conv(2, 9, 10, 40, 72, 3, 3, "normal", (40 * 9) ** -0.25, bias=True, seed=525)
    ref, absacc = orc.conv2d_fprop(X, Wf, pad=(1, 1), bias=cb, epi="clip", epi_args=(0.0, 6.0))
    Y = sg.conv2d_fprop(X.to(DEV), Wf.to(DEV), pad=(1, 1), bias=cb.to(DEV), epi="clip", epi_args=(0.0, 6.0))
    parity.assert_matches(Y, ref, absacc, "conv + bias + clip(0, 6)")
    A = inputs.uniform([3, 72, 136], 535, 1)
    B = inputs.uniform([3, 64, 136], 535, 2)
    ref, absacc = orc.batched_gemm(A, B, epi="leaky_relu", epi_args=(0.01, 0.0))
    D = sg.batched_gemm(A.to(DEV), B.to(DEV), epi="leaky_relu", epi_args=(0.01, 0.0), out_dtype=torch.float32)
    parity.assert_matches(D, ref, absacc, "batched leaky_relu")
    As, Bs = inputs.make_grouped([40, 130], 72, 136, "normal", 136 ** -0.25, seed=545)
    refs, accs = orc.grouped_gemm(As, Bs, epi="mish")
    outs = sg.grouped_gemm([a.to(DEV) for a in As], [b.to(DEV) for b in Bs], epi="mish")
    for g in range(2):
        parity.assert_matches(outs[g], refs[g], accs[g], f"grouped mish {g}")


def test_gemm_activation_form_is_pinned_on_the_fp32_path():
    # K = 1: D = act(x), tolerance 1e-4 |x| -- tight enough to tell tanh-GELU from erf-GELU
    x = torch.linspace(-6, 6, 256, dtype=torch.float64).to(torch.bfloat16).view(-1, 1)
    a = torch.zeros(256, 8, dtype=torch.bfloat16)
    a[:, :1] = x
    b = torch.zeros(8, 8, dtype=torch.bfloat16)
    b[:, 0] = 1
    for epi in ("gelu", "silu", "relu"):
        ref, absacc = orc.gemm(a, b, epi=epi)
        D = sg.gemm(a.to(DEV), b.to(DEV), out_dtype=torch.float32, epi=epi)
        parity.assert_matches(D, ref, absacc, epi)


@pytest.mark.parametrize("scratch", [0, 2])
@pytest.mark.parametrize("tile_n,pair,M,N,K", [(256, 0, 128 * 149, 200, 72), (256, 0, 128 * 149, 190, 72),
                                              (256, 1, 256 * 75, 190, 136), (128, 0, 128 * 149, 136, 72),
                                              (128, 1, 256 * 77, 100, 64), (256, 1, 256 * 75, 192, 1024),
                                              (256, 1, 256 * 98, 256, 192), (256, 0, 128 * 170, 264, 328)])
def test_gemm_tail_wave_is_shared_between_sms(tile_n, pair, M, N, K, scratch):
    # A few tiles more than a whole number of waves.  Without a scratch buffer the planner cuts the last wave's
    # tiles into narrower column slices; with one it cuts their K loop into ranges whose fp32 partial sums the
    # owner of the tile adds up.  Integer inputs: either way the result must be exact.
    sg.enable_scratch(scratch == 2)
    sg.set_tail_mode(1 if scratch == 0 else 2)
    sg.set_tuning(tile_n, pair)
    A = inputs.small_integers([M, K], 313, 1)
    B = inputs.small_integers([N, K], 313, 2)
    ref, _ = orc.gemm(A, B)
    assert float(ref.abs().max()) <= 256
    D, whole = guarded((M, N), torch.bfloat16)
    dA, dB = A.to(DEV), B.to(DEV)
    for _ in range(2):                    # twice: the K-split counters must be back at zero after a launch
        D.fill_(float("nan"))
        sg.gemm(dA, dB, out=D)
        plan = sg.last_launch_plan()
        assert plan["tiles"] > plan["split_begin"], plan
        if not scratch or K <= 64:
            assert plan["tail_split"] > 1, plan            # column slices (a single k-block cannot be cut)
        else:
            assert plan["tail_split"] < -1, plan           # K ranges
        parity.assert_bit_exact(D, ref, f"tail split {plan}")
        assert guards_intact(whole, cols=N)


@pytest.mark.parametrize("tile_n,pair,M,N,K,ks", [
    (256, 1, 256 * 150, 256, 1024, 2),         # 150 pair tiles on 74 pairs: two waves + 2 tiles, 2 ranges of 8 k-blocks
    (256, 1, 256 * 149 + 77, 200, 2048, 4),    # ragged rows and columns, 4 ranges of 8 k-blocks
    (256, 1, 256 * 79, 512, 1536, 3),          # 158 tiles: two waves + 10 tiles, 3 ranges
    (128, 0, 128 * 149, 256, 1024, 2),         # single-CTA tiles: 298 tiles on 148 SMs
    (128, 0, 128 * 149 + 5, 200, 2056, 3),     # 150 x 2 = 300 tiles on 148 SMs, ragged rows and columns, K tail of 8
    (64, 1, 256 * 150, 64, 1024, 2),           # narrow pair tiles
])
def test_k_ranges_with_early_donors_bit_exact(tile_n, pair, M, N, K, ks):
    # The tiles of the last, partial wave have their K loop cut into ks ranges; the first ks - 1 ranges run as the very
    # first items of CTAs of their own and park their sums, which the CTA that runs the last range at the end finds in
    # its accumulator.
    # Integer inputs and fp32 output: whatever the summation order, the result must be exact.  Twice in a row: the
    # arrival counters must be back at zero after a launch.
    sg.set_tuning(tile_n, pair)
    sg.set_option("early_donors", ks)
    try:
        A = inputs.small_integers([M, K], 343, 1)
        B = inputs.small_integers([N, K], 343, 2)
        bias = inputs.small_integers([N], 343, 4, -3, 3)
        ref, _ = orc.gemm(A, B, bias=bias, alpha=2.0, epi="relu")
        dA, dB, db = A.to(DEV), B.to(DEV), bias.to(DEV)
        D, whole = guarded((M, N), torch.float32)
        for _ in range(2):
            D.fill_(float("nan"))
            sg.gemm(dA, dB, bias=db, alpha=2.0, epi="relu", out=D)
            plan = sg.last_launch_plan()
            assert plan["tail_split"] == -ks, plan
            assert plan["split_begin"] > plan["tiles"] - plan["split_begin"], plan      # owner parts sit at the list's end
            parity.assert_bit_exact(D, ref, f"early donors {plan}")
            assert guards_intact(whole, cols=N)
    finally:
        sg.set_option("early_donors", -1)


def test_k_ranges_with_early_donors_conv_and_real_values():
    # the convolution path (151 pair tiles of 256 pixels x 256 filters on 74 pairs; 18 k-blocks in 2 ranges) ...
    sg.set_tuning(256, 1)
    sg.set_option("early_donors", 2)
    try:
        X = inputs.small_integers([4, 98, 98, 128], 353, 6, -1, 1)
        Wf = inputs.small_integers([256, 3, 3, 128], 353, 7, -1, 1) * (inputs.small_integers([256, 3, 3, 128], 354, 7, 0, 2) == 0).to(torch.bfloat16)
        ref, _ = orc.conv2d_fprop(X, Wf, pad=(1, 1))
        Y = sg.conv2d_fprop(X.to(DEV), Wf.to(DEV), pad=(1, 1), out_dtype=torch.float32)
        assert sg.last_launch_plan()["tail_split"] == -2 and sg.last_kernel_name().endswith(", 9>")
        parity.assert_bit_exact(Y.view(-1, 256), ref.reshape(-1, 256), "conv early donors")
        # ... and a dense problem with real values, residual, bias and GELU in bf16
        M, N, K = 256 * 75, 320, 1544                     # 75 x 2 = 150 tiles
        A, B, bias = inputs.make_gemm(M, N, K, "normal", K ** -0.25, bias=True, seed=363)
        C = inputs.normal([M, N], 363, 3)
        ref, absacc = orc.gemm(A, B, C=C, bias=bias, alpha=1.25, beta=0.5, epi="gelu")
        D = sg.gemm(A.to(DEV), B.to(DEV), C=C.to(DEV), bias=bias.to(DEV), alpha=1.25, beta=0.5, epi="gelu")
        assert sg.last_launch_plan()["tail_split"] == -2
        parity.assert_matches(D, ref, absacc, "early donors, real values")
    finally:
        sg.set_option("early_donors", -1)


@pytest.mark.parametrize("tile_n,pair", [(-1, -1), (64, 0), (128, 0), (256, 0), (128, 1), (256, 1)])
@pytest.mark.parametrize("batch,M,N,K", [(1, 256, 256, 8192), (1, 300, 200, 4104), (3, 130, 72, 2048), (1, 17, 264, 16384)])
def test_two_pass_split_k_bit_exact(batch, M, N, K, tile_n, pair):
    # A few tiles and a long K loop: the K loop is cut into many ranges, every part parks its sums, and a second kernel
    # adds them up and runs the epilogue.  Integer inputs with sparse A so that every sum stays exact in bf16 too.
    sg.set_tuning(tile_n, pair)
    A = inputs.small_integers([batch, M, K], 373, 1) * (inputs.small_integers([batch, M, K], 374, 1, 0, 31) == 0).to(torch.bfloat16)
    B = inputs.small_integers([batch, N, K], 373, 2)
    bias = inputs.small_integers([N], 373, 4, -3, 3)
    C = inputs.small_integers([batch, M, N], 373, 3, -2, 2)
    for out_dtype in (torch.bfloat16, torch.float32):
        ref = torch.stack([orc.gemm(A[b], B[b], C=C[b].to(out_dtype), bias=bias, alpha=2.0, beta=1.0, epi="relu")[0] for b in range(batch)])
        assert float(ref.abs().max()) <= 256
        D, whole = guarded((batch, M, N) if N % 8 == 0 else (M, N), out_dtype)
        if batch > 1 or N % 8 == 0:
            for _ in range(2):
                D.fill_(float("nan"))
                if batch == 1:
                    sg.gemm(A[0].to(DEV), B[0].to(DEV), C=C[0].to(out_dtype).to(DEV), bias=bias.to(DEV), alpha=2.0, beta=1.0,
                            epi="relu", out=D[0] if D.dim() == 3 else D)
                else:
                    sg.batched_gemm(A.to(DEV), B.to(DEV), C=C.to(out_dtype).to(DEV), bias=bias.to(DEV), alpha=2.0, beta=1.0,
                                    epi="relu", out=D)
                plan = sg.last_launch_plan()
                assert plan["tail_split"] < -1, plan
                parity.assert_bit_exact(D, ref, f"two-pass split-K {plan}")
                assert guards_intact(whole, cols=N)


def test_two_pass_split_k_real_values_and_part_counts():
    # real values, GELU, fp32 and bf16 outputs, and the number of parts pinned to 2, 5 and "as many as fit"
    M, N, K = 256, 384, 16384 + 8
    A, B, bias = inputs.make_gemm(M, N, K, "normal", K ** -0.25, bias=True, seed=383)
    ref, absacc = orc.gemm(A, B, bias=bias, alpha=0.75, epi="gelu")
    try:
        for parts in (2, 5, -1):
            sg.set_option("two_pass_split_k", parts)
            for out_dtype in (torch.bfloat16, torch.float32):
                D = sg.gemm(A.to(DEV), B.to(DEV), bias=bias.to(DEV), alpha=0.75, epi="gelu", out_dtype=out_dtype)
                plan = sg.last_launch_plan()
                assert plan["tail_split"] < -1 and (parts < 0 or plan["tail_split"] == -parts), plan
                parity.assert_matches(D, ref, absacc, f"two-pass {parts} parts {out_dtype}")
        sg.set_option("two_pass_split_k", 0)            # off: the one-kernel exchange through the scratch
        D = sg.gemm(A.to(DEV), B.to(DEV), bias=bias.to(DEV), alpha=0.75, epi="gelu")
        parity.assert_matches(D, ref, absacc, "one-kernel K ranges")
    finally:
        sg.set_option("two_pass_split_k", -1)


def test_k_split_tail_with_full_epilogue_matches_oracle():
    sg.set_tuning(256, 1)
    sg.set_tail_mode(2)
    M, N, K = 256 * 76, 320, 520                          # 152 tiles on 74 pairs: 4 tail tiles; K tail of 8
    A, B, bias = inputs.make_gemm(M, N, K, "normal", K ** -0.25, bias=True, seed=333)
    C = inputs.normal([M, N], 333, 3)
    ref, absacc = orc.gemm(A, B, C=C, bias=bias, alpha=1.25, beta=0.5, epi="gelu")
    for out_dtype in (torch.bfloat16, torch.float32):
        D = sg.gemm(A.to(DEV), B.to(DEV), C=C.to(out_dtype).to(DEV), bias=bias.to(DEV), alpha=1.25, beta=0.5, epi="gelu",
                    out_dtype=out_dtype)
        assert sg.last_launch_plan()["tail_split"] < -1
        refd, accd = (ref, absacc) if out_dtype == torch.bfloat16 else orc.gemm(A, B, C=C.float(), bias=bias, alpha=1.25, beta=0.5, epi="gelu")
        parity.assert_matches(D, refd, accd, f"K-split tail {out_dtype}")


@pytest.mark.parametrize("out_dtype,N", [(torch.bfloat16, 90), (torch.float32, 90), (torch.float32, 67), (torch.bfloat16, 9)])
def test_ragged_columns_never_touch_memory_past_n(out_dtype, N):
    M, K = 150, 72
    A, B = inputs.small_integers([M, K], 323, 1), inputs.small_integers([N, K], 323, 2)
    ref, _ = orc.gemm(A, B)
    ld = (N + 15) // 8 * 8
    big = torch.full((M, ld), float("nan"), dtype=out_dtype, device=DEV)
    sg.gemm(A.to(DEV), B.to(DEV), out=big[:, :N])
    parity.assert_bit_exact(big[:, :N], ref, "ragged N")
    assert bool(torch.isnan(big[:, N:]).all())
    # the same through the batched and grouped entry points
    bigb = torch.full((2, M, ld), float("nan"), dtype=out_dtype, device=DEV)
    sg.batched_gemm(torch.stack([A, A]).to(DEV), torch.stack([B, B]).to(DEV), out=bigb[:, :, :N])
    assert bool(torch.isnan(bigb[:, :, N:]).all())
    parity.assert_bit_exact(bigb[1, :, :N], ref, "ragged N batched")
    bigg = torch.full((M, ld), float("nan"), dtype=out_dtype, device=DEV)
    sg.grouped_gemm([A.to(DEV)], [B.to(DEV)], outs=[bigg[:, :N]])
    assert bool(torch.isnan(bigg[:, N:]).all())
    parity.assert_bit_exact(bigg[:, :N], ref, "ragged N grouped")


def test_gemm_leading_dimensions_and_k_tail():
    M, N, K = 150, 90, 100                      # K not a multiple of 64, N not a multiple of 8
    bigA = inputs.small_integers([M, K + 28], 303, 1)
    bigB = inputs.small_integers([N, K + 4], 303, 2)
    ref, _ = orc.gemm(bigA[:, :K], bigB[:, :K])
    dA, dB = bigA.to(DEV), bigB.to(DEV)
    bigD = torch.full((M, 104), float("nan"), dtype=torch.bfloat16, device=DEV)
    sg.gemm(dA[:, :K], dB[:, :K], out=bigD[:, :N])
    parity.assert_bit_exact(bigD[:, :N], ref, "padded leading dimensions")
    assert bool(torch.isnan(bigD[:, N:]).all())


def test_gemm_k_zero_and_empty():
    bias = inputs.normal([16], 404, 4)
    A = torch.zeros(40, 0, dtype=torch.bfloat16)
    B = torch.zeros(16, 0, dtype=torch.bfloat16)
    C = inputs.normal([40, 16], 404, 3)
    ref, absacc = orc.gemm(A, B, C=C, bias=bias, beta=2.0, epi="relu")
    dA = torch.zeros(40, 8, dtype=torch.bfloat16, device=DEV)[:, :0]
    dB = torch.zeros(16, 8, dtype=torch.bfloat16, device=DEV)[:, :0]
    D = sg.gemm(dA, dB, C=C.to(DEV), bias=bias.to(DEV), beta=2.0, epi="relu")
    parity.assert_matches(D, ref, absacc, "K == 0")
    launches = sg.launch_count()
    untouched = torch.full((0, 16), 1.0, dtype=torch.bfloat16, device=DEV)
    sg.gemm(torch.zeros(0, 8, dtype=torch.bfloat16, device=DEV), torch.zeros(16, 8, dtype=torch.bfloat16, device=DEV),
            out=untouched)
    assert sg.launch_count() == launches        # M == 0: nothing launched


def test_gemm_beta_zero_never_reads_c():
    M, N, K = 64, 64, 64
    A, B = inputs.small_integers([M, K], 505, 1), inputs.small_integers([N, K], 505, 2)
    ref, _ = orc.gemm(A, B)
    nan_c = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=DEV)
    D = sg.gemm(A.to(DEV), B.to(DEV), C=nan_c, beta=0.0)
    parity.assert_bit_exact(D, ref, "beta == 0 with NaN C")


def test_same_pointers_new_contents_and_side_stream():
    # nothing may be cached by pointer; work must run on the caller's stream, in order
    M, N, K = 256, 128, 192
    dA = torch.empty(M, K, dtype=torch.bfloat16, device=DEV)
    dB = torch.empty(N, K, dtype=torch.bfloat16, device=DEV)
    dD = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
    side = torch.cuda.Stream()
    for seed in (1, 2, 3):
        A, B = inputs.small_integers([M, K], seed, 1), inputs.small_integers([N, K], seed, 2)
        ref, _ = orc.gemm(A, B)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            dA.copy_(A, non_blocking=True)
            dB.copy_(B, non_blocking=True)
            sg.gemm(dA, dB, out=dD)
            doubled = dD.float() * 2          # dependent op queued behind the kernel on the same stream
        side.synchronize()
        parity.assert_bit_exact(dD, ref, f"seed {seed}")
        assert torch.equal(doubled.cpu().double(), 2 * ref)


# ---------------------------------------------------------------------------------------- batched

@pytest.mark.parametrize("tile_n,pair", [(64, 0), (256, 0), (128, 1)])
def test_batched_gemm_bit_exact_with_strides(tile_n, pair):
    sg.set_tuning(tile_n, pair)
    batch, M, N, K = 5, 136, 200, 72
    Apad = inputs.small_integers([batch, M + 8, K + 8], 606, 1)               # padded batch stride and ld
    A = Apad[:, :M, :K]
    B = inputs.small_integers([batch, N, K], 606, 2)
    ref, _ = orc.batched_gemm(A, B)
    D, whole = guarded((batch, M, N), torch.bfloat16)
    sg.batched_gemm(Apad.to(DEV)[:, :M, :K], B.to(DEV), out=D)
    parity.assert_bit_exact(D, ref, "batched")
    assert guards_intact(whole)
    one = sg.batched_gemm(A[:1].to(DEV), B[:1].to(DEV))
    assert torch.equal(one[0].cpu(), sg.gemm(A[0].to(DEV), B[0].to(DEV)).cpu())


def test_batched_gemm_bias_per_batch_and_shared_fp32():
    batch, M, N, K = 3, 64, 72, 128
    A = inputs.uniform([batch, M, K], 707, 1)
    B = inputs.uniform([batch, N, K], 707, 2)
    bias2 = inputs.normal([batch, N], 707, 4)
    C = inputs.normal([batch, M, N], 707, 3).float()
    for bias in (bias2, bias2[0].contiguous()):
        ref, absacc = orc.batched_gemm(A, B, C=C, bias=bias, beta=1.0, epi="gelu")
        D = sg.batched_gemm(A.to(DEV), B.to(DEV), C=C.to(DEV), bias=bias.to(DEV), beta=1.0, epi="gelu",
                            out_dtype=torch.float32)
        parity.assert_matches(D, ref, absacc, f"batched bias dim {bias.dim()}")


# ---------------------------------------------------------------------------------------- grouped

@pytest.mark.parametrize("tile_n,pair", [(128, 0), (256, 0), (256, 1)])
def test_grouped_gemm_ragged_bit_exact(tile_n, pair):
    sg.set_tuning(tile_n, pair)
    Ms = [130, 0, 1, 257, 128, 511]
    N, K = 264, 136
    As = [inputs.small_integers([m, K], 808 + g, 1) for g, m in enumerate(Ms)]
    Bs = [inputs.small_integers([N, K], 808 + g, 2) for g in range(len(Ms))]
    refs, _ = orc.grouped_gemm(As, Bs)
    views, wholes = zip(*[guarded((max(m, 1), N), torch.bfloat16) for m in Ms])
    outs = [v[:m] for v, m in zip(views, Ms)]
    sg.grouped_gemm([a.to(DEV) for a in As], [b.to(DEV) for b in Bs], outs=outs)
    for g, m in enumerate(Ms):
        parity.assert_bit_exact(outs[g], refs[g], f"group {g}")
        assert bool(torch.isnan(wholes[g][:8]).all() and torch.isnan(wholes[g][8 + m:]).all()), f"guards of group {g}"
    # a permutation of the groups permutes the outputs; equal groups reduce to the batched call
    perm = [3, 0, 5]
    outs_p = sg.grouped_gemm([As[i].to(DEV) for i in perm], [Bs[i].to(DEV) for i in perm])
    for j, i in enumerate(perm):
        assert torch.equal(outs_p[j].cpu(), outs[i].cpu())


@pytest.mark.parametrize("scratch", [False, True])
def test_grouped_and_conv_tail_split(scratch):
    sg.enable_scratch(scratch)
    sg.set_tail_mode(2 if scratch else 1)
    sg.set_tuning(256, 0)
    Ms = [128 * 100, 128 * 49, 77]                     # 150 tiles of 128 x 256: two more than a wave of 148
    N, K = 200, 72
    As = [inputs.small_integers([m, K], 818 + g, 1) for g, m in enumerate(Ms)]
    Bs = [inputs.small_integers([N, K], 818 + g, 2) for g in range(len(Ms))]
    refs, _ = orc.grouped_gemm(As, Bs)
    outs = sg.grouped_gemm([a.to(DEV) for a in As], [b.to(DEV) for b in Bs])
    assert sg.last_launch_plan()["tail_split"] not in (0, 1, -1)
    for g in range(len(Ms)):
        parity.assert_bit_exact(outs[g], refs[g], f"group {g} with split tail")
    X = inputs.small_integers([2, 100, 96, 16], 828, 6, -1, 1)
    Wf = inputs.small_integers([256, 3, 3, 16], 828, 7, -1, 1)
    ref, _ = orc.conv2d_fprop(X, Wf, pad=(1, 1))
    Y = sg.conv2d_fprop(X.to(DEV), Wf.to(DEV), pad=(1, 1))
    assert sg.last_launch_plan()["tail_split"] not in (0, 1, -1)
    parity.assert_bit_exact(Y, ref, "conv with split tail")


def test_grouped_gemm_epilogue_bias_and_c():
    Ms = [96, 200, 40]
    N, K = 136, 264
    As, Bs = inputs.make_grouped(Ms, N, K, "normal", K ** -0.25, seed=909)
    biases = [inputs.normal([N], 909 + g, 4) for g in range(len(Ms))]
    Cs = [inputs.normal([m, N], 909 + g, 3) for g, m in enumerate(Ms)]
    refs, accs = orc.grouped_gemm(As, Bs, Cs=Cs, biases=biases, alpha=1.5, beta=0.25, epi="silu")
    outs = sg.grouped_gemm([a.to(DEV) for a in As], [b.to(DEV) for b in Bs], Cs=[c.to(DEV) for c in Cs],
                           biases=[b.to(DEV) for b in biases], alpha=1.5, beta=0.25, epi="silu")
    for g in range(len(Ms)):
        parity.assert_matches(outs[g], refs[g], accs[g], f"group {g}")


def test_grouped_equal_sizes_match_batched():
    groups, M, N, K = 4, 128, 128, 64
    A = inputs.small_integers([groups, M, K], 111, 1).to(DEV)
    B = inputs.small_integers([groups, N, K], 111, 2).to(DEV)
    outs = sg.grouped_gemm(list(A), list(B))
    bat = sg.batched_gemm(A, B)
    for g in range(groups):
        assert torch.equal(outs[g], bat[g])


# ---------------------------------------------------------------------------------------- convolution

CONV_CASES = [
    # N, H, W, C, K, R, S, pad, stride, dil
    (2, 9, 11, 64, 64, 3, 3, (1, 1), (1, 1), (1, 1)),
    (3, 14, 14, 24, 40, 3, 3, (1, 1), (1, 1), (1, 1)),       # C, K not multiples of 64
    (2, 12, 10, 72, 136, 1, 1, (0, 0), (1, 1), (1, 1)),
    (2, 15, 13, 32, 72, 3, 2, (1, 0), (2, 2), (1, 1)),
    (1, 17, 19, 16, 64, 3, 3, (2, 2), (1, 2), (2, 2)),
    (2, 8, 8, 128, 264, 5, 5, (2, 2), (1, 1), (1, 1)),
]


@pytest.mark.parametrize("pair", [0, 1])
@pytest.mark.parametrize("case", CONV_CASES)
def test_conv_integer_inputs_bit_exact(case, pair):
    sg.set_tuning(-1, pair)
    N, H, W, C, K, R, S, pad, stride, dil = case
    X = inputs.small_integers([N, H, W, C], 121, 6, -1, 1)
    Wf = inputs.small_integers([K, R, S, C], 121, 7, -1, 1)
    keep = inputs.small_integers([K, R, S, C], 122, 7, 0, 3) == 0       # thin the filter so sums stay small
    Wf = Wf * keep.to(torch.bfloat16)
    ref, _ = orc.conv2d_fprop(X, Wf, pad=pad, stride=stride, dil=dil)
    assert float(ref.abs().max()) <= 256
    Y, whole = guarded((ref.shape[0] * ref.shape[1] * ref.shape[2], K), torch.bfloat16)
    sg.conv2d_fprop(X.to(DEV), Wf.to(DEV), pad=pad, stride=stride, dil=dil, out=Y.view(ref.shape))
    parity.assert_bit_exact(Y, ref.view(-1, K), f"conv {case}")
    assert guards_intact(whole)


@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float32])
def test_conv_epilogue_bias_relu_and_residual(out_dtype):
    N, H, W, C, K = 2, 10, 12, 72, 80
    X, Wf, bias = inputs.make_conv(N, H, W, C, K, 3, 3, "normal", (C * 9) ** -0.25, bias=True, seed=131)
    Cin = inputs.normal([N, H, W, K], 131, 3).to(out_dtype)
    ref, absacc = orc.conv2d_fprop(X, Wf, pad=(1, 1), Cin=Cin, bias=bias, alpha=0.5, beta=1.0, epi="relu")
    Y = sg.conv2d_fprop(X.to(DEV), Wf.to(DEV), pad=(1, 1), Cin=Cin.to(DEV), bias=bias.to(DEV), alpha=0.5, beta=1.0,
                        epi="relu", out_dtype=out_dtype)
    parity.assert_matches(Y, ref, absacc, f"conv epilogue {out_dtype}")


def test_conv_delta_filter_reproduces_input_on_gpu():
    N, H, W, C = 2, 7, 9, 64
    X = inputs.uniform([N, H, W, C], 141, 6)
    Wf = torch.zeros(C, 3, 3, C, dtype=torch.bfloat16)
    for k in range(C):
        Wf[k, 1, 1, k] = 1
    Y = sg.conv2d_fprop(X.to(DEV), Wf.to(DEV), pad=(1, 1))
    assert torch.equal(Y.cpu(), X)


# ---------------------------------------------------------------------------------------- transpose stage

@pytest.mark.parametrize("in_dtype", [torch.float32, torch.bfloat16, torch.float16])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16, torch.float16])
@pytest.mark.parametrize("shape", [(1, 64, 64), (3, 100, 72), (2, 37, 200), (4, 256, 196), (1, 1, 8), (2, 129, 4)])
def test_transpose_with_dtype_conversion_bit_exact(shape, in_dtype, out_dtype):
    batch, rows, cols = shape
    ld = (cols + 7) // 8 * 8 + 8
    big = (inputs.normal([batch, rows, ld], 616, 1).float() * 1.37).to(in_dtype)          # padded leading dimension
    x = big[:, :, :cols]
    want = orc.transpose(x, out_dtype)
    ld_out = (rows + 7) // 8 * 8 + 8
    out_big = torch.full((batch, cols, ld_out), float("nan"), dtype=out_dtype, device=DEV)
    sg.transpose(big.to(DEV)[:, :, :cols], out=out_big[:, :, :rows])
    parity.assert_bit_exact(out_big[:, :, :rows], want, f"transpose {shape} {in_dtype}->{out_dtype}")
    assert bool(torch.isnan(out_big[:, :, rows:]).all())
    if rows % 8 == 0 and cols % 8 == 0:       # the densely packed form needs 16-byte leading dimensions itself
        assert torch.equal(sg.transpose(x.to(DEV), out_dtype=out_dtype).cpu(), x.permute(0, 2, 1).to(out_dtype))


@pytest.mark.parametrize("in_dtype", [torch.float32, torch.bfloat16, torch.float16])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16, torch.float16])
def test_transpose_many_tiles_per_cta_and_both_kernels(in_dtype, out_dtype):
    # Far more tiles than SMs x ring stages: every CTA of the persistent TMA kernel wraps its stage ring and reuses both
    # output tiles several times; rows and columns end inside a tile (clipped loads and stores).
    batch, rows, cols = 6, 1000, 2072
    x = (inputs.normal([batch, rows, cols], 717, 1).float() * 1.37).to(in_dtype)
    want = orc.transpose(x, out_dtype)
    dx = x.to(DEV)
    out, whole = guarded((batch, cols, rows), out_dtype)
    sg.transpose(dx, out=out)
    assert sg.last_kernel_name().startswith("sg::transpose_tma_kernel")
    parity.assert_bit_exact(out, want, f"TMA transpose {in_dtype}->{out_dtype}")
    assert guards_intact(whole)
    try:
        sg.set_option("transpose_plain", 1)                  # the kernel ragged extents take, on the same problem
        out2 = torch.full((batch, cols, rows), float("nan"), dtype=out_dtype, device=DEV)
        sg.transpose(dx, out=out2)
        assert sg.last_kernel_name().startswith("sg::transpose_kernel")
    finally:
        sg.set_option("transpose_plain", -1)
    assert torch.equal(out2, out)


def test_layout_pipeline_nchw_conv_nchw_and_conv1d():
    # pipeline(transpose(input, NCHW, NHWC, fp32, bf16), conv2d_fprop, transpose(output, NHWC, NCHW, bf16, fp32))
    N, C, H, W, K = 2, 64, 10, 12, 72
    x_nchw = inputs.small_integers([N, C, H, W], 626, 6, -1, 1).float()
    Wf = inputs.small_integers([K, 3, 3, C], 626, 7, -1, 1) * (inputs.small_integers([K, 3, 3, C], 627, 7, 0, 3) == 0).to(torch.bfloat16)
    x_nhwc = sg.nchw_to_nhwc(x_nchw.to(DEV), out_dtype=torch.bfloat16)
    assert torch.equal(x_nhwc.cpu(), x_nchw.permute(0, 2, 3, 1).to(torch.bfloat16))
    y = sg.conv2d_fprop(x_nhwc, Wf.to(DEV), pad=(1, 1), epi="relu")
    y_nchw = sg.nhwc_to_nchw(y, out_dtype=torch.float32)
    ref, _ = orc.conv2d_fprop(x_nchw.permute(0, 2, 3, 1).contiguous().to(torch.bfloat16), Wf, pad=(1, 1), epi="relu")
    parity.assert_bit_exact(y_nchw.permute(0, 2, 3, 1), ref, "NCHW -> conv -> NCHW")
    # the same three stages through the pipeline driver, with a bias and on a side stream
    bias = inputs.small_integers([K], 628, 8, -2, 2)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        y2 = sg.conv2d_fprop_nchw(x_nchw.to(DEV), Wf.to(DEV), pad=(1, 1), bias=bias.to(DEV), epi="relu", stream=side)
    side.synchronize()
    assert y2.dtype == torch.float32 and tuple(y2.shape) == (N, K, H, W)
    ref2, _ = orc.conv2d_fprop(x_nchw.permute(0, 2, 3, 1).contiguous().to(torch.bfloat16), Wf, pad=(1, 1), bias=bias, epi="relu")
    parity.assert_bit_exact(y2.permute(0, 2, 3, 1), ref2, "pipeline driver")
    # conv1d lowered to conv2d with H = 1
    X1 = inputs.small_integers([3, 50, 32], 636, 6, -1, 1)
    W1 = inputs.small_integers([40, 5, 32], 636, 7, -1, 1) * (inputs.small_integers([40, 5, 32], 637, 7, 0, 2) == 0).to(torch.bfloat16)
    ref1, _ = orc.conv2d_fprop(X1.view(3, 1, 50, 32), W1.view(40, 1, 5, 32), pad=(0, 2), stride=(1, 2))
    y1 = sg.conv1d_fprop(X1.to(DEV), W1.to(DEV), pad=2, stride=2)
    parity.assert_bit_exact(y1, ref1.view(3, -1, 40), "conv1d")


# ---------------------------------------------------------------------------------------- fp16 inputs / outputs

@pytest.mark.parametrize("tile_n,pair", [(64, 0), (256, 0), (128, 1), (256, 1)])
@pytest.mark.parametrize("out_dtype", [torch.float16, torch.float32, torch.bfloat16])
def test_fp16_inputs_integer_problem_bit_exact(out_dtype, tile_n, pair):
    sg.set_tuning(tile_n, pair)
    M, N, K = 300, 200, 136
    A = inputs.small_integers([M, K], 717, 1).half()
    B = inputs.small_integers([N, K], 717, 2).half()
    ref, _ = orc.gemm(A, B)
    D = sg.gemm(A.to(DEV), B.to(DEV), out_dtype=out_dtype)
    parity.assert_bit_exact(D, ref, f"fp16 in, {out_dtype} out")


@pytest.mark.parametrize("epi", ["none", "relu", "gelu", "silu"])
def test_fp16_dsl_example_dtype_triple_with_bias_and_residual(epi):
    # the DSL's running example: input=fp16, acc=fp32, output=fp16, with a bias and an activation
    M, N, K = 200, 328, 264
    A = (inputs.normal([M, K], 727, 1).float() * K ** -0.25).half()
    B = (inputs.normal([N, K], 727, 2).float() * K ** -0.25).half()
    bias = inputs.normal([N], 727, 4).half()
    C = inputs.normal([M, N], 727, 3).half()
    ref, absacc = orc.gemm(A, B, C=C, bias=bias, alpha=0.75, beta=-0.5, epi=epi)
    D = sg.gemm(A.to(DEV), B.to(DEV), C=C.to(DEV), bias=bias.to(DEV), alpha=0.75, beta=-0.5, epi=epi, out_dtype=torch.float16)
    parity.assert_matches(D, ref, absacc, f"fp16 {epi}")
    # ragged N (plain-store path), batched, grouped and convolution with fp16 operands
    refr, accr = orc.gemm(A, B[:90], bias=bias[:90].contiguous(), epi=epi)
    big = torch.full((M, 96), float("nan"), dtype=torch.float16, device=DEV)
    sg.gemm(A.to(DEV), B[:90].to(DEV), bias=bias[:90].contiguous().to(DEV), epi=epi, out=big[:, :90])
    parity.assert_matches(big[:, :90], refr, accr, "fp16 ragged N")
    assert bool(torch.isnan(big[:, 90:]).all())


def test_fp16_batched_grouped_and_conv():
    A = (inputs.uniform([3, 72, 136], 737, 1)).half()
    B = (inputs.uniform([3, 64, 136], 737, 2)).half()
    ref, absacc = orc.batched_gemm(A, B, epi="relu")
    parity.assert_matches(sg.batched_gemm(A.to(DEV), B.to(DEV), epi="relu", out_dtype=torch.float16), ref, absacc, "fp16 batched")
    As = [inputs.small_integers([m, 72], 747 + g, 1).half() for g, m in enumerate([130, 40])]
    Bs = [inputs.small_integers([136, 72], 747 + g, 2).half() for g in range(2)]
    refs, _ = orc.grouped_gemm(As, Bs)
    outs = sg.grouped_gemm([a.to(DEV) for a in As], [b.to(DEV) for b in Bs], out_dtype=torch.float16)
    for g in range(2):
        parity.assert_bit_exact(outs[g], refs[g], f"fp16 grouped {g}")
    X = inputs.small_integers([2, 9, 11, 64], 757, 6, -1, 1).half()
    Wf = (inputs.small_integers([72, 3, 3, 64], 757, 7, -1, 1) * (inputs.small_integers([72, 3, 3, 64], 758, 7, 0, 3) == 0).to(torch.bfloat16)).half()
    ref, _ = orc.conv2d_fprop(X, Wf, pad=(1, 1))
    parity.assert_bit_exact(sg.conv2d_fprop(X.to(DEV), Wf.to(DEV), pad=(1, 1), out_dtype=torch.float16), ref, "fp16 conv")


# ---------------------------------------------------------------------------------------- fp8 inputs

@pytest.mark.parametrize("dtype", [torch.float8_e4m3fn, torch.float8_e5m2])
@pytest.mark.parametrize("tile_n,pair", [(64, 0), (128, 0), (256, 0), (128, 1), (256, 1)])
@pytest.mark.parametrize("M,N,K", [(256, 256, 256), (300, 200, 272), (1000, 520, 1040), (129, 72, 16)])
def test_fp8_inputs_integer_problem_bit_exact(M, N, K, tile_n, pair, dtype):
    sg.set_tuning(tile_n, pair)
    A = inputs.small_integers([M, K], 818, 1, -1, 1).float().to(dtype)
    B = inputs.small_integers([N, K], 818, 2, -1, 1).float().to(dtype)
    ref, _ = orc.gemm(A, B)
    assert float(ref.abs().max()) <= 256
    D, whole = guarded((M, N), torch.bfloat16)
    sg.gemm(A.to(DEV), B.to(DEV), out=D)
    parity.assert_bit_exact(D, ref, f"fp8 {dtype} {M}x{N}x{K}")
    assert guards_intact(whole, cols=N)


def test_fp8_real_values_epilogue_batched_grouped_and_conv():
    dt = torch.float8_e4m3fn
    M, N, K = 200, 264, 528
    A = (inputs.normal([M, K], 828, 1).float()).to(dt)
    B = (inputs.normal([N, K], 828, 2).float()).to(dt)
    bias = inputs.normal([N], 828, 4)
    for out_dtype in (torch.bfloat16, torch.float32):
        ref, absacc = orc.gemm(A, B, bias=bias, alpha=K ** -0.5, epi="gelu")
        D = sg.gemm(A.to(DEV), B.to(DEV), bias=bias.to(DEV), alpha=K ** -0.5, epi="gelu", out_dtype=out_dtype)
        parity.assert_matches(D, ref, absacc, f"fp8 gelu {out_dtype}")
    Ab = inputs.small_integers([3, 72, 144], 838, 1, -1, 1).float().to(dt)
    Bb = inputs.small_integers([3, 64, 144], 838, 2, -1, 1).float().to(dt)
    ref, _ = orc.batched_gemm(Ab, Bb)
    parity.assert_bit_exact(sg.batched_gemm(Ab.to(DEV), Bb.to(DEV)), ref, "fp8 batched")
    As = [inputs.small_integers([m, 144], 848 + g, 1, -1, 1).float().to(dt) for g, m in enumerate([130, 40])]
    Bs = [inputs.small_integers([136, 144], 848 + g, 2, -1, 1).float().to(dt) for g in range(2)]
    refs, _ = orc.grouped_gemm(As, Bs)
    outs = sg.grouped_gemm([a.to(DEV) for a in As], [b.to(DEV) for b in Bs])
    for g in range(2):
        parity.assert_bit_exact(outs[g], refs[g], f"fp8 grouped {g}")
    X = inputs.small_integers([2, 9, 11, 144], 858, 6, -1, 1).float().to(torch.float8_e5m2)
    Wf = (inputs.small_integers([72, 3, 3, 144], 858, 7, -1, 1) * (inputs.small_integers([72, 3, 3, 144], 859, 7, 0, 3) == 0).to(torch.bfloat16)).float().to(torch.float8_e5m2)
    ref, _ = orc.conv2d_fprop(X, Wf, pad=(1, 1))
    assert float(ref.abs().max()) <= 256
    parity.assert_bit_exact(sg.conv2d_fprop(X.to(DEV), Wf.to(DEV), pad=(1, 1)), ref, "fp8 conv")
    with pytest.raises(sg.SolgemmError):                       # only the K-contiguous layouts with 8-bit inputs
        sg.gemm(A.to(DEV), torch.zeros(K, N, device=DEV).to(dt), layout_b="row")


@pytest.mark.parametrize("M,chunks", [(1000, 8), (256, 8), (2304, 3), (64, 1)])
def test_gemm_host_pipelined_copies_match_the_oracle(M, chunks):
    N, K = 264, 200
    A, B, bias = inputs.make_gemm(M, N, K, "uniform", 1.0, bias=True, seed=61)
    ref, absacc = orc.gemm(A, B, bias=bias, epi="relu")
    hA, hB, hb = A.pin_memory(), B.pin_memory(), bias.pin_memory()
    hD = torch.full((M, N), float("nan"), dtype=torch.bfloat16).pin_memory()
    scratch = {}
    for _ in range(2):                      # the second call reuses the device buffers of the first
        hD.fill_(float("nan"))
        sg.gemm_host(hA, hB, hD, bias_host=hb, epi="relu", scratch=scratch, chunks=chunks)
        torch.cuda.current_stream().synchronize()
        parity.assert_matches(hD, ref, absacc, f"gemm_host M={M} chunks={chunks}")


def test_gemm_host_residual_other_layouts_padded_rows_and_pageable_memory():
    # column-major A and row-major B with padded leading dimensions, a residual C, fp32 output, small integers (exact);
    # once from pinned and once from pageable host memory; the padding of D_host must stay untouched
    M, N, K = 700, 136, 72
    Ast = inputs.small_integers([K, M + 28], 71, 1)                 # A column-major: [K, M] with lda = M + 28
    Bst = inputs.small_integers([K, N + 8], 71, 2)                  # B row-major:    [K, N] with ldb = N + 8
    C = inputs.small_integers([M, N + 4], 71, 3, -2, 2).float()
    bias = inputs.small_integers([N], 71, 4, -3, 3)
    ref, _ = orc.gemm(Ast[:, :M], Bst[:, :N], C=C[:, :N], bias=bias, alpha=2.0, beta=1.0, layout_a="col", layout_b="row")
    for pin in (True, False):
        place = (lambda t: t.pin_memory()) if pin else (lambda t: t.clone())
        hA, hB, hC, hb = place(Ast), place(Bst), place(C), place(bias)
        hD = place(torch.full((M, N + 12), float("nan"), dtype=torch.float32))
        sg.gemm_host(hA[:, :M], hB[:, :N], hD[:, :N], C_host=hC[:, :N], bias_host=hb, alpha=2.0, beta=1.0, layout_a="col",
                     layout_b="row", chunks=3)
        torch.cuda.current_stream().synchronize()
        parity.assert_bit_exact(hD[:, :N], ref, f"gemm_host layouts pinned={pin}")
        assert bool(torch.isnan(hD[:, N:]).all())


@pytest.mark.parametrize("dtype", [torch.float16, torch.float8_e4m3fn, torch.float8_e5m2, torch.int8, torch.float32])
def test_two_pass_split_k_other_input_types_bit_exact(dtype):
    # the K ranges of a skinny problem through the everything-in-one kernel variant: fp16, fp8, int8 (integer accumulators,
    # converted before they are parked) and fp32-as-tf32 operands; small integers, exact in every type involved
    M, N, K = 200, 264, 8192
    A = (inputs.small_integers([M, K], 393, 1) * (inputs.small_integers([M, K], 394, 1, 0, 15) == 0).to(torch.bfloat16)).float().to(dtype)
    B = inputs.small_integers([N, K], 393, 2).float().to(dtype)
    bias = inputs.small_integers([N], 393, 4, -3, 3).to(orc.bias_dtype_for(dtype))
    ref, _ = orc.gemm(A, B, bias=bias, epi="relu")
    assert float(ref.abs().max()) <= 256
    for out_dtype in (torch.bfloat16, torch.float32):
        D = sg.gemm(A.to(DEV), B.to(DEV), bias=bias.to(DEV), epi="relu", out_dtype=out_dtype)
        assert sg.last_launch_plan()["tail_split"] < -1, sg.last_launch_plan()
        parity.assert_bit_exact(D, ref, f"two-pass {dtype} -> {out_dtype}")


def test_two_pass_split_k_skinny_convolution():
    # a convolution with few output pixels and many input channels: 128 pixels x 136 filters, K = 3 * 3 * 1024
    X = inputs.small_integers([2, 8, 8, 1024], 403, 6, -1, 1) * (inputs.small_integers([2, 8, 8, 1024], 404, 6, 0, 7) == 0).to(torch.bfloat16)
    Wf = inputs.small_integers([136, 3, 3, 1024], 403, 7, -1, 1)
    bias = inputs.small_integers([136], 403, 4, -2, 2)
    ref, _ = orc.conv2d_fprop(X, Wf, pad=(1, 1), bias=bias, epi="relu")
    assert float(ref.abs().max()) <= 256
    Y = sg.conv2d_fprop(X.to(DEV), Wf.to(DEV), pad=(1, 1), bias=bias.to(DEV), epi="relu")
    assert sg.last_launch_plan()["tail_split"] < -1, sg.last_launch_plan()
    parity.assert_bit_exact(Y, ref, "two-pass conv")
