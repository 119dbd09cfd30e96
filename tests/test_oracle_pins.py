"""Pins for the CPU oracle: closed forms, hand-computed cases, invariants and library special cases.

None of these compares the oracle with itself through a retyped formula: each
expected value is either written by hand, a mathematical identity, or comes
from an unrelated library routine (torch fp64 matmul / conv2d / activations).
A plausible mistake in the oracle (dropped term, wrong sign or index,
transposed operand, wrong bias direction, wrong padding) fails at least one.
"""
import math

import pytest
import torch

from oracle import oracle as orc
from paper_2603_29010_b200 import inputs
from tests import parity


def bf(x):
    return torch.tensor(x, dtype=torch.float64).to(torch.bfloat16)


def randi(shape, seed, tid, lo=-3, hi=3):
    return inputs.small_integers(shape, seed, tid, lo, hi)


# ---------------------------------------------------------------- GEMM: hand-written cases

def test_gemm_tiny_hand_computed_tn():
    # A (row-major) = [[1,2,3],[4,5,6]]; B as a matrix (K x N) = [[1,0],[2,1],[0,3]],
    # stored column-major, i.e. as its transpose [N,K] = [[1,2,0],[0,1,3]].
    A = bf([[1, 2, 3], [4, 5, 6]])
    Bt = bf([[1, 2, 0], [0, 1, 3]])
    ref, absacc = orc.gemm(A, Bt, layout_a="row", layout_b="col")
    assert ref.tolist() == [[5.0, 11.0], [14.0, 23.0]]
    assert absacc.tolist() == [[5.0, 11.0], [14.0, 23.0]]


def test_gemm_tiny_hand_computed_all_layouts():
    Am = [[1, -2, 3], [4, 5, -6]]              # M=2, K=3
    Bm = [[1, 0], [2, 1], [0, 3]]              # K=3, N=2
    want = [[-3.0, 7.0], [14.0, -13.0]]
    A_row, A_col = bf(Am), bf(Am).t().contiguous()
    B_row, B_col = bf(Bm), bf(Bm).t().contiguous()
    for la, A in (("row", A_row), ("col", A_col)):
        for lb, B in (("row", B_row), ("col", B_col)):
            ref, _ = orc.gemm(A, B, layout_a=la, layout_b=lb)
            assert ref.tolist() == want, (la, lb)


def test_gemm_scaling_bias_order_hand_computed():
    # acc = [[5, 11]], alpha=2, beta=-1, C=[[1, 3]], bias=[10, -40]:
    # 2*5 - 1 + 10 = 19 ; 2*11 - 3 - 40 = -21 ; bias is NOT multiplied by alpha.
    A = bf([[1, 2, 3]])
    Bt = bf([[1, 2, 0], [0, 1, 3]])
    C = bf([[1, 3]])
    bias = bf([10, -40])
    ref, absacc = orc.gemm(A, Bt, C=C, bias=bias, alpha=2.0, beta=-1.0, epi="bias")
    assert ref.tolist() == [[19.0, -21.0]]
    assert absacc.tolist() == [[10.0 + 1.0 + 10.0, 22.0 + 3.0 + 40.0]]
    ref, _ = orc.gemm(A, Bt, C=C, bias=bias, alpha=2.0, beta=-1.0, epi="relu")
    assert ref.tolist() == [[19.0, 0.0]]


def test_gemm_identity_and_one_hot():
    K = N = 7
    Bt = randi([N, K], 1, 2)                                   # column-major storage of b(k,j) = Bt[j,k]
    eye = torch.eye(K, dtype=torch.bfloat16)
    ref, _ = orc.gemm(eye, Bt)                                 # I . B = B  -> D[i,j] = b(i,j) = Bt[j,i]
    assert torch.equal(ref, Bt.t().double())
    A = randi([5, K], 1, 1)
    onehot = torch.zeros(N, K, dtype=torch.bfloat16)
    onehot[3, 2] = 1                                           # b(2,3) = 1: column 3 of D picks column 2 of A
    ref, _ = orc.gemm(A, onehot)
    want = torch.zeros(5, N, dtype=torch.float64)
    want[:, 3] = A[:, 2].double()
    assert torch.equal(ref, want)


@pytest.mark.parametrize("K", [256, 512, 2304, 4096])
def test_gemm_all_ones_gives_k(K):
    A = torch.ones(3, K, dtype=torch.bfloat16)
    Bt = torch.ones(4, K, dtype=torch.bfloat16)
    ref, absacc = orc.gemm(A, Bt)
    assert torch.equal(ref, torch.full((3, 4), float(K), dtype=torch.float64))
    assert torch.equal(absacc, ref)


def test_gemm_ones_a_gives_column_sums():
    K, N = 33, 9
    Bt = randi([N, K], 2, 2)
    ref, _ = orc.gemm(torch.ones(2, K, dtype=torch.bfloat16), Bt)
    assert torch.equal(ref[0], Bt.double().sum(dim=1))
    assert torch.equal(ref[1], ref[0])


# ---------------------------------------------------------------- GEMM: library and invariants

@pytest.mark.parametrize("la,lb", [("row", "col"), ("row", "row"), ("col", "col"), ("col", "row")])
def test_gemm_matches_torch_fp64_matmul(la, lb):
    M, N, K = 37, 29, 83
    Am = inputs.uniform([M, K], 3, 1)
    Bm = inputs.uniform([K, N], 3, 2)
    A = Am if la == "row" else Am.t().contiguous()
    B = Bm if lb == "row" else Bm.t().contiguous()
    ref, absacc = orc.gemm(A, B, layout_a=la, layout_b=lb)
    want = Am.double() @ Bm.double()
    assert torch.allclose(ref, want, rtol=0, atol=1e-12)
    assert torch.allclose(absacc, Am.double().abs() @ Bm.double().abs(), rtol=0, atol=1e-12)


def test_gemm_transpose_identity_through_layout_flags():
    # (A.B)^T = B^T.A^T : swap operands and flip both layout flags (operand-swap identity).
    M, N, K = 11, 13, 17
    A = randi([M, K], 4, 1)            # row-major A
    Bt = randi([N, K], 4, 2)           # column-major B
    d, _ = orc.gemm(A, Bt, layout_a="row", layout_b="col")
    # B^T is N x K: its row-major storage is exactly Bt.  A^T is K x M: its column-major storage is A.
    dt, _ = orc.gemm(Bt, A, layout_a="row", layout_b="col")
    assert torch.equal(dt, d.t())


def test_gemm_leading_dimensions():
    M, N, K = 6, 5, 12
    bigA = randi([M, K + 8], 5, 1)
    bigB = randi([N, K + 16], 5, 2)
    ref, _ = orc.gemm(bigA[:, :K], bigB[:, :K])
    want, _ = orc.gemm(bigA[:, :K].contiguous(), bigB[:, :K].contiguous())
    assert torch.equal(ref, want)
    assert torch.equal(ref, bigA[:, :K].double() @ bigB[:, :K].double().t())


def test_gemm_alpha_linearity_beta_and_nan_c():
    M, N, K = 8, 8, 16
    A, Bt = randi([M, K], 6, 1), randi([N, K], 6, 2)
    C = randi([M, N], 6, 3)
    base, _ = orc.gemm(A, Bt)
    twice, _ = orc.gemm(A, Bt, alpha=2.0)
    assert torch.equal(twice, 2 * base)
    plus_c, _ = orc.gemm(A, Bt, C=C, beta=1.0)
    assert torch.equal(plus_c, base + C.double())
    c32 = C.float()
    plus_c32, _ = orc.gemm(A, Bt, C=c32, beta=0.5)
    assert torch.equal(plus_c32, base + 0.5 * C.double())
    nan_c = torch.full((M, N), float("nan"), dtype=torch.bfloat16)
    ignored, _ = orc.gemm(A, Bt, C=nan_c, beta=0.0)
    assert torch.equal(ignored, base)


def test_gemm_bias_is_per_column():
    M, N, K = 4, 6, 8
    zeros = torch.zeros(M, K, dtype=torch.bfloat16)
    bias = bf([1, 2, 3, 4, 5, 6])
    ref, _ = orc.gemm(zeros, randi([N, K], 7, 2), bias=bias, epi="bias")
    assert torch.equal(ref, bias.double().expand(M, N))


def test_gemm_k_zero_is_the_empty_sum():
    A = torch.zeros(3, 0, dtype=torch.bfloat16)
    Bt = torch.zeros(2, 0, dtype=torch.bfloat16)
    ref, _ = orc.gemm(A, Bt, bias=bf([1.5, -2]), epi="relu")
    assert ref.tolist() == [[1.5, 0.0]] * 3


def test_gemm_rows_and_points_agree_with_full():
    M, N, K = 19, 7, 31
    A, Bt = inputs.uniform([M, K], 8, 1), inputs.uniform([N, K], 8, 2)
    bias = inputs.normal([N], 8, 4)
    full, facc = orc.gemm(A, Bt, bias=bias, epi="silu")
    part, pacc = orc.gemm(A, Bt, bias=bias, epi="silu", rows=(5, 11))
    assert torch.equal(part, full[5:11]) and torch.equal(pacc, facc[5:11])
    pi, pj = [0, 18, 7, 7], [6, 0, 3, 4]
    pts, ptacc = orc.gemm_points(A, Bt, pi, pj, bias=bias, epi="silu")
    assert torch.equal(pts, full[pi, pj]) and torch.equal(ptacc, facc[pi, pj])


def test_batched_and_grouped_reduce_to_gemm():
    A = randi([3, 5, 8], 9, 1)
    B = randi([3, 4, 8], 9, 2)
    ref, _ = orc.batched_gemm(A, B)
    for b in range(3):
        assert torch.equal(ref[b], A[b].double() @ B[b].double().t())
    one, _ = orc.batched_gemm(A[:1], B[:1])
    assert torch.equal(one[0], orc.gemm(A[0], B[0])[0])
    refs, _ = orc.grouped_gemm([A[0], A[1][:2], A[2][:0]], [B[0], B[1], B[2]])
    assert torch.equal(refs[0], ref[0]) and torch.equal(refs[1], ref[1][:2]) and refs[2].shape == (0, 4)
    # permuting groups permutes outputs
    perm, _ = orc.grouped_gemm([A[1][:2], A[0]], [B[1], B[0]])
    assert torch.equal(perm[0], refs[1]) and torch.equal(perm[1], refs[0])


# ---------------------------------------------------------------- activations

def test_activation_closed_forms():
    assert orc.act("relu", -3.0) == 0.0 and orc.act("relu", 0.0) == 0.0 and orc.act("relu", 2.5) == 2.5
    assert orc.act("none", -3.0) == -3.0 and orc.act("bias", -3.0) == -3.0
    assert orc.act("gelu", 0.0) == 0.0 and orc.act("silu", 0.0) == 0.0
    assert orc.act("silu", 1.0) == pytest.approx(1.0 / (1.0 + math.exp(-1.0)), rel=1e-15)
    assert orc.act("silu", 1.0) == pytest.approx(0.7310585786300049, rel=1e-14)
    assert orc.act("gelu", 1.0) == pytest.approx(0.5 * (1.0 + math.tanh(math.sqrt(2 / math.pi) * 1.044715)), rel=1e-15)
    assert orc.act("gelu", 1.0) == pytest.approx(0.8411919906082768, rel=1e-13)
    # the tanh form, not the erf form (they differ by ~1.5e-4 at x = 1)
    erf_form = 0.5 * (1.0 + math.erf(1.0 / math.sqrt(2.0)))
    assert abs(orc.act("gelu", 1.0) - erf_form) > 1e-4


@pytest.mark.parametrize("x", [0.1, 0.5, 1.0, 2.0, 3.7, 9.0])
def test_activation_odd_part_identities_and_limits(x):
    # gelu(x) - gelu(-x) = x and silu(x) - silu(-x) = x hold exactly in real arithmetic.
    assert orc.act("gelu", x) - orc.act("gelu", -x) == pytest.approx(x, rel=1e-14)
    assert orc.act("silu", x) - orc.act("silu", -x) == pytest.approx(x, rel=1e-14)
    assert orc.act("gelu", 40.0) == 40.0 and abs(orc.act("gelu", -40.0)) == 0.0
    assert orc.act("silu", 50.0) == pytest.approx(50.0, rel=1e-15) and abs(orc.act("silu", -50.0)) < 1e-19


def test_activations_match_torch_library_fp64():
    xs = torch.linspace(-6, 6, 97, dtype=torch.float64)
    for name, fn in (("gelu", lambda t: torch.nn.functional.gelu(t, approximate="tanh")),
                     ("silu", torch.nn.functional.silu), ("relu", torch.relu)):
        got = torch.tensor([orc.act(name, float(x)) for x in xs], dtype=torch.float64)
        assert torch.allclose(got, fn(xs), rtol=1e-13, atol=1e-15), name


def test_further_activations_closed_forms_and_library():
    F = torch.nn.functional
    xs = torch.linspace(-7, 7, 113, dtype=torch.float64)
    table = [("sigmoid", (0, 0), torch.sigmoid), ("tanh", (0, 0), torch.tanh), ("mish", (0, 0), F.mish),
             ("hardswish", (0, 0), F.hardswish), ("leaky_relu", (0.125, 0), lambda t: F.leaky_relu(t, 0.125)),
             ("elu", (1.5, 0), lambda t: F.elu(t, 1.5)), ("clip", (-0.5, 2.0), lambda t: torch.clamp(t, -0.5, 2.0))]
    for name, args, fn in table:
        got = torch.tensor([orc.act(name, float(x), args) for x in xs], dtype=torch.float64)
        assert torch.allclose(got, fn(xs), rtol=1e-13, atol=1e-15), name
    # hand values and identities
    assert orc.act("sigmoid", 0.0) == 0.5 and orc.act("tanh", 0.0) == 0.0 and orc.act("mish", 0.0) == 0.0
    assert orc.act("sigmoid", 2.0) + orc.act("sigmoid", -2.0) == pytest.approx(1.0, rel=1e-15)
    assert orc.act("hardswish", -3.0) == 0.0 and orc.act("hardswish", 3.0) == 3.0 and orc.act("hardswish", 1.0) == pytest.approx(4.0 / 6.0)
    assert orc.act("leaky_relu", -4.0, (0.25, 0)) == -1.0 and orc.act("leaky_relu", 4.0, (0.25, 0)) == 4.0
    assert orc.act("elu", -1.0, (2.0, 0)) == pytest.approx(2.0 * (math.exp(-1.0) - 1.0), rel=1e-15) and orc.act("elu", 3.0, (2.0, 0)) == 3.0
    assert orc.act("clip", 7.0, (0.0, 6.0)) == 6.0 and orc.act("clip", -1.0, (0.0, 6.0)) == 0.0 and orc.act("clip", 2.5, (0.0, 6.0)) == 2.5
    assert orc.act("mish", 1.0) == pytest.approx(math.tanh(math.log(1.0 + math.e)), rel=1e-15)
    assert orc.act("mish", 40.0) == 40.0 and abs(orc.act("mish", -40.0)) < 1e-15
    # the parameters reach the GEMM and convolution entry points
    A, Bt = bf([[1, -2]]), bf([[1, 1], [2, -1]])
    ref, _ = orc.gemm(A, Bt, epi="leaky_relu", epi_args=(0.5, 0))
    assert ref.tolist() == [[-0.5, 4.0]]
    ref, _ = orc.gemm(A, Bt, epi="clip", epi_args=(-0.25, 3.0))
    assert ref.tolist() == [[-0.25, 3.0]]
    X, Wf = bf([[1, -2]]).view(1, 1, 1, 2), bf([[1, 1], [2, -1]]).view(2, 1, 1, 2)
    ref, _ = orc.conv2d_fprop(X, Wf, epi="elu", epi_args=(1.0, 0))
    assert ref.view(-1).tolist() == [pytest.approx(math.expm1(-1.0)), 4.0]


# ---------------------------------------------------------------- convolution

def test_conv_tiny_hand_computed():
    # 1 image, 3x3, 1 channel, values 1..9; 2x2 filter [[1,2],[3,4]], no padding, stride 1.
    X = bf([[1, 2, 3], [4, 5, 6], [7, 8, 9]]).view(1, 3, 3, 1)
    Wf = bf([[1, 2], [3, 4]]).view(1, 2, 2, 1)
    ref, _ = orc.conv2d_fprop(X, Wf)
    # y[0,0] = 1*1 + 2*2 + 4*3 + 5*4 = 37 (cross-correlation: no filter flip)
    assert ref.view(2, 2).tolist() == [[37.0, 47.0], [67.0, 77.0]]
    # stride 2 with padding 1: windows anchored at (-1,-1), (-1,1), (1,-1), (1,1)
    ref, _ = orc.conv2d_fprop(X, Wf, pad=(1, 1), stride=(2, 2))
    assert ref.view(2, 2).tolist() == [[4.0, 3 * 2 + 4 * 3.0], [2 * 4 + 4 * 7.0, 5 + 6 * 2 + 8 * 3 + 9 * 4.0]]
    # dilation 2: taps at rows {0,2} x cols {0,2}
    ref, _ = orc.conv2d_fprop(X, Wf, dil=(2, 2))
    assert ref.view(1).tolist() == [1 * 1 + 3 * 2 + 7 * 3 + 9 * 4.0]


def test_conv_hand_computed_rectangular_two_channels():
    # H=2, W=3, C=2; K=2 filters of size R=1, S=2.  Written out by hand.
    X = bf([[[1, 10], [2, 20], [3, 30]], [[4, 40], [5, 50], [6, 60]]]).view(1, 2, 3, 2)
    Wf = bf([[[1, 0], [0, 1]], [[-1, 1], [2, 0]]]).view(2, 1, 2, 2)     # [K][R=1][S][C]
    ref, _ = orc.conv2d_fprop(X, Wf)
    # k=0: x[.,q,0] + x[.,q+1,1];   k=1: -x[.,q,0] + x[.,q,1] + 2 x[.,q+1,0]
    want = [[[1 + 20.0, -1 + 10 + 4.0], [2 + 30.0, -2 + 20 + 6.0]],
            [[4 + 50.0, -4 + 40 + 10.0], [5 + 60.0, -5 + 50 + 12.0]]]
    assert ref.view(2, 2, 2).tolist() == want


def test_conv_delta_filter_reproduces_input():
    N, H, W, C = 2, 5, 6, 4
    X = randi([N, H, W, C], 10, 6)
    Wf = torch.zeros(C, 3, 3, C, dtype=torch.bfloat16)
    for k in range(C):
        Wf[k, 1, 1, k] = 1
    ref, _ = orc.conv2d_fprop(X, Wf, pad=(1, 1))
    assert torch.equal(ref, X.double())


def test_conv_all_ones_counts_valid_taps():
    C = 3
    X = torch.ones(1, 5, 7, C, dtype=torch.bfloat16)
    Wf = torch.ones(2, 3, 3, C, dtype=torch.bfloat16)
    ref, _ = orc.conv2d_fprop(X, Wf, pad=(1, 1))
    y = ref[0, :, :, 0]
    assert y[2, 3] == 9 * C and y[0, 3] == 6 * C and y[2, 0] == 6 * C and y[0, 0] == 4 * C and y[4, 6] == 4 * C
    assert torch.equal(ref[..., 0], ref[..., 1])


def test_conv_1x1_is_a_gemm():
    N, H, W, C, K = 2, 3, 4, 8, 5
    X = randi([N, H, W, C], 11, 6)
    Wf = randi([K, 1, 1, C], 11, 7)
    bias = bf([1, -2, 3, -4, 5])
    conv, cacc = orc.conv2d_fprop(X, Wf, bias=bias, epi="relu")
    gemm, gacc = orc.gemm(X.view(-1, C), Wf.view(K, C), bias=bias, epi="relu")
    assert torch.equal(conv.view(-1, K), gemm) and torch.equal(cacc.view(-1, K), gacc)


@pytest.mark.parametrize("pad,stride,dil,R,S", [((1, 1), (1, 1), (1, 1), 3, 3), ((0, 2), (2, 1), (1, 1), 2, 3),
                                              ((2, 2), (1, 2), (2, 2), 3, 3), ((0, 0), (3, 3), (1, 1), 1, 1)])
def test_conv_matches_torch_fp64_conv2d(pad, stride, dil, R, S):
    N, H, W, C, K = 2, 9, 8, 5, 4
    X = inputs.uniform([N, H, W, C], 12, 6)
    Wf = inputs.uniform([K, R, S, C], 12, 7)
    ref, absacc = orc.conv2d_fprop(X, Wf, pad=pad, stride=stride, dil=dil)
    want = torch.nn.functional.conv2d(X.double().permute(0, 3, 1, 2), Wf.double().permute(0, 3, 1, 2),
                                      stride=stride, padding=pad, dilation=dil).permute(0, 2, 3, 1)
    assert ref.shape == want.shape
    assert torch.allclose(ref, want, rtol=0, atol=1e-12)
    wabs = torch.nn.functional.conv2d(X.double().abs().permute(0, 3, 1, 2), Wf.double().abs().permute(0, 3, 1, 2),
                                      stride=stride, padding=pad, dilation=dil).permute(0, 2, 3, 1)
    assert torch.allclose(absacc, wabs, rtol=0, atol=1e-12)


def test_conv_shift_equivariance_in_the_interior():
    X = randi([1, 8, 8, 2], 13, 6)
    Wf = randi([3, 3, 3, 2], 13, 7)
    shifted = torch.zeros_like(X)
    shifted[:, :, 1:, :] = X[:, :, :-1, :]
    y, _ = orc.conv2d_fprop(X, Wf, pad=(1, 1))
    ys, _ = orc.conv2d_fprop(shifted, Wf, pad=(1, 1))
    assert torch.equal(ys[:, :, 2:-1, :], y[:, :, 1:-2, :])


def test_conv_beta_bias_and_ranges():
    N, H, W, C, K = 1, 4, 4, 2, 3
    X, Wf = randi([N, H, W, C], 14, 6), randi([K, 3, 3, C], 14, 7)
    Cin = randi([N, H, W, K], 14, 3)
    bias = bf([0.5, -1, 2])
    base, _ = orc.conv2d_fprop(X, Wf, pad=(1, 1))
    full, facc = orc.conv2d_fprop(X, Wf, pad=(1, 1), Cin=Cin, bias=bias, alpha=3.0, beta=2.0, epi="bias")
    assert torch.equal(full, 3 * base + 2 * Cin.double() + bias.double())
    part, _ = orc.conv2d_fprop(X, Wf, pad=(1, 1), Cin=Cin, bias=bias, alpha=3.0, beta=2.0, epi="bias", pixels=(3, 9))
    assert torch.equal(part, full.view(-1, K)[3:9])
    pts, pacc = orc.conv2d_points(X, Wf, [0, 15, 6], [2, 0, 1], pad=(1, 1), Cin=Cin, bias=bias, alpha=3.0, beta=2.0,
                                  epi="bias")
    assert torch.equal(pts, full.view(-1, K)[[0, 15, 6], [2, 0, 1]])
    assert torch.equal(pacc, facc.view(-1, K)[[0, 15, 6], [2, 0, 1]])


def test_conv_output_extent():
    assert orc.conv_out_extent(56, 1, 1, 3, 1) == 56
    assert orc.conv_out_extent(7, 0, 1, 3, 2) == 3
    assert orc.conv_out_extent(7, 1, 2, 3, 2) == 3     # (7 + 2 - 4 - 1) / 2 + 1
    assert orc.conv_out_extent(2, 0, 1, 3, 1) == 0


# ---------------------------------------------------------------- tolerance is not vacuous

def test_tolerance_accepts_bf16_rounding_and_rejects_skipped_work():
    M, N, K = 64, 96, 512
    A, Bt, bias = inputs.make_gemm(M, N, K, "normal", K ** -0.25, bias=True, seed=15)   # outputs ~ N(0,1)
    ref, absacc = orc.gemm(A, Bt, bias=bias, epi="relu")
    parity.assert_matches(ref.to(torch.bfloat16), ref, absacc, "exact result rounded to bf16")
    parity.assert_matches(ref.to(torch.float32), ref, absacc, "exact result rounded to fp32")
    # the "skipped computation step" defects: a dropped 64-wide K block, no bias, no activation
    dropped, _ = orc.gemm(A[:, :K - 64], Bt[:, :K - 64], bias=bias, epi="relu")
    no_bias, _ = orc.gemm(A, Bt, epi="relu")
    no_act, _ = orc.gemm(A, Bt, bias=bias, epi="bias")
    for name, wrong in (("dropped K block", dropped), ("no bias", no_bias), ("no activation", no_act)):
        for dt in (torch.bfloat16, torch.float32):
            assert parity.mismatches(wrong.to(dt), ref, absacc).any(), (name, dt)
    # erf-GELU instead of tanh-GELU is caught on the fp32 path when nothing cancels (K = 1: absacc = |x|)
    x = torch.linspace(-4, 4, 64, dtype=torch.float64).to(torch.bfloat16).view(-1, 1)
    want, wacc = orc.gemm(x, torch.ones(1, 1, dtype=torch.bfloat16), epi="gelu")
    assert torch.equal(wacc, x.double().abs())
    erf = torch.nn.functional.gelu(x.double())
    assert not parity.mismatches(want.float(), want, wacc).any()
    assert parity.mismatches(erf.float(), want, wacc).any()


# ---------------------------------------------------------------- transpose with dtype conversion

def test_transpose_hand_cases_and_rounding_ties():
    x = torch.tensor([[[1.0, 2.0, 3.0], [4.0, 5.0, 6.0]]], dtype=torch.float32)          # [1, 2, 3]
    assert orc.transpose(x, torch.float32).tolist() == [[[1.0, 4.0], [2.0, 5.0], [3.0, 6.0]]]
    # fp32 -> bf16: 8 significant bits; ties go to the even neighbour
    ties = torch.tensor([[[1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, -(1.0 + 2.0 ** -8),
                           3.4028234663852886e38, 3.3895313892515355e38]]], dtype=torch.float32)
    got = orc.transpose(ties, torch.bfloat16).view(-1).tolist()
    assert got[:4] == [1.0, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -7, -1.0]
    assert got[4] == float("inf") and got[5] == 3.3895313892515355e38       # fp32 max rounds up to infinity; bf16 max stays
    nan = orc.transpose(torch.tensor([[[float("nan")]]], dtype=torch.float32), torch.bfloat16)
    assert math.isnan(float(nan))


def test_transpose_fp16_conversions_hand_cases_all_codes_and_library():
    # hand cases of fp32 -> fp16 (11 significant bits, ties to even, subnormal grid 2^-24, overflow at 65520)
    cases = torch.tensor([[[1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 1.0 + 2.0 ** -11 + 2.0 ** -20, -(1.0 + 2.0 ** -11),
                            65519.99, 65520.0, 65504.0, 2.0 ** -24, 2.0 ** -25, 2.0 ** -25 * 1.0001, 3 * 2.0 ** -25,
                            2.0 ** -14 - 2.0 ** -25, 0.0]]], dtype=torch.float32)
    got = orc.transpose(cases, torch.float16).view(-1).tolist()
    assert got[:4] == [1.0, 1.0 + 2.0 ** -9, 1.0 + 2.0 ** -10, -1.0]
    assert got[4] == 65504.0 and got[5] == float("inf") and got[6] == 65504.0
    assert got[7] == 2.0 ** -24 and got[8] == 0.0 and got[9] == 2.0 ** -24 and got[10] == 2.0 ** -23       # ties to even on the subnormal grid
    assert got[11] == 2.0 ** -14 and got[12] == 0.0
    assert math.isnan(float(orc.transpose(torch.tensor([[[float("nan")]]]), torch.float16)))
    # every fp16 code: widening is exact, so fp16 -> fp32 -> fp16 must give the code's own value back
    codes = torch.arange(65536, dtype=torch.int32).to(torch.int16).view(torch.float16).view(1, 256, 256)
    finite = torch.isfinite(codes.float())
    widened = orc.transpose(codes, torch.float32)                       # [1, 256, 256] transposed
    assert torch.equal(widened.permute(0, 2, 1)[finite], codes.double()[finite])
    back = orc.transpose(codes.float(), torch.float16)
    assert torch.equal(back.permute(0, 2, 1)[finite], codes.double()[finite])
    # every bf16 code through bf16 -> fp16 and every fp16 code through fp16 -> bf16 against torch's casts (an unrelated
    # library routine), and random fp32 values through fp32 -> fp16
    bcodes = torch.arange(65536, dtype=torch.int32).to(torch.int16).view(torch.bfloat16).view(1, 256, 256)
    bfin = torch.isfinite(bcodes.float())
    assert torch.equal(orc.transpose(bcodes, torch.float16).permute(0, 2, 1)[bfin], bcodes.to(torch.float16).double()[bfin])
    assert torch.equal(orc.transpose(codes, torch.bfloat16).permute(0, 2, 1)[finite], codes.to(torch.bfloat16).double()[finite])
    g = torch.Generator().manual_seed(5)
    x = torch.randn(2, 64, 48, generator=g) * torch.tensor([1e-7, 1e-3, 1.0, 300.0, 7e4, 1e-5]).repeat(8)
    assert torch.equal(orc.transpose(x, torch.float16), x.permute(0, 2, 1).to(torch.float16).double())


def test_transpose_matches_torch_permute_and_cast():
    x32 = inputs.normal([3, 37, 29], 21, 1).float() * 1.2345 + torch.rand(3, 37, 29, generator=torch.Generator().manual_seed(1)) * 1e-3
    xbf = inputs.uniform([3, 37, 29], 21, 2)
    for x in (x32, xbf):
        for od in (torch.float32, torch.bfloat16):
            want = x.permute(0, 2, 1).contiguous().to(od).double()
            assert torch.equal(orc.transpose(x, od), want), (x.dtype, od)
    padded = x32.new_zeros(3, 37, 40)
    padded[:, :, :29] = x32
    assert torch.equal(orc.transpose(padded[:, :, :29], torch.bfloat16), x32.permute(0, 2, 1).to(torch.bfloat16).double())
    assert orc.transpose_bytes(32, 256, 3136, 4, 2) == 32 * 256 * 3136 * 6


# ---------------------------------------------------------------- fp16 inputs

def test_fp16_inputs_are_widened_exactly():
    # every one of the 65536 binary16 patterns, through the oracle's own decoder (a K = 1 product with 1.0)
    bits = torch.arange(0, 65536, dtype=torch.int32).to(torch.int16).view(torch.float16)
    finite = torch.isfinite(bits)
    col = bits[finite].view(-1, 1)
    one = torch.ones(1, 1, dtype=torch.float16)
    ref, _ = orc.gemm(col, one)
    assert torch.equal(ref.view(-1), col.double().view(-1))            # torch's own widening as the library pin
    assert float(orc.gemm(torch.tensor([[6.103515625e-05]], dtype=torch.float16), one)[0]) == 2.0 ** -14
    assert float(orc.gemm(torch.tensor([[5.960464477539063e-08]], dtype=torch.float16), one)[0]) == 2.0 ** -24   # smallest subnormal
    assert float(orc.gemm(torch.tensor([[65504.0]], dtype=torch.float16), one)[0]) == 65504.0


def test_fp16_gemm_and_conv_match_torch_fp64():
    A = (inputs.uniform([23, 41], 31, 1).float() * 3.3).half()
    Bt = (inputs.uniform([17, 41], 31, 2).float() * 0.7).half()
    bias = inputs.normal([17], 31, 4).half()
    C = inputs.normal([23, 17], 31, 3).half()
    ref, _ = orc.gemm(A, Bt, C=C, bias=bias, alpha=0.5, beta=2.0, epi="bias")
    want = 0.5 * (A.double() @ Bt.double().t()) + 2.0 * C.double() + bias.double()
    assert torch.allclose(ref, want, rtol=0, atol=1e-12)
    X = inputs.uniform([2, 6, 7, 5], 32, 6).half()
    Wf = inputs.uniform([4, 3, 3, 5], 32, 7).half()
    ref, _ = orc.conv2d_fprop(X, Wf, pad=(1, 1))
    want = torch.nn.functional.conv2d(X.double().permute(0, 3, 1, 2), Wf.double().permute(0, 3, 1, 2), padding=1).permute(0, 2, 3, 1)
    assert torch.allclose(ref, want, rtol=0, atol=1e-12)
    with pytest.raises(ValueError):
        orc.gemm(A, Bt.to(torch.bfloat16))


# ---------------------------------------------------------------- 8-bit floating-point inputs

@pytest.mark.parametrize("dtype", [torch.float8_e4m3fn, torch.float8_e5m2])
def test_fp8_inputs_are_widened_exactly(dtype):
    bits = torch.arange(0, 256, dtype=torch.int32).to(torch.uint8).view(dtype)
    wide = bits.float().double()                                    # torch's widening as the library pin
    finite = torch.isfinite(wide)
    col = bits[finite].view(-1, 1)
    ref, _ = orc.gemm(col, torch.ones(1, 1).to(dtype))
    assert torch.equal(ref.view(-1), wide[finite])
    # hand values: largest finite, smallest subnormal, 1.5
    one = torch.ones(1, 1).to(dtype)
    big, tiny = (448.0, 2.0 ** -9) if dtype == torch.float8_e4m3fn else (57344.0, 2.0 ** -16)
    for v in (big, tiny, 1.5, -0.75):
        assert float(orc.gemm(torch.tensor([[v]]).to(dtype), one)[0]) == v


def test_fp8_gemm_with_bf16_bias_matches_torch_fp64():
    A = (inputs.uniform([19, 48], 41, 1).float() * 3).to(torch.float8_e4m3fn)
    Bt = (inputs.uniform([11, 48], 41, 2).float() * 2).to(torch.float8_e4m3fn)
    bias = inputs.normal([11], 41, 4)                               # bf16 bias with 8-bit inputs
    ref, _ = orc.gemm(A, Bt, bias=bias, alpha=0.25, epi="bias")
    want = 0.25 * (A.float().double() @ Bt.float().double().t()) + bias.double()
    assert torch.allclose(ref, want, rtol=0, atol=1e-12)
    X = inputs.uniform([1, 5, 6, 16], 42, 6).to(torch.float8_e5m2)
    Wf = inputs.uniform([4, 3, 3, 16], 42, 7).to(torch.float8_e5m2)
    ref, _ = orc.conv2d_fprop(X, Wf, pad=(1, 1))
    want = torch.nn.functional.conv2d(X.float().double().permute(0, 3, 1, 2), Wf.float().double().permute(0, 3, 1, 2),
                                      padding=1).permute(0, 2, 3, 1)
    assert torch.allclose(ref, want, rtol=0, atol=1e-12)


# ------------------------------------------------------------------------------------------------
# Extended epilogue chain (Table 1c: per_row_scale, per_col_scale, column_broadcast, scale, aux_store, aux_load)
# ------------------------------------------------------------------------------------------------

def test_chain_hand_computed():
    # A = [[1, 2], [3, 4]], B^T = [[1, 0], [1, 1]] (column-major B: rows are columns of B) -> A.B = [[1, 3], [3, 7]]
    A = torch.tensor([[1., 2.], [3., 4.]]).to(torch.bfloat16)
    Bt = torch.tensor([[1., 0.], [1., 1.]]).to(torch.bfloat16)
    C = torch.tensor([[1., -1.], [2., 0.]])
    bias = torch.tensor([0.5, -0.5]).to(torch.bfloat16)
    R = torch.tensor([[10., 20.], [30., 40.]])
    d, aux, mag_d, mag = orc.gemm_ex(A, Bt, alpha=2.0, beta=0.5, C=C, bias=bias, epi="relu",
                                        row_scale=torch.tensor([1., -1.]), col_scale=torch.tensor([2., 0.5]),
                                        row_bias=torch.tensor([0.25, 1.]), post_scale=3.0, aux_load=R)
    # t[0,0] = 2*1*1*2 + 0.5*1 + 0.5 + 0.25 = 5.25      t[0,1] = 2*3*1*0.5 - 0.5 - 0.5 + 0.25 = 2.25
    # t[1,0] = 2*3*(-1)*2 + 1 + 0.5 + 1 = -9.5           t[1,1] = 2*7*(-1)*0.5 + 0 - 0.5 + 1 = -6.5
    assert aux.tolist() == [[5.25, 2.25], [-9.5, -6.5]]
    # D = 3 relu(t) + R
    assert d.tolist() == [[25.75, 26.75], [30.0, 40.0]]
    assert mag.tolist() == [[5.25, 4.25], [14.5, 8.5]]
    assert mag_d.tolist() == [[25.75, 32.75], [73.5, 65.5]]


def test_chain_without_extras_is_the_plain_epilogue():
    A, B, _ = inputs.make_gemm(37, 29, 50, "uniform", 1.0, seed=3)
    C = inputs.uniform([37, 29], 3, 3).to(torch.float32)
    bias = inputs.normal([29], 3, 4)
    for epi in ("none", "gelu", "silu", "tanh"):
        want, want_abs = orc.gemm(A, B, C=C, bias=bias, alpha=0.75, beta=-1.5, epi=epi)
        d, aux, mag_d, mag = orc.gemm_ex(A, B, C=C, bias=bias, alpha=0.75, beta=-1.5, epi=epi)
        torch.testing.assert_close(d, want, rtol=1e-13, atol=1e-13)
        torch.testing.assert_close(mag_d, want_abs, rtol=1e-13, atol=1e-13)
        lin, _ = orc.gemm(A, B, C=C, bias=bias, alpha=0.75, beta=-1.5)
        torch.testing.assert_close(aux, lin, rtol=1e-13, atol=1e-13)


def test_chain_scales_and_row_bias_reduce_to_plain_products():
    M, N, K = 23, 19, 40
    A, B, _ = inputs.make_gemm(M, N, K, "uniform", 1.0, seed=5)          # B is [N, K] (column-major)
    # powers of two scale bf16 values exactly, so the scaled operands are again bf16 matrices
    rs = torch.tensor([2.0 ** ((i % 5) - 2) for i in range(M)])
    cs = torch.tensor([-(2.0 ** ((j % 3) - 1)) for j in range(N)])
    d, _, _, _ = orc.gemm_ex(A, B, row_scale=rs, col_scale=cs)
    As = (A.to(torch.float64) * rs.reshape(M, 1).double()).to(torch.bfloat16)
    Bs = (B.to(torch.float64) * cs.reshape(N, 1).double()).to(torch.bfloat16)
    want, _ = orc.gemm(As, Bs)
    torch.testing.assert_close(d, want, rtol=1e-13, atol=1e-13)
    # a per-row bias is one more k: A' = [A | r], B' = [B | 1]
    r = inputs.uniform([M], 5, 9)                                         # bf16 values
    d, _, _, _ = orc.gemm_ex(A, B, row_bias=r.to(torch.float32))
    A1 = torch.cat([A, r.reshape(M, 1)], dim=1).contiguous()
    B1 = torch.cat([B, torch.ones(N, 1, dtype=torch.bfloat16)], dim=1).contiguous()
    want, _ = orc.gemm(A1, B1)
    torch.testing.assert_close(d, want, rtol=1e-13, atol=1e-13)


def test_chain_post_scale_and_aux_load_follow_the_activation():
    A, B, _ = inputs.make_gemm(9, 11, 16, "uniform", 1.0, seed=8)
    R = inputs.normal([9, 11], 8, 3)
    base, _ = orc.gemm(A, B, epi="gelu")
    d, aux, _, _ = orc.gemm_ex(A, B, epi="gelu", post_scale=-0.5, aux_load=R)
    torch.testing.assert_close(d, -0.5 * base + R.double(), rtol=1e-13, atol=1e-13)
    lin, _ = orc.gemm(A, B)
    torch.testing.assert_close(aux, lin, rtol=0, atol=0)


def test_chain_on_conv_rows_are_pixels_columns_are_channels():
    X, Wf, _ = inputs.make_conv(2, 5, 4, 8, 6, 3, 3, "uniform", 1.0, seed=4)
    cs = torch.tensor([2.0 ** (k % 3) for k in range(6)])
    d, _, _, _ = orc.conv2d_fprop_ex(X, Wf, pad=(1, 1), col_scale=cs, epi="relu")
    Ws = (Wf.to(torch.float64) * cs.reshape(6, 1, 1, 1).double()).to(torch.bfloat16)
    want, _ = orc.conv2d_fprop(X, Ws, pad=(1, 1), epi="relu")
    torch.testing.assert_close(d, want.reshape(-1, 6), rtol=1e-13, atol=1e-13)


# ------------------------------------------------------------------------------------------------
# conv2d_dgrad / conv2d_wgrad (Appendix A.1 operators): the adjoints of the forward convolution
# ------------------------------------------------------------------------------------------------

def test_dgrad_wgrad_hand_computed():
    # N=1, H=W=2, C=K=1, 2x2 filter, no padding -> P=Q=1: y = sum x*w.
    # dx = dy * w (elementwise over the window), dw = dy * x.
    dY = bf([[[[3.0]]]])
    Wf = bf([[[[1.0], [2.0]], [[-1.0], [0.5]]]])
    X = bf([[[[1.0], [2.0]], [[4.0], [-2.0]]]])
    dx, mag = orc.conv2d_dgrad(dY, Wf, (2, 2))
    assert dx.reshape(2, 2).tolist() == [[3.0, 6.0], [-3.0, 1.5]]
    assert mag.reshape(2, 2).tolist() == [[3.0, 6.0], [3.0, 1.5]]
    dw, _ = orc.conv2d_wgrad(dY, X, (2, 2))
    assert dw.reshape(2, 2).tolist() == [[3.0, 6.0], [12.0, -6.0]]
    # 1x3 input, 1x2 filter, pad 1, stride 2 (W direction): outputs q=0 reads w in {-1,0}, q=1 reads w in {1,2}
    dY = bf([[[[1.0], [10.0]]]])                    # [1,1,2,1]
    Wf = bf([[[[2.0], [3.0]]]])                     # [1,1,2,1]
    dx, _ = orc.conv2d_dgrad(dY, Wf, (1, 3), pad=(0, 1), stride=(1, 2))
    assert dx.reshape(3).tolist() == [3.0, 20.0, 30.0]
    X = bf([[[[5.0], [6.0], [7.0]]]])
    dw, _ = orc.conv2d_wgrad(dY, X, (1, 2), pad=(0, 1), stride=(1, 2))
    assert dw.reshape(2).tolist() == [60.0, 75.0]   # tap 0: 10*6 (q=0 is in the halo), tap 1: 1*5 + 10*7


@pytest.mark.parametrize("pad,stride,dil,R,S", [((1, 1), (1, 1), (1, 1), 3, 3), ((0, 2), (2, 1), (1, 2), 2, 3),
                                                ((2, 1), (2, 3), (2, 1), 3, 2), ((0, 0), (1, 1), (1, 1), 1, 1)])
def test_dgrad_wgrad_are_the_adjoints_of_the_forward_oracle(pad, stride, dil, R, S):
    # <conv(X, W), dY> = <X, dgrad(dY, W)> = <W, wgrad(dY, X)>, exactly on small integers
    N_, H, W_, C, K = 2, 7, 6, 3, 4
    X = randi([N_, H, W_, C], 21, 1)
    Wf = randi([K, R, S, C], 21, 2)
    y, _ = orc.conv2d_fprop(X, Wf, pad=pad, stride=stride, dil=dil)
    dY = randi(list(y.shape), 21, 3)
    lhs = float((y * dY.double()).sum())
    dx, _ = orc.conv2d_dgrad(dY, Wf, (H, W_), pad=pad, stride=stride, dil=dil)
    dw, _ = orc.conv2d_wgrad(dY, X, (R, S), pad=pad, stride=stride, dil=dil)
    assert float((dx * X.double()).sum()) == lhs
    assert float((dw * Wf.double()).sum()) == lhs


@pytest.mark.parametrize("pad,stride,dil", [((1, 1), (1, 1), (1, 1)), ((1, 0), (2, 2), (1, 1)), ((2, 2), (1, 2), (2, 1))])
def test_dgrad_wgrad_match_torch_library_gradients(pad, stride, dil):
    N_, H, W_, C, K, R, S = 2, 8, 7, 5, 3, 3, 3
    X, Wf, _ = inputs.make_conv(N_, H, W_, C, K, R, S, "uniform", 1.0, seed=22)
    P = orc.conv_out_extent(H, pad[0], dil[0], R, stride[0])
    Q = orc.conv_out_extent(W_, pad[1], dil[1], S, stride[1])
    dY = inputs.uniform([N_, P, Q, K], 22, 3)
    Cx = inputs.normal([N_, H, W_, C], 22, 4).to(torch.float32)
    dx, _ = orc.conv2d_dgrad(dY, Wf, (H, W_), pad=pad, stride=stride, dil=dil, Cin=Cx, alpha=0.5, beta=2.0)
    dw, _ = orc.conv2d_wgrad(dY, X, (R, S), pad=pad, stride=stride, dil=dil, alpha=-1.5)
    g = dY.double().permute(0, 3, 1, 2)
    want_dx = torch.nn.grad.conv2d_input((N_, C, H, W_), Wf.double().permute(0, 3, 1, 2), g, stride=stride, padding=pad,
                                         dilation=dil).permute(0, 2, 3, 1)
    want_dw = torch.nn.grad.conv2d_weight(X.double().permute(0, 3, 1, 2), (K, C, R, S), g, stride=stride, padding=pad,
                                          dilation=dil).permute(0, 2, 3, 1)
    torch.testing.assert_close(dx, 0.5 * want_dx + 2.0 * Cx.double(), rtol=1e-12, atol=1e-12)
    torch.testing.assert_close(dw, -1.5 * want_dw, rtol=1e-12, atol=1e-12)


def test_dgrad_wgrad_ranges_agree_with_full():
    X, Wf, _ = inputs.make_conv(2, 5, 6, 4, 3, 3, 2, "uniform", 1.0, seed=23)
    dY = inputs.uniform([2, 5, 7, 3], 23, 3)          # pad (1,1): P = 5, Q = 6 + 2 - 1 = 7
    dx, ax = orc.conv2d_dgrad(dY, Wf, (5, 6), pad=(1, 1))
    part, apart = orc.conv2d_dgrad(dY, Wf, (5, 6), pad=(1, 1), pixels=(7, 41))
    assert torch.equal(part, dx.reshape(-1, 4)[7:41]) and torch.equal(apart, ax.reshape(-1, 4)[7:41])
    dw, _ = orc.conv2d_wgrad(dY, X, (3, 2), pad=(1, 1))
    part, _ = orc.conv2d_wgrad(dY, X, (3, 2), pad=(1, 1), filters=(1, 3))
    assert torch.equal(part, dw[1:3])


# ------------------------------------------------------------------------------------------------
# fp32 operands read as tf32 (Appendix A.2: FP32 problems run on TF32 tensor cores)
# ------------------------------------------------------------------------------------------------

def test_tf32_operands_drop_their_low_13_fraction_bits():
    # 1 + 2^-11 + 2^-12 sits above the half-way point between the tf32 neighbours 1 and 1 + 2^-10: a rounding
    # conversion would give 1 + 2^-10, the tensor core's reading (the low 13 bits do not take part) gives 1.
    x = 1.0 + 2.0 ** -11 + 2.0 ** -12
    A = torch.tensor([[x, 1.0 + 2.0 ** -10, -x, 3.0]], dtype=torch.float32)
    B = torch.eye(4, dtype=torch.float32)                        # column-major identity: picks the elements of A
    ref, _ = orc.gemm(A, B)
    assert ref.tolist() == [[1.0, 1.0 + 2.0 ** -10, -1.0, 3.0]]
    # both operands are read that way; the bias (fp32) is used exactly
    bias = torch.tensor([x], dtype=torch.float32)
    ref, _ = orc.gemm(torch.tensor([[x]], dtype=torch.float32), torch.tensor([[x]], dtype=torch.float32), bias=bias)
    assert ref.item() == 1.0 + float(torch.tensor(x, dtype=torch.float32))


def test_tf32_representable_operands_give_the_plain_product():
    A16, B16, _ = inputs.make_gemm(19, 23, 40, "uniform", 1.0, seed=41)       # bf16 values are tf32 values
    want, want_abs = orc.gemm(A16, B16, alpha=0.5, epi="gelu")
    got, got_abs = orc.gemm(A16.float(), B16.float(), alpha=0.5, epi="gelu")
    assert torch.equal(got, want) and torch.equal(got_abs, want_abs)
    X16, W16, _ = inputs.make_conv(2, 6, 5, 4, 3, 3, 3, "uniform", 1.0, seed=42)
    want, _ = orc.conv2d_fprop(X16, W16, pad=(1, 1))
    got, _ = orc.conv2d_fprop(X16.float(), W16.float(), pad=(1, 1))
    assert torch.equal(got, want)


def test_tf32_gemm_matches_torch_fp64_on_masked_operands():
    g = torch.Generator().manual_seed(7)
    A = torch.randn(17, 33, generator=g)
    B = torch.randn(21, 33, generator=g)
    mask = lambda t: (t.view(torch.int32) & -8192).view(torch.float32)     # clear the low 13 bits
    ref, _ = orc.gemm(A, B)
    torch.testing.assert_close(ref, mask(A).double() @ mask(B).double().t(), rtol=1e-13, atol=1e-13)
    assert not torch.allclose(ref, A.double() @ B.double().t(), rtol=0, atol=1e-6)   # the dropped bits are visible


def test_int8_operands_are_plain_integers():
    # hand case incl. the extremes of the type: [[-128, 127]] . [[127], [-128]] = -128*127 + 127*(-128) = -32512
    A = torch.tensor([[-128, 127], [1, 2]], dtype=torch.int8)
    Bt = torch.tensor([[127, -128], [3, -4]], dtype=torch.int8)        # column-major B: rows are columns of B
    ref, absacc = orc.gemm(A, Bt)
    assert ref.tolist() == [[-32512.0, -892.0], [-129.0, -5.0]]
    assert absacc.tolist() == [[32512.0, 892.0], [383.0, 11.0]]
    g = torch.Generator().manual_seed(3)
    A = torch.randint(-128, 128, (13, 40), generator=g, dtype=torch.int8)
    B = torch.randint(-128, 128, (9, 40), generator=g, dtype=torch.int8)
    bias = inputs.normal([9], 3, 4)
    ref, _ = orc.gemm(A, B, bias=bias, alpha=0.5)
    torch.testing.assert_close(ref, 0.5 * (A.double() @ B.double().t()) + bias.double(), rtol=0, atol=0)
    X = torch.randint(-128, 128, (1, 5, 4, 16), generator=g, dtype=torch.int8)
    Wf = torch.randint(-128, 128, (3, 3, 3, 16), generator=g, dtype=torch.int8)
    y, _ = orc.conv2d_fprop(X, Wf, pad=(1, 1))
    want = torch.nn.functional.conv2d(X.double().permute(0, 3, 1, 2), Wf.double().permute(0, 3, 1, 2), padding=1)
    torch.testing.assert_close(y, want.permute(0, 2, 3, 1), rtol=0, atol=0)
