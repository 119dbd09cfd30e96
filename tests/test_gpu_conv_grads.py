"""GPU parity of sg_conv2d_dgrad / sg_conv2d_wgrad against the oracle's definitions."""
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
    sg.poll_status()
    sg.set_tuning(-1, -1)
    sg.set_tail_mode(-1)
    sg.enable_scratch(True)


def extent(size, pad, dil, filt, stride):
    return orc.conv_out_extent(size, pad, dil, filt, stride)


# (N, H, W, C, K, R, S, pad, stride, dil)
GRAD_CASES = [
    (2, 12, 10, 64, 64, 3, 3, (1, 1), (1, 1), (1, 1)),
    (3, 9, 17, 72, 136, 3, 3, (1, 1), (1, 1), (1, 1)),      # ragged channel counts (tails of 8 and 8)
    (1, 20, 20, 128, 64, 1, 1, (0, 0), (1, 1), (1, 1)),
    (2, 11, 13, 64, 96, 3, 2, (2, 0), (1, 1), (2, 1)),      # dilation, asymmetric pads
    (2, 16, 16, 200, 72, 5, 5, (2, 2), (1, 1), (1, 1)),
]
STRIDED = [
    (2, 15, 14, 64, 64, 3, 3, (1, 1), (2, 2), (1, 1)),      # stride 2
    (1, 13, 21, 136, 72, 3, 3, (0, 1), (2, 1), (1, 2)),
    (2, 16, 16, 64, 64, 1, 1, (0, 0), (2, 2), (1, 1)),      # 1x1 stride 2: three of the four output phases get no tap
    (1, 17, 19, 64, 72, 3, 3, (0, 0), (2, 2), (1, 1)),      # the last input row / column is outside every window
    (2, 20, 18, 64, 64, 5, 4, (2, 1), (3, 2), (1, 1)),      # stride 3 x 2
    (1, 21, 20, 72, 64, 3, 3, (2, 2), (2, 2), (2, 2)),      # stride and dilation share a factor
    (1, 23, 9, 64, 64, 4, 2, (1, 0), (4, 1), (1, 1)),       # stride as large as the filter
    (1, 6, 7, 64, 64, 3, 3, (3, 3), (1, 1), (1, 1)),        # pad beyond the filter extent: border windows see padding only
]


def _problem(case, seed, integer):
    N_, H, W, C, K, R, S, pad, stride, dil = case
    P, Q = extent(H, pad[0], dil[0], R, stride[0]), extent(W, pad[1], dil[1], S, stride[1])
    if integer:
        X = inputs.small_integers([N_, H, W, C], seed, 1, -1, 1)
        Wf = inputs.small_integers([K, R, S, C], seed, 2, -1, 1)
        dY = inputs.small_integers([N_, P, Q, K], seed, 3, -1, 1)
    else:
        X, Wf, _ = inputs.make_conv(N_, H, W, C, K, R, S, "normal", 1 / 16., seed=seed)
        dY = inputs.normal([N_, P, Q, K], seed, 3, 1 / 8.)
    return X, Wf, dY


@pytest.mark.parametrize("pair", [0, 1])
@pytest.mark.parametrize("case", GRAD_CASES + STRIDED)
def test_dgrad_integer_inputs_bit_exact(case, pair):
    sg.set_tuning(-1, pair)
    N_, H, W, C, K, R, S, pad, stride, dil = case
    X, Wf, dY = _problem(case, 31, True)
    ref, _ = orc.conv2d_dgrad(dY, Wf, (H, W), pad=pad, stride=stride, dil=dil)
    assert float(ref.abs().max()) < 2 ** 24
    out = torch.full((N_, H, W, C), float("nan"), dtype=torch.float32, device=DEV)
    sg.conv2d_dgrad(dY.to(DEV), Wf.to(DEV), (H, W), pad=pad, stride=stride, dil=dil, out=out)
    parity.assert_bit_exact(out.reshape(-1, C), ref.reshape(-1, C), f"dgrad {case} pair={pair}")


@pytest.mark.parametrize("scratch", [False, True])
@pytest.mark.parametrize("pair", [0, 1])
@pytest.mark.parametrize("case", GRAD_CASES + STRIDED)
def test_wgrad_integer_inputs_bit_exact(case, pair, scratch):
    sg.enable_scratch(scratch)
    sg.set_tuning(-1, pair)
    N_, H, W, C, K, R, S, pad, stride, dil = case
    X, Wf, dY = _problem(case, 32, True)
    ref, _ = orc.conv2d_wgrad(dY, X, (R, S), pad=pad, stride=stride, dil=dil)
    assert float(ref.abs().max()) < 2 ** 24
    out = torch.full((K, R, S, C), float("nan"), dtype=torch.float32, device=DEV)
    sg.conv2d_wgrad(dY.to(DEV), X.to(DEV), (R, S), pad=pad, stride=stride, dil=dil, out=out)
    parity.assert_bit_exact(out.reshape(-1, C), ref.reshape(-1, C), f"wgrad {case} pair={pair} scratch={scratch}")


@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("in_dtype", [torch.bfloat16, torch.float16])
def test_grads_real_values_alpha_beta(in_dtype, out_dtype):
    case = (2, 14, 12, 72, 80, 3, 3, (1, 1), (1, 1), (1, 1))
    N_, H, W, C, K, R, S, pad, stride, dil = case
    X, Wf, dY = (t.to(in_dtype) for t in _problem(case, 33, False))
    Cx = inputs.normal([N_, H, W, C], 33, 5).to(out_dtype)
    Cw = inputs.normal([K, R, S, C], 33, 6).to(out_dtype)
    ref, mag = orc.conv2d_dgrad(dY, Wf, (H, W), pad=pad, Cin=Cx, alpha=0.5, beta=-1.0)
    out = sg.conv2d_dgrad(dY.to(DEV), Wf.to(DEV), (H, W), pad=pad, Cin=Cx.to(DEV), alpha=0.5, beta=-1.0, out_dtype=out_dtype)
    parity.assert_matches(out.reshape(-1, C), ref.reshape(-1, C), mag.reshape(-1, C), "dgrad real")
    ref, mag = orc.conv2d_wgrad(dY, X, (R, S), pad=pad, Cin=Cw, alpha=2.0, beta=0.25)
    out = sg.conv2d_wgrad(dY.to(DEV), X.to(DEV), (R, S), pad=pad, Cin=Cw.to(DEV), alpha=2.0, beta=0.25, out_dtype=out_dtype)
    parity.assert_matches(out.reshape(-1, C), ref.reshape(-1, C), mag.reshape(-1, C), "wgrad real")


def test_grads_are_adjoint_to_the_forward_kernel_on_the_gpu():
    # <fprop(X, W), dY> == <X, dgrad(dY, W)> == <W, wgrad(dY, X)> computed from the three kernels' fp32 outputs
    case = (2, 18, 18, 64, 64, 3, 3, (1, 1), (1, 1), (1, 1))
    N_, H, W, C, K, R, S, pad, stride, dil = case
    X, Wf, dY = (t.to(DEV) for t in _problem(case, 34, True))
    y = sg.conv2d_fprop(X, Wf, pad=pad, out_dtype=torch.float32)
    dx = sg.conv2d_dgrad(dY, Wf, (H, W), pad=pad, out_dtype=torch.float32)
    dw = sg.conv2d_wgrad(dY, X, (R, S), pad=pad, out_dtype=torch.float32)
    lhs = float((y.double() * dY.double()).sum())
    assert float((dx.double() * X.double()).sum()) == lhs
    assert float((dw.double() * Wf.double()).sum()) == lhs


def test_grad_argument_errors_and_empty_sums():
    Wf = torch.zeros((64, 3, 3, 64), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(sg.SolgemmError, match="SG_ERR_UNSUPPORTED"):
        sg.conv2d_dgrad(torch.zeros((1, 1, 1, 64), dtype=torch.bfloat16, device=DEV), Wf, (9, 9), stride=(9, 9))
    with pytest.raises(sg.SolgemmError, match="SG_ERR_INVALID_ARG"):
        sg.conv2d_wgrad(torch.zeros((1, 4, 4, 64), dtype=torch.bfloat16, device=DEV),
                        torch.zeros((1, 4, 4, 64), dtype=torch.bfloat16, device=DEV), (3, 3), pad=(1, 1), dil=(0, 1))
    # an image smaller than the filter has no output pixels: the gradients are beta * Cin
    X = inputs.normal([1, 2, 2, 64], 35, 1).to(DEV)
    dY0 = torch.zeros((1, 0, 0, 64), dtype=torch.bfloat16, device=DEV)
    Cw = inputs.normal([64, 3, 3, 64], 35, 2).to(torch.float32).to(DEV)
    dw = sg.conv2d_wgrad(dY0, X, (3, 3), Cin=Cw, beta=2.0)
    assert torch.equal(dw, 2.0 * Cw)
    Cx = inputs.normal([1, 2, 2, 64], 35, 3).to(torch.float32).to(DEV)
    dx = sg.conv2d_dgrad(dY0, Wf, (2, 2), Cin=Cx, beta=-1.0, out_dtype=torch.float32)
    assert torch.equal(dx, -Cx)


def test_wgrad_long_pixel_contraction_is_cut_into_k_ranges():
    # few output tiles, 8192 pixels to sum over: with the scratch lent the planner shares each tile's contraction
    case = (8, 32, 32, 64, 128, 3, 3, (1, 1), (1, 1), (1, 1))
    N_, H, W, C, K, R, S, pad, stride, dil = case
    X, Wf, dY = _problem(case, 36, True)
    ref, _ = orc.conv2d_wgrad(dY, X, (R, S), pad=pad)
    out = sg.conv2d_wgrad(dY.to(DEV), X.to(DEV), (R, S), pad=pad)
    assert sg.last_launch_plan()["tail_split"] < 0, sg.last_launch_plan()
    parity.assert_bit_exact(out.reshape(-1, C), ref.reshape(-1, C), "wgrad k ranges")
    Xr, _, dYr = _problem(case, 37, False)
    ref, mag = orc.conv2d_wgrad(dYr, Xr, (R, S), pad=pad)
    out = sg.conv2d_wgrad(dYr.to(DEV), Xr.to(DEV), (R, S), pad=pad)
    parity.assert_matches(out.reshape(-1, C), ref.reshape(-1, C), mag.reshape(-1, C), "wgrad k ranges real")


@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float32])
def test_strided_dgrad_real_values_with_residual(out_dtype):
    # stride 2: four launches, each writing its own pixels of dX (and reading the same pixels of Cin)
    case = (2, 19, 18, 72, 80, 3, 3, (1, 1), (2, 2), (1, 1))
    N_, H, W, C, K, R, S, pad, stride, dil = case
    X, Wf, dY = _problem(case, 38, False)
    Cx = inputs.normal([N_, H, W, C], 38, 5).to(out_dtype)
    ref, mag = orc.conv2d_dgrad(dY, Wf, (H, W), pad=pad, stride=stride, Cin=Cx, alpha=1.5, beta=0.5)
    out = torch.full((N_, H, W, C), float("nan"), dtype=out_dtype, device=DEV)
    sg.conv2d_dgrad(dY.to(DEV), Wf.to(DEV), (H, W), pad=pad, stride=stride, Cin=Cx.to(DEV), alpha=1.5, beta=0.5, out=out)
    parity.assert_matches(out.reshape(-1, C), ref.reshape(-1, C), mag.reshape(-1, C), "strided dgrad")
