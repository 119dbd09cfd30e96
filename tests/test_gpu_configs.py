"""GPU parity on the five benchmark configurations at their full sizes.

Small configurations are compared on every element.  For the large ones the
oracle computes every row next to a tile edge of the first / last tiles plus
seeded random points spread over the whole output (never a prefix), and the
whole output is additionally checked for finiteness and against a tighter
self-imposed bound on the sampled points.
"""
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
CFG = inputs.CONFIGS


@pytest.fixture(autouse=True)
def _clean_status():
    sg.set_tuning(-1, -1)
    yield
    torch.cuda.synchronize()
    sg.poll_status()


def sample_points(rows, cols, count, seed):
    pi = inputs.integers(count, seed, 11, 0, rows - 1)
    pj = inputs.integers(count, seed, 12, 0, cols - 1)
    return pi, pj


def check_points(D, ref, absacc, pi, pj, what):
    got = D[torch.as_tensor(pi, device=D.device), torch.as_tensor(pj, device=D.device)]
    parity.assert_matches(got, ref, absacc, what)
    # tighter than the stated tolerance: one bf16 rounding of the result plus fp32 accumulation noise
    err = (got.cpu().double() - ref).abs()
    tight = 2.0 ** -8 * ref.abs() + 1e-4 * absacc + 1e-30
    assert bool((err <= tight).all()), f"{what}: sampled points outside the tight bound"


def test_c1_gemm_256_every_element():
    c = CFG["c1_gemm_256"]
    A, B, _ = inputs.make_gemm(c["M"], c["N"], c["K"], c["dist"], c["scale"])
    ref, absacc = orc.gemm(A, B)
    D = sg.gemm(A.to(DEV), B.to(DEV))
    parity.assert_matches(D, ref, absacc, "c1")


@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float32])
def test_c2_gemm_4096_bias_relu(out_dtype):
    c = CFG["c2_gemm_4096_bias_relu"]
    A, B, bias = inputs.make_gemm(c["M"], c["N"], c["K"], c["dist"], c["scale"], bias=True, device=DEV)
    D = sg.gemm(A, B, bias=bias, epi=c["epi"], out_dtype=out_dtype)
    assert bool(torch.isfinite(D).all()) and bool((D >= 0).all())
    hA, hB, hb = A.cpu(), B.cpu(), bias.cpu()
    for r0 in (0, 120, 2040, 4088):                      # rows on both sides of tile edges, first and last tiles
        ref, absacc = orc.gemm(hA, hB, bias=hb, epi=c["epi"], rows=(r0, r0 + 8))
        parity.assert_matches(D[r0:r0 + 8], ref, absacc, f"c2 rows {r0}")
    pi, pj = sample_points(c["M"], c["N"], 4096, 7)
    ref, absacc = orc.gemm_points(hA, hB, pi, pj, bias=hb, epi=c["epi"])
    check_points(D, ref, absacc, pi, pj, "c2 sampled")


def test_c3_batched_gelu_every_element():
    c = CFG["c3_batched_128x256x256x512_gelu"]
    A, B, _ = inputs.make_gemm(c["M"], c["N"], c["K"], c["dist"], c["scale"], batch=c["batch"])
    ref, absacc = orc.batched_gemm(A, B, epi=c["epi"])
    D = sg.batched_gemm(A.to(DEV), B.to(DEV), epi=c["epi"])
    parity.assert_matches(D, ref, absacc, "c3")
    D32 = sg.batched_gemm(A.to(DEV), B.to(DEV), epi=c["epi"], out_dtype=torch.float32)
    parity.assert_matches(D32, ref, absacc, "c3 fp32 out")


def test_c4_conv_bias_relu():
    c = CFG["c4_conv_32x56x56x256_k256_3x3_bias_relu"]
    X, Wf, bias = inputs.make_conv(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["dist"], c["scale"],
                                   bias=True, device=DEV)
    Y = sg.conv2d_fprop(X, Wf, pad=c["pad"], bias=bias, epi=c["epi"])
    assert bool(torch.isfinite(Y).all()) and bool((Y >= 0).all())
    hX, hW, hb = X.cpu(), Wf.cpu(), bias.cpu()
    PQ = 56 * 56
    Yf = Y.view(-1, c["K"])
    # image corners and borders, a tile edge (pixel 128), an image boundary, the very last pixels
    for p0 in (0, 50, 120, PQ - 8, PQ + 48, 17 * PQ + 1000, 32 * PQ - 16):
        ref, absacc = orc.conv2d_fprop(hX, hW, pad=c["pad"], bias=hb, epi=c["epi"], pixels=(p0, p0 + 16))
        parity.assert_matches(Yf[p0:p0 + 16], ref, absacc, f"c4 pixels {p0}")
    ppix, pk = sample_points(32 * PQ, c["K"], 2048, 9)
    ref, absacc = orc.conv2d_points(hX, hW, ppix, pk, pad=c["pad"], bias=hb, epi=c["epi"])
    check_points(Yf, ref, absacc, ppix, pk, "c4 sampled")


def test_c5_grouped_silu():
    c = CFG["c5_grouped_16xMx4096x4096_silu"]
    Ms = inputs.grouped_sizes(c["groups"], c["M_lo"], c["M_hi"])
    assert all(c["M_lo"] <= m <= c["M_hi"] for m in Ms)
    As, Bs = inputs.make_grouped(Ms, c["N"], c["K"], c["dist"], c["scale"], device=DEV)
    outs = sg.grouped_gemm(As, Bs, epi=c["epi"])
    for g, m in enumerate(Ms):
        assert outs[g].shape == (m, c["N"]) and bool(torch.isfinite(outs[g]).all())
        hA, hB = As[g].cpu(), Bs[g].cpu()
        last = max(m - 4, 0)
        for r0, r1 in ((0, 2), (last, m)):               # first rows and the ragged last rows of every group
            ref, absacc = orc.gemm(hA, hB, epi=c["epi"], rows=(r0, r1))
            parity.assert_matches(outs[g][r0:r1], ref, absacc, f"c5 group {g} rows {r0}:{r1}")
        pi, pj = sample_points(m, c["N"], 256, 100 + g)
        ref, absacc = orc.gemm_points(hA, hB, pi, pj, epi=c["epi"])
        check_points(outs[g], ref, absacc, pi, pj, f"c5 group {g} sampled")


def test_c4_sized_conv_gradients():
    # the gradients of the benchmark convolution at its full size, in the configuration bench.py --widened times
    c = CFG["c4_conv_32x56x56x256_k256_3x3_bias_relu"]
    N_, H, W, C, K, R, S = c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"]
    X = inputs.normal([N_, H, W, C], 70, 1, device=DEV)
    dY = inputs.normal([N_, H, W, K], 70, 3, 1 / 16., device=DEV)
    Wf = inputs.normal([K, R, S, C], 70, 2, 1 / 48., device=DEV)
    hX, hdY, hW = X.cpu(), dY.cpu(), Wf.cpu()
    dX = sg.conv2d_dgrad(dY, Wf, (H, W), pad=c["pad"])
    assert bool(torch.isfinite(dX).all())
    PQ = H * W
    dXf = dX.view(-1, C)
    for p0 in (0, 52, 124, PQ - 6, 9 * PQ + 1500, N_ * PQ - 8):      # corners, a tile edge, an image boundary, the end
        ref, absacc = orc.conv2d_dgrad(hdY, hW, (H, W), pad=c["pad"], pixels=(p0, p0 + 8))
        parity.assert_matches(dXf[p0:p0 + 8], ref, absacc, f"c4 dgrad pixels {p0}")
    sg.enable_scratch(True)                                             # (the environment may have turned lending off)
    dW = sg.conv2d_wgrad(dY, X, (R, S), pad=c["pad"])                  # fp32, K ranges through the scratch
    assert sg.last_launch_plan()["tail_split"] < 0 and bool(torch.isfinite(dW).all())
    for k0 in (0, 131, K - 1):                                          # first tile, across the pair's second CTA, last row
        ref, absacc = orc.conv2d_wgrad(hdY, hX, (R, S), pad=c["pad"], filters=(k0, k0 + 1))
        parity.assert_matches(dW[k0:k0 + 1].reshape(-1, C), ref.reshape(-1, C), absacc.reshape(-1, C), f"c4 wgrad filter {k0}")
