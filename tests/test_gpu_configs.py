"""GPU parity on the five benchmark configurations at their full sizes, in the launch configuration bench.py times.

c1, c2, c3 and c4 are compared with the oracle on EVERY output element (the oracle runs once per configuration and
serves both output types).  c5 (about 1.1e12 MACs) is compared on every row within one row of a group edge or of a
128-row tile edge, plus a seeded 2 % sample of each group's rows spread over the whole group -- never a prefix.
On top of the stated tolerance every compared element must meet a tighter self-imposed bound (one rounding of the
result in the output type plus fp32 accumulation noise), because config 2's products are small against its bias.
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
    sg.set_option("gemv_small_log2", -1)      # the launch configuration bench.py times: the library's own choice of path
    sg.set_option("gemv_max_vectors", -1)
    yield
    torch.cuda.synchronize()
    sg.poll_status()


def sample_points(rows, cols, count, seed):
    pi = inputs.integers(count, seed, 11, 0, rows - 1)
    pj = inputs.integers(count, seed, 12, 0, cols - 1)
    return pi, pj


def assert_tight(got, ref, absacc, what):
    """Tighter than the stated tolerance: one rounding of the result in the output type (2^-8 relative for bf16; the fp32
    path is already judged on that scale) plus fp32 accumulation noise on the scale of the terms summed."""
    parity.assert_matches(got, ref, absacc, what)
    err = (got.detach().cpu().double().reshape(ref.shape) - ref).abs()
    tight = 2.0 ** -8 * ref.abs() + 1e-4 * absacc + 1e-30
    bad = err > tight
    assert not bool(bad.any()), f"{what}: {int(bad.sum())} of {bad.numel()} elements outside the tight bound"


def check_points(D, ref, absacc, pi, pj, what):
    got = D[torch.as_tensor(pi, device=D.device), torch.as_tensor(pj, device=D.device)]
    assert_tight(got, ref, absacc, what)


_REFS = {}


def reference(name, fn):
    """One oracle run per configuration and test session (the reference does not depend on the output type)."""
    if name not in _REFS:
        _REFS[name] = fn()
    return _REFS[name]


def test_c1_gemm_256_every_element():
    c = CFG["c1_gemm_256"]
    A, B, _ = inputs.make_gemm(c["M"], c["N"], c["K"], c["dist"], c["scale"])
    ref, absacc = orc.gemm(A, B)
    D = sg.gemm(A.to(DEV), B.to(DEV))
    assert "gemv_mma_kernel" in sg.last_kernel_name()      # (a product this small runs on the warp-level MMA kernel)
    parity.assert_matches(D, ref, absacc, "c1")
    assert_tight(D, ref, absacc, "c1")
    # and through the tensor-core tiles, which a forced tile shape keeps it on
    sg.set_tuning(64, 0)
    D = sg.gemm(A.to(DEV), B.to(DEV))
    assert "contract_kernel" in sg.last_kernel_name()
    parity.assert_matches(D, ref, absacc, "c1 on the tiles")


@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float32])
def test_c2_gemm_4096_bias_relu(out_dtype):
    c = CFG["c2_gemm_4096_bias_relu"]
    A, B, bias = inputs.make_gemm(c["M"], c["N"], c["K"], c["dist"], c["scale"], bias=True, device=DEV)
    D = sg.gemm(A, B, bias=bias, epi=c["epi"], out_dtype=out_dtype)
    plan = sg.last_launch_plan()
    assert plan["tile_n"] == 256 and plan["cta_pair"] == 1          # the configuration bench.py times
    assert bool(torch.isfinite(D).all()) and bool((D >= 0).all())
    ref, absacc = reference("c2", lambda: orc.gemm(A.cpu(), B.cpu(), bias=bias.cpu(), epi=c["epi"]))
    assert_tight(D, ref, absacc, f"c2 every element, {out_dtype}")


def test_c3_batched_gelu_every_element():
    c = CFG["c3_batched_128x256x256x512_gelu"]
    A, B, _ = inputs.make_gemm(c["M"], c["N"], c["K"], c["dist"], c["scale"], batch=c["batch"])
    ref, absacc = orc.batched_gemm(A, B, epi=c["epi"])
    D = sg.batched_gemm(A.to(DEV), B.to(DEV), epi=c["epi"])
    parity.assert_matches(D, ref, absacc, "c3")
    D32 = sg.batched_gemm(A.to(DEV), B.to(DEV), epi=c["epi"], out_dtype=torch.float32)
    parity.assert_matches(D32, ref, absacc, "c3 fp32 out")


@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float32])
def test_c4_conv_bias_relu(out_dtype):
    c = CFG["c4_conv_32x56x56x256_k256_3x3_bias_relu"]
    X, Wf, bias = inputs.make_conv(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["dist"], c["scale"],
                                   bias=True, device=DEV)
    Y = sg.conv2d_fprop(X, Wf, pad=c["pad"], bias=bias, epi=c["epi"], out_dtype=out_dtype)
    assert bool(torch.isfinite(Y).all()) and bool((Y >= 0).all())
    ref, absacc = reference("c4", lambda: orc.conv2d_fprop(X.cpu(), Wf.cpu(), pad=c["pad"], bias=bias.cpu(), epi=c["epi"]))
    assert_tight(Y.view(-1, c["K"]), ref.reshape(-1, c["K"]), absacc.reshape(-1, c["K"]), f"c4 every element, {out_dtype}")


def test_c5_grouped_silu():
    c = CFG["c5_grouped_16xMx4096x4096_silu"]
    Ms = inputs.grouped_sizes(c["groups"], c["M_lo"], c["M_hi"])
    assert all(c["M_lo"] <= m <= c["M_hi"] for m in Ms)
    As, Bs = inputs.make_grouped(Ms, c["N"], c["K"], c["dist"], c["scale"], device=DEV)
    outs = sg.grouped_gemm(As, Bs, epi=c["epi"])
    compared = 0
    for g, m in enumerate(Ms):
        assert outs[g].shape == (m, c["N"]) and bool(torch.isfinite(outs[g]).all())
        # every row within one row of the group's edges and of every 128-row tile edge ...
        rows = {r for r in range(m) if r % 128 in (0, 1, 127)} | {0, 1, m - 2, m - 1}
        # ... plus a seeded 2 % of the group's rows, spread over the whole group
        rows |= set(inputs.integers(max(1, (m + 49) // 50), 300 + g, 13, 0, m - 1))
        idx = torch.tensor(sorted(r for r in rows if 0 <= r < m))
        compared += len(idx)
        # the oracle's product of the selected rows of A_g with B_g (each output row depends on its own row of A only)
        ref, absacc = orc.gemm(As[g].cpu()[idx].contiguous(), Bs[g].cpu(), epi=c["epi"])
        assert_tight(outs[g][idx.to(DEV)], ref, absacc, f"c5 group {g}: {len(idx)} rows at tile and group edges + sample")
    assert compared >= sum(Ms) // 25


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
