"""GPU parity of fp32 operands contracted on the TF32 tensor-core path."""
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
    yield
    torch.cuda.synchronize()
    sg.poll_status()
    sg.set_tuning(-1, -1)


def test_tensor_core_reads_fp32_operands_as_truncated_tf32():
    # the oracle's reading of the operand type, checked on the hardware: 1 + 2^-11 + 2^-12 must count as 1
    x = 1.0 + 2.0 ** -11 + 2.0 ** -12
    A = torch.zeros((128, 32), dtype=torch.float32)
    A[:, 0] = x
    A[:, 1] = 1.0 + 2.0 ** -10
    B = torch.zeros((64, 32), dtype=torch.float32)
    B[0, 0] = 1.0
    B[1, 1] = 1.0
    B[2, 0] = x
    D = sg.gemm(A.to(DEV), B.to(DEV), out_dtype=torch.float32).cpu()
    assert float(D[5, 0]) == 1.0, f"operand bits below tf32 are not dropped: got {float(D[5, 0])!r}"
    assert float(D[5, 1]) == 1.0 + 2.0 ** -10
    assert float(D[5, 2]) == 1.0
    ref, _ = orc.gemm(A, B)
    parity.assert_bit_exact(D, ref, "tf32 truncation")


@pytest.mark.parametrize("tile_n,pair", [(64, 0), (128, 0), (256, 0), (128, 1), (256, 1)])
@pytest.mark.parametrize("M,N,K", [(256, 256, 256), (300, 200, 132), (1000, 520, 1036), (129, 72, 4)])
def test_tf32_integer_problem_bit_exact(M, N, K, tile_n, pair):
    sg.set_tuning(tile_n, pair)
    A = inputs.small_integers([M, K], 71, 1).float()
    B = inputs.small_integers([N, K], 71, 2).float()
    ref, _ = orc.gemm(A, B)
    D = torch.full((M, N), float("nan"), dtype=torch.float32, device=DEV)
    sg.gemm(A.to(DEV), B.to(DEV), out=D)
    parity.assert_bit_exact(D, ref, f"tf32 gemm {M}x{N}x{K} tile_n={tile_n} pair={pair}")


@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_tf32_real_values_epilogue_batched_grouped_and_conv(out_dtype):
    g = torch.Generator().manual_seed(5)
    M, N, K = 333, 264, 520
    A = torch.randn(M, K, generator=g)
    B = torch.randn(N, K, generator=g) / 16
    bias = torch.randn(N, generator=g)
    C = torch.randn(M, N, generator=g).to(out_dtype)
    ref, absacc = orc.gemm(A, B, C=C, bias=bias, alpha=0.5, beta=0.25, epi="gelu")
    D = sg.gemm(A.to(DEV), B.to(DEV), C=C.to(DEV), bias=bias.to(DEV), alpha=0.5, beta=0.25, epi="gelu", out_dtype=out_dtype)
    parity.assert_matches(D, ref, absacc, "tf32 gemm")
    # batched with a per-batch bias
    Ab = torch.randn(3, 130, 96, generator=g)
    Bb = torch.randn(3, 72, 96, generator=g) / 8
    bb = torch.randn(3, 72, generator=g)
    Db = sg.batched_gemm(Ab.to(DEV), Bb.to(DEV), bias=bb.to(DEV), epi="relu", out_dtype=out_dtype)
    for i in range(3):
        ref, absacc = orc.gemm(Ab[i], Bb[i], bias=bb[i], epi="relu")
        parity.assert_matches(Db[i], ref, absacc, f"tf32 batch {i}")
    # grouped
    Ms = [100, 0, 257]
    As = [torch.randn(m, 64, generator=g) for m in Ms]
    Bs = [torch.randn(40, 64, generator=g) / 8 for _ in Ms]
    outs = sg.grouped_gemm([a.to(DEV) for a in As], [b.to(DEV) for b in Bs], epi="silu", out_dtype=out_dtype)
    for a, b, o in zip(As, Bs, outs):
        if a.shape[0]:
            ref, absacc = orc.gemm(a, b, epi="silu")
            parity.assert_matches(o, ref, absacc, "tf32 grouped")
    # convolution
    X = torch.randn(2, 9, 8, 36, generator=g)
    Wf = torch.randn(40, 3, 3, 36, generator=g) / 18
    bc = torch.randn(40, generator=g)
    ref, absacc = orc.conv2d_fprop(X, Wf, pad=(1, 1), bias=bc, epi="relu")
    Y = sg.conv2d_fprop(X.to(DEV), Wf.to(DEV), pad=(1, 1), bias=bc.to(DEV), epi="relu", out_dtype=out_dtype)
    parity.assert_matches(Y.reshape(-1, 40), ref.reshape(-1, 40), absacc.reshape(-1, 40), "tf32 conv")


def test_tf32_argument_rules():
    A = torch.zeros((128, 128), dtype=torch.float32, device=DEV)
    with pytest.raises(sg.SolgemmError, match="SG_ERR_UNSUPPORTED"):
        sg.gemm(A, A, layout_a="col", layout_b="col")
    odd = torch.zeros((128, 66), dtype=torch.float32, device=DEV)
    with pytest.raises(sg.SolgemmError, match="SG_ERR_ALIGNMENT"):
        sg.gemm(odd, odd)                                     # leading dimension 66 elements = 264 bytes
