"""GPU parity of signed 8-bit integer operands (32-bit integer accumulation, floating-point epilogue)."""
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


def _rand8(shape, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randint(-128, 128, shape, generator=g, dtype=torch.int8)


@pytest.mark.parametrize("tile_n,pair", [(64, 0), (128, 0), (256, 0), (128, 1), (256, 1)])
@pytest.mark.parametrize("M,N,K", [(256, 256, 256), (300, 200, 272), (1000, 520, 1024), (129, 72, 16)])
def test_int8_full_range_is_exact_in_fp32_output(M, N, K, tile_n, pair):
    # |sum| <= 1024 * 128 * 128 = 2^24: every accumulator converts to fp32 exactly
    sg.set_tuning(tile_n, pair)
    A, B = _rand8((M, K), 81), _rand8((N, K), 82)
    ref, _ = orc.gemm(A, B)
    D = torch.full((M, N), float("nan"), dtype=torch.float32, device=DEV)
    sg.gemm(A.to(DEV), B.to(DEV), out=D)
    parity.assert_bit_exact(D, ref, f"int8 gemm {M}x{N}x{K} tile_n={tile_n} pair={pair}")


def test_int8_extremes_and_sign():
    A = torch.full((128, 128), -128, dtype=torch.int8)
    B = torch.full((64, 128), -128, dtype=torch.int8)
    B[1] = 127
    D = sg.gemm(A.to(DEV), B.to(DEV), out_dtype=torch.float32).cpu()
    assert float(D[0, 0]) == 128.0 * 128 * 128 and float(D[3, 1]) == -128.0 * 127 * 128


@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float32])
def test_int8_dequantising_epilogue_batched_grouped_and_conv(out_dtype):
    M, N, K = 333, 264, 528
    A, B = _rand8((M, K), 83), _rand8((N, K), 84)
    bias = inputs.normal([N], 83, 4)
    rs = (torch.rand(M, generator=torch.Generator().manual_seed(1)) + 0.5) / 128
    cs = (torch.rand(N, generator=torch.Generator().manual_seed(2)) + 0.5) / 128
    d, aux, mag_d, mag = orc.gemm_ex(A, B, bias=bias, row_scale=rs, col_scale=cs, alpha=1 / 16., epi="gelu")
    D = sg.gemm(A.to(DEV), B.to(DEV), bias=bias.to(DEV), alpha=1 / 16., epi="gelu", out_dtype=out_dtype,
                ex=dict(row_scale=rs.to(DEV), col_scale=cs.to(DEV)))
    parity.assert_matches(D, d, mag_d, "int8 dequantised gemm")
    Ab, Bb = _rand8((3, 130, 96), 85), _rand8((3, 72, 96), 86)
    Db = sg.batched_gemm(Ab.to(DEV), Bb.to(DEV), alpha=2.0 ** -10, epi="relu", out_dtype=out_dtype)
    for i in range(3):
        ref, absacc = orc.gemm(Ab[i], Bb[i], alpha=2.0 ** -10, epi="relu")
        parity.assert_matches(Db[i], ref, absacc, f"int8 batch {i}")
    Ms = [100, 0, 257]
    As = [_rand8((m, 64), 87 + i) for i, m in enumerate(Ms)]
    Bs = [_rand8((48, 64), 90 + i) for i in range(3)]
    outs = sg.grouped_gemm([a.to(DEV) for a in As], [b.to(DEV) for b in Bs], alpha=2.0 ** -12, out_dtype=out_dtype)
    for a, b, o in zip(As, Bs, outs):
        if a.shape[0]:
            ref, absacc = orc.gemm(a, b, alpha=2.0 ** -12)
            parity.assert_matches(o, ref, absacc, "int8 grouped")
    X, Wf = _rand8((2, 9, 8, 48), 93), _rand8((40, 3, 3, 48), 94)
    bc = inputs.normal([40], 93, 4)
    ref, absacc = orc.conv2d_fprop(X, Wf, pad=(1, 1), bias=bc, alpha=2.0 ** -12, epi="relu")
    Y = sg.conv2d_fprop(X.to(DEV), Wf.to(DEV), pad=(1, 1), bias=bc.to(DEV), alpha=2.0 ** -12, epi="relu", out_dtype=out_dtype)
    parity.assert_matches(Y.reshape(-1, 40), ref.reshape(-1, 40), absacc.reshape(-1, 40), "int8 conv")
