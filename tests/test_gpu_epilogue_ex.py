"""GPU parity of the extended epilogue chain (sg_gemm_ex / sg_conv2d_fprop_ex) against the oracle's chain."""
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


def _vec(n, seed, tid, kind="uniform"):
    """An fp32 vector whose values are bf16-representable (so that it is the same number on both sides)."""
    gen = inputs.uniform if kind == "uniform" else inputs.normal
    return gen([n], seed, tid).to(torch.float32)


@pytest.mark.parametrize("tile_n,pair", [(64, 0), (128, 0), (256, 0), (128, 1), (256, 1)])
@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float32, torch.float16])
def test_gemm_ex_integer_chain_is_bit_exact(out_dtype, tile_n, pair):
    # integers, power-of-two scales: every intermediate is exact in fp32 and in the output type
    sg.set_tuning(tile_n, pair)
    M, N, K = 300, 200, 72
    A = inputs.small_integers([M, K], 41, 1, -2, 2)
    B = inputs.small_integers([N, K], 41, 2, -2, 2)
    rs = torch.tensor([2.0 ** (i % 2) for i in range(M)])
    cs = torch.tensor([(-1.0) ** j * 2.0 ** (j % 2 - 1) for j in range(N)])
    rb = inputs.small_integers([M], 41, 6, -4, 4).to(torch.float32)
    bias = inputs.small_integers([N], 41, 4, -4, 4)
    R = inputs.small_integers([M, N], 41, 7, -8, 8).to(out_dtype)
    d, aux, _, _ = orc.gemm_ex(A, B, bias=bias, row_scale=rs, col_scale=cs, row_bias=rb, epi="relu", post_scale=0.5, aux_load=R)
    assert float(aux.abs().max()) <= 256 and float(d.abs().max()) <= 256
    D = torch.full((M, N), float("nan"), dtype=out_dtype, device=DEV)
    AUX = torch.full((M, N), float("nan"), dtype=out_dtype, device=DEV)
    sg.gemm(A.to(DEV), B.to(DEV), bias=bias.to(DEV), out=D, epi="relu",
            ex=dict(row_scale=rs.to(DEV), col_scale=cs.to(DEV), row_bias=rb.to(DEV), post_scale=0.5,
                    aux_load=R.to(DEV), aux_store=AUX))
    parity.assert_bit_exact(D, d, "gemm_ex D")
    parity.assert_bit_exact(AUX, aux, "gemm_ex aux_store")


@pytest.mark.parametrize("epi", ["none", "gelu", "silu", "clip"])
@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float32])
def test_gemm_ex_real_values_ragged_and_each_member_alone(out_dtype, epi):
    M, N, K = 333, 200, 264
    A, B, bias = inputs.make_gemm(M, N, K, "uniform", 1.0, bias=True, seed=12)
    C = inputs.normal([M, N], 12, 3).to(out_dtype)
    R = inputs.normal([M, N], 12, 7).to(out_dtype)
    rs, cs, rb = _vec(M, 12, 8), _vec(N, 12, 9), _vec(M, 12, 10, "normal")
    full = dict(row_scale=rs, col_scale=cs, row_bias=rb, post_scale=1.5, aux_load=R)
    cases = [full] + [{k: v} for k, v in full.items()] + [dict()]
    args = (-1.0, 2.0) if epi == "clip" else (0.0, 0.0)
    for members in cases:
        d, aux, mag_d, mag = orc.gemm_ex(A, B, C=C, bias=bias, alpha=0.125, beta=0.5, epi=epi, epi_args=args, **members)
        D = torch.full((M, N), float("nan"), dtype=out_dtype, device=DEV)
        AUX = torch.full((M, N), float("nan"), dtype=out_dtype, device=DEV)
        ex = {k: (v.to(DEV) if torch.is_tensor(v) else v) for k, v in members.items()}
        ex["aux_store"] = AUX
        sg.gemm(A.to(DEV), B.to(DEV), C=C.to(DEV), bias=bias.to(DEV), out=D, alpha=0.125, beta=0.5, epi=epi, epi_args=args, ex=ex)
        parity.assert_matches(D, d, mag_d, f"gemm_ex D {sorted(members)} {epi}")
        parity.assert_matches(AUX, aux, mag, f"gemm_ex aux {sorted(members)} {epi}")


@pytest.mark.parametrize("out_dtype,N", [(torch.bfloat16, 90), (torch.float32, 67)])
def test_gemm_ex_ragged_columns_stay_inside_n(out_dtype, N):
    M, K = 140, 64
    ld = (N + 15) // 8 * 8
    A, B, _ = inputs.make_gemm(M, N, K, "uniform", 1.0, seed=14)
    cs = _vec(ld, 14, 9)[:N].contiguous()
    R = inputs.normal([M, ld], 14, 7).to(out_dtype)
    d, aux, mag_d, mag = orc.gemm_ex(A, B, col_scale=cs, aux_load=R[:, :N], epi="tanh")
    Dw = torch.full((M, ld), float("nan"), dtype=out_dtype, device=DEV)
    Aw = torch.full((M, ld), float("nan"), dtype=out_dtype, device=DEV)
    cs_dev = torch.full((ld,), float("nan"), dtype=torch.float32, device=DEV)
    cs_dev[:N] = cs
    Rd = R.to(DEV)
    Rd[:, N:] = float("nan")
    sg.gemm(A.to(DEV), B.to(DEV), out=Dw[:, :N], epi="tanh", ex=dict(col_scale=cs_dev[:N], aux_load=Rd[:, :N], aux_store=Aw[:, :N]))
    parity.assert_matches(Dw[:, :N], d, mag_d, "ragged D")
    parity.assert_matches(Aw[:, :N], aux, mag, "ragged aux")
    assert bool(torch.isnan(Dw[:, N:]).all()) and bool(torch.isnan(Aw[:, N:]).all())


def test_gemm_ex_null_is_plain_gemm_and_k_split_tail():
    M, N, K = 256, 256, 4096                 # a long K with few tiles: the planner cuts K into ranges
    A, B, bias = inputs.make_gemm(M, N, K, "normal", 1 / 64., bias=True, seed=15)
    rs = _vec(M, 15, 8)
    d, aux, mag_d, mag = orc.gemm_ex(A, B, bias=bias, row_scale=rs, epi="relu")
    D = torch.empty((M, N), dtype=torch.float32, device=DEV)
    AUX = torch.empty_like(D)
    sg.gemm(A.to(DEV), B.to(DEV), bias=bias.to(DEV), out=D, epi="relu", ex=dict(row_scale=rs.to(DEV), aux_store=AUX))
    parity.assert_matches(D, d, mag_d, "k-split D")
    parity.assert_matches(AUX, aux, mag, "k-split aux")
    plain = sg.gemm(A.to(DEV), B.to(DEV), bias=bias.to(DEV), epi="relu", out_dtype=torch.float32)
    same = sg.gemm(A.to(DEV), B.to(DEV), bias=bias.to(DEV), epi="relu", out_dtype=torch.float32, ex=dict())
    assert torch.equal(plain, same)


@pytest.mark.parametrize("pair", [0, 1])
def test_conv_ex_per_channel_scale_residual_and_aux(pair):
    sg.set_tuning(-1, pair)
    N_, H, W, C, K = 3, 20, 17, 64, 96
    X, Wf, bias = inputs.make_conv(N_, H, W, C, K, 3, 3, "normal", 1 / 24., bias=True, seed=16)
    P, Q = H, W
    cs = _vec(K, 16, 9)
    rb = _vec(N_ * P * Q, 16, 10)
    R = inputs.normal([N_, P, Q, K], 16, 7)
    d, aux, mag_d, mag = orc.conv2d_fprop_ex(X, Wf, pad=(1, 1), bias=bias, col_scale=cs, row_bias=rb, epi="relu",
                                             post_scale=2.0, aux_load=R.reshape(-1, K))
    Y = torch.full((N_, P, Q, K), float("nan"), dtype=torch.bfloat16, device=DEV)
    AUX = torch.full((N_, P, Q, K), float("nan"), dtype=torch.bfloat16, device=DEV)
    sg.conv2d_fprop(X.to(DEV), Wf.to(DEV), pad=(1, 1), bias=bias.to(DEV), out=Y, epi="relu",
                    ex=dict(col_scale=cs.to(DEV), row_bias=rb.to(DEV), post_scale=2.0, aux_load=R.to(DEV), aux_store=AUX))
    parity.assert_matches(Y.reshape(-1, K), d, mag_d, "conv_ex Y")
    parity.assert_matches(AUX.reshape(-1, K), aux, mag, "conv_ex aux")


def test_ex_argument_errors():
    A, B, _ = inputs.make_gemm(128, 64, 64, "uniform", 1.0, seed=17)
    A, B = A.to(DEV), B.to(DEV)
    v = torch.zeros(130, dtype=torch.float32, device=DEV)
    with pytest.raises(sg.SolgemmError, match="SG_ERR_ALIGNMENT"):
        sg.gemm(A, B, ex=dict(col_scale=v[1:65]))
    narrow = torch.zeros((128, 32), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(sg.SolgemmError, match="SG_ERR_INVALID_ARG"):
        sg.gemm(A, B, ex=dict(aux_store=narrow))
    with pytest.raises(sg.SolgemmError, match="SG_ERR_INVALID_ARG"):
        sg.gemm(A, B, ex=dict(post_scale=float("inf")))
