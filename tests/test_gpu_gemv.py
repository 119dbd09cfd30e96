"""GPU parity of matrix-vector products (a GEMM with N = 1 or M = 1), which run as a stream over the matrix."""
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
    sg.set_option("gemv_max_vectors", -1)        # this module tests the library's own choice of path
    sg.set_option("gemv_small_log2", -1)
    sg.set_option("no_gemv", -1)
    yield
    torch.cuda.synchronize()
    sg.poll_status()
    sg.set_option("gemv_max_vectors", -1)
    sg.set_option("gemv_small_log2", -1)
    sg.set_option("no_gemv", -1)


def _took_vector_path():
    return sg.last_launch_plan()["tile_n"] == 0


# rows x K: many rows, few rows with a long K (K ranges over a cluster), ragged row blocks, one row, tiny
SHAPES = [(4096, 4096), (64, 65536), (1003, 1024), (8, 40000), (1, 4096), (3, 8), (300, 2056), (7, 262144)]


@pytest.mark.parametrize("R,K", SHAPES)
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16, torch.float32])
def test_matrix_times_vector_integer_values_bit_exact(R, K, dtype):
    # small integers: every partial sum is exact in fp32 whatever the order, so the result must match to the bit
    W = inputs.small_integers([R, K], 90, 1, lo=-2, hi=2).to(dtype)
    x = inputs.small_integers([1, K], 90, 2, lo=-2, hi=2).to(dtype)
    ref, _ = orc.gemm(W, x)
    D = torch.full((R, 1), float("nan"), dtype=torch.float32, device=DEV)
    sg.gemm(W.to(DEV), x.to(DEV), out=D)
    assert _took_vector_path()
    parity.assert_bit_exact(D, ref, f"gemv {R}x{K} {dtype}")
    # the vector on the left: (1 x K) . (R x K)^T
    ref_t, _ = orc.gemm(x, W)
    Dt = torch.full((1, R), float("nan"), dtype=torch.float32, device=DEV)
    sg.gemm(x.to(DEV), W.to(DEV), out=Dt)
    assert _took_vector_path()
    parity.assert_bit_exact(Dt, ref_t, f"vector-matrix {R}x{K} {dtype}")


@pytest.mark.parametrize("R,K", [(4096, 4096), (257, 33000), (5, 100008)])
@pytest.mark.parametrize("dtype,out_dtype", [(torch.bfloat16, torch.bfloat16), (torch.float16, torch.float16),
                                             (torch.float32, torch.float32), (torch.bfloat16, torch.float32)])
@pytest.mark.parametrize("epi", ["none", "gelu", "relu"])
def test_matrix_times_vector_real_values_with_epilogue(R, K, dtype, out_dtype, epi):
    g = torch.Generator().manual_seed(R + K)
    W = (torch.randn(R, K, generator=g) / 8).to(dtype)
    x = (torch.randn(1, K, generator=g) / 8).to(dtype)
    C = torch.randn(R, 1, generator=g).to(out_dtype)
    bias1 = torch.randn(1, generator=g).to(dtype)
    ref, absacc = orc.gemm(W, x, C=C, bias=bias1, alpha=0.75, beta=0.5, epi=epi)
    D = sg.gemm(W.to(DEV), x.to(DEV), C=C.to(DEV), bias=bias1.to(DEV), alpha=0.75, beta=0.5, epi=epi, out_dtype=out_dtype)
    assert _took_vector_path()
    parity.assert_matches(D, ref, absacc, f"gemv {R}x{K} {dtype} {epi}")
    # vector on the left: the bias is per output column, the residual a row
    biasR = torch.randn(R, generator=g).to(dtype)
    Ct = torch.randn(1, R, generator=g).to(out_dtype)
    ref, absacc = orc.gemm(x, W, C=Ct, bias=biasR, alpha=-1.25, beta=2.0, epi=epi)
    D = sg.gemm(x.to(DEV), W.to(DEV), C=Ct.to(DEV), bias=biasR.to(DEV), alpha=-1.25, beta=2.0, epi=epi, out_dtype=out_dtype)
    assert _took_vector_path()
    parity.assert_matches(D, ref, absacc, f"vector-matrix {R}x{K} {dtype} {epi}")


@pytest.mark.parametrize("nvec", [2, 3, 4, 5, 8])
@pytest.mark.parametrize("R,K", [(4096, 4096), (130, 66000), (5, 1000), (37, 264)])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16, torch.float32])
def test_several_vectors_in_one_pass(R, K, nvec, dtype):
    # 16-bit inputs: up to eight vectors (warp-level MMAs); fp32 inputs: up to four (FMA kernel)
    if dtype == torch.float32 and nvec > 4:
        pytest.skip("more than four fp32 vectors run on the tiles")
    g = torch.Generator().manual_seed(R + K + nvec)
    out_dtype = torch.float32 if dtype == torch.float32 else dtype
    W = (torch.randn(R, K, generator=g) / 8).to(dtype)
    X = (torch.randn(nvec, K, generator=g) / 8).to(dtype)
    # matrix on the left: D [R, nvec], bias per vector
    C = torch.randn(R, nvec, generator=g).to(out_dtype)
    bias = torch.randn(nvec, generator=g).to(dtype)
    ref, absacc = orc.gemm(W, X, C=C, bias=bias, alpha=0.5, beta=-1.0, epi="tanh")
    D = sg.gemm(W.to(DEV), X.to(DEV), C=C.to(DEV), bias=bias.to(DEV), alpha=0.5, beta=-1.0, epi="tanh", out_dtype=out_dtype)
    assert _took_vector_path()
    parity.assert_matches(D, ref, absacc, f"{R}x{K} times {nvec} vectors {dtype}")
    # vectors on the left (a decode batch): D [nvec, R], bias per matrix row
    Ct = torch.randn(nvec, R, generator=g).to(out_dtype)
    biasR = torch.randn(R, generator=g).to(dtype)
    ref, absacc = orc.gemm(X, W, C=Ct, bias=biasR, beta=0.5, epi="silu")
    D = sg.gemm(X.to(DEV), W.to(DEV), C=Ct.to(DEV), bias=biasR.to(DEV), beta=0.5, epi="silu", out_dtype=out_dtype)
    assert _took_vector_path()
    parity.assert_matches(D, ref, absacc, f"{nvec} vectors times {R}x{K} {dtype}")
    # small integers: exact
    Wi = inputs.small_integers([R, K], 91, 1, lo=-2, hi=2).to(dtype)
    Xi = inputs.small_integers([nvec, K], 91, 2, lo=-2, hi=2).to(dtype)
    ref, _ = orc.gemm(Xi, Wi)
    Di = torch.full((nvec, R), float("nan"), dtype=torch.float32, device=DEV)
    sg.gemm(Xi.to(DEV), Wi.to(DEV), out=Di)
    parity.assert_bit_exact(Di, ref, f"{nvec} integer vectors times {R}x{K} {dtype}")


def test_several_vectors_with_a_ragged_k():
    # K is no multiple of 8: the FMA kernel (up to four vectors), rows padded to 16 bytes
    g = torch.Generator().manual_seed(21)
    R, K, ld = 300, 1003, 1008
    Wp = (torch.randn(R, ld, generator=g) / 4).to(torch.bfloat16)
    Xp = (torch.randn(3, ld, generator=g) / 4).to(torch.bfloat16)
    ref, absacc = orc.gemm(Xp[:, :K], Wp[:, :K], epi="relu")
    D = sg.gemm(Xp.to(DEV)[:, :K], Wp.to(DEV)[:, :K], epi="relu")
    assert _took_vector_path()
    parity.assert_matches(D, ref, absacc, "three vectors, K = 1003")


def test_padded_rows_strided_outputs_and_a_column_vector_operand():
    g = torch.Generator().manual_seed(11)
    R, K, ld = 517, 1003, 1008                         # K is no multiple of a 16-byte vector; rows padded to one
    Wp = (torch.randn(R, ld, generator=g) / 4).to(torch.bfloat16)
    W = Wp[:, :K]
    xcol = (torch.randn(K, 1, generator=g) / 4).to(torch.bfloat16)     # a K x 1 row-major B
    Cp = torch.randn(R, 4, generator=g).to(torch.bfloat16)
    ref, absacc = orc.gemm(W, xcol, layout_b="row", C=Cp[:, :1], beta=1.0, epi="silu")
    Dp = torch.full((R, 3), 7.0, dtype=torch.bfloat16, device=DEV)
    sg.gemm(Wp.to(DEV)[:, :K], xcol.to(DEV), layout_b="row", C=Cp.to(DEV)[:, :1], beta=1.0,
            epi="silu", out=Dp[:, :1])
    assert _took_vector_path()
    parity.assert_matches(Dp[:, :1], ref, absacc, "padded gemv")
    assert bool((Dp[:, 1:] == 7.0).all()), "the neighbours of a strided output column were written"


def test_results_do_not_depend_on_the_run():
    g = torch.Generator().manual_seed(3)
    W = torch.randn(100, 70000, generator=g).to(torch.bfloat16).to(DEV)
    x = torch.randn(1, 70000, generator=g).to(torch.bfloat16).to(DEV)
    first = sg.gemm(W, x, out_dtype=torch.float32).clone()
    for _ in range(5):
        assert torch.equal(sg.gemm(W, x, out_dtype=torch.float32), first)


def test_other_forms_still_go_through_the_tiles():
    g = torch.Generator().manual_seed(4)
    sg.set_option("gemv_small_log2", 0)           # (a product this small would otherwise go to the MMA kernel whole)
    A = torch.randn(256, 64, generator=g).to(torch.bfloat16)
    B33 = torch.randn(33, 64, generator=g).to(torch.bfloat16)
    out = torch.empty(256, 40, dtype=torch.bfloat16, device=DEV)
    sg.gemm(A.to(DEV), B33.to(DEV), out=out[:, :33])
    assert not _took_vector_path()
    ref, absacc = orc.gemm(A, B33)
    parity.assert_matches(out[:, :33], ref, absacc, "N = 33")
    # nine vectors against a matrix too large for the many-vector form of the kernel (more than 48 MB)
    sg.set_option("gemv_small_log2", -1)
    Wbig = torch.randn(6200, 4096, generator=g).to(torch.bfloat16)
    X9 = torch.randn(9, 4096, generator=g).to(torch.bfloat16)
    D9 = sg.gemm(X9.to(DEV), Wbig.to(DEV))
    assert not _took_vector_path()
    parity.assert_matches(D9[:, :64], *[t[:, :64] for t in orc.gemm(X9, Wbig[:64])], "nine vectors, large matrix")
    # ... or with more groups of eight than are resident at once (512 row blocks x 3 groups)
    sg.gemm(torch.zeros(20, 2048, dtype=torch.bfloat16, device=DEV), torch.zeros(8192, 2048, dtype=torch.bfloat16, device=DEV))
    assert not _took_vector_path()
    # a K x 2 row-major B is not a pair of contiguous vectors
    Brow = torch.randn(64, 8, generator=g).to(torch.bfloat16)
    sg.gemm(A.to(DEV), Brow.to(DEV)[:, :2], layout_b="row", out=out[:, :2])
    assert not _took_vector_path()
    ref, absacc = orc.gemm(A, Brow[:, :2], layout_b="row")
    parity.assert_matches(out[:, :2], ref, absacc, "N = 2, row-major B")


@pytest.mark.parametrize("M", [9, 16, 32, 33, 64, 65])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
def test_few_rows_against_a_large_matrix_on_the_tiles(M, dtype):
    # 9..64 rows: the tensor-core tiles with only 32 or 64 rows of A loaded per stage; 65: the full A tile
    # (a matrix this small would go to the matrix-vector kernels with up to 32 rows: keep those to eight vectors here)
    sg.set_option("gemv_max_vectors", 8)
    sg.set_option("gemv_small_log2", 0)
    g = torch.Generator().manual_seed(100 + M)
    N, K = 1080, 2056
    A = (torch.randn(M, K, generator=g) / 8).to(dtype)
    W = (torch.randn(N, K, generator=g) / 8).to(dtype)
    C = torch.randn(M, N, generator=g).to(dtype)
    bias = torch.randn(N, generator=g).to(dtype)
    ref, absacc = orc.gemm(A, W, C=C, bias=bias, alpha=1.5, beta=0.5, epi="gelu")
    D = sg.gemm(A.to(DEV), W.to(DEV), C=C.to(DEV), bias=bias.to(DEV), alpha=1.5, beta=0.5, epi="gelu", out_dtype=dtype)
    assert not _took_vector_path()
    parity.assert_matches(D, ref, absacc, f"{M} rows x {N} x {K} {dtype}")
    # exact on integers, through every tile width
    Ai = inputs.small_integers([M, K], 92, 1).to(dtype)
    Wi = inputs.small_integers([N, K], 92, 2).to(dtype)
    refi, _ = orc.gemm(Ai, Wi)
    for tile_n in (64, 128, 256):
        sg.set_tuning(tile_n, 0)
        Di = torch.full((M, N), float("nan"), dtype=torch.float32, device=DEV)
        sg.gemm(Ai.to(DEV), Wi.to(DEV), out=Di)
        parity.assert_bit_exact(Di, refi, f"{M} integer rows, tile width {tile_n}")
    sg.set_tuning(-1, -1)
    sg.set_option("gemv_max_vectors", -1)


def test_few_rows_batched():
    g = torch.Generator().manual_seed(77)
    batch, M, N, K = 3, 20, 200, 264
    A = (torch.randn(batch, M, K, generator=g) / 4).to(torch.bfloat16)
    W = (torch.randn(batch, N, K, generator=g) / 4).to(torch.bfloat16)
    bias = torch.randn(batch, N, generator=g).to(torch.bfloat16)
    D = sg.batched_gemm(A.to(DEV), W.to(DEV), bias=bias.to(DEV), epi="relu")
    for b in range(batch):
        ref, absacc = orc.gemm(A[b], W[b], bias=bias[b], epi="relu")
        parity.assert_matches(D[b], ref, absacc, f"few rows, batch {b}")


@pytest.mark.parametrize("K", [8, 24, 200, 1000, 1016, 4104])
@pytest.mark.parametrize("nvec", [3, 8])
@pytest.mark.parametrize("R", [1, 17, 100])
def test_several_vectors_k_not_a_multiple_of_a_warp_step(R, K, nvec):
    # K % 32 != 0: the last step of a warp is partly past the end of the row (lanes there must contribute zeros
    # while the whole warp still executes the tensor-core instruction)
    W = inputs.small_integers([R, K], 93, 1, lo=-2, hi=2)
    X = inputs.small_integers([nvec, K], 93, 2, lo=-2, hi=2)
    ref, _ = orc.gemm(X, W)
    D = torch.full((nvec, R), float("nan"), dtype=torch.float32, device=DEV)
    sg.gemm(X.to(DEV), W.to(DEV), out=D)
    assert _took_vector_path()
    parity.assert_bit_exact(D, ref, f"{nvec} vectors times {R}x{K}")
    ref, _ = orc.gemm(W, X)
    D = torch.full((R, nvec), float("nan"), dtype=torch.float32, device=DEV)
    sg.gemm(W.to(DEV), X.to(DEV), out=D)
    assert _took_vector_path()
    parity.assert_bit_exact(D, ref, f"{R}x{K} times {nvec} vectors")


@pytest.mark.parametrize("nvec", [9, 12, 16, 17, 24, 31, 32])
@pytest.mark.parametrize("R,K", [(512, 1024), (130, 4104), (37, 264), (2048, 2048), (5, 72)])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
@pytest.mark.parametrize("form", ["groups of eight", "blocks in one CTA"])
def test_nine_to_32_vectors(R, K, nvec, dtype, form):
    # the library's own choice: groups of eight vectors along the grid (CTAs that share rows of the matrix are neighbours);
    # with the vector limit pinned to 32: blocks of eight vectors inside one CTA (two up to 16 vectors, four up to 32)
    g = torch.Generator().manual_seed(R + K + nvec)
    W = (torch.randn(R, K, generator=g) / 8).to(dtype)
    X = (torch.randn(nvec, K, generator=g) / 8).to(dtype)
    fewer = min(nvec, R)                      # the operand with fewer rows supplies the vectors
    blocks = 1
    if form == "blocks in one CTA":
        sg.set_option("gemv_max_vectors", 32)
        blocks = 1 if fewer <= 8 else (2 if fewer <= 16 else 4)
    # vectors on the left (a decode batch): D [nvec, R], bias per matrix row, residual
    Ct = torch.randn(nvec, R, generator=g).to(dtype)
    biasR = torch.randn(R, generator=g).to(dtype)
    ref, absacc = orc.gemm(X, W, C=Ct, bias=biasR, alpha=0.75, beta=0.5, epi="silu")
    D = sg.gemm(X.to(DEV), W.to(DEV), C=Ct.to(DEV), bias=biasR.to(DEV), alpha=0.75, beta=0.5, epi="silu", out_dtype=dtype)
    assert _took_vector_path() and sg.last_kernel_name().endswith(f", {blocks}>"), sg.last_kernel_name()
    parity.assert_matches(D, ref, absacc, f"{nvec} vectors times {R}x{K} {dtype}")
    # matrix on the left: D [R, nvec], bias per vector, fp32 output inside NaN guard columns
    bias = torch.randn(nvec, generator=g).to(dtype)
    ref, absacc = orc.gemm(W, X, bias=bias, epi="gelu")
    whole = torch.full((R, 40), float("nan"), dtype=torch.float32, device=DEV)
    sg.gemm(W.to(DEV), X.to(DEV), bias=bias.to(DEV), epi="gelu", out=whole[:, :nvec])
    assert _took_vector_path()
    parity.assert_matches(whole[:, :nvec], ref, absacc, f"{R}x{K} times {nvec} vectors {dtype}")
    assert bool(torch.isnan(whole[:, nvec:]).all())
    # small integers: exact, both forms
    Wi = inputs.small_integers([R, K], 95, 1, lo=-2, hi=2).to(dtype)
    Xi = inputs.small_integers([nvec, K], 95, 2, lo=-2, hi=2).to(dtype)
    refi, _ = orc.gemm(Xi, Wi)
    Di = torch.full((nvec, R), float("nan"), dtype=torch.float32, device=DEV)
    sg.gemm(Xi.to(DEV), Wi.to(DEV), out=Di)
    parity.assert_bit_exact(Di, refi, f"{nvec} integer vectors times {R}x{K} {dtype}")
    refi, _ = orc.gemm(Wi, Xi)
    Di = torch.full((R, nvec), float("nan"), dtype=torch.float32, device=DEV)
    sg.gemm(Wi.to(DEV), Xi.to(DEV), out=Di)
    parity.assert_bit_exact(Di, refi, f"{R}x{K} times {nvec} integer vectors {dtype}")


def test_many_vectors_match_the_tiles_bit_for_bit_on_integers():
    # the same product through both paths of the library
    W = inputs.small_integers([700, 1544], 96, 1, lo=-2, hi=2)
    X = inputs.small_integers([20, 1544], 96, 2, lo=-2, hi=2)
    a = sg.gemm(X.to(DEV), W.to(DEV), out_dtype=torch.float32)
    assert _took_vector_path()
    sg.set_option("no_gemv", 1)
    b = sg.gemm(X.to(DEV), W.to(DEV), out_dtype=torch.float32)
    sg.set_option("no_gemv", -1)
    assert not _took_vector_path()
    assert torch.equal(a, b)


SMALL = [(256, 256, 256), (128, 128, 128), (300, 200, 136), (129, 72, 8), (384, 384, 1024), (64, 64, 4096), (512, 64, 512),
         (33, 77, 4104), (100, 100, 2048), (40, 1000, 264)]


@pytest.mark.parametrize("M,N,K", SMALL)
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
def test_small_products_run_on_the_mma_kernel(M, N, K, dtype):
    # groups of 32 rows of the operand with fewer rows along the grid's second dimension: a small GEMM without tiles
    g = torch.Generator().manual_seed(M + N + K)
    A = (torch.randn(M, K, generator=g) / 8).to(dtype)
    B = (torch.randn(N, K, generator=g) / 8).to(dtype)
    C = torch.randn(M, N, generator=g).to(dtype)
    bias = torch.randn(N, generator=g).to(dtype)
    ref, absacc = orc.gemm(A, B, C=C, bias=bias, alpha=0.75, beta=0.5, epi="gelu")
    whole = torch.full((M + 4, (N + 15) // 8 * 8), float("nan"), dtype=dtype, device=DEV)
    out = whole[2:2 + M, :N]
    sg.gemm(A.to(DEV), B.to(DEV), C=C.to(DEV), bias=bias.to(DEV), alpha=0.75, beta=0.5, epi="gelu", out=out)
    assert _took_vector_path() and "gemv_mma_kernel" in sg.last_kernel_name(), sg.last_kernel_name()
    parity.assert_matches(out, ref, absacc, f"small product {M}x{N}x{K} {dtype}")
    assert bool(torch.isnan(whole[:2]).all()) and bool(torch.isnan(whole[2 + M:]).all()) and bool(torch.isnan(whole[:, N:]).all())
    # exact on small integers, fp32 out; and the same bits as the tiles give
    Ai = inputs.small_integers([M, K], 97, 1, lo=-2, hi=2).to(dtype)
    Bi = inputs.small_integers([N, K], 97, 2, lo=-2, hi=2).to(dtype)
    refi, _ = orc.gemm(Ai, Bi)
    Di = sg.gemm(Ai.to(DEV), Bi.to(DEV), out_dtype=torch.float32)
    assert _took_vector_path()
    parity.assert_bit_exact(Di, refi, f"small integer product {M}x{N}x{K} {dtype}")
    sg.set_option("gemv_small_log2", 0)
    sg.set_option("gemv_max_vectors", 8)
    Dt = torch.empty(M, (N + 7) // 8 * 8, dtype=torch.float32, device=DEV)[:, :N]      # (the tiles want 16-byte row pitches)
    sg.gemm(Ai.to(DEV), Bi.to(DEV), out=Dt)
    assert not _took_vector_path() or min(M, N) <= 8
    assert torch.equal(Di, Dt)


def test_products_too_large_for_the_small_form_use_the_tiles():
    for M, N, K in [(512, 512, 512), (256, 1024, 256), (400, 400, 400), (256, 256, 4096)]:
        A = torch.zeros(M, K, dtype=torch.bfloat16, device=DEV)
        B = torch.zeros(N, K, dtype=torch.bfloat16, device=DEV)
        sg.gemm(A, B)
        assert not _took_vector_path(), (M, N, K)


def test_forced_tile_shapes_keep_small_products_on_the_tiles():
    A = torch.zeros(256, 256, dtype=torch.bfloat16, device=DEV)
    sg.set_tuning(64, 0)
    sg.gemm(A, A)
    assert not _took_vector_path()
    sg.set_tuning(-1, -1)
    sg.gemm(A, A)
    assert _took_vector_path()
