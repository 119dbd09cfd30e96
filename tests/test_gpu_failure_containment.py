"""Failure containment of the contraction kernel, exercised without hanging or faulting anything.

Every device-side wait of the kernel is bounded; when one runs out the kernel records where, every role leaves, the
CTA frees its TMEM and returns, and the status word stays set until `sg_poll_status` reports and clears it -- launches
in between are no-ops that leave their outputs untouched.  Two forms are tested:

* the word is written from the HOST (a test hook), so nothing waits on anything: launches must be no-ops, the poll
  must report once and then be clean, and the same calls must then compute exactly;
* the bound of the waits is shortened to a few hundred nanoseconds, far below the time the first operand tile needs
  to arrive, so a wait that would have succeeded gives up: the kernel returns by itself, the word is set, and after
  the poll the same call is bit-exact (TMEM was freed, no barrier state survives a launch).
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
NAN = float("nan")


@pytest.fixture(autouse=True)
def _restore():
    sg.set_tuning(-1, -1)
    sg.set_tail_mode(-1)
    sg.set_option("wait_limit_ns", -1)
    sg.enable_scratch(True)
    yield
    sg.set_option("wait_limit_ns", -1)
    sg.set_tail_mode(-1)
    torch.cuda.synchronize()
    try:
        sg.poll_status()
    except sg.SolgemmError:
        pass                                          # a failed test must not leave the word set for the next one
    sg.enable_scratch(True)


def _expect_timeout():
    torch.cuda.synchronize()
    with pytest.raises(sg.SolgemmError) as e:
        sg.poll_status()
    assert sg.STATUS_NAMES[e.value.status] == "SG_ERR_TIMEOUT"
    sg.poll_status()                                  # the report cleared the word: the second poll is clean
    return str(e.value)


def test_set_status_word_makes_launches_no_ops_until_polled():
    # dense (specialised kernel variant), grouped, and a skinny long-K problem whose K loop is cut into ranges
    A, B = inputs.small_integers([300, 200], 901, 1), inputs.small_integers([264, 200], 901, 2)
    Ms = [130, 0, 257]
    gA = [inputs.small_integers([m, 136], 902 + g, 1) for g, m in enumerate(Ms)]
    gB = [inputs.small_integers([72, 136], 902 + g, 2) for g in range(len(Ms))]
    kA, kB = inputs.small_integers([256, 8192], 903, 1, 0, 1), inputs.small_integers([256, 8192], 903, 2, -1, 1)
    dA, dB, dkA, dkB = A.to(DEV), B.to(DEV), kA.to(DEV), kB.to(DEV)
    dgA, dgB = [a.to(DEV) for a in gA], [b.to(DEV) for b in gB]

    def run_all():
        D = torch.full((300, 264), NAN, dtype=torch.bfloat16, device=DEV)
        G = [torch.full((m, 72), NAN, dtype=torch.bfloat16, device=DEV) for m in Ms]
        Kd = torch.full((256, 256), NAN, dtype=torch.float32, device=DEV)
        sg.gemm(dA, dB, out=D)
        sg.grouped_gemm(dgA, dgB, outs=G)
        sg.gemm(dkA, dkB, out=Kd)
        ksplit_plan = sg.last_launch_plan()
        torch.cuda.synchronize()
        return D, G, Kd, ksplit_plan

    torch.cuda.synchronize()
    sg.test_set_status_word((3 << 24) | 77)           # "epilogue, barrier 77", as a wait that ran out would leave it
    launches = sg.launch_count()
    D, G, Kd, plan = run_all()
    assert sg.launch_count() > launches               # the kernels were launched ...
    assert plan["tail_split"] < -1, plan              # (the long-K problem was planned with K ranges)
    assert bool(torch.isnan(D).all()) and bool(torch.isnan(Kd).all())        # ... and wrote nothing
    assert all(bool(torch.isnan(g).all()) for g in G)
    msg = _expect_timeout()
    assert "epilogue" in msg and "77" in msg

    D, G, Kd, plan = run_all()                        # the same calls now compute, exactly
    parity.assert_bit_exact(D, orc.gemm(A, B)[0], "dense after the poll")
    for g, m in enumerate(Ms):
        if m:
            parity.assert_bit_exact(G[g], orc.gemm(gA[g], gB[g])[0], f"group {g} after the poll")
    parity.assert_bit_exact(Kd, orc.gemm(kA, kB)[0], "K ranges after the poll")
    sg.poll_status()


@pytest.mark.parametrize("tile_n,pair", [(-1, -1), (128, 0), (256, 1)])
def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_exact(tile_n, pair):
    # One or a few tiles with a very long K loop (about a millisecond): the epilogue warps wait for the accumulator all
    # that time, the MMA thread waits for every operand stage.  With a bound of 300 ns the first of those waits that
    # is looked at gives up.  No K ranges and no tail slices, so the only waits are the pipeline's own barriers.
    sg.enable_scratch(False)
    sg.set_tail_mode(0)
    sg.set_tuning(tile_n, pair)
    M, N, K = 256, 256, 131072
    A = inputs.small_integers([M, K], 911, 1, 0, 1).to(DEV)
    B = inputs.small_integers([N, K], 911, 2, -1, 1).to(DEV)
    D = torch.full((M, N), NAN, dtype=torch.float32, device=DEV)
    torch.cuda.synchronize()
    sg.set_option("wait_limit_ns", 300)
    sg.gemm(A, B, out=D)
    torch.cuda.synchronize()                          # returns: the kernel left by itself
    sg.set_option("wait_limit_ns", -1)
    D2 = torch.full((M, N), NAN, dtype=torch.float32, device=DEV)
    sg.gemm(A, B, out=D2)                             # the word is still set: a no-op
    torch.cuda.synchronize()
    assert bool(torch.isnan(D2).all())
    msg = _expect_timeout()
    assert any(role in msg for role in ("producer", "mma", "epilogue")), msg
    # a launch that gave up must not have stored a complete result
    ref = orc.gemm(A.cpu(), B.cpu())[0]
    assert not torch.equal(torch.nan_to_num(D.cpu().double(), nan=-1e30), ref)
    # after the poll: TMEM was freed and no barrier state survived, the same call is exact
    for _ in range(2):
        D3 = torch.full((M, N), NAN, dtype=torch.float32, device=DEV)
        sg.gemm(A, B, out=D3)
        torch.cuda.synchronize()
        sg.poll_status()
        parity.assert_bit_exact(D3, ref, "after a timed-out launch")


def test_matrix_vector_and_small_product_kernels_store_nothing_while_the_word_is_set():
    sg.set_option("gemv_small_log2", -1)              # the library's own choice of path
    sg.set_option("gemv_max_vectors", -1)
    W = inputs.small_integers([1000, 520], 921, 1)
    X = inputs.small_integers([3, 520], 921, 2)       # three vectors: the matrix-vector kernels
    A = inputs.small_integers([256, 264], 922, 1)
    B = inputs.small_integers([200, 264], 922, 2)     # a small product: the warp-level MMA kernel with groups of vectors
    dW, dX, dA, dB = W.to(DEV), X.to(DEV), A.to(DEV), B.to(DEV)

    def run_all():
        Dv = torch.full((3, 1000), NAN, dtype=torch.float32, device=DEV)
        Ds = torch.full((256, 200), NAN, dtype=torch.float32, device=DEV)
        sg.gemm(dX, dW, out=Dv)
        assert sg.last_launch_plan()["tile_n"] == 0
        sg.gemm(dA, dB, out=Ds)
        assert sg.last_launch_plan()["tile_n"] == 0 and "gemv_mma_kernel" in sg.last_kernel_name()
        torch.cuda.synchronize()
        return Dv, Ds

    torch.cuda.synchronize()
    sg.test_set_status_word((3 << 24) | 5)
    Dv, Ds = run_all()
    assert bool(torch.isnan(Dv).all()) and bool(torch.isnan(Ds).all())
    _expect_timeout()
    Dv, Ds = run_all()
    parity.assert_bit_exact(Dv, orc.gemm(X, W)[0], "vectors after the poll")
    parity.assert_bit_exact(Ds, orc.gemm(A, B)[0], "small product after the poll")
    sg.poll_status()
