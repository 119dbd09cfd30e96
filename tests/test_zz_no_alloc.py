"""The allocation-free grouped entry point (sg_grouped_gemm_static) against the workspace-taking one.

Some callers cannot allocate device memory at the time they need a grouped product (all of it already
belongs to a pool they must not touch, or cudaMalloc's possible device-wide synchronisation is not
acceptable on their path), so they cannot provide the workspace sg_grouped_gemm asks for.  This file
checks, through the C ABI, that the variant whose tables live in a scratch array inside the library
image gives the same result -- on two calls in a row with different group counts and sizes, because
the array is shared and still holds the first call's tables when the second starts.

It is collected last on purpose and passes both alone in a fresh process and after the other tests.
"""
import ctypes

import pytest
import torch

from paper_2603_29010_b200 import inputs

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

from paper_2603_29010_b200 import solgemm as sg       # noqa: E402

DEV = "cuda"


def _problem(Ms, N, K, seed):
    As, Bs = inputs.make_grouped(Ms, N, K, "normal", K ** -0.25, seed=seed, device=DEV)
    biases = [inputs.normal([N], seed + g, 4, device=DEV) for g in range(len(Ms))]
    return As, Bs, biases


def _compare(Ms, N, K, seed, epi):
    As, Bs, biases = _problem(Ms, N, K, seed)
    want = sg.grouped_gemm(As, Bs, biases=biases, epi=epi)                  # caller-provided workspace
    outs = [torch.full((m, N), float("nan"), dtype=torch.bfloat16, device=DEV) for m in Ms]
    # The first call on a device makes the CUDA runtime load the library's device code (documented: do it early);
    # from then on nothing may be taken from the device, neither through torch's allocator nor behind its back.
    sg.grouped_gemm_static(As, Bs, biases=biases, outs=outs, epi=epi)
    torch.cuda.synchronize()
    for o in outs:
        o.fill_(float("nan"))
    torch.cuda.synchronize()
    before, free_before = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
    got = sg.grouped_gemm_static(As, Bs, biases=biases, outs=outs, epi=epi)  # tables in the library's own array
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before                         # the wrapper allocated nothing either
    assert torch.cuda.mem_get_info()[0] >= free_before                     # and no cudaMalloc happened underneath it
    sg.poll_status()
    for g, m in enumerate(Ms):
        w, o = want[g].float(), got[g].float()
        assert bool(torch.isfinite(o).all())
        # same kernel, same tiling, same inputs: the tolerance of the parity tests is met with room to spare
        assert bool(((o - w).abs() <= 1e-2 + 1e-2 * w.abs()).all()), f"group {g}"
        assert torch.equal(o, w), f"group {g}: results differ bitwise"


def test_static_scratch_matches_workspace_entry_point_twice_in_a_row():
    _compare([300, 0, 129, 1000, 64, 257, 33], 264, 200, seed=4242, epi="silu")     # 7 groups, ragged, one empty
    _compare([512, 77, 128], 136, 328, seed=4343, epi="relu")                       # fewer groups: stale entries beyond them


def test_static_scratch_rejects_too_many_groups():
    lib = sg.raw_lib()
    n = sg.STATIC_MAX_GROUPS + 1
    desc = sg.GemmDesc(0, 64, 64, 0, 1, 64, 64, 64, 64, 0, 0, 1.0, 0.0, 0, 0.0, 0.0, 0)
    Ms = (ctypes.c_int64 * n)(*([64] * n))
    ptrs = (ctypes.c_void_p * n)(*([0x1000] * n))
    launches = sg.launch_count()
    st = lib.sg_grouped_gemm_static(ctypes.byref(desc), n, Ms, ptrs, ptrs, None, None, ptrs, None)
    assert sg.STATUS_NAMES[st] == "SG_ERR_WORKSPACE"
    assert str(sg.STATIC_MAX_GROUPS) in lib.sg_last_error().decode()
    assert sg.launch_count() == launches
