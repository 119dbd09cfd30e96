import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200, sm_100a)")


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")


@pytest.fixture(autouse=True)
def _tile_kernel_by_default(request):
    """GPU tests exercise the tensor-core tile kernel unless they ask otherwise: small products and products with nine to
    32 rows or columns would by default run on the warp-level MMA kernels of the matrix-vector path, which have tests of
    their own (and the random sweep runs every case both ways).  A test that wants the library's own choice sets the two
    options back to -1."""
    if request.node.get_closest_marker("gpu") is None:
        yield
        return
    import torch
    if not torch.cuda.is_available():
        yield
        return
    from paper_2603_29010_b200 import solgemm as sg
    sg.set_option("gemv_small_log2", 0)
    sg.set_option("gemv_max_vectors", 8)
    yield
    sg.set_option("gemv_small_log2", -1)
    sg.set_option("gemv_max_vectors", -1)
