"""The oracle's Speed-of-Light calculator against the paper's printed worked report and hand counts."""
import os

import pytest

from oracle import oracle as orc


def load_golden(path):
    vals = {}
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, rest = line.split("=", 1)
        vals[key.strip()] = rest.split("|")[0].strip()
    return vals


@pytest.fixture(scope="module")
def g(golden_dir):
    return load_golden(os.path.join(golden_dir, "sol_report_gemm4096.txt"))


def rounds_to(value, printed: str) -> bool:
    """True if `value` agrees with the digits the paper printed to within one unit of the last digit.

    The report derives its figures from already-rounded intermediates (682.6 is 1.374e11 / 2.013e8,
    while the exact ratio is 682.67), so rounding and truncation of the exact value are both accepted.
    """
    decimals = len(printed.split(".")[1]) if "." in printed else 0
    return abs(value - float(printed)) < 10 ** (-decimals)


def test_counts_match_the_printed_report_exactly(g):
    n, eb = int(g["n"]), int(g["elem_bytes"])
    assert orc.gemm_flops(n, n, n) == int(g["total_flops"])
    assert orc.gemm_bytes(n, n, n, eb, eb) == int(g["total_bytes"])


def test_tf32_bound_matches_the_printed_report(g):
    n, eb = int(g["n"]), int(g["elem_bytes"])
    r = orc.sol_bound(orc.gemm_flops(n, n, n), orc.gemm_bytes(n, n, n, eb, eb),
                      float(g["peak_tf32_flops"]), float(g["peak_bytes_per_s"]),
                      float(g["sm_clock_mhz"]), float(g["sm_clock_max_mhz"]),
                      float(g["mem_clock_mhz"]), float(g["mem_clock_max_mhz"]))
    assert r["flops"] == int(g["total_flops"]) and r["bytes"] == int(g["total_bytes"])
    assert rounds_to(r["ai"], g["arithmetic_intensity"])
    assert rounds_to(r["eff_peak_flops"] / float(g["peak_tf32_flops"]), g["sm_clock_ratio"])
    # the report multiplies by the ratio already rounded to 4 decimals (0.7576): allow that last-digit slack
    assert abs(r["eff_peak_flops"] / 1e12 - float(g["eff_peak_tf32_tflops"])) < 0.02
    assert rounds_to(r["eff_bytes_per_s"] / 1e12, g["eff_bandwidth_tbs"])
    assert rounds_to(r["t_compute_s"] * 1e3, g["t_compute_tf32_ms"])
    assert rounds_to(r["t_mem_s"] * 1e3, g["t_mem_ms"])
    assert rounds_to(r["t_sol_s"] * 1e3, g["t_sol_tf32_ms"])
    assert abs(r["ridge"] - float(g["ridge_tf32"])) < 0.06
    assert r["compute_bound"] is (g["bottleneck"] == "compute")
    assert r["t_sol_s"] == max(r["t_compute_s"], r["t_mem_s"])


def test_fp16_augmentation_matches_the_printed_report(g):
    n, eb = int(g["n"]), int(g["elem_bytes"])
    r = orc.sol_bound(orc.gemm_flops(n, n, n), orc.gemm_bytes(n, n, n, eb, eb),
                      float(g["peak_fp16_flops"]), float(g["peak_bytes_per_s"]),
                      float(g["sm_clock_mhz"]), float(g["sm_clock_max_mhz"]),
                      float(g["mem_clock_mhz"]), float(g["mem_clock_max_mhz"]))
    assert abs(r["eff_peak_flops"] / 1e12 - float(g["eff_peak_fp16_tflops"])) < 0.02
    assert rounds_to(r["t_sol_s"] * 1e3, g["t_sol_fp16_ms"])
    assert rounds_to(r["t_mem_s"] * 1e3, g["t_mem_ms"])
    assert r["compute_bound"]


def test_memory_bound_case_and_unscaled_clocks():
    # 1 GFLOP over 1 GB at 100 TFLOP/s and 1 TB/s: T_c = 10 us, T_m = 1 ms -> memory bound.
    r = orc.sol_bound(10 ** 9, 10 ** 9, 100e12, 1e12)
    assert r["t_compute_s"] == pytest.approx(1e-5) and r["t_mem_s"] == pytest.approx(1e-3)
    assert r["t_sol_s"] == r["t_mem_s"] and not r["compute_bound"]
    assert r["ai"] == 1.0 and r["ridge"] == pytest.approx(100.0)
    assert r["eff_peak_flops"] == 100e12 and r["eff_bytes_per_s"] == 1e12
    # halving the SM clock doubles T_compute and leaves T_mem alone
    h = orc.sol_bound(10 ** 9, 10 ** 9, 100e12, 1e12, 900, 1800)
    assert h["t_compute_s"] == pytest.approx(2e-5) and h["t_mem_s"] == r["t_mem_s"]


def test_hand_counts_for_the_benchmark_problems():
    # counted by hand from the shapes: 2 bytes per bf16 element, each tensor once
    assert orc.gemm_flops(256, 256, 256) == 33_554_432
    assert orc.gemm_bytes(256, 256, 256) == 393_216
    assert orc.gemm_flops(4096, 4096, 4096) == 137_438_953_472
    assert orc.gemm_bytes(4096, 4096, 4096, has_bias=True) == 3 * 33_554_432 + 8_192
    assert 128 * orc.gemm_flops(256, 256, 512) == 8_589_934_592
    assert 128 * orc.gemm_bytes(256, 256, 512) == 83_886_080
    conv = dict(N=32, H=56, W=56, C=256, K=256, R=3, S=3, pad=(1, 1))
    assert orc.conv_flops(**conv) == 118_380_036_096          # 2 * 100352 * 256 * 2304, halo taps included
    assert orc.conv_bytes(**conv, has_bias=True) == 2 * 51_380_224 + 1_179_648 + 512
    m = 1000
    assert orc.gemm_flops(m, 4096, 4096) == 33_554_432 * m
    assert orc.gemm_bytes(m, 4096, 4096) == 16_384 * m + 33_554_432
    assert orc.gemm_bytes(8, 8, 8, has_c=True) == 4 * 128
    assert orc.gemm_bytes(8, 8, 8, eb_out=4) == 2 * 128 + 256
