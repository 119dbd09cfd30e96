"""Element-by-element comparison of a computed result with the oracle's fp64 reference.

bf16 output:  |D - ref| <= 1e-2 + 1e-2 |ref|                      (every element)
fp16 output:  |D - ref| <= 1e-3 + 1e-3 |ref| + 1e-4 * absacc      (one fp16 rounding is 2^-11 = 4.9e-4 relative;
              the last term is the fp32 path's bound for the accumulation)
fp32 output:  |D - ref| <= 1e-4 * absacc,  absacc = |alpha| sum|a||b| + |beta c| + |bias|
              (relative to the magnitude of the terms summed, so that results
              near zero from cancellation are judged on the dot product's scale)
"""
from __future__ import annotations

import torch

BF16_ATOL = 1e-2
BF16_RTOL = 1e-2
F32_RTOL = 1e-4


def allowed_error(ref: torch.Tensor, absacc: torch.Tensor, out_dtype: torch.dtype) -> torch.Tensor:
    if out_dtype == torch.bfloat16:
        return BF16_ATOL + BF16_RTOL * ref.abs()
    if out_dtype == torch.float16:
        return 1e-3 + 1e-3 * ref.abs() + F32_RTOL * absacc
    if out_dtype == torch.float32:
        return F32_RTOL * absacc
    raise ValueError(out_dtype)


def mismatches(D: torch.Tensor, ref: torch.Tensor, absacc: torch.Tensor) -> torch.Tensor:
    """Boolean mask of elements outside the tolerance (NaN/Inf in D always count)."""
    d = D.detach().to("cpu").to(torch.float64).reshape(ref.shape)
    err = (d - ref).abs()
    bad = err > allowed_error(ref, absacc, D.dtype)
    return bad | ~torch.isfinite(d)


def assert_matches(D: torch.Tensor, ref: torch.Tensor, absacc: torch.Tensor, what: str = "") -> None:
    bad = mismatches(D, ref, absacc)
    if bad.any():
        d = D.detach().to("cpu").to(torch.float64).reshape(ref.shape)
        idx = bad.nonzero()[:8].tolist()
        shown = [(tuple(i), float(d[tuple(i)]), float(ref[tuple(i)])) for i in idx]
        raise AssertionError(f"{what}: {int(bad.sum())} of {bad.numel()} elements outside tolerance; "
                             f"first (index, got, want): {shown}")


def assert_bit_exact(D: torch.Tensor, ref: torch.Tensor, what: str = "") -> None:
    """For integer-valued problems whose every partial sum is exact in fp32 and in the output type."""
    d = D.detach().to("cpu").to(torch.float64).reshape(ref.shape)
    bad = d != ref
    if bad.any():
        idx = bad.nonzero()[:8].tolist()
        shown = [(tuple(i), float(d[tuple(i)]), float(ref[tuple(i)])) for i in idx]
        raise AssertionError(f"{what}: {int(bad.sum())} of {bad.numel()} elements differ; "
                             f"first (index, got, want): {shown}")
