"""Seeded synthetic inputs shared by the CUDA library's callers and by the CPU oracle's callers.

This module holds DATA GENERATION ONLY: a counter-based hash, two value
distributions and the shapes of the benchmark problems.  It contains none of
the method's arithmetic (no products, no epilogue, no convolution indexing) and
imports neither the CUDA binding nor the oracle.

Generator.  Element ``i`` of tensor ``tensor_id`` under ``seed`` is derived from

    h(c) = splitmix64((seed XOR tensor_id * 0x9E3779B97F4A7C15) + c)

* ``uniform``:  (h(i) >> 40) * 2^-23 - 1, i.e. U(-1, 1) on a 2^-23 grid (exact in fp32);
* ``normal``:   Box-Muller on u1 = ((h(2i) >> 11) + 1) * 2^-53, u2 = (h(2i+1) >> 11) * 2^-53,
                z = sqrt(-2 ln u1) cos(2 pi u2), evaluated in fp64;
* ``integers``: lo + (h(i) >> 11) mod (hi - lo + 1).

The value is scaled, then rounded to bf16 (round to nearest even).  The same
bf16 bits are handed to both sides of every comparison.  The integer hash is
identical on CPU and GPU; the fp64 log/cos of ``normal`` may differ in the last
place between devices, so a comparison always generates on ONE device and copies.
"""
from __future__ import annotations

import math
from typing import Dict, List, Sequence

import torch

BASE_SEED = 260329010
TENSOR_IDS = {"A": 1, "B": 2, "C": 3, "bias": 4, "M": 5, "X": 6, "Wf": 7}

_MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_MUL1 = 0xBF58476D1CE4E5B9
_MUL2 = 0x94D049BB133111EB


def _signed(x: int) -> int:
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


def splitmix64_scalar(x: int) -> int:
    """Reference scalar form on Python integers (unsigned 64-bit result)."""
    x = (x + _GOLDEN) & _MASK64
    z = x
    z = ((z ^ (z >> 30)) * _MUL1) & _MASK64
    z = ((z ^ (z >> 27)) * _MUL2) & _MASK64
    return z ^ (z >> 31)


def _lsr(x: torch.Tensor, k: int) -> torch.Tensor:
    """Logical shift right of int64 lanes (torch's >> on int64 is arithmetic)."""
    return (x >> k) & ((1 << (64 - k)) - 1)


def _splitmix64(x: torch.Tensor) -> torch.Tensor:
    """Vector form on int64 lanes with two's-complement wrap-around; same bits as the scalar form."""
    z = x + _signed(_GOLDEN)
    z = (z ^ _lsr(z, 30)) * _signed(_MUL1)
    z = (z ^ _lsr(z, 27)) * _signed(_MUL2)
    return z ^ _lsr(z, 31)


def _stream_base(seed: int, tensor_id: int) -> int:
    return _signed((seed ^ ((tensor_id * _GOLDEN) & _MASK64)) & _MASK64)


def _hash(seed: int, tensor_id: int, counters: torch.Tensor) -> torch.Tensor:
    return _splitmix64(counters + _stream_base(seed, tensor_id))


_CHUNK = 1 << 24


def _fill(shape: Sequence[int], fn, device) -> torch.Tensor:
    n = int(math.prod(shape))
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    for start in range(0, n, _CHUNK):
        idx = torch.arange(start, min(start + _CHUNK, n), dtype=torch.int64, device=device)
        out[start:start + idx.numel()] = fn(idx).to(torch.bfloat16)
    return out.view(*shape)


def uniform(shape: Sequence[int], seed: int, tensor_id: int, scale: float = 1.0, device="cpu") -> torch.Tensor:
    """bf16 tensor of U(-1,1) * scale."""
    def fn(idx):
        h = _hash(seed, tensor_id, idx)
        return (_lsr(h, 40).to(torch.float64) * 2.0 ** -23 - 1.0) * scale
    return _fill(shape, fn, device)


def normal(shape: Sequence[int], seed: int, tensor_id: int, scale: float = 1.0, device="cpu") -> torch.Tensor:
    """bf16 tensor of N(0,1) * scale."""
    def fn(idx):
        u1 = (_lsr(_hash(seed, tensor_id, 2 * idx), 11) + 1).to(torch.float64) * 2.0 ** -53
        u2 = _lsr(_hash(seed, tensor_id, 2 * idx + 1), 11).to(torch.float64) * 2.0 ** -53
        return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos(2.0 * math.pi * u2) * scale
    return _fill(shape, fn, device)


def small_integers(shape: Sequence[int], seed: int, tensor_id: int, lo: int = -1, hi: int = 1,
                   device="cpu") -> torch.Tensor:
    """bf16 tensor of integers in [lo, hi]: sums of their products stay exact in fp32 and in bf16."""
    def fn(idx):
        h = _hash(seed, tensor_id, idx)
        return (_lsr(h, 11) % (hi - lo + 1) + lo).to(torch.float64)
    return _fill(shape, fn, device)


def integers(count: int, seed: int, tensor_id: int, lo: int, hi: int) -> List[int]:
    """``count`` Python integers drawn uniformly from the closed range [lo, hi]."""
    base = (seed ^ ((tensor_id * _GOLDEN) & _MASK64)) & _MASK64
    return [lo + (splitmix64_scalar((base + i) & _MASK64) >> 11) % (hi - lo + 1) for i in range(count)]


# ---- the benchmark problems (shapes, distributions, epilogues) -------------------------------------
# Synthetic stand-ins for the paper's workload families: square GEMM, GEMM + bias + ReLU, batched
# matmul with a fused activation, an NHWC 3x3 convolution, and a ragged expert-MLP grouped GEMM.
# All GEMM operands use the K-contiguous pair "A row-major, B column-major".

CONFIGS: Dict[str, dict] = {
    "c1_gemm_256": dict(op="gemm", M=256, N=256, K=256, dist="uniform", scale=1.0, bias=False, epi="none"),
    "c2_gemm_4096_bias_relu": dict(op="gemm", M=4096, N=4096, K=4096, dist="normal", scale=1.0 / 64.0,
                                   bias=True, epi="relu"),
    "c3_batched_128x256x256x512_gelu": dict(op="batched", batch=128, M=256, N=256, K=512, dist="uniform",
                                            scale=1.0, bias=False, epi="gelu"),
    "c4_conv_32x56x56x256_k256_3x3_bias_relu": dict(op="conv", N=32, H=56, W=56, C=256, K=256, R=3, S=3,
                                                    pad=(1, 1), stride=(1, 1), dil=(1, 1), dist="normal",
                                                    scale=1.0 / 48.0, bias=True, epi="relu"),
    "c5_grouped_16xMx4096x4096_silu": dict(op="grouped", groups=16, M_lo=128, M_hi=4096, N=4096, K=4096,
                                           dist="normal", scale=1.0 / 64.0, bias=False, epi="silu"),
}


def _draw(dist: str):
    return {"uniform": uniform, "normal": normal}[dist]


def make_gemm(M, N, K, dist="uniform", scale=1.0, bias=False, seed=BASE_SEED, device="cpu", batch=None):
    """A [M,K] (row-major) and B [N,K] (column-major storage) (+ leading batch), bias [N] ~ N(0,1)."""
    lead = [] if batch is None else [batch]
    A = _draw(dist)(lead + [M, K], seed, TENSOR_IDS["A"], scale, device)
    B = _draw(dist)(lead + [N, K], seed, TENSOR_IDS["B"], scale, device)
    b = normal([N], seed, TENSOR_IDS["bias"], 1.0, device) if bias else None
    return A, B, b


def grouped_sizes(groups: int, lo: int, hi: int, seed: int = BASE_SEED) -> List[int]:
    return integers(groups, seed, TENSOR_IDS["M"], lo, hi)


def make_grouped(Ms: Sequence[int], N, K, dist="normal", scale=1.0, seed=BASE_SEED, device="cpu"):
    """Per group g: A_g [M_g,K], B_g [N,K]; every group draws from its own stream."""
    As = [_draw(dist)([m, K], seed + 1000 * (g + 1), TENSOR_IDS["A"], scale, device) for g, m in enumerate(Ms)]
    Bs = [_draw(dist)([N, K], seed + 1000 * (g + 1), TENSOR_IDS["B"], scale, device) for g in range(len(Ms))]
    return As, Bs


def make_conv(N, H, W, C, K, R, S, dist="normal", scale=1.0, bias=False, seed=BASE_SEED, device="cpu"):
    """X in NHWC, filter in KRSC, bias [K] ~ N(0,1)."""
    X = _draw(dist)([N, H, W, C], seed, TENSOR_IDS["X"], scale, device)
    Wf = _draw(dist)([K, R, S, C], seed, TENSOR_IDS["Wf"], scale, device)
    b = normal([K], seed, TENSOR_IDS["bias"], 1.0, device) if bias else None
    return X, Wf, b
