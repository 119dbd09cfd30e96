"""The seeded input generators: reproducible bits, documented distributions, no method arithmetic."""
import torch

from paper_2603_29010_b200 import inputs


def test_vector_hash_equals_scalar_hash():
    seed, tid = inputs.BASE_SEED, 3
    idx = torch.tensor([0, 1, 2, 12345, 2 ** 40 + 7], dtype=torch.int64)
    got = inputs._hash(seed, tid, idx).tolist()
    base = (seed ^ ((tid * 0x9E3779B97F4A7C15) & (2 ** 64 - 1))) & (2 ** 64 - 1)
    for i, h in zip(idx.tolist(), got):
        want = inputs.splitmix64_scalar((base + i) & (2 ** 64 - 1))
        assert (h & (2 ** 64 - 1)) == want
    # published splitmix64 test vector: state 0 -> first output 0xE220A8397B1DCDAF
    assert inputs.splitmix64_scalar(0) == 0xE220A8397B1DCDAF


def test_generators_are_deterministic_and_distinct_per_tensor():
    a1 = inputs.uniform([64, 33], 7, 1)
    a2 = inputs.uniform([64, 33], 7, 1)
    b = inputs.uniform([64, 33], 7, 2)
    assert a1.dtype == torch.bfloat16 and torch.equal(a1, a2) and not torch.equal(a1, b)
    assert float(a1.float().abs().max()) <= 1.0


def test_distributions_have_the_stated_moments():
    u = inputs.uniform([1 << 16], 1, 1).double()
    assert abs(float(u.mean())) < 0.02 and abs(float(u.var()) - 1.0 / 3.0) < 0.01
    z = inputs.normal([1 << 16], 1, 2, scale=0.5).double()
    assert abs(float(z.mean())) < 0.01 and abs(float(z.std()) - 0.5) < 0.01
    k = inputs.small_integers([1 << 12], 1, 3, -1, 1).double()
    assert set(k.tolist()) == {-1.0, 0.0, 1.0}


def test_grouped_sizes_cover_the_closed_range():
    ms = inputs.grouped_sizes(16, 128, 4096)
    assert len(ms) == 16 and all(128 <= m <= 4096 for m in ms) and ms == inputs.grouped_sizes(16, 128, 4096)
    many = inputs.integers(20000, 5, 5, 0, 3)
    assert set(many) == {0, 1, 2, 3}


def test_benchmark_configs_have_the_stated_shapes():
    c = inputs.CONFIGS
    assert len(c) == 5
    assert c["c2_gemm_4096_bias_relu"]["M"] == 4096 and c["c2_gemm_4096_bias_relu"]["epi"] == "relu"
    A, B, bias = inputs.make_gemm(8, 16, 24, bias=True)
    assert A.shape == (8, 24) and B.shape == (16, 24) and bias.shape == (16,)
    X, Wf, b = inputs.make_conv(2, 5, 6, 8, 4, 3, 3, bias=True)
    assert X.shape == (2, 5, 6, 8) and Wf.shape == (4, 3, 3, 8) and b.shape == (4,)
