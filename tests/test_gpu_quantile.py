"""GPU parity of lgn_quantile (the high quantile that estimates the cut k of the
truncated lognormal) against the oracle's sort-based order statistic: the value bit
for bit, the nonzero count exactly."""
import numpy as np
import pytest
import torch

from gpu_helpers import np_bits
from paper_2006_08173_b200 import synth

pytestmark = pytest.mark.gpu

DTYPES = [torch.float32, torch.bfloat16]


def check(lgn, oracle, g, q):
    got = lgn.lgn_quantile(g, q)
    g_np = np_bits(g)
    st = oracle.stats(g_np)
    _, want = oracle.quantile_k(g_np, q, st["mu"], max(st["sigma"], 1e-6))
    assert got["nnz"] == st["nnz"]
    assert np.float32(got["value"]).tobytes() == np.float32(want).tobytes(), (got, want, q)


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("n", [1, 3, 1023, 2 ** 20 + 7, 5_000_001])
def test_quantile_parity(lgn, oracle, dtype, n):
    g = synth.lognormal_tensor(n, -12.0, 2.0, 0.4, seed=n % 83, dtype=dtype, device="cuda")
    for q in (0.0, 0.5, 0.997, 1.0):
        check(lgn, oracle, g, q)


@pytest.mark.parametrize("dtype", DTYPES)
def test_quantile_parity_bracket_path(lgn, oracle, dtype):
    """From 2^24 elements the selection reads the tensor once, around a bracket taken from a sample."""
    g = synth.lognormal_tensor(2 ** 24 + 5, -12.0, 2.0, 0.4, seed=17, dtype=dtype, device="cuda")
    for q in (0.0, 0.003, 0.5, 0.9, 0.997, 0.99999, 1.0):
        check(lgn, oracle, g, q)
    g = synth.lognormal_tensor(2 ** 26 + 8 * 3 + 1, -9.0, 3.0, 0.7, seed=18, dtype=dtype, device="cuda")
    check(lgn, oracle, g, 0.997)


@pytest.mark.parametrize("dtype", DTYPES)
def test_quantile_when_the_bracket_fails(lgn, oracle, dtype):
    """Inputs on which the one-read selection has to give up (more elements inside the bracket than its
    list holds; a sample without a nonzero element) and the two-pass selection answers instead."""
    n = 2 ** 24 + 11
    gen = torch.Generator(device="cuda").manual_seed(3)
    # all values equal; all values in one bin of the upper 15 bits; every value distinct in a narrow band
    const = torch.full((n,), -3.0, device="cuda").to(dtype)
    const[::3] = 0
    band = (1.0 + torch.rand(n, device="cuda", generator=gen) / 128.0).to(dtype)
    for g in (const, band):
        for q in (0.5, 0.997):
            check(lgn, oracle, g, q)
    # a handful of nonzero elements that the sample is unlikely to meet
    sparse = torch.zeros(n, dtype=dtype, device="cuda")
    sparse[torch.tensor([5, 77_777, 1_000_003, 14_999_999, n - 1], device="cuda")] = torch.tensor([0.5, -2.0, 1e-3, 8.0, -0.25], device="cuda").to(dtype)
    for q in (0.0, 0.5, 1.0):
        check(lgn, oracle, sparse, q)
    # magnitudes in increasing order (the sample still represents them), and in two populations far apart
    ramp = synth.lognormal_tensor(n, -12.0, 2.0, 0.2, seed=4, dtype=dtype, device="cuda")
    ramp = ramp[torch.argsort(ramp.float().abs())].contiguous()
    check(lgn, oracle, ramp, 0.997)
    two = torch.cat([synth.lognormal_tensor(n // 2, -20.0, 1.0, 0.1, seed=5, dtype=dtype, device="cuda"),
                     synth.lognormal_tensor(n - n // 2, 2.0, 0.5, 0.0, seed=6, dtype=dtype, device="cuda")])
    for q in (0.4, 0.5, 0.6):
        check(lgn, oracle, two, q)


@pytest.mark.parametrize("dtype", DTYPES)
def test_quantile_special_inputs(lgn, oracle, dtype):
    z = torch.zeros(70_000, dtype=dtype, device="cuda")
    assert lgn.lgn_quantile(z, 0.997) == {"value": 0.0, "nnz": 0}
    assert lgn.lgn_quantile(torch.zeros(0, dtype=dtype, device="cuda"), 0.5) == {"value": 0.0, "nnz": 0}
    # many equal values; negative values; fp32 subnormals; a heavy tail
    g = torch.tensor([3.0, -3.0, 3.0, 0.0, -0.0, 0.5, -7.0] * 1000, dtype=dtype, device="cuda")
    for q in (0.1, 0.5, 0.9, 1.0):
        check(lgn, oracle, g, q)
    for kw in [dict(mu=-85.0, sigma=4.0, p=0.3), dict(mu=-12.0, sigma=4.0, p=0.5), dict(mu=3.0, sigma=2.0, p=0.5, clip=1e4)]:
        g = synth.lognormal_tensor(300_003, kw["mu"], kw["sigma"], kw["p"], seed=9, dtype=dtype, device="cuda", clip=kw.get("clip"))
        for q in (0.003, 0.997):
            check(lgn, oracle, g, q)


def test_k_of_a_lognormal_tensor(lgn, oracle):
    """End to end: statistics and quantile from the library give the cut k in sigmas."""
    g = synth.lognormal_tensor(4_000_000, -12.0, 2.0, 0.5, seed=1, device="cuda")
    st = lgn.lgn_stats(g)
    v = lgn.lgn_quantile(g, 0.997)["value"]
    k = (np.log(v) - st["mu"]) / st["sigma"]
    assert abs(k - 2.748) < 0.03                                   # the 0.997 quantile of a normal
    c = lgn.lgn_cosine_similarity(st["mu"], st["sigma"], k, lgn.lgn_threshold(st["mu"], st["sigma"], 0.5, 0.9))
    assert 0.9 < c < 1.0


def test_quantile_errors(lgn):
    g = torch.ones(64, device="cuda")
    ws = torch.empty(lgn.lgn_quantile_workspace_bytes(), dtype=torch.uint8, device="cuda")
    for q in (-0.1, 1.5, float("nan")):
        with pytest.raises(lgn.LgnError):
            lgn.lgn_quantile(g, q, ws)
    with pytest.raises(lgn.LgnError):
        lgn.lgn_quantile(g, 0.5, ws[:1024])
