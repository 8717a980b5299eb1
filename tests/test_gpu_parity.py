"""GPU parity: every entry point of the C ABI against the CPU oracle on the
same seeded inputs.  Integer/bit outputs must be identical; mu and sigma within
1e-5 relative."""
import math

import numpy as np
import pytest
import torch

from gpu_helpers import (assert_same_bits, assert_same_codes, assert_stats_close, np_bits,
                         oracle_layer)
from paper_2006_08173_b200 import synth

pytestmark = pytest.mark.gpu

DTYPES = [torch.float32, torch.bfloat16]
SIZES = [1, 3, 1023, 16384, 16385, 2 ** 20 + 7]          # below a vector, ragged tails, several tiles


def make(n, dtype, mu=-12.0, sigma=2.0, p=0.4, seed=0, **kw):
    return synth.lognormal_tensor(n, mu, sigma, p, seed, dtype=dtype, device="cuda", **kw)


# ------------------------------------------------------------------ lgn_stats
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("n", SIZES + [5_000_000])
def test_stats_parity(lgn, oracle, dtype, n):
    g = make(n, dtype, seed=n % 97)
    got = lgn.lgn_stats(g)
    want = oracle.stats(np_bits(g))
    assert_stats_close(got, want)
    assert got["sum_ln"] == pytest.approx(want["mu"] * want["nnz"], rel=1e-5, abs=1e-9)


@pytest.mark.parametrize("dtype", DTYPES)
def test_stats_special_inputs(lgn, oracle, dtype):
    z = torch.zeros(40_000, dtype=dtype, device="cuda")
    assert lgn.lgn_stats(z) == {"n": 40_000, "nnz": 0, "sum_ln": 0.0, "sum_ln2": 0.0, "mu": 0.0, "sigma": 0.0}
    e = torch.zeros(0, dtype=dtype, device="cuda")
    assert lgn.lgn_stats(e)["n"] == 0
    # negative zeros are zeros; powers of two have exact logs
    g = torch.tensor([2.0, -4.0, 8.0, 0.0, -0.0], dtype=dtype, device="cuda")
    st = lgn.lgn_stats(g)
    assert st["nnz"] == 3
    assert st["mu"] == pytest.approx(2 * math.log(2), rel=1e-6)
    assert st["sigma"] == pytest.approx(math.log(2) * math.sqrt(2 / 3), rel=1e-5)
    # heavy tail, subnormal range, large magnitudes, mixture
    for kw in [dict(mu=-12.0, sigma=4.0, p=0.5), dict(mu=-85.0, sigma=4.0, p=0.3),
               dict(mu=3.0, sigma=2.0, p=0.5, clip=1e4),
               dict(mu=0.0, sigma=1.0, p=0.5, mixture=[(-14.0, 1.5), (-8.0, 1.5)])]:
        g = make(2 ** 20 + 7, dtype, seed=5, **kw)
        assert_stats_close(lgn.lgn_stats(g), oracle.stats(np_bits(g)))


def test_stats_is_deterministic(lgn):
    g = make(3_000_001, torch.float32, seed=1)
    a = lgn.lgn_stats(g)
    for _ in range(3):
        assert lgn.lgn_stats(g) == a


# ------------------------------------------------------------------ lgn_prune
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("n", SIZES)
def test_prune_parity(lgn, oracle, dtype, n):
    g = make(n, dtype, seed=n % 89 + 1)
    g_np = np_bits(g)
    st = oracle.stats(g_np)
    for S, seed in [(0.8, 1), (0.5, 2 ** 40 + 3), (0.99, 7)]:
        tau = oracle.threshold(st["mu"], st["sigma"], st["zero_frac"], S) if st["nnz"] else 0.0
        out = lgn.lgn_prune(g, tau, seed)
        dt = oracle.BF16 if dtype == torch.bfloat16 else oracle.F32
        ref = oracle.prune(g_np, oracle.snap_tau(tau, dt), seed)
        assert_same_bits(out, ref)


@pytest.mark.parametrize("dtype", DTYPES)
def test_prune_edge_thresholds(lgn, oracle, dtype):
    g = make(100_003, dtype, mu=-85.0, sigma=4.0, p=0.3, seed=3)     # reaches fp32 subnormals
    g_np = np_bits(g)
    dt = oracle.BF16 if dtype == torch.bfloat16 else oracle.F32
    for tau in (0.0, 1e-45, 1e-38, 1e-30, 1e30, 1e39):
        assert_same_bits(lgn.lgn_prune(g, tau, 11), oracle.prune(g_np, oracle.snap_tau(tau, dt), 11))
    # tau = 0 is the identity (up to the sign of zero)
    out = lgn.lgn_prune(g, 0.0, 1)
    assert torch.equal(out, torch.where(g == 0, torch.zeros_like(g), g))


# ------------------------------------------------------------------ lgn_quantize
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("nbits", [4, 5, 6, 7, 8])
def test_quantize_parity_all_formats(lgn, oracle, dtype, nbits):
    n = 2 ** 15 + 13
    g = make(n, dtype, mu=-12.0, sigma=3.0, p=0.3, seed=nbits)
    g_np = np_bits(g)
    for n2 in range(1, nbits):
        n1 = nbits - 1 - n2
        fmt = {"nbits": nbits, "exp_bits": n2, "man_bits": n1, "scale_exp": -17}
        for rounding, seed in [(0, 0), (1, 5)]:
            packed = lgn.lgn_quantize(g, fmt, rounding, seed)
            ref = oracle.pack(oracle.quantize(g_np, n2, n1, -17, rounding, seed), nbits)
            assert packed.numel() >= ref.size
            assert_same_codes(packed, ref)


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("n", SIZES)
def test_quantize_parity_sizes(lgn, oracle, dtype, n):
    g = make(n, dtype, seed=n % 83 + 2)
    g_np = np_bits(g)
    for nbits, n2, rounding in [(6, 4, 1), (5, 4, 0), (5, 3, 1), (6, 5, 0), (7, 4, 1), (8, 5, 1), (4, 3, 1)]:
        n1 = nbits - 1 - n2
        fmt = {"nbits": nbits, "exp_bits": n2, "man_bits": n1, "scale_exp": -17}
        packed = lgn.lgn_quantize(g, fmt, rounding, 2 ** 33 + 1)
        assert_same_codes(packed, oracle.pack(oracle.quantize(g_np, n2, n1, -17, rounding, 2 ** 33 + 1), nbits))


@pytest.mark.parametrize("dtype", DTYPES)
def test_quantize_extreme_scales(lgn, oracle, dtype):
    n = 70_001
    for mu, sigma, e_s in [(-85.0, 4.0, -123), (-85.0, 4.0, -140), (3.0, 2.0, 4), (-12.0, 2.0, 60), (-12.0, 2.0, -80)]:
        g = make(n, dtype, mu=mu, sigma=sigma, p=0.2, seed=9, clip=1e4 if mu > 0 else None)
        g_np = np_bits(g)
        for nbits, n2 in [(6, 5), (6, 4), (5, 4), (8, 2), (4, 1)]:
            n1 = nbits - 1 - n2
            fmt = {"nbits": nbits, "exp_bits": n2, "man_bits": n1, "scale_exp": e_s}
            for rounding in (0, 1):
                packed = lgn.lgn_quantize(g, fmt, rounding, 3)
                assert_same_codes(packed, oracle.pack(oracle.quantize(g_np, n2, n1, e_s, rounding, 3), nbits))
