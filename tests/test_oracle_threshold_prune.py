"""Pins for the oracle's sparsity <-> threshold closed form (Eq. 6-8) and for
stochastic pruning (Eq. 5)."""
import math

import numpy as np
import pytest
import torch
from scipy import integrate, stats as sps

from paper_2006_08173_b200 import synth


# ------------------------------------------------------------------ Eq. 6-8
@pytest.mark.parametrize("sigma", [0.3, 1.0, 2.0, 3.5, 5.5])
@pytest.mark.parametrize("u", [-6.0, -1.0, 0.0, 0.8, 2.5, 7.0])
def test_eq8_equals_quadrature_of_eq6(oracle, sigma, u):
    """Eq. 6: S = E_eps[ CDF_lognormal(alpha*eps) ], eps ~ U[0,1]; here with
    mu = 0, alpha = e^u, a library lognormal CDF and adaptive quadrature."""
    alpha = math.exp(u)
    cdf = lambda e: sps.lognorm.cdf(alpha * e, s=sigma)
    ref, err = integrate.quad(cdf, 0.0, 1.0, epsabs=1e-13, epsrel=1e-12, limit=400)
    assert oracle.sparsity_of(u, sigma) == pytest.approx(ref, abs=5e-10)


def test_eq8_monte_carlo(oracle):
    rs = np.random.RandomState(5)
    n = 4_000_000
    for mu, sigma, S in [(-12.0, 2.0, 2.0 / 3.0), (0.0, 3.0, 0.9), (-5.0, 1.5, 0.5)]:
        tau = oracle.threshold(mu, sigma, 0.0, S)
        x = np.exp(mu + sigma * rs.standard_normal(n))
        eps = rs.random_sample(n)
        got = np.mean(x < tau * eps)
        assert abs(got - S) < 4 * math.sqrt(S * (1 - S) / n)


@pytest.mark.parametrize("S", [1e-6, 0.01, 0.5, 0.8, 0.85, 0.99, 1 - 1e-9])
@pytest.mark.parametrize("sigma", [1e-3, 0.5, 2.0, 4.0, 8.0])
def test_threshold_inverts_eq8(oracle, S, sigma):
    mu = -7.25
    tau = oracle.threshold(mu, sigma, 0.0, S)
    u = math.log(tau) - mu
    assert oracle.sparsity_of(u, sigma) == pytest.approx(S, rel=1e-9, abs=1e-13)


def test_threshold_small_sigma_limit(oracle):
    # all magnitudes equal e^mu: S = 1 - e^mu/alpha for alpha >= e^mu
    for S in (0.1, 0.5, 0.9):
        tau = oracle.threshold(1.5, 0.0, 0.0, S)
        assert tau == pytest.approx(math.exp(1.5) / (1 - S), rel=1e-5)


def test_threshold_monotone_in_sparsity_and_scales_with_mu(oracle):
    taus = [oracle.threshold(-12.0, 2.0, 0.0, S) for S in np.linspace(0.05, 0.95, 19)]
    assert all(b > a for a, b in zip(taus, taus[1:]))
    assert oracle.threshold(-10.0, 2.0, 0.0, 0.7) == pytest.approx(
        math.exp(2.0) * oracle.threshold(-12.0, 2.0, 0.0, 0.7), rel=1e-12)


def test_threshold_bimodal_adjustment(oracle):
    mu, sigma = -12.0, 2.0
    for l, S in [(0.4, 0.8), (0.5, 0.85), (0.3, 0.31)]:
        Sp = (S - l) / (1 - l)
        assert l + (1 - l) * Sp == pytest.approx(S, rel=1e-15)
        assert oracle.threshold(mu, sigma, l, S) == oracle.threshold(mu, sigma, 0.0, Sp)
    assert oracle.threshold(mu, sigma, 0.5, 0.5) == 0.0      # already sparse enough
    assert oracle.threshold(mu, sigma, 0.6, 0.5) == 0.0
    assert oracle.threshold(mu, sigma, 1.0, 0.5) == 0.0      # all-zero tensor
    assert oracle.threshold(mu, sigma, 0.0, 0.0) == 0.0
    for bad in [(0.0, 1.0), (0.0, -0.1), (1.5, 0.5), (-0.1, 0.5)]:
        with pytest.raises(ValueError):
            oracle.threshold(mu, sigma, bad[0], bad[1])


def test_snap_tau_matches_library_roundings(oracle):
    rs = np.random.RandomState(0)
    for tau in np.exp(rs.uniform(-40, 40, 200)):
        assert oracle.snap_tau(tau, oracle.F32) == float(np.float32(tau))
        ref = float(torch.tensor(float(np.float32(tau))).to(torch.bfloat16).to(torch.float64))
        assert oracle.snap_tau(tau, oracle.BF16) == ref
    assert oracle.snap_tau(1e60, oracle.F32) == float(np.finfo(np.float32).max)
    assert oracle.snap_tau(1e60, oracle.BF16) == float(torch.finfo(torch.bfloat16).max)
    assert oracle.snap_tau(0.0, oracle.BF16) == 0.0


# ------------------------------------------------------------------ Eq. 5
H_HALF = 0x7FFF            # eps = (h + 1) / 2^16 = 1/2


def test_prune_hand_cases(oracle):
    cases = [                     # x, tau, h, expected
        (0.6, 1.0, H_HALF, 1.0),
        (0.4, 1.0, H_HALF, 0.0),
        (-0.5, 1.0, H_HALF, -1.0),          # |x| == alpha*eps is kept
        (1.0, 1.0, H_HALF, 1.0),            # |x| == alpha maps to alpha
        (-1.5, 1.0, H_HALF, -1.5),
        (0.0, 1.0, 0, 0.0),                 # zero stays zero whatever eps
        (2.0 ** -16, 1.0, 0, 1.0),          # eps = 2^-16, the smallest
        (2.0 ** -17, 1.0, 0, 0.0),
        (0.99999, 1.0, 0xFFFF, 0.0),        # eps = 1: only |x| == alpha survives
        (1.0, 1.0, 0xFFFF, 1.0),
        (3.0, 0.0, H_HALF, 3.0),            # tau = 0: identity
        (0.0, 0.0, H_HALF, 0.0),
    ]
    for x, tau, h, want in cases:
        assert oracle.prune_one(float(np.float32(x)), tau, h) == float(np.float32(want))
    assert math.copysign(1.0, oracle.prune_one(-0.0, 1.0, 0)) == 1.0      # -0 -> +0 when pruning
    assert math.copysign(1.0, oracle.prune_one(-0.0, 0.0, 0)) == -1.0     # tau = 0 changes nothing at all


def test_prune_threshold_product_is_rounded_to_fp32(oracle):
    tau = float(np.float32(1.0 + 2 ** -23))
    h = 0x5554
    eps = (h + 1) / 2 ** 16
    thr32 = float(np.float32(tau) * np.float32(eps))            # numpy's fp32 multiply
    exact = tau * eps
    assert thr32 != exact
    lo, hi = min(thr32, exact), max(thr32, exact)
    x = float(np.float32(thr32))
    assert oracle.prune_one(x, tau, h) == tau                   # at the rounded product: kept
    below = float(np.nextafter(np.float32(thr32), np.float32(0)))
    assert oracle.prune_one(below, tau, h) == 0.0


def test_prune_keep_probability_enumerated_over_all_draws(oracle):
    """Eq. 5 on the grid eps = (h+1)/2^16: over all 2^16 values of h an element with
    0 < |x| <= alpha is kept exactly floor(2^16 |x| / alpha) times (alpha a power of two, so
    alpha*eps is exact), hence E[T(x)] = alpha * floor(2^16 |x|/alpha) / 2^16 lies in
    (|x| - alpha 2^-16, |x|]: the bias of the 16-bit grid, against the exact unbiasedness
    of a continuous eps.  For a full-mantissa alpha the one fp32 rounding of alpha*eps can
    move the count by at most one."""
    hs = np.arange(1 << 16, dtype=np.uint16)
    for alpha in (1.0, 2.0 ** -14, 2.0 ** 10):
        for ratio in (2.0 ** -16, 3 * 2.0 ** -16, 0.1, 1 / 3, 0.5, 0.75 - 2.0 ** -20, 0.999, 1.0):
            x = float(np.float32(alpha * ratio))
            g = np.full(1 << 16, -x, dtype=np.float32)
            out = oracle.prune_with_bits(g, alpha, hs)
            kept = int(np.count_nonzero(out))
            assert kept == math.floor((1 << 16) * (x / alpha)), (alpha, ratio)
            assert np.all(out[out != 0] == np.float32(-alpha))
            mean = -float(out.astype(np.float64).mean())
            assert x - alpha * 2.0 ** -16 < mean <= x
        below = float(np.float32(alpha * 2.0 ** -17))                   # under the smallest alpha*eps: never kept
        assert np.count_nonzero(oracle.prune_with_bits(np.full(1 << 16, below, dtype=np.float32), alpha, hs)) == 0
    alpha = float(np.float32(1.2345678))
    for ratio in (0.1, 0.37, 0.9):
        x = float(np.float32(alpha * ratio))
        kept = int(np.count_nonzero(oracle.prune_with_bits(np.full(1 << 16, x, dtype=np.float32), alpha, hs)))
        assert abs(kept - (1 << 16) * x / alpha) <= 1.0 + 1e-9


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_prune_three_value_property(oracle, dtype):
    n = 200_000
    t = synth.lognormal_tensor(n, -12.0, 2.0, 0.4, seed=2, dtype=dtype)
    g = synth.as_numpy_bits(t)
    st = oracle.stats(g)
    code = oracle.BF16 if dtype == torch.bfloat16 else oracle.F32
    tau = oracle.snap_tau(oracle.threshold(st["mu"], st["sigma"], st["zero_frac"], 0.8), code)
    out = oracle.prune(g, tau, seed=1)
    x = t.to(torch.float64).numpy()
    y = synth.from_numpy_bits(out).to(torch.float64).numpy()
    big = np.abs(x) > tau
    assert np.array_equal(y[big], x[big])
    small = ~big
    assert np.all(np.isin(y[small], [0.0, tau, -tau]))
    nz = small & (y != 0)
    assert np.array_equal(np.sign(y[nz]), np.sign(x[nz]))
    assert np.all(y[x == 0] == 0)
    # the seeded path is the supplied-bits path fed by the generator
    assert np.array_equal(out, oracle.prune_with_bits(g, tau, oracle.rand16_fill(1, 0, n)))
    # element i depends on its global index only
    assert np.array_equal(out[1000:1300], oracle.prune(g[1000:1300], tau, seed=1, first=1000))


def test_prune_is_unbiased(oracle):
    """E[T(x)] = x for |x| <= alpha: checked per magnitude bin on positive inputs."""
    n = 2_000_000
    t = synth.lognormal_tensor(n, -12.0, 2.0, 0.0, seed=4).abs()
    g = synth.as_numpy_bits(t)
    tau = oracle.snap_tau(oracle.threshold(-12.0, 2.0, 0.0, 0.8), oracle.F32)
    y = oracle.prune(g, tau, seed=9).astype(np.float64)
    x = g.astype(np.float64)
    assert abs(y.sum() - x.sum()) < 4 * math.sqrt(np.sum(np.where(x < tau, x * (tau - x), 0.0)))
    edges = tau * np.array([0.0, 0.01, 0.05, 0.2, 0.5, 0.8, 1.0])
    for lo, hi in zip(edges[:-1], edges[1:]):
        m = (x > lo) & (x <= hi)
        sd = math.sqrt(np.sum(x[m] * (tau - x[m])))
        assert abs(y[m].sum() - x[m].sum()) < 4 * sd


@pytest.mark.parametrize("mu,sigma,l,S", [(-12.0, 2.0, 0.4, 0.8), (-10.0, 3.0, 0.5, 0.85),
                                          (-14.0, 1.5, 0.3, 0.5), (-9.0, 2.5, 0.0, 0.99)])
def test_prune_achieves_requested_sparsity(oracle, mu, sigma, l, S):
    n = 4_000_000
    g = synth.as_numpy_bits(synth.lognormal_tensor(n, mu, sigma, l, seed=6))
    st = oracle.stats(g)
    tau = oracle.snap_tau(oracle.threshold(st["mu"], st["sigma"], st["zero_frac"], S), oracle.F32)
    out = oracle.prune(g, tau, seed=3)
    achieved = oracle.count_zeros(out) / n
    assert achieved == np.mean(out == 0)
    assert abs(achieved - S) < 1e-3


def test_prune_tau_zero_is_identity(oracle):
    g = synth.as_numpy_bits(synth.lognormal_tensor(10_000, -12.0, 2.0, 0.5, seed=8))
    g[:3] = [-0.0, 0.0, -1e-30]
    out = oracle.prune(g, 0.0, seed=1)
    assert np.array_equal(out.view(np.uint32), g.view(np.uint32))
