"""Pins for the oracle's cosine-similarity closed form, its inverse, the heterogeneous
sparsity allocation and the quantile that estimates the cut k (appendix "Cosine
similarity and heterogeneous stochastic pruning")."""
import math

import numpy as np
import pytest

import oracle


def truncated_lognormal(n, sigma, k, seed, mu=0.0):
    """exp(mu + sigma z), z ~ N(0,1) redrawn until z <= k."""
    rs = np.random.RandomState(seed)
    z = rs.standard_normal(int(n * 1.2) + 1000)
    z = z[z <= k][:n]
    assert z.size == n
    sign = np.where(rs.rand(n) < 0.5, -1.0, 1.0)
    return (sign * np.exp(mu + sigma * z)).astype(np.float32)


@pytest.mark.parametrize("sigma,k", [(1.0, 3.0), (2.0, 2.75), (3.0, 3.0), (3.0, 2.0)])
@pytest.mark.parametrize("S", [0.5, 0.8, 0.95])
def test_closed_form_tracks_simulation(sigma, k, S):
    """The appendix compares analysis and simulation (its sigma = 3 and 5 figure): prune a
    truncated lognormal sample with Eq. 5 and measure the cosine between input and output."""
    n, mu = 2_000_000, -3.0
    x = truncated_lognormal(n, sigma, k, seed=int(10 * sigma + k + 100 * S), mu=mu)
    u = math.log(oracle.threshold(mu, sigma, 0.0, S)) - mu
    if u > k * sigma:
        pytest.skip("threshold above the cut")
    tau = oracle.snap_tau(math.exp(mu + u), oracle.F32)
    t = oracle.prune(x, tau, seed=3).astype(np.float64)
    xd = x.astype(np.float64)
    measured = float(xd @ t / math.sqrt((xd @ xd) * (t @ t)))
    want = oracle.cosine_similarity(u, sigma, k)
    # the sums are dominated by the few largest elements: the tolerance follows the tail weight
    tol = 0.004 if sigma <= 2.0 else 0.02
    assert abs(measured - want) < tol
    assert want <= 1.0


def test_limits_and_monotonicity():
    for sigma, k in [(1.0, 3.0), (3.0, 3.0), (5.0, 2.5)]:
        assert oracle.cosine_similarity(-200.0, sigma, k) == pytest.approx(1.0, abs=1e-12)
        us = np.linspace(-10 * sigma, k * sigma, 60)
        cs = [oracle.cosine_similarity(float(u), sigma, k) for u in us]
        assert all(a >= b - 1e-15 for a, b in zip(cs, cs[1:]))           # more pruning, smaller cosine
        assert cs[-1] < 1.0
        # a wider cut (more large elements kept in the model) gives a larger cosine at the same threshold
        assert oracle.cosine_similarity(1.0, sigma, k + 1.0) > oracle.cosine_similarity(1.0, sigma, k)


def test_threshold_for_cosine_is_the_inverse():
    for sigma, k in [(1.5, 3.0), (3.0, 2.75), (4.0, 3.0)]:
        for c in (0.999, 0.98, 0.95, 0.9):
            u = oracle.threshold_for_cosine(c, sigma, k)
            if u < k * sigma:
                assert oracle.cosine_similarity(u, sigma, k) == pytest.approx(c, abs=1e-12)
            else:
                assert oracle.cosine_similarity(u, sigma, k) >= c
    assert oracle.threshold_for_cosine(0.0, 2.0, 3.0) == pytest.approx(6.0)   # no floor: up to the cut


def test_allocation_by_hand():
    """Two deep layers with floors, two shallow layers that compensate."""
    n = [1_000, 3_000, 16_000, 80_000]
    sigma = [3.0, 3.0, 2.0, 2.0]
    l = [0.0, 0.5, 0.4, 0.3]
    k = [3.0, 3.0, 3.0, 3.0]
    S = 0.9
    # layer 0: a floor so low that S already satisfies it -> keeps S
    u0 = math.log(oracle.threshold(0.0, 3.0, 0.0, S))
    c0 = oracle.cosine_similarity(u0, 3.0, 3.0)
    # layer 1: a floor above its cosine at S -> lowered to the threshold that reaches the floor
    u1 = math.log(oracle.threshold(0.0, 3.0, 0.5, S))
    c1 = oracle.cosine_similarity(u1, 3.0, 3.0)
    floor1 = c1 + 0.5 * (1.0 - c1)
    out, mean = oracle.allocate_sparsity(n, sigma, l, k, [c0 - 0.01, floor1], S, 0.98)
    assert out[0] == S
    u1p = oracle.threshold_for_cosine(floor1, 3.0, 3.0)
    want1 = 0.5 + 0.5 * oracle.sparsity_of(u1p, 3.0)
    assert out[1] == pytest.approx(want1, rel=1e-12) and out[1] < S
    rest = (S * sum(n) - n[0] * out[0] - n[1] * out[1]) / (n[2] + n[3])
    assert out[2] == out[3] == pytest.approx(rest, rel=1e-12) and rest > S
    assert mean == pytest.approx(S, rel=1e-12)                              # the budget is kept
    assert sum(a * b for a, b in zip(n, out)) / sum(n) == pytest.approx(S, rel=1e-12)


def test_allocation_cap_and_degenerate_cases():
    n = [50_000, 50_000, 10_000]
    out, mean = oracle.allocate_sparsity(n, [3.0, 3.0, 2.0], [0.0, 0.0, 0.0], [3.0] * 3, [0.9999, 0.9999], 0.9, 0.97)
    assert out[2] == 0.97 and mean < 0.9                                    # the cap binds: budget missed, as the appendix warns
    assert out[0] < 0.9 and out[1] < 0.9
    # no floors at all: the homogeneous scheme
    out, mean = oracle.allocate_sparsity(n, [3.0, 3.0, 2.0], [0.1, 0.2, 0.3], [3.0] * 3, [], 0.8, 0.98)
    assert out == [0.8, 0.8, 0.8] and mean == pytest.approx(0.8)
    # a deep layer already sparser than S keeps S (nothing to prune there, nothing to lower)
    out, _ = oracle.allocate_sparsity([10, 10], [2.0, 2.0], [0.95, 0.0], [3.0, 3.0], [0.99], 0.9, 0.98)
    assert out[0] == 0.9


def test_quantile_k():
    x = np.array([0.0, 1.0, -2.0, 4.0, 0.0, 8.0, -16.0], dtype=np.float32)     # nonzeros: 1 2 4 8 16
    k, v = oracle.quantile_k(x, 0.6, mu=math.log(4.0), sigma=math.log(2.0))    # r = ceil(0.6*5) = 3 -> 4
    assert v == 4.0 and k == pytest.approx(0.0, abs=1e-15)
    k, v = oracle.quantile_k(x, 1.0, mu=math.log(4.0), sigma=math.log(2.0))
    assert v == 16.0 and k == pytest.approx(2.0, rel=1e-15)
    k, v = oracle.quantile_k(x, 0.0, mu=0.0, sigma=1.0)
    assert v == 1.0
    # on a large lognormal sample the 0.997 quantile sits near 2.75 sigma
    rs = np.random.RandomState(0)
    g = np.exp(-12.0 + 2.0 * rs.standard_normal(1_000_000)).astype(np.float32)
    st = oracle.stats(g)
    k, _ = oracle.quantile_k(g, 0.997, st["mu"], st["sigma"])
    assert abs(k - 2.748) < 0.03
    assert oracle.quantile_k(np.zeros(5, dtype=np.float32), 0.5, 0.0, 1.0) == (0.0, 0.0)
