"""Pins for the oracle's random-bit generator and its lognormal statistics."""
import math

import numpy as np
import pytest
import torch

from conftest import golden_lines
from paper_2006_08173_b200 import synth


# ------------------------------------------------------------------ generator
def test_philox_known_answers(oracle):
    rows = golden_lines("philox4x32_10_kat.txt")
    assert len(rows) == 3
    for r in rows:
        w = [int(x, 16) for x in r]
        out = oracle.philox4x32(w[0:4], w[4:6], 10)
        assert [int(x) for x in out] == w[6:10]


def test_philox_rounds_compose(oracle):
    """The 7-round function the method uses is the same bijection stopped
    earlier: three more rounds, with the key advanced by seven Weyl steps, must
    reproduce the 10-round known answers."""
    W0, W1 = 0x9E3779B9, 0xBB67AE85
    for r in golden_lines("philox4x32_10_kat.txt"):
        w = [int(x, 16) for x in r]
        mid = oracle.philox4x32(w[0:4], w[4:6], 7)
        key7 = [(w[4] + 7 * W0) & 0xFFFFFFFF, (w[5] + 7 * W1) & 0xFFFFFFFF]
        out = oracle.philox4x32([int(x) for x in mid], key7, 3)
        assert [int(x) for x in out] == w[6:10]
    assert oracle.PHILOX_ROUNDS == 7


def test_rand16_is_a_pure_function_of_seed_and_index(oracle):
    seed = 0x1234_5678_9ABC_DEF0
    first = (1 << 35) + 5                      # crosses the 32-bit boundary of the block counter
    a = oracle.rand16_fill(seed, first, 64)
    for j in (0, 1, 2, 3, 10, 11, 17, 63):
        i = first + j
        blk = i >> 3
        ref = oracle.philox4x32([blk & 0xFFFFFFFF, blk >> 32, 0, 0],
                                [seed & 0xFFFFFFFF, seed >> 32], oracle.PHILOX_ROUNDS)
        word = int(ref[(i >> 1) & 3])
        want = (word >> 16) if (i & 1) else (word & 0xFFFF)
        assert int(a[j]) == want == oracle.rand16(seed, i)
    # chunking does not matter
    b = np.concatenate([oracle.rand16_fill(seed, first, 10), oracle.rand16_fill(seed, first + 10, 54)])
    assert np.array_equal(a, b)
    assert not np.array_equal(a, oracle.rand16_fill(seed + 1, first, 64))


def test_rand16_uniformity(oracle):
    n = 1 << 21
    h = oracle.rand16_fill(1, 0, n).astype(np.int64)
    eps = h / 2.0 ** 16
    assert abs(eps.mean() - (0.5 - 2.0 ** -17)) < 4 * math.sqrt(1 / 12 / n)
    assert abs(eps.var() - 1 / 12) < 4 * math.sqrt(1 / 180 / n)
    for field in (h >> 8, h & 0xFF):                          # top and bottom byte
        counts = np.bincount(field, minlength=256)
        chi2 = ((counts - n / 256) ** 2 / (n / 256)).sum()
        assert chi2 < 255 + 5 * math.sqrt(2 * 255)
    for lag in (1, 2, 8):                                     # neighbours, word mates, block mates
        c = np.corrcoef(eps[:-lag], eps[lag:])[0, 1]
        assert abs(c) < 4 / math.sqrt(n)
    # consecutive seeds give unrelated streams
    g = oracle.rand16_fill(2, 0, n).astype(np.float64)
    assert abs(np.corrcoef(eps, g)[0, 1]) < 4 / math.sqrt(n)


# ------------------------------------------------------------------ statistics
def test_stats_powers_of_two(oracle):
    g = np.array([2.0, -4.0, 8.0, 0.0, -0.0], dtype=np.float32)
    st = oracle.stats(g)
    ln2 = math.log(2.0)
    assert st["n"] == 5 and st["nnz"] == 3
    assert st["mu"] == pytest.approx(2 * ln2, rel=1e-15)
    assert st["sigma"] == pytest.approx(ln2 * math.sqrt(2.0 / 3.0), rel=1e-14)   # population std
    assert st["zero_frac"] == pytest.approx(0.4, rel=1e-15)


def test_stats_population_not_sample_std(oracle):
    st = oracle.stats(np.array([1.0, 4.0], dtype=np.float32))
    assert st["mu"] == pytest.approx(math.log(2.0), rel=1e-15)
    assert st["sigma"] == pytest.approx(math.log(2.0), rel=1e-15)


def test_stats_natural_log_of_magnitude_sign_ignored(oracle):
    g = np.array([math.e, -math.e ** 3], dtype=np.float64).astype(np.float32)
    st = oracle.stats(g)
    assert st["mu"] == pytest.approx(2.0, abs=1e-7)       # fp32 rounding of e, e^3
    assert st["sigma"] == pytest.approx(1.0, abs=1e-7)


def test_stats_subnormal_and_extremes(oracle):
    g = np.array([2.0 ** -140, 2.0 ** 100], dtype=np.float32)
    st = oracle.stats(g)
    assert st["mu"] == pytest.approx(-20 * math.log(2.0), rel=1e-14)
    assert st["sigma"] == pytest.approx(120 * math.log(2.0), rel=1e-14)


def test_stats_degenerate(oracle):
    st = oracle.stats(np.zeros(7, dtype=np.float32))
    assert (st["nnz"], st["mu"], st["sigma"], st["zero_frac"]) == (0, 0.0, 0.0, 1.0)
    st = oracle.stats(np.zeros(0, dtype=np.float32))
    assert (st["n"], st["nnz"], st["zero_frac"]) == (0, 0, 0.0)
    st = oracle.stats(np.array([-3.0], dtype=np.float32))
    assert st["mu"] == pytest.approx(math.log(3.0), rel=1e-15) and st["sigma"] == 0.0


def test_stats_bf16_equals_fp32_of_same_values(oracle):
    t = synth.lognormal_tensor(50_000, -12.0, 2.0, 0.4, seed=3, dtype=torch.bfloat16)
    a = oracle.stats(synth.as_numpy_bits(t))
    b = oracle.stats(synth.as_numpy_bits(t.to(torch.float32)))
    assert a == b


@pytest.mark.parametrize("mu,sigma,p", [(-12.0, 2.0, 0.4), (-9.5, 3.0, 0.0), (0.0, 1.0, 0.6)])
def test_stats_recover_generator_parameters(oracle, mu, sigma, p):
    n = 2_000_000
    g = synth.as_numpy_bits(synth.lognormal_tensor(n, mu, sigma, p, seed=11))
    st = oracle.stats(g)
    nnz = st["nnz"]
    assert abs(st["zero_frac"] - p) <= 4 * math.sqrt(max(p * (1 - p), 1e-12) / n)
    assert abs(st["mu"] - mu) <= 4 * sigma / math.sqrt(nnz)
    assert abs(st["sigma"] - sigma) <= 4 * sigma / math.sqrt(2 * nnz)
