"""Pins for the oracle's FP-format closed form (Eq. 4, Table 2) and its FP
quantiser (Eq. 1-2, Algorithm 1)."""
import math
from fractions import Fraction

import numpy as np
import pytest
import torch

from conftest import golden_lines
from paper_2006_08173_b200 import synth

FORMATS = [(N, n2) for N in range(4, 9) for n2 in range(1, N)]
RTN, SR = 0, 1


def fmt_str(f):
    return "1-%d-%d" % (f["exp_bits"], f["man_bits"])


# ------------------------------------------------------------------ Eq. 4 / Table 2
def test_table2_formats(oracle):
    rows = {r[0]: r for r in golden_lines("table2_fp_formats.txt")}
    # ImageNet row (sigma 3 - 5.5): every cell at the midpoint of the range.
    r = rows["imagenet"]
    mid = 0.5 * (float(r[1]) + float(r[2]))
    for k, N in enumerate(range(4, 9)):
        assert fmt_str(oracle.fp_format(-12.0, mid, 1000, N)) == r[3 + k]
    # Cifar100 row (sigma 2.5 - 4.5): FP4, FP5, FP6, FP8 at the midpoint; the FP7
    # cell (1-4-2) is the minimiser in the lower part of the range only.
    r = rows["cifar100"]
    lo, hi = float(r[1]), float(r[2])
    mid = 0.5 * (lo + hi)
    for k, N in enumerate(range(4, 9)):
        sigma = lo + 0.25 if N == 7 else mid
        assert lo <= sigma <= hi
        assert fmt_str(oracle.fp_format(-12.0, sigma, 1000, N)) == r[3 + k]
    # and over each whole range the cell is among the minimisers found
    for name in ("cifar100", "imagenet"):
        r = rows[name]
        for k, N in enumerate(range(4, 9)):
            found = {fmt_str(oracle.fp_format(0.0, s, 10, N))
                     for s in np.linspace(float(r[1]), float(r[2]), 41)}
            assert r[3 + k] in found


def test_eq4_in_range_limit_uses_printed_constants(oracle):
    """Range much wider than the data: only the mantissa term is left,
    E|eps| * E[1/m] = (Delta/4) * 0.721 with Delta = 2^-n1."""
    c = {r[0]: float(r[1]) for r in golden_lines("eq4_constants.txt")}
    for n1 in range(0, 4):
        eta = oracle.expected_rel_err(0.5, n1, 6)
        assert eta == pytest.approx(c["E_abs_eps_over_delta"] * 2.0 ** -n1 * c["E_inv_mantissa"], rel=1e-3)
        assert eta == pytest.approx(2.0 ** -n1 / (8 * math.log(2)), rel=1e-12)
    # E[1/m] for m = 2^U, U ~ U[0,1], by quadrature
    from scipy import integrate
    val, _ = integrate.quad(lambda t: 2.0 ** -t, 0, 1)
    assert val == pytest.approx(1 / (2 * math.log(2)), rel=1e-12)
    assert val == pytest.approx(c["E_inv_mantissa"], abs=5e-4)


def test_eq4_out_of_range_limit(oracle):
    """Data much wider than the range: half the mass underflows (error 1),
    half is clipped (error -> 1), so the expected relative error -> 1."""
    assert oracle.expected_rel_err(25.0, 2, 1) == pytest.approx(1.0, abs=0.08)
    # and the three terms are each probabilities/expectations in [0, 1]
    for sigma in (0.5, 1, 2, 3, 5, 8):
        for N, n2 in FORMATS:
            e = oracle.expected_rel_err(sigma, N - 1 - n2, n2)
            assert 0.0 < e < 1.0


def test_eq4_by_quadrature_of_its_three_cases(oracle):
    """The three cases of the derivation integrated numerically over the
    base-2 exponent E ~ N(0, s^2), s = sigma/ln 2."""
    from scipy import integrate, stats as sps
    for sigma, n1, n2 in [(2.0, 1, 4), (3.0, 0, 5), (1.0, 2, 3), (5.0, 2, 5), (4.0, 0, 3)]:
        s = sigma / math.log(2)
        Emax = 2.0 ** (n2 - 1)
        pdf = lambda e: sps.norm.pdf(e, scale=s)
        in_range = sps.norm.cdf(Emax / s) - sps.norm.cdf(-Emax / s)
        mant = in_range * (2.0 ** -n1 / 4) / (2 * math.log(2))
        clip, _ = integrate.quad(lambda e: (1 - 2.0 ** (Emax - e)) * pdf(e), Emax, Emax + 40 * s,
                                 epsabs=1e-14, epsrel=1e-12, limit=400)
        under = sps.norm.cdf(-Emax / s)
        assert oracle.expected_rel_err(sigma, n1, n2) == pytest.approx(mant + clip + under, rel=1e-8)


def test_eq4_tracks_simulation(oracle):
    """Quantise lognormal samples (sigma = 1, 3, 5; FP8; every n2) with the
    oracle's own quantiser and compare the mean relative error with Eq. 4.

    Eq. 4 models the representable exponents as -E_max..E_max (2 E_max + 1
    binades); a real n2-bit exponent field that also has to encode zero holds
    2 E_max - 1 of them (-E_max+1..E_max-1).  So the two agree closely where
    the range is not what limits the error, the simulation is the larger of
    the two where it is, and its minimiser needs at most one more exponent bit."""
    rs = np.random.RandomState(1)
    n = 200_000
    for sigma in (1.0, 3.0, 5.0):
        s = sigma / math.log(2)
        x = np.exp(sigma * rs.standard_normal(n)).astype(np.float32)
        sim, ana = [], []
        for n2 in range(1, 8):
            n1 = 7 - n2
            codes = oracle.quantize_with_bits(x, n2, n1, 0, RTN)
            xq = np.array([oracle.decode(c, n2, n1, 0) for c in range(256)])[codes]
            sim.append(np.mean(np.abs(xq - x) / x))
            ana.append(oracle.expected_rel_err(sigma, n1, n2))
            if 2 ** (n2 - 1) - 1 >= 4.5 * s:                 # range wider than +-4.5 std
                assert sim[-1] == pytest.approx(ana[-1], rel=0.08)   # uniform-noise model, coarsest at n1 = 0
            else:
                assert sim[-1] > 0.97 * ana[-1]
        assert int(np.argmin(sim)) - int(np.argmin(ana)) in (0, 1)


def test_format_scale_and_degenerate(oracle):
    ln2 = math.log(2)
    for k in (-20, -17, 0, 3):
        assert oracle.fp_format(k * ln2, 2.0, 5, 6)["scale_exp"] == k
        assert oracle.fp_format((k + 0.49) * ln2, 2.0, 5, 6)["scale_exp"] == k
        assert oracle.fp_format((k + 0.51) * ln2, 2.0, 5, 6)["scale_exp"] == k + 1
    assert oracle.fp_format(-12.0, 2.0, 0, 6) == {"nbits": 6, "exp_bits": 1, "man_bits": 4, "scale_exp": 0}
    for bad in (3, 9):
        with pytest.raises(ValueError):
            oracle.fp_format(-12.0, 2.0, 10, bad)
    f = oracle.fp_format(-12.0, 2.0, 10, 6)
    assert 1 + f["exp_bits"] + f["man_bits"] == 6


# ------------------------------------------------------------------ quantiser: brute force
@pytest.mark.parametrize("N,n2", FORMATS)
def test_every_code_of_every_format(oracle, N, n2):
    n1 = N - 1 - n2
    Emax = 2 ** (n2 - 1)
    e_s = -3
    vals = [oracle.decode(c, n2, n1, e_s) for c in range(2 ** N)]
    half = 2 ** (N - 1)
    pos = vals[:half]
    assert all(v == 0.0 for v in pos[: 2 ** n1])                       # exponent field 0 is zero
    grid = pos[2 ** n1:]
    assert all(b > a for a, b in zip(grid, grid[1:]))                  # code order = value order
    assert grid[0] == 2.0 ** (1 - Emax + e_s)                          # smallest normal
    assert grid[-1] == (2 - 2.0 ** -n1) * 2.0 ** (Emax - 1 + e_s)      # largest code
    assert len(grid) == (2 ** n2 - 1) * 2 ** n1
    assert vals[half + 2 ** n1:] == [-v for v in grid]
    # idempotent under both roundings, any random bits
    for c in range(2 ** n1, half):
        for rnd, h in ((RTN, 0), (SR, 0), (SR, 0xFFFF)):
            assert oracle.quantize_one(vals[c], n2, n1, e_s, rnd, h) == c
            assert oracle.quantize_one(-vals[c], n2, n1, e_s, rnd, h) == c + half
    assert oracle.quantize_one(0.0, n2, n1, e_s, RTN) == 0
    assert oracle.quantize_one(-0.0, n2, n1, e_s, SR, 123) == 0
    # midpoints between neighbours: below -> lower, above -> upper, tie -> even mantissa
    for c in range(2 ** n1, half - 1):
        a, b = vals[c], vals[c + 1]
        mid = np.float32((a + b) / 2)
        assert float(mid) == (a + b) / 2
        assert oracle.quantize_one(float(np.nextafter(mid, np.float32(0))), n2, n1, e_s, RTN) == c
        assert oracle.quantize_one(float(np.nextafter(mid, np.float32(np.inf))), n2, n1, e_s, RTN) == c + 1
        # tie: the even mantissa integer wins; with no mantissa bits the only integer is 0 (down)
        assert oracle.quantize_one(float(mid), n2, n1, e_s, RTN) == (c if (n1 == 0 or c % 2 == 0) else c + 1)
    # clipping: everything from half a step above the largest code upward -> largest code
    top = half - 1
    for x in (grid[-1] * (1 + 2.0 ** -(n1 + 1)), grid[-1] * 2, grid[-1] * 1e6, 2.0 ** (Emax + e_s)):
        for rnd, h in ((RTN, 0), (SR, 0), (SR, 0xFFFF)):
            assert oracle.quantize_one(float(np.float32(x)), n2, n1, e_s, rnd, h) == top
    # underflow: E <= -Emax means |x| < smallest normal; nearest flushes all of it
    mn = grid[0]
    for x in (mn * (1 - 2.0 ** -24), mn * 0.75, mn * 0.5, mn * 1e-6):
        assert oracle.quantize_one(float(np.float32(x)), n2, n1, e_s, RTN) == 0


@pytest.mark.parametrize("N,n2", FORMATS)
def test_round_to_nearest_is_nearest_grid_point(oracle, N, n2):
    n1 = N - 1 - n2
    Emax = 2 ** (n2 - 1)
    e_s = 2
    half = 2 ** (N - 1)
    grid = np.array([oracle.decode(c, n2, n1, e_s) for c in range(2 ** n1, half)])
    rs = np.random.RandomState(N * 10 + n2)
    x = (2.0 ** rs.uniform(1 - Emax + e_s, Emax + e_s + 0.5, 4000)).astype(np.float32)
    x = x[x >= grid[0]]
    codes = oracle.quantize_with_bits(x, n2, n1, e_s, RTN)
    got = np.array([oracle.decode(int(c), n2, n1, e_s) for c in codes])
    dist = np.abs(grid[None, :] - x.astype(np.float64)[:, None])
    best = dist.min(axis=1)
    assert np.array_equal(np.abs(got - x), best)          # exact: fp64 holds all of these


def test_stochastic_rounding_probabilities_are_exact(oracle):
    """All 2^16 values of an element's random bits for one x: the count that
    rounds up is the dropped fraction, cut to 16 bits."""
    for (n2, n1, f) in [(4, 1, 0x2ABCDE), (5, 0, 0x000001), (5, 0, 0x000100), (3, 4, 0x7FFFFF), (2, 3, 0x400000),
                        (4, 1, 0x3FFFFF), (4, 1, 0x400000)]:
        d = 23 - n1
        bits = np.uint32(0x3F800000 | f)                  # x in [1,2), E = 0
        x = np.full(2 ** 16, bits, dtype=np.uint32).view(np.float32)
        h = np.arange(2 ** 16, dtype=np.uint16)
        codes = oracle.quantize_with_bits(x, n2, n1, 0, SR, h)
        lo_code = oracle.quantize_one(float(x[0]), n2, n1, 0, SR, 0)
        ups = int(np.sum(codes != lo_code))
        frac = Fraction(f % (2 ** d), 2 ** d)             # position between the two neighbours
        assert ups == int(frac * 2 ** 16)                 # floor(frac * 2^16)
        assert np.all(np.diff((codes != lo_code).astype(int)) >= 0)      # up exactly for the largest h
        if ups:
            (hi_code,) = set(np.unique(codes)) - {lo_code}
            step = oracle.decode(hi_code, n2, n1, 0) - oracle.decode(lo_code, n2, n1, 0)
            assert step == 2.0 ** -n1


def test_underflow_flushes_under_both_roundings(oracle):
    """Eq. 2 as printed: E <= -E_max gives 0, whatever the rounding mode and the
    random bits; the smallest normal itself is kept."""
    for n2, n1, e_s in [(4, 1, 0), (5, 0, -17), (3, 2, -140), (2, 3, 5)]:
        Emax = 2 ** (n2 - 1)
        mn = 2.0 ** (1 - Emax + e_s)
        one = 1 << n1
        for frac in (0.999999, 0.75, 0.5, 2.0 ** -10):
            x = float(np.float32(mn * frac))
            if x == 0.0 or x >= mn:
                continue
            for h in (0, 1, 0x8000, 0xFFFF):
                assert oracle.quantize_one(x, n2, n1, e_s, SR, h) == 0
                assert oracle.quantize_one(-x, n2, n1, e_s, SR, h) == 0
            assert oracle.quantize_one(x, n2, n1, e_s, RTN, 0) == 0
        for h in (0, 0xFFFF):
            assert oracle.quantize_one(mn, n2, n1, e_s, SR, h) == one


def test_stochastic_rounding_is_unbiased(oracle):
    rs = np.random.RandomState(3)
    n = 400_000
    n2, n1, e_s = 4, 1, -17
    x = (2.0 ** rs.uniform(-7 + e_s, 6 + e_s, n)).astype(np.float32)       # inside the range: E in [-7, 6]
    codes = oracle.quantize(x, n2, n1, e_s, SR, seed=5)
    dec = np.array([oracle.decode(c, n2, n1, e_s) for c in range(64)])[codes]
    binade = 2.0 ** np.floor(np.log2(x.astype(np.float64)))
    step = np.maximum(binade * 2.0 ** -n1, 0)          # in range: one mantissa step
    rel = (dec - x) / step                              # each term has variance <= 1/4
    assert abs(rel.mean()) < 4 * 0.5 / math.sqrt(n)


def test_quantize_subnormal_input_and_bf16(oracle):
    # fp32 subnormals, scaled into range by a very negative layer scale
    n2, n1 = 5, 0
    x = np.array([2.0 ** -140, 1.75 * 2.0 ** -135, -(2.0 ** -149)], dtype=np.float32)
    codes = oracle.quantize_with_bits(x, n2, n1, -140, RTN)
    assert [oracle.decode(int(c), n2, n1, -140) for c in codes] == [2.0 ** -140, 2.0 ** -134, -(2.0 ** -149)]
    # bf16 tensors quantise exactly like the fp32 tensors holding the same values
    t = synth.lognormal_tensor(20_000, -12.0, 2.0, 0.5, seed=7, dtype=torch.bfloat16)
    a = oracle.quantize(synth.as_numpy_bits(t), 4, 1, -17, SR, seed=2)
    b = oracle.quantize(synth.as_numpy_bits(t.to(torch.float32)), 4, 1, -17, SR, seed=2)
    assert np.array_equal(a, b)
    assert np.all(a[(t == 0).numpy()] == 0)


@pytest.mark.parametrize("nbits", [4, 5, 6, 7, 8])
@pytest.mark.parametrize("n", [0, 1, 3, 5, 16, 31, 1001])
def test_pack_is_a_little_endian_bit_stream(oracle, nbits, n):
    rs = np.random.RandomState(n + nbits)
    codes = rs.randint(0, 2 ** nbits, n).astype(np.uint8)
    packed = oracle.pack(codes, nbits)
    want_bytes = (n * nbits + 7) // 8
    assert packed.size == (want_bytes + 3) // 4 * 4 == oracle.packed_bytes(n, nbits)
    big = 0
    for i, c in enumerate(codes):
        big |= int(c) << (i * nbits)
    assert int.from_bytes(packed.tobytes(), "little") == big          # pad bits are zero
    assert np.array_equal(oracle.unpack(packed, n, nbits), codes)
