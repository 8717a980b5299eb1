"""Pins for the oracle's bi-modal statistics (appendix "Algorithm for bi-modal lognormal
pruning", steps 1-4) and for the scale taken from the tensor's maximum (Algorithm 1)."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2006_08173_b200 import synth


def bits(t):
    return synth.as_numpy_bits(t).reshape(-1)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_masked_stats_by_hand(dtype):
    """Right mode = entries 0, 2, 3, 4; entry 4 is exactly zero and has no logarithm.
    log2 of the rest: 1, 3, 4 -> mean 8/3, variance 14/9 (population)."""
    g = bits(torch.tensor([2.0, 4.0, -8.0, 16.0, 0.0, 32.0], dtype=dtype))
    st = oracle.stats_masked(g, np.array([1, 0, 1, 7, 255, 0], dtype=np.uint8))
    assert (st["n"], st["nnz"], st["n_right"]) == (6, 3, 4)
    assert st["zero_frac"] == pytest.approx(1.0 - 4.0 / 6.0, rel=1e-15)
    assert st["mu"] == pytest.approx(math.log(2) * 8.0 / 3.0, rel=1e-14)
    assert st["sigma"] == pytest.approx(math.log(2) * math.sqrt(14.0 / 9.0), rel=1e-14)
    # an empty right mode: nothing to measure, everything is left mode
    st = oracle.stats_masked(g, np.zeros(6, dtype=np.uint8))
    assert (st["nnz"], st["n_right"], st["mu"], st["sigma"], st["zero_frac"]) == (0, 0, 0.0, 0.0, 1.0)


def test_masked_stats_recover_the_right_mode():
    n, l = 2_000_000, 0.55
    g, mask = synth.bimodal_tensor(n, -10.0, 1.5, -18.0, 1.0, l, seed=3)
    st = oracle.stats_masked(bits(g), mask.numpy())
    nr = st["n_right"]
    assert abs(st["zero_frac"] - l) < 4 * math.sqrt(l * (1 - l) / n)
    assert abs(st["mu"] + 10.0) < 4 * 1.5 / math.sqrt(nr)
    assert abs(st["sigma"] - 1.5) < 4 * 1.5 / math.sqrt(2 * nr)
    # the mask matters: over the whole tensor the two modes smear into one wide lump
    whole = oracle.stats(bits(g))
    assert whole["sigma"] > 3.0 and whole["mu"] < -13.0


@pytest.mark.parametrize("S", [0.7, 0.8, 0.9, 0.97])
def test_bimodal_procedure_reaches_the_requested_sparsity(S):
    """Steps (1)-(4): threshold from the right mode's parameters and S' = (S-l)/(1-l),
    applied to the whole tensor.  With the left mode three orders of magnitude below
    the right one nearly all of it falls under alpha*eps, so the total is S."""
    n, l = 1_000_000, 0.5
    g, mask = synth.bimodal_tensor(n, -9.0, 1.5, -17.0, 1.0, l, seed=11)
    g_np = bits(g)
    st = oracle.stats_masked(g_np, mask.numpy())
    tau = oracle.snap_tau(oracle.threshold(st["mu"], st["sigma"], st["zero_frac"], S), oracle.F32)
    out = oracle.prune(g_np, tau, seed=5)
    achieved = oracle.count_zeros(out) / n
    assert abs(achieved - S) < 4 * math.sqrt(S * (1 - S) / n) + 4e-3
    # and the survivors of the left mode are rare
    left_kept = np.count_nonzero(out[mask.numpy() == 0]) / (n * l)
    assert left_kept < 0.01


def test_bimodal_low_sparsity_falls_short_as_the_paper_reports():
    """Just above l the threshold is low, part of the left mode survives, and the
    achieved sparsity is below the request."""
    n, l, S = 1_000_000, 0.5, 0.55
    g, mask = synth.bimodal_tensor(n, -9.0, 1.5, -13.0, 1.5, l, seed=12)
    g_np = bits(g)
    st = oracle.stats_masked(g_np, mask.numpy())
    tau = oracle.snap_tau(oracle.threshold(st["mu"], st["sigma"], st["zero_frac"], S), oracle.F32)
    achieved = oracle.count_zeros(oracle.prune(g_np, tau, seed=5)) / n
    assert achieved < S - 0.01


def test_scale_from_max_by_hand():
    """e_s = floor(log2 max) - (E_max - 1): the maximum's exponent becomes E_max - 1."""
    assert oracle.scale_exp_from_max(1.0, 4) == 0 - 7
    assert oracle.scale_exp_from_max(1.0 - 2.0 ** -24, 4) == -1 - 7
    assert oracle.scale_exp_from_max(1.5 * 2.0 ** -20, 4) == -20 - 7
    assert oracle.scale_exp_from_max(1.5 * 2.0 ** -20, 5) == -20 - 15
    assert oracle.scale_exp_from_max(2.0 ** -140, 3) == -140 - 3          # an fp32 subnormal maximum
    assert oracle.scale_exp_from_max(1e4, 1) == 13 - 0
    assert oracle.max_abs(np.array([0.5, -3.0, 2.0, 0.0], dtype=np.float32)) == 3.0
    assert oracle.max_abs(np.array([0x3F00, 0xC040, 0x8000], dtype=np.uint16)) == 3.0   # bf16 0.5, -3, -0


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("nbits", [4, 5, 6, 8])
@pytest.mark.parametrize("sigma", [1.0, 2.0, 4.0])
def test_the_largest_element_stays_representable(dtype, nbits, sigma):
    g = bits(synth.lognormal_tensor(50_000, -12.0, sigma, 0.4, seed=nbits, dtype=dtype))
    st = oracle.stats(g)
    mx = oracle.max_abs(g)
    f = oracle.fp_format_max_scale(st["mu"], st["sigma"], st["nnz"], nbits, mx)
    Emax = 2 ** (f["exp_bits"] - 1)
    m, ex = math.frexp(mx / 2.0 ** f["scale_exp"])
    assert ex - 1 == Emax - 1                                   # top binade, by construction of the scale
    # no element is clipped before rounding; the maximum decodes within one mantissa step
    x = (g.astype(np.float64) if g.dtype == np.float32
         else (g.astype(np.uint32) << 16).view(np.float32).astype(np.float64))
    assert np.all(np.abs(x) / 2.0 ** f["scale_exp"] < 2.0 ** Emax)
    code = oracle.quantize_one(mx, f["exp_bits"], f["man_bits"], f["scale_exp"], oracle.ROUND_NEAREST)
    back = oracle.decode(code, f["exp_bits"], f["man_bits"], f["scale_exp"])
    assert abs(back - mx) <= mx * 2.0 ** -f["man_bits"]
    # the centred scale of the same split clips where this one does not (wide tensors, narrow formats)
    c = oracle.fp_format(st["mu"], st["sigma"], st["nnz"], nbits)
    clipped_centred = np.count_nonzero(np.abs(x) / 2.0 ** c["scale_exp"] >= 2.0 ** Emax)
    if sigma >= 4.0 and nbits <= 5:
        assert clipped_centred > 0
