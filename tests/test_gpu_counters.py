"""The apply pass's counters (n_zero_out, n_snapped, n_saturated, n_underflow of the layer
result) against counts taken from the oracle's own output of the same layer."""
import numpy as np
import pytest
import torch

from gpu_helpers import np_bits
from paper_2006_08173_b200 import synth

pytestmark = pytest.mark.gpu

SIZES = [1, 1023, 32768, 2 ** 20 + 7, 3_000_001]


def magnitudes(a):
    """|x| of float32 values or of bf16 patterns, as float64."""
    if a.dtype == np.uint16:
        return np.abs((a.astype(np.uint32) << 16).view(np.float32).astype(np.float64))
    return np.abs(a.astype(np.float64))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_prune_counters(lgn, oracle, dtype):
    code = oracle.BF16 if dtype == torch.bfloat16 else oracle.F32
    gs = [synth.lognormal_tensor(n, -12.0 + k, 2.0, 0.1 * k, seed=60 + k, dtype=dtype, device="cuda") for k, n in enumerate(SIZES)]
    sts = [oracle.stats(np_bits(g)) for g in gs]
    outs = [torch.empty_like(g) for g in gs]
    S = [0.0, 0.5, 0.8, 0.9, 0.99]
    layers = [lgn.make_layer(g, o, lgn.MODE_PRUNE, S=s, seed=7 + k, mu_override=st["mu"], sigma_override=st["sigma"], counters=True)
              for k, (g, o, s, st) in enumerate(zip(gs, outs, S, sts))]
    ws = lgn.new_workspace(SIZES, "cuda")
    res = lgn.new_results(len(gs), "cuda")
    for _ in range(2):                                     # the second call starts from a used record
        lgn.lgn_compress_layers(layers, res, ws)
        torch.cuda.synchronize()
    for k, (g, o, s, st, r) in enumerate(zip(gs, outs, S, sts, lgn.read_results(res, len(gs)))):
        tau = oracle.snap_tau(oracle.threshold(st["mu"], st["sigma"], st["zero_frac"], s), code) if st["nnz"] else 0.0
        assert r["status"] == 0 and r["tau"] == tau
        gn = np_bits(g)
        ref = oracle.prune(gn, tau, 7 + k)
        assert np.array_equal(np_bits(o).view(np.uint8), ref.view(np.uint8))
        a_in, a_out = magnitudes(gn), magnitudes(ref)
        assert r["n_zero_out"] == int(np.count_nonzero(a_out == 0)), k
        assert r["n_snapped"] == int(np.count_nonzero((a_out != 0) & (a_in <= tau))), k
        assert r["n_saturated"] == 0 and r["n_underflow"] == 0


@pytest.mark.parametrize("rounding", [0, 1])
@pytest.mark.parametrize("nbits", [5, 6, 8])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_quantise_counters(lgn, oracle, dtype, nbits, rounding):
    # sigma up to 4: both ends of the format's range are reached
    gs = [synth.lognormal_tensor(n, -12.0 + k, 1.5 + 0.6 * k, 0.1 * k, seed=80 + k, dtype=dtype, device="cuda") for k, n in enumerate(SIZES)]
    sts = [oracle.stats(np_bits(g)) for g in gs]
    outs = [torch.empty(max(16, lgn.lgn_codes_bytes(g.numel(), nbits)), dtype=torch.uint8, device="cuda") for g in gs]
    layers = [lgn.make_layer(g, o, lgn.MODE_QUANTIZE, nbits=nbits, rounding=rounding, seed=3 + k,
                             mu_override=st["mu"], sigma_override=st["sigma"], counters=(k == 0))   # one layer asking is enough
              for k, (g, o, st) in enumerate(zip(gs, outs, sts))]
    ws = lgn.new_workspace(SIZES, "cuda")
    res = lgn.new_results(len(gs), "cuda")
    lgn.lgn_compress_layers(layers, res, ws)
    torch.cuda.synchronize()
    seen_sat = seen_under = 0
    for k, (g, o, st, r) in enumerate(zip(gs, outs, sts, lgn.read_results(res, len(gs)))):
        fmt = oracle.fp_format(st["mu"], st["sigma"], st["nnz"], nbits)
        assert r["status"] == 0 and r["fmt"] == fmt
        codes = oracle.quantize(np_bits(g), fmt["exp_bits"], fmt["man_bits"], fmt["scale_exp"], rounding, 3 + k)
        ref = oracle.pack(codes, nbits)
        assert np.array_equal(o.cpu().numpy()[:ref.size], ref)
        mag = codes & ((1 << (nbits - 1)) - 1)
        top = (1 << (nbits - 1)) - 1
        zero_codes = int(np.count_nonzero(mag == 0))
        assert r["n_zero_out"] == zero_codes, k
        assert r["n_saturated"] == int(np.count_nonzero(mag == top)), k
        assert r["n_underflow"] == zero_codes - (st["n"] - st["nnz"]), k
        assert r["n_snapped"] == 0
        seen_sat += r["n_saturated"]
        seen_under += r["n_underflow"]
    assert seen_sat > 0 and seen_under > 0                 # the cases do exercise both counters


def test_counters_stay_zero_when_nobody_asks(lgn):
    g = synth.lognormal_tensor(500_000, -12.0, 2.0, 0.4, seed=5, device="cuda")
    o = torch.empty_like(g)
    ws = lgn.new_workspace([g.numel()], "cuda")
    res = lgn.new_results(1, "cuda")
    lgn.lgn_compress_layers([lgn.make_layer(g, o, lgn.MODE_PRUNE, S=0.8, seed=1)], res, ws)
    torch.cuda.synchronize()
    r = lgn.read_results(res, 1)[0]
    assert r["status"] == 0
    assert (r["n_zero_out"], r["n_snapped"], r["n_saturated"], r["n_underflow"]) == (0, 0, 0, 0)


def test_mixed_group_counts_too(lgn, oracle):
    """Layers that differ in type and mode run through the general kernel, which always counts."""
    a = synth.lognormal_tensor(400_003, -11.0, 2.0, 0.3, seed=11, device="cuda")
    b = synth.lognormal_tensor(250_001, -9.0, 3.0, 0.5, seed=12, dtype=torch.bfloat16, device="cuda")
    oa = torch.empty_like(a)
    ob = torch.empty(lgn.lgn_codes_bytes(b.numel(), 6), dtype=torch.uint8, device="cuda")
    sa, sb = oracle.stats(np_bits(a)), oracle.stats(np_bits(b))
    layers = [lgn.make_layer(a, oa, lgn.MODE_PRUNE, S=0.85, seed=1, mu_override=sa["mu"], sigma_override=sa["sigma"]),
              lgn.make_layer(b, ob, lgn.MODE_QUANTIZE, nbits=6, rounding=1, seed=2, mu_override=sb["mu"], sigma_override=sb["sigma"])]
    ws = lgn.new_workspace([a.numel(), b.numel()], "cuda")
    res = lgn.new_results(2, "cuda")
    lgn.lgn_compress_layers(layers, res, ws)
    torch.cuda.synchronize()
    ra, rb = lgn.read_results(res, 2)
    assert ra["n_zero_out"] == int((oa == 0).sum())
    fmt = oracle.fp_format(sb["mu"], sb["sigma"], sb["nnz"], 6)
    codes = oracle.quantize(np_bits(b), fmt["exp_bits"], fmt["man_bits"], fmt["scale_exp"], 1, 2)
    assert rb["n_zero_out"] == int(np.count_nonzero((codes & 31) == 0))
    assert rb["n_saturated"] == int(np.count_nonzero((codes & 31) == 31))
