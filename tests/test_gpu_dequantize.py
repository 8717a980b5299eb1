"""GPU parity of lgn_dequantize (Algorithm 1, X_Q = 2^e_s Q_FP) against the oracle's
decoder: every output element bit for bit, both output types."""
import numpy as np
import pytest
import torch

from gpu_helpers import assert_same_bits, np_bits
from paper_2006_08173_b200 import synth

pytestmark = pytest.mark.gpu

OUT_DTYPES = [torch.float32, torch.bfloat16]
FORMATS = [(nb, n2, nb - 1 - n2) for nb in range(4, 9) for n2 in range(1, nb)]


def run(lgn, packed_np, n, fmt, odt):
    codes = torch.from_numpy(packed_np.copy()).cuda() if packed_np.size else torch.zeros(16, dtype=torch.uint8, device="cuda")
    out = torch.full((n,), float("nan"), dtype=odt, device="cuda")
    lgn.lgn_dequantize(codes, n, fmt, out)
    torch.cuda.synchronize()
    return out


@pytest.mark.parametrize("odt", OUT_DTYPES)
@pytest.mark.parametrize("nbits,n2,n1", FORMATS)
def test_random_codes_of_every_format(lgn, oracle, odt, nbits, n2, n1):
    """Uniformly random codes (zero-field codes with sign and mantissa bits included),
    a size that spans tiles and leaves a ragged tail."""
    n = 3 * 8192 + 1234 + nbits
    fmt = {"nbits": nbits, "exp_bits": n2, "man_bits": n1, "scale_exp": -17}
    codes = np.random.RandomState(100 * nbits + n2).randint(0, 1 << nbits, size=n).astype(np.uint8)
    packed = oracle.pack(codes, nbits)
    want = oracle.dequantize(packed, n, fmt, oracle.BF16 if odt == torch.bfloat16 else oracle.F32)
    assert_same_bits(run(lgn, packed, n, fmt, odt), want)


@pytest.mark.parametrize("odt", OUT_DTYPES)
@pytest.mark.parametrize("n", [0, 1, 3, 7, 8, 9, 1023, 8191, 8192, 8193, 2 ** 20 + 7])
def test_sizes(lgn, oracle, odt, n):
    for nbits, n2 in [(6, 4), (5, 3)]:
        fmt = {"nbits": nbits, "exp_bits": n2, "man_bits": nbits - 1 - n2, "scale_exp": 3}
        codes = np.random.RandomState(n % 1000 + nbits).randint(0, 1 << nbits, size=n).astype(np.uint8)
        packed = oracle.pack(codes, nbits)
        want = oracle.dequantize(packed, n, fmt, oracle.BF16 if odt == torch.bfloat16 else oracle.F32)
        got = run(lgn, packed, n, fmt, odt)
        if n:
            assert_same_bits(got, want)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("nbits,rounding", [(6, 1), (5, 0), (8, 1), (4, 0)])
def test_round_trip_through_the_library(lgn, oracle, dtype, nbits, rounding):
    """lgn_quantize -> lgn_dequantize equals oracle quantise -> oracle decode, and every
    in-range element comes back within one mantissa step of its value."""
    n = 200_003
    g = synth.lognormal_tensor(n, -12.0, 2.0, 0.4, 11, dtype=dtype, device="cuda")
    g_np = np_bits(g)
    st = oracle.stats(g_np)
    fmt = oracle.fp_format(st["mu"], st["sigma"], st["nnz"], nbits)
    codes = lgn.lgn_quantize(g, fmt, rounding, 5)
    for odt in OUT_DTYPES:
        out = torch.empty(n, dtype=odt, device="cuda")
        lgn.lgn_dequantize(codes, n, fmt, out)
        ref_codes = oracle.quantize(g_np, fmt["exp_bits"], fmt["man_bits"], fmt["scale_exp"], rounding, 5)
        want = oracle.dequantize(oracle.pack(ref_codes, nbits), n, fmt, oracle.BF16 if odt == torch.bfloat16 else oracle.F32)
        assert_same_bits(out, want)
    x = g.float().cpu().numpy().astype(np.float64)
    y = out.float().cpu().numpy().astype(np.float64)
    Emax = 2 ** (fmt["exp_bits"] - 1)
    lo, hi = 2.0 ** (1 - Emax + fmt["scale_exp"]), 2.0 ** (Emax + fmt["scale_exp"])
    inr = (np.abs(x) >= lo) & (np.abs(x) < hi / 2)
    assert inr.mean() > 0.3
    step = 2.0 ** (np.floor(np.log2(np.abs(x[inr]))) - fmt["man_bits"])
    assert np.all(np.abs(y[inr] - x[inr]) <= step * (1 + 1e-12))
    assert np.all(np.sign(y[inr]) == np.sign(x[inr]))


def test_after_the_grouped_call(lgn, oracle):
    """Codes written by lgn_compress_layers, decoded with the format it reports."""
    n = 70_001
    g = synth.lognormal_tensor(n, -10.0, 2.5, 0.5, 4, dtype=torch.bfloat16, device="cuda")
    out_q = torch.empty(lgn.lgn_codes_bytes(n, 6) + 16, dtype=torch.uint8, device="cuda")
    res = lgn.new_results(1, g.device)
    ws = lgn.new_workspace([n], g.device)
    lgn.lgn_compress_layers([lgn.make_layer(g, out_q, lgn.MODE_QUANTIZE, nbits=6, rounding=lgn.ROUND_STOCHASTIC, seed=9)], res, ws)
    fmt = lgn.read_results(res, 1)[0]["fmt"]
    out = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    lgn.lgn_dequantize(out_q, n, fmt, out)
    packed = out_q.cpu().numpy()[:lgn.lgn_codes_bytes(n, 6)]
    assert_same_bits(out, oracle.dequantize(packed, n, fmt, oracle.BF16))


def test_canary_and_errors(lgn, oracle):
    n, nbits = 8192 + 5, 6
    fmt = {"nbits": 6, "exp_bits": 4, "man_bits": 1, "scale_exp": 0}
    codes = np.random.RandomState(1).randint(0, 64, size=n).astype(np.uint8)
    packed = torch.from_numpy(oracle.pack(codes, nbits)).cuda()
    buf = torch.full((n + 64,), 7.0, dtype=torch.float32, device="cuda")
    lgn.lgn_dequantize(packed, n, fmt, buf[:n])
    torch.cuda.synchronize()
    assert bool((buf[n:] == 7.0).all())                        # nothing written past n
    out = torch.empty(n, dtype=torch.float32, device="cuda")
    for bad, code in [({"nbits": 3, "exp_bits": 1, "man_bits": 1, "scale_exp": 0}, 2),
                      ({"nbits": 9, "exp_bits": 4, "man_bits": 4, "scale_exp": 0}, 2),
                      ({"nbits": 6, "exp_bits": 3, "man_bits": 1, "scale_exp": 0}, 1),
                      ({"nbits": 6, "exp_bits": 4, "man_bits": 1, "scale_exp": -130}, 2),    # below the normal range
                      ({"nbits": 6, "exp_bits": 4, "man_bits": 1, "scale_exp": 121}, 2)]:    # above it
        with pytest.raises(lgn.LgnError) as e:
            lgn.lgn_dequantize(packed, n, bad, out)
        assert e.value.code == code
    with pytest.raises(lgn.LgnError):                          # misaligned output
        lgn.lgn_dequantize(packed, n - 1, fmt, buf[1:n])
