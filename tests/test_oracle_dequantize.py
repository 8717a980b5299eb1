"""Pins for the oracle's decoder of packed code streams (Algorithm 1: X_Q = 2^e_s Q_FP)."""
import numpy as np
import pytest

import oracle

FORMATS = [(nb, n2, nb - 1 - n2) for nb in range(4, 9) for n2 in range(1, nb)]


@pytest.mark.parametrize("nbits,n2,n1", FORMATS)
def test_every_code_against_the_value_formula(nbits, n2, n1):
    """Eq. 1-2: sign, exponent field f (0 = zero), mantissa m -> (-1)^s (1 + m 2^-n1) 2^(f - E_max + e_s)."""
    e_s = -9
    fmt = {"nbits": nbits, "exp_bits": n2, "man_bits": n1, "scale_exp": e_s}
    codes = np.arange(1 << nbits, dtype=np.uint8)
    packed = oracle.pack(codes, nbits)
    for odt, npdt in ((oracle.F32, np.float32), (oracle.BF16, np.uint16)):
        got = oracle.dequantize(packed, codes.size, fmt, odt)
        for c in range(1 << nbits):
            s, f, m = c >> (nbits - 1), (c >> n1) & ((1 << n2) - 1), c & ((1 << n1) - 1)
            want = 0.0 if f == 0 else (-1.0) ** s * (1.0 + m / 2.0 ** n1) * 2.0 ** (f - 2 ** (n2 - 1) + e_s)
            if odt == oracle.F32:
                assert float(got[c]) == want and (want != 0.0 or got.view(np.uint32)[c] == 0)
            else:
                bits = np.array([want], dtype=np.float32).view(np.uint32)[0]
                assert bits & 0xFFFF == 0                           # exact in bf16
                assert int(got[c]) == int(bits >> 16)


@pytest.mark.parametrize("nbits,n2,n1", [(6, 4, 1), (5, 3, 1), (8, 5, 2), (4, 2, 1)])
def test_nearest_quantisation_of_a_decoded_value_is_the_code(nbits, n2, n1):
    e_s = 3
    fmt = {"nbits": nbits, "exp_bits": n2, "man_bits": n1, "scale_exp": e_s}
    codes = np.arange(1 << nbits, dtype=np.uint8)
    vals = oracle.dequantize(oracle.pack(codes, nbits), codes.size, fmt, oracle.F32)
    for c in range(1 << nbits):
        f = (c >> n1) & ((1 << n2) - 1)
        back = oracle.quantize_one(float(vals[c]), n2, n1, e_s, 0)
        assert back == (c if f != 0 else 0)                        # every zero-field code means 0


def test_stream_positions():
    """Code i occupies bits [6i, 6i+6): a tensor of distinct codes comes back in order."""
    fmt = {"nbits": 6, "exp_bits": 4, "man_bits": 1, "scale_exp": 0}
    rs = np.random.RandomState(0)
    codes = rs.randint(0, 64, size=1000).astype(np.uint8)
    vals = oracle.dequantize(oracle.pack(codes, 6), 1000, fmt, oracle.F32)
    want = np.array([oracle.decode(int(c), 4, 1, 0) for c in codes], dtype=np.float32)
    assert np.array_equal(vals, want)
