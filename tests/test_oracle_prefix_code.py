"""Pins for the oracle's prefix code (appendix "Encoding"): the paper's code
table on a hand-written example, losslessness, the length identity, and the
compression the appendix states for synthetic lognormal data."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2006_08173_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "prefix_code_table.txt")


def table():
    words, claims = {}, []
    for line in open(GOLDEN):
        f = line.split()
        if not f or f[0].startswith("#"):
            continue
        if f[0] == "claim":
            claims.append((float(f[1]), float(f[2])))
        else:
            words[f[0]] = f[1]
    return words, claims


def stream_bits(stream, nbits):
    return "".join(str((int(stream[k >> 5]) >> (k & 31)) & 1) for k in range(nbits))


def lsb_first(pattern, width):
    return "".join(str((pattern >> k) & 1) for k in range(width))


def test_code_table_on_a_worked_example_fp32():
    w, _ = table()
    alpha = 0.25
    v = np.array([0.0, alpha, -alpha, 1.5, 0.0, -3.0], dtype=np.float32)
    pat = v.view(np.uint32)
    want = (w["zero"] + w["plus_alpha"] + w["minus_alpha"] + w["fp_value"] + lsb_first(int(pat[3]), 32)
            + w["zero"] + w["fp_value"] + lsb_first(int(pat[5]), 32))
    stream, off = oracle.prefix_encode(v, alpha)
    assert list(off) == [0, (len(want) + 31) // 32]
    got = stream_bits(stream, 32 * len(stream))
    assert got[:len(want)] == want
    assert set(got[len(want):]) <= {"0"}                      # padding to a whole word


def test_code_table_on_a_worked_example_bf16():
    w, _ = table()
    alpha_bits = 0x3E80                                        # 0.25
    v = np.array([alpha_bits | 0x8000, 0, 0x3FC0, alpha_bits], dtype=np.uint16)
    want = w["minus_alpha"] + w["zero"] + w["fp_value"] + lsb_first(0x3FC0, 16) + w["plus_alpha"]
    stream, off = oracle.prefix_encode(v, 0.25)
    assert stream_bits(stream, len(want)) == want
    assert int(off[-1]) == (len(want) + 31) // 32


def test_classes():
    assert oracle.prefix_class(0, oracle.F32, 0.5) == 0
    assert oracle.prefix_class(0x80000000, oracle.F32, 0.5) == 3          # -0 is not the zero code: lossless
    assert oracle.prefix_class(0x3F000000, oracle.F32, 0.5) == 1
    assert oracle.prefix_class(0xBF000000, oracle.F32, 0.5) == 2
    assert oracle.prefix_class(0x3F000001, oracle.F32, 0.5) == 3
    assert oracle.prefix_class(0x3F000000, oracle.F32, 0.0) == 3          # no alpha codes without a threshold
    assert oracle.prefix_class(0x3F00, oracle.BF16, 0.5) == 1
    assert oracle.prefix_class(0xBF00, oracle.BF16, 0.5) == 2
    assert oracle.prefix_class(0x8000, oracle.BF16, 0.5) == 3


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("n", [0, 1, 5, 2047, 2048, 2049, 3 * 2048 + 77])
def test_round_trip_and_length(dtype, n):
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    g = synth.as_numpy_bits(synth.lognormal_tensor(n, -9.0, 2.0, 0.4, seed=n + 3, dtype=tdt, device="cpu"))
    tau = oracle.snap_tau(2e-4, oracle.F32 if dtype == "f32" else oracle.BF16)
    v = oracle.prune(g, tau, seed=11)
    if n >= 5:
        v = v.copy()
        v.view(np.uint32 if dtype == "f32" else np.uint16)[2] = 0x80000000 if dtype == "f32" else 0x8000   # a -0
    stream, off = oracle.prefix_encode(v, tau)
    dt = oracle.F32 if dtype == "f32" else oracle.BF16
    back = oracle.prefix_decode(stream, off, n, dt, tau)
    raw = np.uint32 if dtype == "f32" else np.uint16
    assert np.array_equal(back.view(raw), v.view(raw))
    # length: per block ceil((n0 + 3 n_alpha + (2 + width) n_fp) / 32) words
    width = 32 if dtype == "f32" else 16
    pats = v.view(raw).astype(np.uint64)
    sign = 0x80000000 if dtype == "f32" else 0x8000
    tp = int(np.array([tau], dtype=np.float32).view(np.uint32)[0]) >> (0 if dtype == "f32" else 16)
    zero = pats == 0
    alpha = ((pats & (sign - 1)) == tp) & ~zero
    bits = np.where(zero, 1, np.where(alpha, 3, 2 + width))
    words = 0
    for b in range(oracle.prefix_blocks(n)):
        assert int(off[b]) == words
        words += (int(bits[b * 2048:(b + 1) * 2048].sum()) + 31) // 32
    assert int(off[-1]) == words == len(stream)
    assert len(stream) <= oracle.prefix_bound_words(n, dt)


def test_no_threshold_is_still_lossless():
    g = synth.as_numpy_bits(synth.lognormal_tensor(5000, -3.0, 1.0, 0.2, seed=5, dtype=torch.float32, device="cpu"))
    stream, off = oracle.prefix_encode(g, 0.0)
    assert np.array_equal(oracle.prefix_decode(stream, off, g.size, oracle.F32, 0.0).view(np.uint32), g.view(np.uint32))


def test_compression_stated_in_the_appendix():
    """Synthetic lognormal tensor, sigma = 2 (the middle of the range the paper
    reports for neural gradients), FP32 values: the appendix puts the code at
    about 4 bits per value at 80 % sparsity and 2 bits at 90 %."""
    _, claims = table()
    n = 1 << 20
    g = synth.as_numpy_bits(synth.lognormal_tensor(n, -10.0, 2.0, 0.0, seed=1, dtype=torch.float32, device="cpu"))
    st = oracle.stats(g)
    for S, bits_claimed in claims:
        tau = oracle.snap_tau(oracle.threshold(st["mu"], st["sigma"], st["zero_frac"], S), oracle.F32)
        v = oracle.prune(g, tau, seed=3)
        stream, _ = oracle.prefix_encode(v, tau)
        bits = 32.0 * len(stream) / n
        assert abs(bits - bits_claimed) < 0.15 * bits_claimed + 0.1, (S, bits)
