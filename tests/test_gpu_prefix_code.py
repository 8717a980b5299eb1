"""Prefix code (appendix "Encoding") on the GPU against the oracle: offsets and
stream words bit for bit, fused with Eq. 5 and on an already pruned tensor, both
types, ragged and empty tensors, a stream that does not fit, and the decoder."""
import ctypes as C

import numpy as np
import pytest
import torch

from gpu_helpers import np_bits
from paper_2006_08173_b200 import synth

pytestmark = pytest.mark.gpu


def encode(lgn, g, tau, seed, apply_prune, capacity=None, tau_from=None):
    n = g.numel()
    cap = lgn.lgn_prefix_bound_words(n, lgn.dtype_code(g)) if capacity is None else capacity
    stream = torch.full((max(cap, 1),), 0x5A5A5A5A, dtype=torch.int32, device="cuda")[:cap]
    off = torch.full((lgn.lgn_prefix_blocks(n) + 1,), -1, dtype=torch.int64, device="cuda")
    ws = torch.empty(lgn.lgn_prefix_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    lgn.lgn_prefix_encode(g, tau, seed, apply_prune, stream, off, ws, tau_from_dev=tau_from)
    torch.cuda.synchronize()
    return stream.cpu().numpy().view(np.uint32), off.cpu().numpy().view(np.uint64)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("n", [0, 1, 7, 2048, 2049, 5 * 2048 + 13, 300_000])
def test_fused_prune_and_encode_matches_oracle(lgn, oracle, dtype, n):
    g = synth.lognormal_tensor(n, -9.0, 2.0, 0.4, seed=n + 1, dtype=dtype, device="cuda")
    odt = oracle.F32 if dtype == torch.float32 else oracle.BF16
    tau = oracle.snap_tau(3e-4, odt)
    want_stream, want_off = oracle.prefix_encode(oracle.prune(np_bits(g), tau, seed=17), tau)
    stream, off = encode(lgn, g, tau, 17, True)
    assert np.array_equal(off, want_off)
    words = int(off[-1])
    assert np.array_equal(stream[:words], want_stream)
    # decoder: back to the pruned tensor
    out = torch.empty_like(g)
    s_dev = torch.from_numpy(stream[:max(words, 1)].view(np.int32).copy()).cuda()[:words]
    lgn.lgn_prefix_decode(s_dev, torch.from_numpy(off.view(np.int64).copy()).cuda(), out, tau)
    torch.cuda.synchronize()
    assert np.array_equal(np_bits(out).view(np.uint8), oracle.prune(np_bits(g), tau, seed=17).view(np.uint8))
    assert np.array_equal(np_bits(lgn.lgn_prune(g, tau, 17)).view(np.uint8), np_bits(out).view(np.uint8))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_encode_of_a_pruned_tensor_and_odd_values(lgn, oracle, dtype):
    n = 40_000
    g = synth.lognormal_tensor(n, -5.0, 1.5, 0.3, seed=9, dtype=dtype, device="cuda")
    odt = oracle.F32 if dtype == torch.float32 else oracle.BF16
    tau = oracle.snap_tau(5e-3, odt)
    v = oracle.prune(np_bits(g), tau, seed=2).copy()
    raw = v.view(np.uint32 if dtype == torch.float32 else np.uint16)
    raw[3] = 0x80000000 if dtype == torch.float32 else 0x8000           # -0: travels as a value
    raw[4] = 0x00000001                                                 # smallest subnormal pattern
    raw[2047] = 0xFF7FFFFF if dtype == torch.float32 else 0xFF7F        # most negative finite
    v_dev = synth.from_numpy_bits(v, "cuda")
    want_stream, want_off = oracle.prefix_encode(v, tau)
    stream, off = encode(lgn, v_dev, tau, 0, False)
    assert np.array_equal(off, want_off) and np.array_equal(stream[:int(off[-1])], want_stream)
    # no threshold: everything nonzero is a value
    want_stream, want_off = oracle.prefix_encode(v, 0.0)
    stream, off = encode(lgn, v_dev, 0.0, 0, False)
    assert np.array_equal(off, want_off) and np.array_equal(stream[:int(off[-1])], want_stream)


def test_stream_that_does_not_fit_is_reported_not_overrun(lgn, oracle):
    n = 50_000
    g = synth.lognormal_tensor(n, -9.0, 2.0, 0.4, seed=4, dtype=torch.float32, device="cuda")
    tau = oracle.snap_tau(3e-4, oracle.F32)
    want_stream, want_off = oracle.prefix_encode(oracle.prune(np_bits(g), tau, seed=1), tau)
    cap = int(want_off[10])                                             # room for ten blocks only
    guard = torch.full((cap + 64,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    off = torch.empty(lgn.lgn_prefix_blocks(n) + 1, dtype=torch.int64, device="cuda")
    ws = torch.empty(lgn.lgn_prefix_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    lgn.lgn_prefix_encode(g, tau, 1, True, guard[:cap], off, ws)
    torch.cuda.synchronize()
    assert int(off[-1]) == int(want_off[-1]) > cap                      # the caller can tell
    got = guard.cpu().numpy().view(np.uint32)
    assert np.array_equal(got[:cap], want_stream[:cap])
    assert (got[cap:] == 0x5A5A5A5A).all()                              # nothing written past the capacity


def test_threshold_taken_from_a_layer_result_on_the_device(lgn, oracle):
    n = 200_000
    g = synth.lognormal_tensor(n, -11.0, 2.5, 0.5, seed=6, dtype=torch.float32, device="cuda")
    out = torch.empty_like(g)
    ws = lgn.new_workspace([n], g.device)
    res = lgn.new_results(1, g.device)
    lgn.lgn_compress_layers([lgn.make_layer(g, out, lgn.MODE_PRUNE, S=0.85, seed=5)], res, ws)
    stream, off = encode(lgn, g, 123.0, 5, True, tau_from=res.data_ptr())   # the host value is ignored
    tau = lgn.read_results(res, 1)[0]["tau"]
    want_stream, want_off = oracle.prefix_encode(np_bits(out), tau)     # the pruned tensor the grouped call wrote
    assert np.array_equal(off, want_off) and np.array_equal(stream[:int(off[-1])], want_stream)
    bits = 32.0 * int(off[-1]) / n
    assert bits < 4.0                                                    # 85 % sparsity: a few bits per value


def test_bad_arguments(lgn):
    g = torch.zeros(4096, device="cuda")
    off = torch.zeros(3, dtype=torch.int64, device="cuda")
    ws = torch.empty(lgn.lgn_prefix_workspace_bytes(4096), dtype=torch.uint8, device="cuda")
    stream = torch.zeros(8192, dtype=torch.int32, device="cuda")
    with pytest.raises(lgn.LgnError):
        lgn.lgn_prefix_encode(g, -1.0, 0, True, stream, off, ws)
    with pytest.raises(lgn.LgnError):
        lgn.lgn_prefix_encode(g, 1.0, 0, True, stream, off, ws[:16])
    with pytest.raises(ValueError):
        lgn.lgn_prefix_encode(g, 1.0, 0, True, stream, off[:2], ws)
