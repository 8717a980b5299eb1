"""Shared helpers of the GPU parity tests: run the oracle for one layer and
compare the library's outputs with it."""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import torch

from paper_2006_08173_b200 import synth

REL_TOL = 1e-5      # mu / sigma: relative to the oracle's fp64 value


def np_bits(t):
    return synth.as_numpy_bits(t).reshape(-1)


# The oracle's C functions release the interpreter lock: host threads run it in parallel.
THREADS = max(1, len(os.sched_getaffinity(0)))


def on_threads(fn, jobs):
    with ThreadPoolExecutor(THREADS) as ex:
        return list(ex.map(lambda j: fn(*j), jobs))


def oracle_stats_whole(oracle, tensors):
    """oracle.stats of every tensor over all of its elements, one tensor at a time on the
    host (a device tensor is copied, measured, and its host copy dropped)."""
    def one(g):
        return oracle.stats(np_bits(g))
    return on_threads(one, [(g,) for g in tensors])


def windows_of(n, tile, rs, width=65536, seams=3, rand=3, full_below=3_000_000):
    """Windows [lo, hi) of a tensor of n elements: the whole tensor when small; else its
    first and last `width` elements, windows straddling tile seams (at the start, in the
    middle and near the end of the tensor) and random ones.  Starts are multiples of 8."""
    if n <= full_below:
        return [(0, n)]
    w = [(0, width), (n - width - (n - width) % 8, n)]
    ntiles = n // tile
    for k in sorted(set([1, ntiles // 2, max(1, ntiles - 1)]))[:seams]:
        lo = k * tile - width // 2
        if 0 <= lo and lo + width <= n:
            w.append((lo, lo + width))
    for x in rs.randint(0, (n - width) // 8, rand):
        w.append((int(x) * 8, int(x) * 8 + width))
    return w


def oracle_layer(orc, g_np, mode, *, S=0.0, nbits=6, rounding=0, seed=0):
    """stats -> closed form -> apply, all in the oracle."""
    dt = orc.BF16 if g_np.dtype == np.uint16 else orc.F32
    st = orc.stats(g_np)
    res = {"stats": st}
    if mode == "prune":
        # a tensor with no nonzero entry has nothing to prune: tau = 0
        tau = orc.snap_tau(orc.threshold(st["mu"], st["sigma"], st["zero_frac"], S), dt) if st["nnz"] else 0.0
        res["tau"] = tau
        res["out"] = orc.prune(g_np, tau, seed)
    else:
        fmt = orc.fp_format(st["mu"], st["sigma"], st["nnz"], nbits)
        res["fmt"] = fmt
        codes = orc.quantize(g_np, fmt["exp_bits"], fmt["man_bits"], fmt["scale_exp"], rounding, seed)
        res["codes"] = codes
        res["packed"] = orc.pack(codes, nbits)
    return res


def assert_stats_close(got, want, n_for_tol=None):
    """nnz exact; mu and sigma within REL_TOL of the oracle.  mu's error is
    measured against max(|mu|, sigma): a mean of logs can sit arbitrarily close
    to zero, and sigma is the scale on which it is known at all."""
    assert got["n"] == want["n"]
    assert got["nnz"] == want["nnz"]
    scale = max(abs(want["mu"]), want["sigma"])
    assert abs(got["mu"] - want["mu"]) <= REL_TOL * scale
    assert abs(got["sigma"] - want["sigma"]) <= REL_TOL * max(want["sigma"], 1e-300) or want["sigma"] == 0.0 and got["sigma"] <= 1e-6


def assert_same_bits(t_gpu, ref_np):
    got = np_bits(t_gpu)
    assert got.dtype == ref_np.dtype and got.shape == ref_np.reshape(-1).shape
    if not np.array_equal(got.view(np.uint16 if got.dtype == np.uint16 else np.uint32),
                          ref_np.reshape(-1).view(np.uint16 if got.dtype == np.uint16 else np.uint32)):
        bad = np.nonzero(got.view(np.uint8).reshape(got.size, -1).any(axis=1)
                         != ref_np.reshape(-1).view(np.uint8).reshape(got.size, -1).any(axis=1))[0]
        diff = np.nonzero(got != ref_np.reshape(-1))[0]
        raise AssertionError(f"{diff.size} of {got.size} elements differ; first at {diff[:5]}: "
                             f"got {got[diff[:5]]} want {ref_np.reshape(-1)[diff[:5]]} (zero-pattern diffs {bad.size})")


def assert_same_codes(packed_gpu, packed_ref):
    a = packed_gpu.cpu().numpy()[:packed_ref.size]
    if not np.array_equal(a, packed_ref):
        diff = np.nonzero(a != packed_ref)[0]
        raise AssertionError(f"{diff.size} of {a.size} packed bytes differ; first at byte {diff[:8]}")
