"""The bench workload at its full size (ResNet-18 shapes, batch 256, fp32,
635.8 M elements, per-layer sparsity), in the launch configuration bench.py
times: one lgn_compress_layers call over all 20 layers.  Statistics of every
layer are compared with the oracle's over the whole tensor; outputs are compared
bit for bit on sampled windows of every layer (and in full on the small layers)
with the oracle's mu/sigma fed in; properties that hold at any size are checked
over every element on the device."""
import numpy as np
import pytest
import torch

import bench
from gpu_helpers import assert_stats_close, np_bits, on_threads, windows_of
from paper_2006_08173_b200 import synth

pytestmark = pytest.mark.gpu


def launch(lgn, w, specs, tensors, overrides=None):
    outs = [torch.empty_like(g) for g in tensors]
    layers = []
    for k, (g, o, s) in enumerate(zip(tensors, outs, specs)):
        ov = overrides[k] if overrides else (None, None)
        layers.append(lgn.make_layer(g, o, lgn.MODE_PRUNE, S=s.sparsity, seed=1000 + k,
                                     mu_override=ov[0], sigma_override=ov[1]))
    ws = lgn.new_workspace([g.numel() for g in tensors], tensors[0].device)
    res = lgn.new_results(len(tensors), tensors[0].device)
    lgn.lgn_compress_layers(layers, res, ws)
    torch.cuda.synchronize()
    return outs, lgn.read_results(res, len(tensors))


def test_bench_workload_full_size(lgn, oracle):
    w, specs = bench.workload_specs("resnet18_bs256_fp32_prune", 256, 0)
    tensors = synth.make_layers(specs, torch.float32, "cuda")
    assert sum(t.numel() for t in tensors) == 635_830_272

    # (a) free-running: statistics of every layer against the oracle over the whole tensor
    outs, res = launch(lgn, w, specs, tensors)
    ref_stats = []
    for g, r in zip(tensors, res):
        st = oracle.stats(np_bits(g))
        ref_stats.append(st)
        assert r["status"] == 0
        assert_stats_close(r, st)
    # properties over every element, on the device
    for g, o, r, s in zip(tensors, outs, res, specs):
        tau = r["tau"]
        a = g.abs()
        assert bool(torch.equal(o[a > tau], g[a > tau]))                         # above alpha: unchanged
        small = a <= tau
        vals = o[small]
        assert bool(((vals == 0) | (vals.abs() == tau)).all())                   # else 0 or +-alpha
        keep = small & (o != 0)
        assert bool((torch.sign(o[keep]) == torch.sign(g[keep])).all())
        achieved = float((o == 0).sum()) / o.numel()
        zero_in = 1.0 - r["nnz"] / r["n"]
        want = max(s.sparsity, zero_in)                  # a layer already sparser than asked is left alone
        if zero_in >= s.sparsity:
            assert tau == 0.0 and bool(torch.equal(o, g))
        assert abs(achieved - want) < 1e-3 + 5 * (want * (1 - want) / o.numel()) ** 0.5

    # (b) oracle's mu/sigma fed in: thresholds identical, outputs bit-exact on samples
    ov = [(st["mu"], st["sigma"]) for st in ref_stats]
    outs, res = launch(lgn, w, specs, tensors, overrides=ov)
    rs = np.random.RandomState(0)
    for k, (g, o, r, s, st) in enumerate(zip(tensors, outs, res, specs, ref_stats)):
        tau = oracle.snap_tau(oracle.threshold(st["mu"], st["sigma"], st["zero_frac"], s.sparsity), oracle.F32)
        assert r["tau"] == tau
        n = g.numel()
        # the small layers in full; about 3.5 M elements of every other layer: its first and
        # last half million, windows across tile seams and random ones
        windows = windows_of(n, 32768, rs, width=1 << 19, full_below=7_000_000)

        def one(lo, hi, g=g, o=o, tau=tau, k=k):
            ref = oracle.prune(np_bits(g[lo:hi]), tau, 1000 + k, first=lo)
            return np.array_equal(np_bits(o[lo:hi]).view(np.uint32), ref.view(np.uint32))
        for (lo, hi), ok in zip(windows, on_threads(one, windows)):
            assert ok, (k, lo, hi)


@pytest.mark.parametrize("mode", ["quant", "prune"])
def test_bf16_group_with_large_queue_items(lgn, oracle, mode):
    """A bf16 group large enough (1.4 GB of input) for the library to hand out two
    sub-tiles per queue item: ResNet-50 shapes at batch 64, one grouped call.  Every
    layer's statistics against the oracle; codes / pruned values bit for bit on windows
    that straddle item and tile boundaries, and on the smallest layers in full."""
    name = "resnet50_bs256_bf16_fp6" if mode == "quant" else "resnet50_bs256_bf16_prune"
    w, specs = bench.workload_specs(name, 64, 0)
    tensors = synth.make_layers(specs, torch.bfloat16, "cuda")
    assert sum(t.numel() for t in tensors) * 2 > 8 * 592 * (128 << 10)
    dev = tensors[0].device
    ref_stats = [oracle.stats(np_bits(g)) for g in tensors]
    if mode == "quant":
        outs = [torch.empty(lgn.lgn_codes_bytes(g.numel(), 6) + 16, dtype=torch.uint8, device=dev) for g in tensors]
        layers = [lgn.make_layer(g, o, lgn.MODE_QUANTIZE, nbits=6, rounding=lgn.ROUND_STOCHASTIC, seed=500 + k,
                                 mu_override=st["mu"], sigma_override=st["sigma"])
                  for k, (g, o, st) in enumerate(zip(tensors, outs, ref_stats))]
    else:
        outs = [torch.empty_like(g) for g in tensors]
        layers = [lgn.make_layer(g, o, lgn.MODE_PRUNE, S=s.sparsity, seed=500 + k,
                                 mu_override=st["mu"], sigma_override=st["sigma"])
                  for k, (g, o, s, st) in enumerate(zip(tensors, outs, specs, ref_stats))]
    ws = lgn.new_workspace([g.numel() for g in tensors], dev)
    res = lgn.new_results(len(tensors), dev)
    lgn.lgn_compress_layers(layers, res, ws)
    torch.cuda.synchronize()
    results = lgn.read_results(res, len(tensors))
    rs = np.random.RandomState(1)
    for k, (g, o, r, s, st) in enumerate(zip(tensors, outs, results, specs, ref_stats)):
        assert r["status"] == 0
        assert_stats_close(r, st)
        n = g.numel()
        if n <= 2_000_000:
            windows = [(0, n)]
        else:
            starts = [0, 65536 - 4096, 2 * 65536 - 4096, n - 8192] + [int(x) // 8 * 8 for x in rs.randint(0, n - 8192, 2)]
            windows = [(a, a + 8192) for a in starts]
        if mode == "quant":
            fmt = oracle.fp_format(st["mu"], st["sigma"], st["nnz"], 6)
            assert r["fmt"] == fmt
            got_all = o.cpu().numpy()
            for lo, hi in windows:                        # windows start on multiples of 8 elements = 6 bytes
                codes = oracle.quantize(np_bits(g[lo:hi]), fmt["exp_bits"], fmt["man_bits"], fmt["scale_exp"], 1, 500 + k, first=lo)
                ref = oracle.pack(codes, 6)
                nbytes = (hi - lo) * 6 // 8
                assert np.array_equal(got_all[lo * 6 // 8: lo * 6 // 8 + nbytes], ref[:nbytes]), (k, lo)
        else:
            tau = oracle.snap_tau(oracle.threshold(st["mu"], st["sigma"], st["zero_frac"], s.sparsity), oracle.BF16) if st["nnz"] else 0.0
            assert r["tau"] == tau
            for lo, hi in windows:
                ref = oracle.prune(np_bits(g[lo:hi]), tau, 500 + k, first=lo)
                assert np.array_equal(np_bits(o[lo:hi]), ref), (k, lo)
