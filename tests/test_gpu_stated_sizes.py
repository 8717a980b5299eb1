"""The configurations at the sizes they are stated at, against the oracle.

* ResNet-50 shapes at batch 256 in bf16 (53 tensors, 2.845 G elements, 5.7 GB): FP5 and
  FP6, round-to-nearest and stochastic, one grouped call each.  Statistics of every layer
  against the oracle over the whole tensor; formats equal; packed codes bit for bit on
  windows of every layer that cover its first and last tile, tile seams and random places
  (small layers in full).
* Single flat tensors of 2^28 and 2^30 elements, fp32 and bf16, pruning and FP6: statistics
  against the oracle over the WHOLE tensor (not a slice), outputs bit for bit on windows that
  include the first and the last tile and the element where the packed stream passes bit
  2^32.
* Index arithmetic beyond 32 bits: an fp32 tensor whose bytes pass 4 GiB, a bf16 tensor of
  more than 2^32 elements, and a bf16 tensor of more than 2^35 elements (the counter of the
  random-bit generator, element index / 8, then needs its second word).

The oracle runs on host threads (its C functions release the interpreter lock), one layer
or window per task.
"""
import numpy as np
import pytest
import torch

import bench
from gpu_helpers import assert_stats_close, np_bits, on_threads, oracle_stats_whole, windows_of
from paper_2006_08173_b200 import synth

pytestmark = pytest.mark.gpu

def check_codes(oracle, g, codes_np, fmt, nbits, rounding, seed, windows, tag):
    def one(lo, hi):
        c = oracle.quantize(np_bits(g[lo:hi]), fmt["exp_bits"], fmt["man_bits"], fmt["scale_exp"], rounding, seed, first=lo)
        ref = oracle.pack(c, nbits)
        nbytes = ((hi - lo) * nbits + 7) // 8               # lo is a multiple of 8: the window starts on a byte;
                                                            # only a window that ends the tensor can end inside one
        b0 = lo * nbits // 8
        return np.array_equal(codes_np(b0, nbytes), ref[:nbytes])
    for (lo, hi), ok in zip(windows, on_threads(one, windows)):
        assert ok, (tag, lo, hi)


def check_pruned(oracle, g, o, tau, seed, windows, tag):
    def one(lo, hi):
        ref = oracle.prune(np_bits(g[lo:hi]), tau, seed, first=lo)
        got = np_bits(o[lo:hi])
        return np.array_equal(got.view(np.uint8), ref.view(np.uint8))
    for (lo, hi), ok in zip(windows, on_threads(one, windows)):
        assert ok, (tag, lo, hi)


# --------------------------------------------------------------------------- config 3 at batch 256
@pytest.fixture(scope="module")
def resnet50_bs256(oracle):
    w, specs = bench.workload_specs("resnet50_bs256_bf16_fp6", 256, 0)
    tensors = synth.make_layers(specs, torch.bfloat16, "cuda")
    assert len(tensors) == 53 and sum(t.numel() for t in tensors) == 2_845_179_904
    ref_stats = oracle_stats_whole(oracle, tensors)
    yield specs, tensors, ref_stats
    del tensors
    torch.cuda.empty_cache()


@pytest.mark.parametrize("nbits,rounding", [(6, 1), (6, 0), (5, 1), (5, 0)])
def test_resnet50_batch256_bf16_quantise(lgn, oracle, resnet50_bs256, nbits, rounding):
    specs, tensors, ref_stats = resnet50_bs256
    dev = tensors[0].device
    outs = [torch.full((lgn.lgn_codes_bytes(g.numel(), nbits) + 16,), 0xA5, dtype=torch.uint8, device=dev) for g in tensors]
    ws = lgn.new_workspace([g.numel() for g in tensors], dev)

    # free-running call: statistics and formats from the library's own mu, sigma
    res = lgn.new_results(len(tensors), dev)
    layers = [lgn.make_layer(g, o, lgn.MODE_QUANTIZE, nbits=nbits, rounding=rounding, seed=700 + k)
              for k, (g, o) in enumerate(zip(tensors, outs))]
    lgn.lgn_compress_layers(layers, res, ws)
    torch.cuda.synchronize()
    for k, (r, st) in enumerate(zip(lgn.read_results(res, len(tensors)), ref_stats)):
        assert r["status"] == 0, k
        assert_stats_close(r, st)

    # the oracle's mu, sigma fed in: formats equal, codes bit for bit
    layers = [lgn.make_layer(g, o, lgn.MODE_QUANTIZE, nbits=nbits, rounding=rounding, seed=700 + k,
                             mu_override=st["mu"], sigma_override=st["sigma"])
              for k, (g, o, st) in enumerate(zip(tensors, outs, ref_stats))]
    lgn.lgn_compress_layers(layers, res, ws)
    torch.cuda.synchronize()
    results = lgn.read_results(res, len(tensors))
    rs = np.random.RandomState(nbits * 2 + rounding)
    for k, (g, o, r, st) in enumerate(zip(tensors, outs, results, ref_stats)):
        assert r["status"] == 0
        fmt = oracle.fp_format(st["mu"], st["sigma"], st["nnz"], nbits)
        assert r["fmt"] == fmt, k
        n = g.numel()
        nb = lgn.lgn_codes_bytes(n, nbits)
        assert bool((o[nb:] == 0xA5).all()), k                       # nothing written past the stream
        wins = windows_of(n, 65536, rs)

        def codes_np(b0, nbytes, o=o):
            return o[b0:b0 + nbytes].cpu().numpy()
        check_codes(oracle, g, codes_np, fmt, nbits, rounding, 700 + k, wins, ("layer", k))


def test_resnet50_batch256_bf16_prune(lgn, oracle, resnet50_bs256):
    _, tensors, ref_stats = resnet50_bs256
    _, specs = bench.workload_specs("resnet50_bs256_bf16_prune", 256, 0)
    dev = tensors[0].device
    outs = [torch.empty_like(g) for g in tensors]
    ws = lgn.new_workspace([g.numel() for g in tensors], dev)
    res = lgn.new_results(len(tensors), dev)
    layers = [lgn.make_layer(g, o, lgn.MODE_PRUNE, S=s.sparsity, seed=900 + k, mu_override=st["mu"], sigma_override=st["sigma"])
              for k, (g, o, s, st) in enumerate(zip(tensors, outs, specs, ref_stats))]
    lgn.lgn_compress_layers(layers, res, ws)
    torch.cuda.synchronize()
    rs = np.random.RandomState(3)
    for k, (g, o, r, s, st) in enumerate(zip(tensors, outs, lgn.read_results(res, len(tensors)), specs, ref_stats)):
        assert r["status"] == 0
        assert_stats_close(r, st)
        tau = oracle.snap_tau(oracle.threshold(st["mu"], st["sigma"], st["zero_frac"], s.sparsity), oracle.BF16)
        assert r["tau"] == tau, k
        check_pruned(oracle, g, o, tau, 900 + k, windows_of(g.numel(), 65536, rs), ("layer", k))
        achieved = float((o == 0).sum()) / o.numel()
        want = max(s.sparsity, st["zero_frac"])
        assert abs(achieved - want) < 2e-3, k                         # bf16 magnitudes are coarse: ties at alpha


# --------------------------------------------------------------------------- config 4 at 2^28 and 2^30
_STATS_CACHE = {}


def flat_case(lgn, oracle, n, dtype, mode, seed, extra_windows=()):
    g = synth.lognormal_tensor(n, -12.0, 2.0, 0.5, seed, dtype, "cuda")
    key = (n, str(dtype), seed)                         # the same seeded tensor serves pruning and FP6
    if key not in _STATS_CACHE:
        _STATS_CACHE[key] = oracle.stats(np_bits(g))    # over the whole tensor
    st = _STATS_CACHE[key]
    dev = g.device
    tile = 65536 if dtype == torch.bfloat16 else 32768
    ws = lgn.new_workspace([n], dev)
    res = lgn.new_results(1, dev)
    rs = np.random.RandomState(seed)
    wins = windows_of(n, tile, rs) + [w for w in extra_windows if w[1] <= n]
    code = oracle.BF16 if dtype == torch.bfloat16 else oracle.F32
    if mode == "prune":
        o = torch.empty_like(g)
        for ov in (False, True):                        # free-running (statistics), then the oracle's mu, sigma fed in
            layer = lgn.make_layer(g, o, lgn.MODE_PRUNE, S=0.85, seed=77, mu_override=st["mu"] if ov else None,
                                   sigma_override=st["sigma"] if ov else None)
            lgn.lgn_compress_layers([layer], res, ws)
            torch.cuda.synchronize()
            r = lgn.read_results(res, 1)[0]
            assert r["status"] == 0
            assert_stats_close(r, st)
        tau = oracle.snap_tau(oracle.threshold(st["mu"], st["sigma"], st["zero_frac"], 0.85), code)
        assert r["tau"] == tau
        check_pruned(oracle, g, o, tau, 77, wins, (n, str(dtype)))
        achieved = float((o == 0).sum()) / n
        assert abs(achieved - 0.85) < 1e-3 + (2e-3 if dtype == torch.bfloat16 else 0.0)
    else:
        nb = lgn.lgn_codes_bytes(n, 6)
        o = torch.full((nb + 16,), 0xA5, dtype=torch.uint8, device=dev)
        for ov in (False, True):
            layer = lgn.make_layer(g, o, lgn.MODE_QUANTIZE, nbits=6, rounding=lgn.ROUND_STOCHASTIC, seed=77,
                                   mu_override=st["mu"] if ov else None, sigma_override=st["sigma"] if ov else None)
            lgn.lgn_compress_layers([layer], res, ws)
            torch.cuda.synchronize()
            r = lgn.read_results(res, 1)[0]
            assert r["status"] == 0
            assert_stats_close(r, st)
        fmt = oracle.fp_format(st["mu"], st["sigma"], st["nnz"], 6)
        assert r["fmt"] == fmt
        assert bool((o[nb:] == 0xA5).all())
        check_codes(oracle, g, lambda b0, m: o[b0:b0 + m].cpu().numpy(), fmt, 6, 1, 77, wins, (n, str(dtype)))


BIT32 = (1 << 32) // 6 // 8 * 8           # the element in whose neighbourhood the FP6 stream passes bit 2^32


@pytest.mark.parametrize("mode", ["prune", "fp6"])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("log2n", [28, 30])
def test_flat_tensor_at_stated_size(lgn, oracle, log2n, dtype, mode):
    extra = [(BIT32 - 32768, BIT32 + 32768)] if mode == "fp6" else []
    flat_case(lgn, oracle, 1 << log2n, dtype, mode, seed=log2n, extra_windows=extra)
    torch.cuda.empty_cache()


# --------------------------------------------------------------------------- beyond 32-bit offsets and indices
@pytest.mark.parametrize("mode", ["prune", "fp6"])
def test_fp32_tensor_whose_bytes_pass_4_GiB(lgn, oracle, mode):
    n = (1 << 30) + (1 << 20) + 7                     # ragged, 4.3 GB
    at = 1 << 30                                      # element at byte offset 2^32
    flat_case(lgn, oracle, n, torch.float32, mode, seed=5, extra_windows=[(at - 32768, at + 32768)])
    torch.cuda.empty_cache()


def tiled_bf16(n, seed):
    """n bf16 elements: a seeded lognormal block of 2^26 elements repeated (index arithmetic is
    what these sizes test; the values only have to be ordinary)."""
    block = synth.lognormal_tensor(1 << 26, -12.0, 2.0, 0.5, seed, torch.bfloat16, "cuda")
    g = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    for lo in range(0, n, block.numel()):
        m = min(block.numel(), n - lo)
        g[lo:lo + m] = block[:m]
    return g, block


@pytest.mark.parametrize("mode", ["prune", "fp6"])
def test_bf16_tensor_of_more_than_2p32_elements(lgn, oracle, mode):
    n = (1 << 32) + (1 << 20) + 8                     # 8.6 GB
    g, block = tiled_bf16(n, seed=6)
    st = oracle.stats(np_bits(block))                 # any mu, sigma serve as the override
    dev = g.device
    ws = lgn.new_workspace([n], dev)
    res = lgn.new_results(1, dev)
    at = 1 << 32
    wins = [(0, 65536), (at - 65536, at + 65536), (n - 65536 - 8, n), (at + (1 << 19), at + (1 << 19) + 65536)]
    if mode == "prune":
        o = torch.empty_like(g)
        layer = lgn.make_layer(g, o, lgn.MODE_PRUNE, S=0.85, seed=3, mu_override=st["mu"], sigma_override=st["sigma"])
        lgn.lgn_compress_layers([layer], res, ws)
        torch.cuda.synchronize()
        r = lgn.read_results(res, 1)[0]
        assert r["status"] == 0 and r["n"] == n
        reps, rem = divmod(n, block.numel())
        assert r["nnz"] == reps * st["nnz"] + int((block[:rem] != 0).sum())
        zero_frac = 1.0 - r["nnz"] / n
        tau = oracle.snap_tau(oracle.threshold(st["mu"], st["sigma"], zero_frac, 0.85), oracle.BF16)
        assert r["tau"] == tau
        check_pruned(oracle, g, o, tau, 3, wins, "2^32+")
    else:
        nb = lgn.lgn_codes_bytes(n, 6)
        o = torch.full((nb + 16,), 0xA5, dtype=torch.uint8, device=dev)
        layer = lgn.make_layer(g, o, lgn.MODE_QUANTIZE, nbits=6, rounding=1, seed=3, mu_override=st["mu"], sigma_override=st["sigma"])
        lgn.lgn_compress_layers([layer], res, ws)
        torch.cuda.synchronize()
        r = lgn.read_results(res, 1)[0]
        fmt = oracle.fp_format(st["mu"], st["sigma"], st["nnz"], 6)
        assert r["status"] == 0 and r["fmt"] == fmt
        assert bool((o[nb:] == 0xA5).all())
        check_codes(oracle, g, lambda b0, m: o[b0:b0 + m].cpu().numpy(), fmt, 6, 1, 3, wins, "2^32+")
    del g, o
    torch.cuda.empty_cache()


def test_bf16_tensor_of_more_than_2p35_elements_cached_format(lgn, oracle):
    """lgn_quantize (cached format) on 2^35 + 2^17 bf16 elements (64 GiB in, 24 GiB out): past
    element 2^35 the generator's block counter, element index / 8, is 2^32 or more."""
    free, _ = torch.cuda.mem_get_info()
    n = (1 << 35) + (1 << 17)
    if free < 2 * n + lgn.lgn_codes_bytes(n, 6) + (4 << 30):
        pytest.skip("needs 92 GB of free device memory")
    g, block = tiled_bf16(n, seed=7)
    st = oracle.stats(np_bits(block))
    fmt = oracle.fp_format(st["mu"], st["sigma"], st["nnz"], 6)
    nb = lgn.lgn_codes_bytes(n, 6)
    o = torch.empty(nb + 16, dtype=torch.uint8, device="cuda")
    o[nb:] = 0xA5
    lgn.lgn_quantize(g, fmt, lgn.ROUND_STOCHASTIC, 11, o)
    torch.cuda.synchronize()
    at = 1 << 35
    wins = [(0, 32768), (at - 32768, at + 32768), (n - 32768, n), ((1 << 34) + 8, (1 << 34) + 8 + 32768)]
    assert bool((o[nb:] == 0xA5).all())
    check_codes(oracle, g, lambda b0, m: o[b0:b0 + m].cpu().numpy(), fmt, 6, 1, 11, wins, "2^35+")
    del g, o
    torch.cuda.empty_cache()
