"""CPU-only checks of the C ABI: the library loads, exports what include/lgn.h
declares, rejects bad arguments on the host, and its host-side closed forms
agree with the oracle's."""
import ctypes as C
import math
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "lgn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lgn_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lgn):
    names = declared_functions()
    assert {"lgn_stats", "lgn_threshold", "lgn_fp_format", "lgn_prune", "lgn_quantize",
            "lgn_compress_layers"} <= set(names)
    for name in names:
        assert hasattr(lgn.raw(), name), name


def test_struct_sizes_match_header(lgn):
    assert C.sizeof(lgn.StatsT) == 48
    assert C.sizeof(lgn.FpFormatT) == 16
    assert C.sizeof(lgn.LayerT) == 96
    assert C.sizeof(lgn.LayerResultT) == 120


def test_status_strings(lgn):
    seen = {lgn.raw().lgn_status_string(c).decode() for c in range(6)}
    assert len(seen) == 6
    assert lgn.raw().lgn_status_string(77).decode() == "unknown status"


def test_sizes(lgn, oracle):
    for nbits in range(4, 9):
        for n in (0, 1, 3, 5, 1023, 2 ** 20 + 7, 2 ** 30):
            assert lgn.lgn_codes_bytes(n, nbits) == oracle.packed_bytes(n, nbits)
    assert lgn.lgn_codes_bytes(10, 3) == 0 and lgn.lgn_codes_bytes(10, 9) == 0
    w1 = lgn.lgn_workspace_bytes([2 ** 20])
    w2 = lgn.lgn_workspace_bytes([2 ** 30])
    w3 = lgn.lgn_workspace_bytes([2 ** 20] * 53)
    assert 0 < w1 < w2 and w1 < w3
    assert w1 % 256 == 0
    assert lgn.lgn_workspace_bytes([]) > 0
    assert lgn.lgn_workspace_bytes([2 ** 50]) == 0           # too large: reported as 0
    # launches per grouped call: one set-up launch up to about 110 layers, then one more per 112 or so
    assert lgn.lgn_launches_per_call(0) == 0
    assert [lgn.lgn_launches_per_call(L) for L in (1, 20, 53, 100)] == [2, 2, 2, 2]
    counts = [lgn.lgn_launches_per_call(L) for L in range(1, 400)]
    assert counts == sorted(counts) and counts[-1] == 5


@pytest.mark.parametrize("sigma", [1e-3, 0.3, 1.0, 1.5, 2.0, 3.0, 4.0, 5.5, 8.0, 25.0, 40.0])
def test_threshold_agrees_with_oracle(lgn, oracle, sigma):
    for mu in (-85.0, -12.0, 0.0, 3.0):
        for l, S in [(0.0, 1e-6), (0.0, 0.5), (0.4, 0.8), (0.5, 0.85), (0.3, 0.99), (0.0, 1 - 1e-9),
                     (0.5, 0.5), (0.6, 0.5), (1.0, 0.5), (0.0, 0.0)]:
            a = lgn.lgn_threshold(mu, sigma, l, S)
            b = oracle.threshold(mu, sigma, l, S)
            assert a == pytest.approx(b, rel=2e-12, abs=0.0)
            for dt in (lgn.F32, lgn.BF16):
                assert lgn.lgn_snap_threshold(a, dt) == oracle.snap_tau(b, dt)


def test_threshold_rejects_bad_arguments(lgn):
    for args in [(0.0, 1.0, 0.0, 1.0), (0.0, 1.0, 0.0, -0.1), (0.0, 1.0, 1.5, 0.5), (0.0, 1.0, -0.1, 0.5),
                 (float("nan"), 1.0, 0.0, 0.5), (0.0, -1.0, 0.0, 0.5), (0.0, float("inf"), 0.0, 0.5)]:
        with pytest.raises(lgn.LgnError) as e:
            lgn.lgn_threshold(*args)
        assert e.value.code == 1
    assert lgn.raw().lgn_threshold(0.0, 1.0, 0.0, 0.5, None) == 1
    assert math.isnan(lgn.lgn_snap_threshold(-1.0, lgn.F32))
    assert math.isnan(lgn.lgn_snap_threshold(1.0, 7))


def test_snap_threshold_agrees_with_oracle(lgn, oracle):
    rs = np.random.RandomState(0)
    for tau in list(np.exp(rs.uniform(-100, 88, 500))) + [0.0, 1e39, 3.4e38, 2.0 ** -149, 2.0 ** -150, 1e-46]:
        for dt in (lgn.F32, lgn.BF16):
            assert lgn.lgn_snap_threshold(float(tau), dt) == oracle.snap_tau(float(tau), dt)


def test_fp_format_agrees_with_oracle(lgn, oracle):
    for nbits in range(4, 9):
        for sigma in np.concatenate([np.linspace(0.05, 9.0, 180), [1e-9, 25.0, 60.0]]):
            for mu in (-85.3, -12.0, -0.2, 0.0, 0.35, 4.0):
                assert lgn.lgn_fp_format(mu, float(sigma), nbits) == oracle.fp_format(mu, float(sigma), 1, nbits)


def test_fp_format_rejects_bad_arguments(lgn):
    for nbits in (3, 9, 0, -1):
        with pytest.raises(lgn.LgnError) as e:
            lgn.lgn_fp_format(0.0, 1.0, nbits)
        assert e.value.code == 2
    with pytest.raises(lgn.LgnError):
        lgn.lgn_fp_format(float("nan"), 1.0, 6)
    assert lgn.raw().lgn_fp_format(0.0, 1.0, 6, None) == 1


def test_device_entry_points_reject_bad_arguments_before_any_cuda_call(lgn):
    """Fake, never dereferenced addresses: every call must return on the host."""
    R = lgn.raw()
    A, B, W = 0x10000, 0x90000, 0x200000                 # 16-byte aligned, disjoint
    fmt = lgn.FpFormatT(6, 4, 1, -17)
    INVALID, UNSUPPORTED, WORKSPACE = 1, 2, 3
    # prune
    assert R.lgn_prune(None, B, 100, 0, 1.0, 0, None) == INVALID
    assert R.lgn_prune(A, None, 100, 0, 1.0, 0, None) == INVALID
    assert R.lgn_prune(A + 4, B, 100, 0, 1.0, 0, None) == INVALID          # misaligned
    assert R.lgn_prune(A, A + 64, 100, 0, 1.0, 0, None) == INVALID         # overlap
    assert R.lgn_prune(A, B, 100, 5, 1.0, 0, None) == INVALID              # dtype
    assert R.lgn_prune(A, B, 100, 0, -1.0, 0, None) == INVALID
    assert R.lgn_prune(A, B, 100, 0, float("nan"), 0, None) == INVALID
    assert R.lgn_prune(A, B, 0, 0, 1.0, 0, None) == 0                      # empty: nothing to do
    # quantize
    assert R.lgn_quantize(A, B, 100, 0, None, 0, 0, None) == INVALID
    assert R.lgn_quantize(A, B, 100, 0, C.byref(lgn.FpFormatT(9, 5, 3, 0)), 0, 0, None) == UNSUPPORTED
    assert R.lgn_quantize(A, B, 100, 0, C.byref(lgn.FpFormatT(6, 4, 2, 0)), 0, 0, None) == INVALID
    assert R.lgn_quantize(A, B, 100, 0, C.byref(lgn.FpFormatT(6, 0, 5, 0)), 0, 0, None) == INVALID
    assert R.lgn_quantize(A, B, 100, 0, C.byref(fmt), 3, 0, None) == INVALID
    assert R.lgn_quantize(A, B + 2, 100, 0, C.byref(fmt), 0, 0, None) == INVALID
    assert R.lgn_quantize(A, B, 0, 0, C.byref(fmt), 0, 0, None) == 0
    # stats
    ws_need = lgn.lgn_workspace_bytes([100])
    assert R.lgn_stats(A, 100, 0, None, W, ws_need, None) == INVALID
    assert R.lgn_stats(None, 100, 0, B, W, ws_need, None) == INVALID
    assert R.lgn_stats(A, 100, 0, B, None, ws_need, None) == INVALID
    assert R.lgn_stats(A, 100, 0, B, W, ws_need - 1, None) == WORKSPACE
    assert R.lgn_stats(A, 2 ** 50, 0, B, W, 2 ** 40, None) == UNSUPPORTED
    # grouped
    def layer(**kw):
        d = dict(g=A, out=B, n=100, dt=0, mode=0, S=0.8, nbits=6, rounding=0, seed=0,
                 use_override=0, scale_mode=0, mu_override=0.0, sigma_override=0.0, right_mode=None,
                 counters=0, reserved=0)
        d.update(kw)
        return lgn.LayerT(*[d[f[0]] for f in lgn.LayerT._fields_])
    def call(l, ws_bytes=None, res=0x300000, n=1):
        arr = (lgn.LayerT * 1)(l)
        return R.lgn_compress_layers(arr, n, res, W, ws_need if ws_bytes is None else ws_bytes, None)
    assert call(layer(S=1.0)) == INVALID
    assert call(layer(S=-0.5)) == INVALID
    assert call(layer(mode=7)) == INVALID
    assert call(layer(mode=2)) == INVALID                  # the internal statistics-only mode is not public
    assert call(layer(mode=1, nbits=3)) == UNSUPPORTED
    assert call(layer(mode=1, rounding=2)) == INVALID
    assert call(layer(out=None)) == INVALID
    assert call(layer(g=A + 8)) == INVALID
    assert call(layer(use_override=1, sigma_override=-1.0)) == INVALID
    assert call(layer(use_override=1, mu_override=float("nan"), sigma_override=1.0)) == INVALID
    assert call(layer(right_mode=0x400000 + 8)) == INVALID            # mask: 16-byte aligned
    assert call(layer(right_mode=B + 16)) == INVALID                  # the output would overwrite the mask
    assert call(layer(mode=1, right_mode=0x400000)) == INVALID        # a mask belongs to pruning
    assert call(layer(scale_mode=1)) == INVALID                       # a scale mode belongs to quantisation
    assert call(layer(mode=1, scale_mode=2)) == INVALID
    assert call(layer(reserved=3)) == INVALID                         # must be zero
    assert call(layer(), ws_bytes=16) == WORKSPACE
    assert call(layer(), res=None) == INVALID
    assert call(layer(), n=-1) == INVALID
    assert call(layer(), n=0) == 0


def test_quantile_rejects_bad_arguments_before_any_cuda_call(lgn):
    R = lgn.raw()
    A, O, W = 0x10000, 0x90000, 0x200000
    need = lgn.lgn_quantile_workspace_bytes()
    INVALID, UNSUPPORTED, WORKSPACE = 1, 2, 3
    assert R.lgn_quantile(A, 100, 0, 1.5, O, W, need, None) == INVALID
    assert R.lgn_quantile(A + 8, 100, 0, 0.5, O, W, need, None) == INVALID
    assert R.lgn_quantile(A, 100, 0, 0.5, O + 8, W, need, None) == INVALID
    assert R.lgn_quantile(A, 100, 0, 0.5, O, W, need - 1, None) == WORKSPACE
    # the bins are 32-bit counters: a tensor that could overflow one is refused
    assert R.lgn_quantile(A, 2 ** 32, 1, 0.5, O, W, need, None) == UNSUPPORTED
    assert R.lgn_quantile(A, 2 ** 40, 0, 0.5, O, W, need, None) == UNSUPPORTED


def test_dequantize_rejects_bad_arguments_before_any_cuda_call(lgn):
    R = lgn.raw()
    A, B = 0x10000, 0x90000
    INVALID, UNSUPPORTED = 1, 2
    ok = lgn.FpFormatT(6, 4, 1, -17)
    assert R.lgn_dequantize(A, 100, None, 0, B, None) == INVALID
    assert R.lgn_dequantize(A, 100, C.byref(lgn.FpFormatT(3, 1, 1, 0)), 0, B, None) == UNSUPPORTED
    assert R.lgn_dequantize(A, 100, C.byref(lgn.FpFormatT(6, 4, 2, 0)), 0, B, None) == INVALID
    assert R.lgn_dequantize(A, 100, C.byref(ok), 2, B, None) == INVALID                              # output type
    assert R.lgn_dequantize(A, 100, C.byref(lgn.FpFormatT(6, 4, 1, -120)), 0, B, None) == UNSUPPORTED  # subnormal codes
    assert R.lgn_dequantize(A, 100, C.byref(lgn.FpFormatT(6, 4, 1, 121)), 0, B, None) == UNSUPPORTED   # codes beyond fp32
    assert R.lgn_dequantize(None, 100, C.byref(ok), 0, B, None) == INVALID
    assert R.lgn_dequantize(A, 100, C.byref(ok), 0, None, None) == INVALID
    assert R.lgn_dequantize(A, 100, C.byref(ok), 0, B + 16, None) == INVALID                         # out: 32-byte aligned
    assert R.lgn_dequantize(A + 4, 100, C.byref(ok), 0, B, None) == INVALID
    assert R.lgn_dequantize(A, 100, C.byref(ok), 0, A + 64, None) == INVALID                         # overlap
    assert R.lgn_dequantize(A, 2 ** 50, C.byref(ok), 0, B, None) == UNSUPPORTED
    assert R.lgn_dequantize(None, 0, C.byref(ok), 0, None, None) == 0                                # empty


def test_scale_from_max(lgn, oracle):
    for mx in [1.0, 1.0 - 2.0 ** -24, 3.0e-6, 2.0 ** -140, 1e4, 65504.0, 2.0 ** -20 * 1.5]:
        for n2 in range(1, 8):
            assert lgn.lgn_scale_from_max(mx, n2) == oracle.scale_exp_from_max(mx, n2)
    for bad in [(0.0, 4), (-1.0, 4), (float("inf"), 4), (float("nan"), 4), (1.0, 0), (1.0, 8)]:
        with pytest.raises(lgn.LgnError) as e:
            lgn.lgn_scale_from_max(*bad)
        assert e.value.code == 1
    assert lgn.raw().lgn_scale_from_max(1.0, 4, None) == 1


def test_cosine_similarity_agrees_with_oracle(lgn, oracle):
    for sigma in (0.5, 1.0, 2.0, 3.0, 5.0):
        for k in (2.0, 2.75, 3.0, 4.0):
            for mu in (-12.0, 0.0):
                for u in np.linspace(-6 * sigma, k * sigma, 25):
                    got = lgn.lgn_cosine_similarity(mu, sigma, k, float(np.exp(mu + u)))
                    u_eff = float(np.log(np.exp(mu + u)) - mu)            # what the library sees after exp/log
                    if u_eff > k * sigma:
                        continue
                    assert got == pytest.approx(oracle.cosine_similarity(u_eff, sigma, k), rel=1e-11)
    for bad in [(0.0, 1.0, 3.0, 0.0), (0.0, 1.0, 3.0, -1.0), (0.0, 1.0, 3.0, float("inf")), (float("nan"), 1.0, 3.0, 1.0),
                (0.0, -1.0, 3.0, 1.0), (0.0, 1.0, 3.0, float(np.exp(3.5)))]:
        with pytest.raises(lgn.LgnError) as e:
            lgn.lgn_cosine_similarity(*bad)
        assert e.value.code == 1
    assert lgn.raw().lgn_cosine_similarity(0.0, 1.0, 3.0, 1.0, None) == 1


def test_allocate_sparsity_agrees_with_oracle(lgn, oracle):
    rs = np.random.RandomState(3)
    for trial in range(40):
        L = int(rs.randint(1, 21))
        deep = int(rs.randint(0, L + 1))
        n = [int(x) for x in rs.randint(1_000, 5_000_000, L)]
        sigma = [float(x) for x in rs.uniform(1.0, 4.0, L)]
        l = [float(x) for x in rs.uniform(0.0, 0.7, L)]
        k = [float(x) for x in rs.uniform(2.0, 3.5, L)]
        floors = [float(x) for x in rs.uniform(0.9, 0.9999, deep)]
        S, cap = float(rs.choice([0.6, 0.8, 0.9, 0.95])), 0.98
        want, want_mean = oracle.allocate_sparsity(n, sigma, l, k, floors, S, cap)
        layers = [dict(n=n[i], sigma=sigma[i], zero_frac=l[i], k=k[i], min_cos=floors[i] if i < deep else 0.0)
                  for i in range(L)]
        got, got_mean = lgn.lgn_allocate_sparsity(layers, deep, S, cap)
        assert got == pytest.approx(want, rel=1e-10, abs=1e-12)
        assert got_mean == pytest.approx(want_mean, rel=1e-10)
    with pytest.raises(lgn.LgnError):
        lgn.lgn_allocate_sparsity([dict(n=1, sigma=1.0, zero_frac=0.0)], 2, 0.5, 0.9)       # more deep layers than layers
    with pytest.raises(lgn.LgnError):
        lgn.lgn_allocate_sparsity([dict(n=1, sigma=1.0, zero_frac=0.0)], 0, 0.95, 0.9)      # cap below S
    with pytest.raises(lgn.LgnError):
        lgn.lgn_allocate_sparsity([dict(n=1, sigma=1.0, zero_frac=1.5)], 0, 0.5, 0.9)
    assert lgn.lgn_allocate_sparsity([], 0, 0.5, 0.9) == ([], 0.0)


def test_lgn_log_prints_host_decisions():
    """LGN_LOG=1: one "[lgn] " line per host-side decision on stderr; nothing without it."""
    import os, subprocess, sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = ("from paper_2006_08173_b200 import binding as lgn\n"
            "print(lgn.lgn_threshold(-12.0, 2.0, 0.4, 0.8))\n"
            "print(lgn.lgn_fp_format(-12.0, 2.0, 6)['exp_bits'])\n")
    def run(env_extra):
        env = dict(os.environ); env.pop("LGN_LOG", None); env.update(env_extra)
        return subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=300)
    quiet = run({})
    assert quiet.returncode == 0 and "[lgn]" not in quiet.stderr
    assert "[lgn]" not in run({"LGN_LOG": "0"}).stderr
    loud = run({"LGN_LOG": "1"})
    assert loud.returncode == 0 and loud.stdout == quiet.stdout
    lines = [l for l in loud.stderr.splitlines() if l.startswith("[lgn] ")]
    assert any(l.startswith("[lgn] threshold: mu=-12 sigma=2 zero fraction=0.4") and "S'=0.66666" in l and "tau=" in l for l in lines)
    assert any(l.startswith("[lgn] format: mu=-12 sigma=2 nbits=6 -> 1-") for l in lines)
