"""GPU parity of the grouped single-launch path (statistics -> closed form on
the device -> apply) against the oracle, on the workload shapes of the paper's
setting: one small tensor, a ResNet-18-shaped group pruned with per-layer
sparsity, a ResNet-50-shaped bf16 group quantised to FP5/FP6, and the
edge-case stress set."""
import numpy as np
import pytest
import torch

from gpu_helpers import (assert_same_bits, assert_same_codes, assert_stats_close, np_bits,
                         oracle_layer)
from paper_2006_08173_b200 import synth

pytestmark = pytest.mark.gpu


def run_group(lgn, tensors, specs, overrides=None):
    """specs: list of dicts(mode='prune'|'quant', S, nbits, rounding, seed).
    Returns (outputs, results)."""
    dev = tensors[0].device
    outs, layers = [], []
    for k, (g, sp) in enumerate(zip(tensors, specs)):
        ov = overrides[k] if overrides else (None, None)
        if sp["mode"] == "prune":
            out = torch.empty_like(g)
            layers.append(lgn.make_layer(g, out, lgn.MODE_PRUNE, S=sp["S"], seed=sp["seed"],
                                         mu_override=ov[0], sigma_override=ov[1]))
        else:
            nb = lgn.lgn_codes_bytes(g.numel(), sp["nbits"])
            out = torch.full((max(16, nb) + 16,), 0xAB, dtype=torch.uint8, device=dev)   # canary tail
            layers.append(lgn.make_layer(g, out, lgn.MODE_QUANTIZE, nbits=sp["nbits"], rounding=sp["rounding"],
                                         seed=sp["seed"], mu_override=ov[0], sigma_override=ov[1]))
        outs.append(out)
    ws = lgn.new_workspace([g.numel() for g in tensors], dev)
    ws.fill_(0xCD)                                                   # the library must not rely on zeros
    res = lgn.new_results(len(tensors), dev)
    lgn.lgn_compress_layers(layers, res, ws)
    torch.cuda.synchronize()
    return outs, lgn.read_results(res, len(tensors))


def check_group(lgn, oracle, tensors, specs):
    """Two runs: (a) free-running: stats within tolerance; (b) with the oracle's
    mu/sigma fed in: thresholds, formats and every output bit identical."""
    refs = []
    for g, sp in zip(tensors, specs):
        refs.append(oracle_layer(oracle, np_bits(g), sp["mode"] if sp["mode"] == "prune" else "quant",
                                 S=sp.get("S", 0.0), nbits=sp.get("nbits", 6),
                                 rounding=sp.get("rounding", 0), seed=sp["seed"]))
    outs, res = run_group(lgn, tensors, specs)
    for r, ref in zip(res, refs):
        assert r["status"] == 0
        assert_stats_close(r, ref["stats"])
    ov = [(ref["stats"]["mu"], ref["stats"]["sigma"]) for ref in refs]
    outs, res = run_group(lgn, tensors, specs, overrides=ov)
    for g, sp, out, r, ref in zip(tensors, specs, outs, res, refs):
        assert r["status"] == 0
        assert_stats_close(r, ref["stats"])                  # measured stats are still reported
        if sp["mode"] == "prune":
            assert r["tau"] == ref["tau"]
            assert_same_bits(out, ref["out"])
        else:
            assert r["fmt"] == ref["fmt"]
            assert_same_codes(out, ref["packed"])
            nb = lgn.lgn_codes_bytes(g.numel(), sp["nbits"])
            assert bool((out[max(16, nb):] == 0xAB).all())     # nothing written past the stream
    return outs, res, refs


# ------------------------------------------------------------------ one small tensor
def test_single_small_tensor_prune_and_fp6(lgn, oracle):
    g = synth.lognormal_tensor(8 * 64 * 32 * 32, -12.0, 2.0, 0.40, seed=0, device="cuda").reshape(8, 64, 32, 32)
    outs, res, refs = check_group(lgn, oracle, [g, g],
                                  [dict(mode="prune", S=0.80, seed=1),
                                   dict(mode="quant", nbits=6, rounding=1, seed=1)])
    assert res[1]["fmt"] == {"nbits": 6, "exp_bits": 4, "man_bits": 1, "scale_exp": -17}
    # end to end, no override: requested sparsity reached
    outs, res = run_group(lgn, [g], [dict(mode="prune", S=0.80, seed=1)])
    achieved = float((outs[0] == 0).float().mean())
    assert abs(achieved - 0.80) < 1e-3 + 4 * (0.8 * 0.2 / g.numel()) ** 0.5


# ------------------------------------------------------------------ ResNet-18-shaped group, fp32, per-layer S
def test_resnet18_shaped_group_prune(lgn, oracle):
    specs = synth.resnet18_prune_workload(batch=4, seed=0)            # same 20 shapes, small batch
    tensors = synth.make_layers(specs, torch.float32, "cuda")
    assert len(tensors) == 20
    lspecs = [dict(mode="prune", S=s.sparsity, seed=100 + k) for k, s in enumerate(specs)]
    outs, res, refs = check_group(lgn, oracle, tensors, lspecs)
    outs, res = run_group(lgn, tensors, lspecs)
    for out, s in zip(outs, specs):
        achieved = float((out == 0).float().mean())
        assert abs(achieved - s.sparsity) < 1e-3 + 5 * (s.sparsity * (1 - s.sparsity) / out.numel()) ** 0.5


# ------------------------------------------------------------------ ResNet-50-shaped group, bf16, FP5/FP6
@pytest.mark.parametrize("nbits", [5, 6])
@pytest.mark.parametrize("rounding", [0, 1])
def test_resnet50_shaped_group_quantize(lgn, oracle, nbits, rounding):
    specs = synth.resnet50_quant_workload(batch=1, seed=0)            # same 53 shapes, batch 1
    tensors = synth.make_layers(specs, torch.bfloat16, "cuda")
    assert len(tensors) == 53
    lspecs = [dict(mode="quant", nbits=nbits, rounding=rounding, seed=7 + k) for k in range(53)]
    outs, res, refs = check_group(lgn, oracle, tensors, lspecs)
    seen = {(r["fmt"]["exp_bits"], r["fmt"]["man_bits"]) for r in res}
    assert len(seen) >= 2                                             # per-layer formats really differ


# ------------------------------------------------------------------ mixed group
def test_mixed_modes_dtypes_and_empty_layers(lgn, oracle):
    mk = lambda n, dt, seed, **kw: synth.lognormal_tensor(n, kw.pop("mu", -12.0), kw.pop("sigma", 2.0),
                                                          kw.pop("p", 0.4), seed, dtype=dt, device="cuda", **kw)
    tensors = [mk(100_003, torch.float32, 1), mk(0, torch.float32, 2), mk(1, torch.bfloat16, 3),
               mk(40_000, torch.bfloat16, 4, sigma=3.0), mk(3, torch.float32, 5), mk(65_537, torch.bfloat16, 6),
               torch.zeros(20_000, device="cuda"), mk(1023, torch.float32, 8)]
    specs = [dict(mode="prune", S=0.7, seed=1), dict(mode="prune", S=0.5, seed=2),
             dict(mode="quant", nbits=6, rounding=1, seed=3), dict(mode="quant", nbits=5, rounding=0, seed=4),
             dict(mode="prune", S=0.5, seed=5), dict(mode="prune", S=0.9, seed=6),
             dict(mode="quant", nbits=4, rounding=1, seed=7), dict(mode="quant", nbits=8, rounding=1, seed=8)]
    check_group(lgn, oracle, tensors, specs)


def test_many_layers_in_one_call(lgn, oracle):
    """150 small layers in one call: the descriptors of that many layers no longer
    fit one set-up launch (its parameter block holds about 110 layers), so this
    call takes two; every layer is still checked in full against the oracle."""
    L = 150
    assert lgn.lgn_launches_per_call(L) == 3 and lgn.lgn_launches_per_call(100) == 2
    tensors, specs = [], []
    for k in range(L):
        dt = torch.bfloat16 if k % 3 == 2 else torch.float32
        tensors.append(synth.lognormal_tensor(500 + 37 * k, -14.0 + 0.03 * k, 1.5 + 0.01 * k, 0.3, 100 + k,
                                              dtype=dt, device="cuda"))
        if k % 2:
            specs.append(dict(mode="quant", nbits=5 + (k % 4 == 3), rounding=(k // 2) % 2, seed=k))
        else:
            specs.append(dict(mode="prune", S=(0.5, 0.7, 0.85, 0.9)[(k // 2) % 4], seed=k))
    check_group(lgn, oracle, tensors, specs)


def test_call_is_ordered_after_earlier_work_on_its_stream(lgn):
    """The compute kernel may become resident while the set-up launch before it still
    runs; it must all the same see what earlier kernels on the stream wrote.  The
    input is overwritten by copies enqueued right before the call, with no
    synchronisation in between, and the output must be that of the new contents."""
    n = 2 ** 25 + 5
    a = synth.lognormal_tensor(n, -12.0, 2.0, 0.4, 31, device="cuda")
    b = synth.lognormal_tensor(n, -10.0, 2.5, 0.2, 32, device="cuda")
    specs = [dict(mode="prune", S=0.8, seed=9)]
    (want,), (want_res,) = run_group(lgn, [b.clone()], specs)
    g = a.clone()
    torch.cuda.synchronize()
    for _ in range(3):
        g.copy_(a)
        g.copy_(b)                                   # still running when the call below is enqueued
        (got,), (res,) = run_group(lgn, [g], specs)
        assert res["status"] == 0 and res["tau"] == want_res["tau"]
        assert torch.equal(got.view(torch.int32), want.view(torch.int32))


# ------------------------------------------------------------------ edge-case stress
EDGE_INPUTS = [
    dict(n=1), dict(n=3), dict(n=1023), dict(n=2 ** 20 + 7),
    dict(n=50_000, p=1.0),                                            # all zero
    dict(n=2 ** 18 + 1, sigma=4.0),                                   # heavy tail
    dict(n=2 ** 18 + 1, mu=-85.0, sigma=4.0, p=0.3),                  # into the fp32 subnormals
    dict(n=2 ** 18 + 1, mu=3.0, sigma=2.0, clip=1e4),                 # up to 1e4
    dict(n=2 ** 18 + 1, mixture=[(-14.0, 1.5), (-8.0, 1.5)]),         # two-component mixture
]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("case", range(len(EDGE_INPUTS)))
def test_edge_cases(lgn, oracle, dtype, case):
    kw = dict(EDGE_INPUTS[case])
    n = kw.pop("n")
    g = synth.lognormal_tensor(n, kw.pop("mu", -12.0), kw.pop("sigma", 2.0), kw.pop("p", 0.5), seed=case,
                               dtype=dtype, device="cuda", **kw)
    tensors = [g] * 7
    specs = [dict(mode="prune", S=0.0, seed=1), dict(mode="prune", S=0.5, seed=2), dict(mode="prune", S=0.99, seed=3),
             dict(mode="quant", nbits=5, rounding=0, seed=4), dict(mode="quant", nbits=5, rounding=1, seed=5),
             dict(mode="quant", nbits=6, rounding=0, seed=6), dict(mode="quant", nbits=6, rounding=1, seed=7)]
    if n <= 3:
        # mu/sigma of one to three samples: population std, compared with a looser absolute guard
        # (checked bit-for-bit below with the oracle's values fed in)
        refs = [oracle_layer(oracle, np_bits(g), sp["mode"] if sp["mode"] == "prune" else "quant",
                             S=sp.get("S", 0.0), nbits=sp.get("nbits", 6), rounding=sp.get("rounding", 0),
                             seed=sp["seed"]) for sp in specs]
        ov = [(r["stats"]["mu"], r["stats"]["sigma"]) for r in refs]
        outs, res = run_group(lgn, tensors, specs, overrides=ov)
        for sp, out, r, ref in zip(specs, outs, res, refs):
            assert r["nnz"] == ref["stats"]["nnz"]
            assert abs(r["mu"] - ref["stats"]["mu"]) <= 1e-5 * max(abs(ref["stats"]["mu"]), 1.0)
            assert abs(r["sigma"] - ref["stats"]["sigma"]) <= 1e-4
            if sp["mode"] == "prune":
                assert r["tau"] == ref["tau"]
                assert_same_bits(out, ref["out"])
            else:
                assert r["fmt"] == ref["fmt"]
                assert_same_codes(out, ref["packed"])
    else:
        check_group(lgn, oracle, tensors, specs)


def test_grouped_path_is_deterministic(lgn):
    specs = synth.resnet18_prune_workload(batch=2, seed=3)
    tensors = synth.make_layers(specs, torch.float32, "cuda")
    lspecs = [dict(mode="prune", S=s.sparsity, seed=k) for k, s in enumerate(specs)]
    o1, r1 = run_group(lgn, tensors, lspecs)
    for _ in range(3):
        o2, r2 = run_group(lgn, tensors, lspecs)
        assert r1 == r2
        assert all(torch.equal(a, b) for a, b in zip(o1, o2))


def test_host_buffer_form_in_several_groups(lgn):
    """Enough input (5 x 40 MB) for the host form to run its layers in three pipelined
    groups, of mixed kinds: every output and result must be what one grouped call on
    device tensors gives."""
    n = 10_000_000
    gs = [synth.lognormal_tensor(n + 1000 * k, -12.0 + k, 2.0, 0.4, seed=40 + k) for k in range(5)]
    kinds = [dict(mode=lgn.MODE_PRUNE, S=0.8), dict(mode=lgn.MODE_QUANTIZE, nbits=6, rounding=lgn.ROUND_STOCHASTIC),
             dict(mode=lgn.MODE_PRUNE, S=0.6), dict(mode=lgn.MODE_PRUNE, S=0.9),
             dict(mode=lgn.MODE_QUANTIZE, nbits=5, rounding=lgn.ROUND_NEAREST)]

    def out_like(g, kd, device):
        if kd["mode"] == lgn.MODE_PRUNE:
            return torch.empty(g.shape, dtype=g.dtype, device=device)
        return torch.zeros(lgn.lgn_codes_bytes(g.numel(), kd["nbits"]), dtype=torch.uint8, device=device)

    hin = [g.pin_memory() for g in gs]
    hout = [out_like(g, kd, "cpu").pin_memory() for g, kd in zip(gs, kinds)]
    hl = [lgn.make_host_layer(a, b, kd["mode"], seed=7 + k, **{x: y for x, y in kd.items() if x != "mode"})
          for k, (a, b, kd) in enumerate(zip(hin, hout, kinds))]
    buf = torch.empty(lgn.lgn_host_staging_bytes(hl) + 256, dtype=torch.uint8, device="cuda")
    buf = buf[(-buf.data_ptr()) % 256:]
    res_h = lgn.lgn_compress_layers_host(hl, buf)

    dg = [g.cuda() for g in gs]
    dout = [out_like(g, kd, "cuda") for g, kd in zip(dg, kinds)]
    dl = [lgn.make_layer(a, b, kd["mode"], seed=7 + k, **{x: y for x, y in kd.items() if x != "mode"})
          for k, (a, b, kd) in enumerate(zip(dg, dout, kinds))]
    res = lgn.new_results(5, "cuda")
    lgn.lgn_compress_layers(dl, res, lgn.new_workspace([g.numel() for g in dg], "cuda"))
    torch.cuda.synchronize()
    res_d = lgn.read_results(res, 5)
    for k in range(5):
        assert res_h[k]["status"] == 0
        for key in ("n", "nnz", "tau", "fmt"):
            assert res_h[k][key] == res_d[k][key], (k, key)
        assert abs(res_h[k]["mu"] - res_d[k]["mu"]) <= 1e-9 * abs(res_d[k]["mu"])
        assert torch.equal(hout[k].view(torch.uint8), dout[k].cpu().view(torch.uint8)), k
