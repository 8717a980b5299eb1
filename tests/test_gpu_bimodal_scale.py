"""GPU parity of the two variants of the grouped call: bi-modal pruning driven by a
right-mode mask (appendix "Algorithm for bi-modal lognormal pruning") and the scale
taken from the tensor's maximum (Algorithm 1), against the oracle."""
import numpy as np
import pytest
import torch

from gpu_helpers import REL_TOL, assert_same_bits, assert_same_codes, np_bits
from paper_2006_08173_b200 import synth

pytestmark = pytest.mark.gpu

DTYPES = [torch.float32, torch.bfloat16]
SIZES = [1, 3, 1023, 40_000, 2 ** 20 + 7]


def close(got, want):
    assert got["nnz"] == want["nnz"]
    scale = max(abs(want["mu"]), want["sigma"], 1e-300)
    small = want["nnz"] <= 3                                   # one to three samples: 1e-5 of max(|mu|, 1), 1e-4 absolute on sigma
    assert abs(got["mu"] - want["mu"]) <= REL_TOL * (max(abs(want["mu"]), 1.0) if small else scale)
    assert abs(got["sigma"] - want["sigma"]) <= (1e-4 if small else REL_TOL * max(want["sigma"], 1e-300)) \
        or (want["sigma"] == 0.0 and got["sigma"] <= 1e-6)


def one_call(lgn, layers, n_per_layer, dev):
    ws = lgn.new_workspace(n_per_layer, dev)
    ws.fill_(0xCD)
    res = lgn.new_results(len(layers), dev)
    lgn.lgn_compress_layers(layers, res, ws)
    torch.cuda.synchronize()
    return lgn.read_results(res, len(layers))


def oracle_max_f32(oracle, g_np):
    return float(np.float32(oracle.max_abs(g_np)))


# ------------------------------------------------------------------ bi-modal pruning
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("n", SIZES)
def test_bimodal_prune_parity(lgn, oracle, dtype, n):
    g, mask = synth.bimodal_tensor(n, -9.0, 1.5, -17.0, 1.0, 0.5, seed=n % 91, dtype=dtype, device="cuda")
    g_np, m_np = np_bits(g), mask.cpu().numpy()
    st = oracle.stats_masked(g_np, m_np)
    dt = oracle.BF16 if dtype == torch.bfloat16 else oracle.F32
    for S in (0.8, 0.97):
        # free-running: the library's own statistics
        out = torch.empty_like(g)
        r = one_call(lgn, [lgn.make_layer(g, out, lgn.MODE_PRUNE, S=S, seed=3, right_mode=mask)], [n], g.device)[0]
        assert r["status"] == 0 and r["n_right_mode"] == st["n_right"] and r["n"] == n
        close(r, st)
        assert r["max_abs"] == oracle_max_f32(oracle, g_np)
        # with the oracle's mu, sigma: threshold and every output bit identical
        out = torch.empty_like(g)
        r = one_call(lgn, [lgn.make_layer(g, out, lgn.MODE_PRUNE, S=S, seed=3, right_mode=mask,
                                          mu_override=st["mu"], sigma_override=st["sigma"])], [n], g.device)[0]
        tau = oracle.snap_tau(oracle.threshold(st["mu"], st["sigma"], st["zero_frac"], S), dt) if st["nnz"] else 0.0
        assert r["tau"] == tau
        assert_same_bits(out, oracle.prune(g_np, tau, 3))


def test_bimodal_prune_reaches_the_requested_sparsity(lgn):
    n = 4_000_000
    g, mask = synth.bimodal_tensor(n, -9.0, 1.5, -17.0, 1.0, 0.5, seed=2, device="cuda")
    out = torch.empty_like(g)
    r = one_call(lgn, [lgn.make_layer(g, out, lgn.MODE_PRUNE, S=0.85, seed=8, right_mode=mask)], [n], g.device)[0]
    achieved = float((out == 0).float().mean())
    assert abs(achieved - 0.85) < 5e-3
    # without the mask the two modes are fitted as one wide lognormal and the sparsity misses
    out2 = torch.empty_like(g)
    one_call(lgn, [lgn.make_layer(g, out2, lgn.MODE_PRUNE, S=0.85, seed=8)], [n], g.device)
    assert abs(float((out2 == 0).float().mean()) - 0.85) > 2e-2


def test_mask_edge_cases(lgn, oracle):
    n = 70_001
    g, _ = synth.bimodal_tensor(n, -9.0, 1.5, -17.0, 1.0, 0.5, seed=4, device="cuda")
    g_np = np_bits(g)
    for mask in (torch.zeros(n, dtype=torch.uint8, device="cuda"),            # no right mode: nothing measured
                 torch.ones(n, dtype=torch.bool, device="cuda"),              # all right mode: same as no mask
                 (torch.arange(n, device="cuda") % 3 == 0).to(torch.uint8) * 200):
        st = oracle.stats_masked(g_np, mask.cpu().numpy().astype(np.uint8))
        out = torch.empty_like(g)
        r = one_call(lgn, [lgn.make_layer(g, out, lgn.MODE_PRUNE, S=0.9, seed=1, right_mode=mask,
                                          mu_override=st["mu"], sigma_override=st["sigma"])], [n], g.device)[0]
        assert r["n_right_mode"] == st["n_right"] and r["nnz"] == st["nnz"]
        tau = oracle.snap_tau(oracle.threshold(st["mu"], st["sigma"], st["zero_frac"], 0.9), oracle.F32) if st["nnz"] else 0.0
        assert r["tau"] == tau
        assert_same_bits(out, oracle.prune(g_np, tau, 1))
    # a right-mode entry that is exactly zero counts in l but not in mu, sigma
    g2 = g.clone()
    g2[::5] = 0.0
    mask = torch.ones(n, dtype=torch.uint8, device="cuda")
    st = oracle.stats_masked(np_bits(g2), mask.cpu().numpy())
    r = one_call(lgn, [lgn.make_layer(g2, torch.empty_like(g2), lgn.MODE_PRUNE, S=0.5, seed=1, right_mode=mask)], [n], g.device)[0]
    assert r["n_right_mode"] == n and r["nnz"] == st["nnz"] < n
    close(r, st)


# ------------------------------------------------------------------ scale from the maximum
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("n", SIZES)
def test_max_scale_quantise_parity(lgn, oracle, dtype, n):
    g = synth.lognormal_tensor(n, -12.0, 2.5, 0.4, seed=n % 89 + 2, dtype=dtype, device="cuda")
    g_np = np_bits(g)
    st = oracle.stats(g_np)
    mx = oracle.max_abs(g_np)
    for nbits, rounding in [(6, 1), (5, 0), (4, 1), (8, 0)]:
        out = torch.full((max(16, lgn.lgn_codes_bytes(n, nbits)) + 16,), 0xAB, dtype=torch.uint8, device="cuda")
        r = one_call(lgn, [lgn.make_layer(g, out, lgn.MODE_QUANTIZE, nbits=nbits, rounding=rounding, seed=6,
                                          scale_mode=lgn.SCALE_FROM_MAX, mu_override=st["mu"],
                                          sigma_override=st["sigma"])], [n], g.device)[0]
        assert r["status"] == 0
        assert r["max_abs"] == float(np.float32(mx))
        fmt = oracle.fp_format_max_scale(st["mu"], st["sigma"], st["nnz"], nbits, mx)
        assert r["fmt"] == fmt
        if st["nnz"]:
            assert lgn.lgn_scale_from_max(mx, fmt["exp_bits"]) == fmt["scale_exp"]
        ref = oracle.pack(oracle.quantize(g_np, fmt["exp_bits"], fmt["man_bits"], fmt["scale_exp"], rounding, 6), nbits)
        assert_same_codes(out, ref)
        assert bool((out[max(16, lgn.lgn_codes_bytes(n, nbits)):] == 0xAB).all())


@pytest.mark.parametrize("dtype", DTYPES)
def test_max_scale_extremes(lgn, oracle, dtype):
    cases = [synth.lognormal_tensor(50_001, -85.0, 4.0, 0.3, seed=1, dtype=dtype, device="cuda"),     # subnormal range
             synth.lognormal_tensor(50_001, 3.0, 2.0, 0.5, seed=2, dtype=dtype, device="cuda", clip=1e4),
             torch.zeros(9_000, dtype=dtype, device="cuda"),
             torch.tensor([0.0, -2.0 ** -20, 0.0], dtype=dtype, device="cuda")]
    for g in cases:
        n = g.numel()
        g_np = np_bits(g)
        st = oracle.stats(g_np)
        mx = oracle.max_abs(g_np)
        out = torch.empty(max(16, lgn.lgn_codes_bytes(n, 6)), dtype=torch.uint8, device="cuda")
        r = one_call(lgn, [lgn.make_layer(g, out, lgn.MODE_QUANTIZE, nbits=6, rounding=1, seed=2,
                                          scale_mode=lgn.SCALE_FROM_MAX, mu_override=st["mu"],
                                          sigma_override=st["sigma"])], [n], g.device)[0]
        fmt = oracle.fp_format_max_scale(st["mu"], st["sigma"], st["nnz"], 6, mx)
        assert r["fmt"] == fmt
        ref = oracle.pack(oracle.quantize(g_np, fmt["exp_bits"], fmt["man_bits"], fmt["scale_exp"], 1, 2), 6)
        assert_same_codes(out, ref)


# ------------------------------------------------------------------ a mixed group, and the host-buffer form
def test_mixed_group(lgn, oracle):
    dev = torch.device("cuda")
    gb, mask = synth.bimodal_tensor(150_003, -9.0, 1.5, -17.0, 1.0, 0.45, seed=5, dtype=torch.bfloat16, device="cuda")
    gp = synth.lognormal_tensor(90_000, -11.0, 2.0, 0.4, seed=6, device="cuda")
    gq = synth.lognormal_tensor(120_001, -13.0, 3.0, 0.5, seed=7, dtype=torch.bfloat16, device="cuda")
    ob, op = torch.empty_like(gb), torch.empty_like(gp)
    oq1 = torch.empty(lgn.lgn_codes_bytes(gq.numel(), 5) + 16, dtype=torch.uint8, device=dev)
    oq2 = torch.empty(lgn.lgn_codes_bytes(gq.numel(), 5) + 16, dtype=torch.uint8, device=dev)
    sb = oracle.stats_masked(np_bits(gb), mask.cpu().numpy())
    sp, sq = oracle.stats(np_bits(gp)), oracle.stats(np_bits(gq))
    layers = [lgn.make_layer(gb, ob, lgn.MODE_PRUNE, S=0.9, seed=1, right_mode=mask, mu_override=sb["mu"], sigma_override=sb["sigma"]),
              lgn.make_layer(gp, op, lgn.MODE_PRUNE, S=0.7, seed=2, mu_override=sp["mu"], sigma_override=sp["sigma"]),
              lgn.make_layer(gq, oq1, lgn.MODE_QUANTIZE, nbits=5, rounding=1, seed=3, scale_mode=lgn.SCALE_FROM_MAX,
                             mu_override=sq["mu"], sigma_override=sq["sigma"]),
              lgn.make_layer(gq, oq2, lgn.MODE_QUANTIZE, nbits=5, rounding=1, seed=3, mu_override=sq["mu"], sigma_override=sq["sigma"])]
    res = one_call(lgn, layers, [gb.numel(), gp.numel(), gq.numel(), gq.numel()], dev)
    assert [r["status"] for r in res] == [0, 0, 0, 0]
    tb = oracle.snap_tau(oracle.threshold(sb["mu"], sb["sigma"], sb["zero_frac"], 0.9), oracle.BF16)
    tp = oracle.snap_tau(oracle.threshold(sp["mu"], sp["sigma"], sp["zero_frac"], 0.7), oracle.F32)
    assert res[0]["tau"] == tb and res[1]["tau"] == tp
    assert_same_bits(ob, oracle.prune(np_bits(gb), tb, 1))
    assert_same_bits(op, oracle.prune(np_bits(gp), tp, 2))
    f1 = oracle.fp_format_max_scale(sq["mu"], sq["sigma"], sq["nnz"], 5, oracle.max_abs(np_bits(gq)))
    f2 = oracle.fp_format(sq["mu"], sq["sigma"], sq["nnz"], 5)
    assert res[2]["fmt"] == f1 and res[3]["fmt"] == f2 and f1["scale_exp"] != f2["scale_exp"]
    for out, f in ((oq1, f1), (oq2, f2)):
        assert_same_codes(out, oracle.pack(oracle.quantize(np_bits(gq), f["exp_bits"], f["man_bits"], f["scale_exp"], 1, 3), 5))
    assert res[1]["max_abs"] == 0.0 and res[1]["n_right_mode"] == 0          # not measured for plain layers


def test_host_buffer_form_with_a_mask(lgn, oracle):
    n = 100_003
    g, mask = synth.bimodal_tensor(n, -9.0, 1.5, -17.0, 1.0, 0.5, seed=9)
    gh, mh = g.pin_memory(), mask.pin_memory()
    oh = torch.empty_like(gh).pin_memory()
    layers = [lgn.make_host_layer(gh, oh, lgn.MODE_PRUNE, S=0.8, seed=4, right_mode=mh)]
    buf = torch.empty(lgn.lgn_host_staging_bytes(layers) + 256, dtype=torch.uint8, device="cuda")
    buf = buf[(-buf.data_ptr()) % 256:]
    r = lgn.lgn_compress_layers_host(layers, buf)[0]
    st = oracle.stats_masked(np_bits(g), mask.numpy())
    assert r["n_right_mode"] == st["n_right"]
    close(r, st)
    assert_same_bits(oh, oracle.prune(np_bits(g), r["tau"], 4))
