"""Failure detection without a fault: a device-side wait whose condition never
comes true must run out, report LGN_ERR_TIMEOUT for the layer it belongs to, let
the other layers finish, and leave the context usable."""
import time

import numpy as np
import pytest
import torch

from gpu_helpers import np_bits
from paper_2006_08173_b200 import synth

pytestmark = pytest.mark.gpu


def test_wait_runs_out_and_is_reported(lgn, oracle):
    a = synth.lognormal_tensor(300_000, -12.0, 2.0, 0.4, seed=31, device="cuda")
    b = synth.lognormal_tensor(200_000, -10.0, 2.5, 0.5, seed=32, device="cuda")
    oa = torch.full_like(a, 7.0)
    ob = torch.empty_like(b)
    layers = [lgn.make_layer(a, oa, lgn.MODE_PRUNE, S=0.8, seed=1),
              lgn.make_layer(b, ob, lgn.MODE_PRUNE, S=0.9, seed=2)]
    ws = lgn.new_workspace([a.numel(), b.numel()], a.device)
    res = lgn.new_results(2, a.device)
    t0 = time.time()
    lgn.lgn_selftest_wait_expires(layers, res, ws)
    torch.cuda.synchronize()                                   # returns: nothing hung
    elapsed = time.time() - t0
    r = lgn.read_results(res, 2)
    assert r[0]["status"] == 5                                 # LGN_ERR_TIMEOUT
    assert r[1]["status"] == 0
    assert 0.05 < elapsed < 30.0
    assert bool((oa == 7.0).all())                             # the timed-out layer wrote nothing
    # the other layer is complete and right
    st = oracle.stats(np_bits(b))
    assert r[1]["nnz"] == st["nnz"]
    res2 = lgn.new_results(2, a.device)
    ob2 = torch.empty_like(b)
    oa2 = torch.empty_like(a)
    layers2 = [lgn.make_layer(a, oa2, lgn.MODE_PRUNE, S=0.8, seed=1),
               lgn.make_layer(b, ob2, lgn.MODE_PRUNE, S=0.9, seed=2)]
    lgn.lgn_compress_layers(layers2, res2, ws)                 # the context and the workspace are still good
    torch.cuda.synchronize()
    r2 = lgn.read_results(res2, 2)
    assert r2[0]["status"] == 0 and r2[1]["status"] == 0
    assert torch.equal(ob, ob2)
    assert abs(float((oa2 == 0).float().mean()) - 0.8) < 5e-3


def test_a_time_out_stays_with_its_own_layer(lgn):
    """Four layers; layer 0 never completes.  Layer 1 is large enough (120 MB) for the
    queue to place the statistics of layers 2 and 3 behind layer 0's apply tiles, so they
    are still to run when layer 0's waiters give up: they, and layer 1, must come back
    LGN_OK and bit for bit what a normal call writes."""
    sizes = [1_000_000, 30_000_000, 8_000_000, 8_000_003]
    gs = [synth.lognormal_tensor(n, -12.0 + k, 2.0, 0.4, seed=40 + k, device="cuda") for k, n in enumerate(sizes)]
    S = [0.8, 0.7, 0.9, 0.85]

    def run(call):
        outs = [torch.full_like(g, 7.0) for g in gs]
        layers = [lgn.make_layer(g, o, lgn.MODE_PRUNE, S=s, seed=10 + k) for k, (g, o, s) in enumerate(zip(gs, outs, S))]
        ws = lgn.new_workspace(sizes, "cuda")
        res = lgn.new_results(len(gs), "cuda")
        call(layers, res, ws)
        torch.cuda.synchronize()
        return outs, lgn.read_results(res, len(gs))

    good_out, good = run(lgn.lgn_compress_layers)
    assert all(r["status"] == 0 for r in good)
    t0 = time.time()
    outs, r = run(lgn.lgn_selftest_wait_expires)
    assert time.time() - t0 < 30.0
    assert r[0]["status"] == 5 and bool((outs[0] == 7.0).all())
    for k in (1, 2, 3):
        assert r[k]["status"] == 0, k
        assert r[k] == good[k]
        assert torch.equal(outs[k].view(torch.int32), good_out[k].view(torch.int32)), k
