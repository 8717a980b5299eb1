"""Globally consistent statistics across data-parallel ranks: the host-side combine and
the all-reduce step, run as two gloo ranks on CPU.  Each rank holds half of a tensor;
the combined (mu, sigma) must be the oracle's statistics of the whole tensor."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def local_sums(orc, g_np):
    """What lgn_stats reports for a tensor, formed from the oracle's mean and deviation."""
    st = orc.stats(g_np)
    return {"n": st["n"], "nnz": st["nnz"], "sum_ln": st["mu"] * st["nnz"],
            "sum_ln2": (st["sigma"] ** 2 + st["mu"] ** 2) * st["nnz"]}


def test_combine_stats_matches_the_whole_tensor(lgn, oracle):
    from paper_2006_08173_b200 import synth
    g = synth.as_numpy_bits(synth.lognormal_tensor(300_001, -12.0, 2.0, 0.4, seed=5))
    cuts = [0, 1, 70_000, 70_000, 210_017, 300_001]                 # includes an empty part and a one-element part
    parts = [local_sums(oracle, g[a:b]) for a, b in zip(cuts[:-1], cuts[1:])]
    got = lgn.lgn_combine_stats(parts)
    want = oracle.stats(g)
    assert got["n"] == want["n"] and got["nnz"] == want["nnz"]
    assert got["mu"] == pytest.approx(want["mu"], rel=1e-12)
    assert got["sigma"] == pytest.approx(want["sigma"], rel=1e-10)
    assert lgn.lgn_combine_stats([]) == {"n": 0, "nnz": 0, "sum_ln": 0.0, "sum_ln2": 0.0, "mu": 0.0, "sigma": 0.0}
    with pytest.raises(lgn.LgnError):
        lgn.lgn_combine_stats([{"n": 1, "nnz": 2, "sum_ln": 0.0, "sum_ln2": 0.0}])
    with pytest.raises(lgn.LgnError):
        lgn.lgn_combine_stats([{"n": 2, "nnz": 1, "sum_ln": float("nan"), "sum_ln2": 0.0}])
    assert lgn.raw().lgn_combine_stats(None, 0, None) == 1


def _rank_main(rank, world, port, ret):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle as orc
        from paper_2006_08173_b200 import binding as lgn
        from paper_2006_08173_b200 import global_stats, synth
        layers = [synth.as_numpy_bits(synth.lognormal_tensor(n, mu, sg, p, seed=k))
                  for k, (n, mu, sg, p) in enumerate([(200_000, -12.0, 2.0, 0.4), (50_001, -9.0, 1.5, 0.0), (64, -14.0, 3.0, 0.5)])]
        mine = [g[rank::world] for g in layers]                      # this rank's slice of every layer
        combined = global_stats.allreduce_stats([local_sums(orc, g) for g in mine])
        ok = True
        for c, g in zip(combined, layers):
            want = orc.stats(g)
            ok &= c["n"] == want["n"] and c["nnz"] == want["nnz"]
            ok &= abs(c["mu"] - want["mu"]) <= 1e-12 * abs(want["mu"])
            ok &= abs(c["sigma"] - want["sigma"]) <= 1e-10 * want["sigma"]
            # every rank derives the same threshold and format from the combined record
            tau = lgn.lgn_threshold(c["mu"], c["sigma"], 1.0 - c["nnz"] / c["n"], 0.8)
            ok &= tau == orc.threshold(want["mu"], want["sigma"], want["zero_frac"], 0.8) or \
                abs(tau / orc.threshold(want["mu"], want["sigma"], want["zero_frac"], 0.8) - 1.0) < 1e-9
            taus = [None] * world
            dist.all_gather_object(taus, tau)
            ok &= len(set(taus)) == 1
        ok &= global_stats.rank_seed(7, 0) != global_stats.rank_seed(7, 1)
        ret[rank] = bool(ok)
    finally:
        dist.destroy_process_group()


def test_allreduce_stats_two_gloo_ranks(lgn, oracle):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    ret = ctx.Manager().dict()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, ret)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=240)
        assert p.exitcode == 0
    assert dict(ret) == {0: True, 1: True}
