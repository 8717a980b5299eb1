"""Two grouped calls (and a prefix encoder) in flight at once on different streams, each
with its own workspace.  The persistent kernels size their grids to fill the GPU, so the
second kernel's CTAs become resident only as the first one's retire: every device-side wait
must still end, because a CTA only ever waits for work that a running CTA of its own kernel
has already taken.  All outputs must equal those of the same calls run one after the other."""
import numpy as np
import pytest
import torch

from paper_2006_08173_b200 import synth

pytestmark = pytest.mark.gpu


def group(lgn, tensors, mode, **kw):
    outs = []
    layers = []
    for k, g in enumerate(tensors):
        if mode == lgn.MODE_PRUNE:
            o = torch.empty_like(g)
        else:
            o = torch.zeros(lgn.lgn_codes_bytes(g.numel(), kw["nbits"]), dtype=torch.uint8, device=g.device)
        outs.append(o)
        layers.append(lgn.make_layer(g, o, mode, seed=11 + k, **kw))
    ws = lgn.new_workspace([g.numel() for g in tensors], tensors[0].device)
    res = lgn.new_results(len(tensors), tensors[0].device)
    return layers, outs, ws, res


def test_two_grouped_calls_and_an_encoder_overlap(lgn):
    a = [synth.lognormal_tensor(6_000_000 + 777 * k, -12.0, 2.0, 0.4, seed=k, device="cuda") for k in range(4)]
    b = [synth.lognormal_tensor(5_000_000 + 333 * k, -10.0, 2.5, 0.5, seed=10 + k, dtype=torch.bfloat16, device="cuda") for k in range(4)]
    c = synth.lognormal_tensor(3_000_001, -9.0, 2.0, 0.4, seed=99, device="cuda")

    def run(streams):
        la, oa, wa, ra = group(lgn, a, lgn.MODE_PRUNE, S=0.85)
        lb, ob, wb, rb = group(lgn, b, lgn.MODE_QUANTIZE, nbits=6, rounding=lgn.ROUND_STOCHASTIC)
        n = c.numel()
        sd = torch.zeros(lgn.lgn_prefix_bound_words(n, lgn.F32), dtype=torch.int32, device="cuda")
        od = torch.zeros(lgn.lgn_prefix_blocks(n) + 1, dtype=torch.int64, device="cuda")
        wc = torch.empty(lgn.lgn_prefix_workspace_bytes(n), dtype=torch.uint8, device="cuda")
        torch.cuda.synchronize()
        for rep in range(3):                                   # several rounds, so that the kernels really overlap
            lgn.lgn_compress_layers(la, ra, wa, stream=streams[0])
            lgn.lgn_compress_layers(lb, rb, wb, stream=streams[1])
            lgn.lgn_prefix_encode(c, 3e-4, 5, True, sd, od, wc, stream=streams[2])
        torch.cuda.synchronize()
        ra_, rb_ = lgn.read_results(ra, 4), lgn.read_results(rb, 4)
        assert all(r["status"] == 0 for r in ra_ + rb_)
        words = int(od[-1].item())
        assert 0 < words <= sd.numel()
        return ([o.clone() for o in oa], [o.clone() for o in ob], sd[:words].clone(), od.clone(),
                [(r["nnz"], r["mu"], r["sigma"], r["tau"], r["fmt"]) for r in ra_ + rb_])

    one = torch.cuda.current_stream()
    seq = run([one, one, one])
    par = run([torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()])
    for x, y in zip(seq[0] + seq[1], par[0] + par[1]):
        assert torch.equal(x.view(torch.uint8), y.view(torch.uint8))
    assert torch.equal(seq[2], par[2]) and torch.equal(seq[3], par[3])
    assert seq[4] == par[4]
