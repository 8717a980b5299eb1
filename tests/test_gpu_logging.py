"""LGN_LOG=1 on a GPU machine: the host side reports which kernel, tile size, grid and queue a grouped
call takes, and which selection path a quantile takes; the results are the same with and without it."""
import os
import re
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CODE = """
import torch
from paper_2006_08173_b200 import binding as lgn, synth
g = synth.lognormal_tensor(300_001, -12.0, 2.0, 0.4, seed=3, device="cuda")
h = synth.lognormal_tensor(70_000, -10.0, 1.5, 0.2, seed=4, device="cuda")
outs = [torch.empty_like(g), torch.empty_like(h)]
layers = [lgn.make_layer(g, outs[0], lgn.MODE_PRUNE, S=0.8, seed=1), lgn.make_layer(h, outs[1], lgn.MODE_PRUNE, S=0.5, seed=2)]
ws = lgn.new_workspace([g.numel(), h.numel()], "cuda")
res = lgn.new_results(2, "cuda")
lgn.lgn_compress_layers(layers, res, ws)
torch.cuda.synchronize()
print([r["tau"] for r in lgn.read_results(res, 2)], int(outs[0].count_nonzero()), int(outs[1].count_nonzero()))
print(lgn.lgn_quantile(g, 0.997))
big = synth.lognormal_tensor(2 ** 24 + 3, -12.0, 2.0, 0.4, seed=5, dtype=torch.bfloat16, device="cuda")
print(lgn.lgn_quantile(big, 0.997))
try:
    lgn.lgn_compress_layers([lgn.make_layer(g, outs[0], lgn.MODE_PRUNE, S=1.5, seed=1)], res, ws)
except lgn.LgnError as e:
    print("refused", e.code)
"""


def run(extra):
    env = dict(os.environ)
    env.pop("LGN_LOG", None)
    env.update(extra)
    return subprocess.run([sys.executable, "-c", CODE], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)


def test_log_lines_of_a_grouped_call_and_a_quantile():
    quiet, loud = run({}), run({"LGN_LOG": "1"})
    assert quiet.returncode == 0 and loud.returncode == 0, (quiet.stderr[-2000:], loud.stderr[-2000:])
    assert "[lgn]" not in quiet.stderr
    assert loud.stdout == quiet.stdout                               # logging changes no result
    lines = [l for l in loud.stderr.splitlines() if l.startswith("[lgn] ")]
    grouped = [l for l in lines if l.startswith("[lgn] grouped call: 2 layers, 370001 elements; kernel: specialised")]
    assert len(grouped) == 1
    assert "of fp32" in grouped[0] and "x 256 threads" in grouped[0] and "counters off" in grouped[0]
    tile = int(re.search(r"tiles of (\d+) elements", grouped[0]).group(1))
    assert tile in (8192, 32768)                                     # a call this small takes the small tiles
    items = 2 * (-(-300_001 // tile) + -(-70_000 // tile))           # every tile once for statistics, once for apply
    assert f"{items} queue items in" in grouped[0]
    assert any("quantile: n=300001 fp32" in l and "radix selection (tensor below 2^24 elements)" in l for l in lines)
    assert any("quantile: n=16777219 bf16" in l and "one read around a bracket from a sample" in l for l in lines)
    assert any("quantile: sample of 2097152 elements" in l for l in lines)
    assert any("layer 0 of 1 refused: " in l and "S=1.5" in l for l in lines)
