"""The multi-rank plumbing of bench.py on CPU (gloo, world size 2): the path has
no exchange step, every rank runs its own replica, and only the timing is
reduced (max over ranks)."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, %(root)r)
import torch
import bench
world, rank, local = bench.dist_setup(2)
assert world == 2 and rank == int(os.environ["RANK"])
bench.barrier(world)
slowest = bench.max_over_ranks(1.5 + rank, world, torch.device("cpu"))
w, specs = bench.workload_specs("resnet18_bs256_fp32_prune", 256, rank)
bench.barrier(world)
print(json.dumps({"rank": rank, "slowest": slowest, "layers": len(specs),
                  "mu0": specs[0].mu, "seed0": specs[0].data_seed,
                  "elements": sum(s.numel for s in specs)}))
import torch.distributed as dist
dist.destroy_process_group()
"""


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_ranks_reduce_only_the_timing():
    port = free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER % {"root": ROOT}], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda d: d["rank"])
    assert [o["slowest"] for o in outs] == [2.5, 2.5]                 # max over ranks, seen by both
    assert outs[0]["layers"] == outs[1]["layers"] == 20
    assert outs[0]["elements"] == outs[1]["elements"] == 635_830_272  # weak scaling: same work per rank
    assert outs[0]["seed0"] != outs[1]["seed0"] and outs[0]["mu0"] != outs[1]["mu0"]   # its own micro-batch


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
               MASTER_PORT=str(free_port()), CUDA_VISIBLE_DEVICES="")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "3"], env=env, capture_output=True, text=True, timeout=180)
    assert p.returncode == 0 and p.stdout.strip() == ""               # exits without work, prints nothing
    env0 = dict(os.environ, CUDA_VISIBLE_DEVICES="")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "3", "--ref-sample-elems", "2000000", "--batch", "8"],
                       env=env0, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0, p.stderr[-2000:]
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
