#!/usr/bin/env python
"""Benchmark of the fused statistics -> closed form -> apply path.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One step = one grouped call (lgn_compress_layers) over every tensor of the
workload.  The default workload is the ResNet-18 backward pass at batch 256 in
fp32: 20 conv-output gradient tensors, 635.8 M elements, pruned with per-layer
sparsity.  Inputs are synthetic (seeded lognormal magnitudes with exact zeros)
and resident in HBM before the clock starts.  With N > 1 (torchrun) every rank
runs its own replica of the workload (its own micro-batch); there is no
data-path exchange between ranks.

Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2006_08173_b200 import synth  # noqa: E402

FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0

# algorithmic bytes per element: read for the statistics, read again for the
# apply pass, write the result
def bytes_per_elem(dtype_bytes: int, mode: str, nbits: int = 6) -> float:
    return 2 * dtype_bytes + (dtype_bytes if mode == "prune" else nbits / 8.0)


WORKLOADS = {
    # name: (builder, dtype, mode, nbits, rounding)
    "resnet18_bs256_fp32_prune": dict(net="resnet18", dtype="f32", mode="prune"),
    "resnet18_bs256_fp32_fp6": dict(net="resnet18", dtype="f32", mode="quant", nbits=6, rounding=1),
    "resnet50_bs256_bf16_fp6": dict(net="resnet50", dtype="bf16", mode="quant", nbits=6, rounding=1),
    "resnet50_bs256_bf16_fp5": dict(net="resnet50", dtype="bf16", mode="quant", nbits=5, rounding=1),
    "resnet50_bs256_bf16_prune": dict(net="resnet50", dtype="bf16", mode="prune"),
}
for _dt in ("fp32", "bf16"):
    for _lg in (20, 24, 26, 28, 30):
        WORKLOADS[f"flat_2p{_lg}_{_dt}_prune"] = dict(net="flat", log2n=_lg, dtype="f32" if _dt == "fp32" else "bf16",
                                                      mode="prune")
        WORKLOADS[f"flat_2p{_lg}_{_dt}_fp6"] = dict(net="flat", log2n=_lg, dtype="f32" if _dt == "fp32" else "bf16",
                                                    mode="quant", nbits=6, rounding=1)


# Steps next to the path (not bench lines: timed for the tables in profiles/):
# the decoder of a packed code stream and the prefix-code encoder, on flat tensors.
for _lg in (26, 28):
    for _odt in ("fp32", "bf16"):
        WORKLOADS[f"dequant_fp6_to_{_odt}_2p{_lg}"] = dict(net="aux", kind="dequant", log2n=_lg, nbits=6,
                                                           dtype="f32" if _odt == "fp32" else "bf16", mode="dequant")
    for _dt in ("fp32", "bf16"):
        WORKLOADS[f"bimodal_prune_{_dt}_2p{_lg}"] = dict(net="aux", kind="bimodal", log2n=_lg,
                                                         dtype="f32" if _dt == "fp32" else "bf16", mode="prune")
        WORKLOADS[f"max_scale_fp6_{_dt}_2p{_lg}"] = dict(net="aux", kind="maxscale", log2n=_lg, nbits=6,
                                                         dtype="f32" if _dt == "fp32" else "bf16", mode="quant")
        for _k in ("stats", "apply_prune", "apply_fp6"):           # the entry points of the steady-state iterations
            WORKLOADS[f"{_k}_{_dt}_2p{_lg}"] = dict(net="aux", kind=_k, log2n=_lg, nbits=6,
                                                    dtype="f32" if _dt == "fp32" else "bf16", mode=_k)
        WORKLOADS[f"quantile_{_dt}_2p{_lg}"] = dict(net="aux", kind="quantile", log2n=_lg,
                                                    dtype="f32" if _dt == "fp32" else "bf16", mode="quantile")
        WORKLOADS[f"prefix_decode_{_dt}_2p{_lg}"] = dict(net="aux", kind="prefix", decode=True, log2n=_lg,
                                                         dtype="f32" if _dt == "fp32" else "bf16", mode="prefix")
        WORKLOADS[f"prefix_encode_{_dt}_2p{_lg}"] = dict(net="aux", kind="prefix", log2n=_lg,
                                                         dtype="f32" if _dt == "fp32" else "bf16", mode="prefix")
for _dt in ("fp32", "bf16"):
    WORKLOADS[f"quantile_{_dt}_2p30"] = dict(net="aux", kind="quantile", log2n=30,
                                             dtype="f32" if _dt == "fp32" else "bf16", mode="quantile")


def workload_specs(name: str, batch: int, seed: int):
    w = WORKLOADS[name]
    if w["net"] == "resnet18":
        specs = synth.resnet18_prune_workload(batch, seed)
    elif w["net"] == "resnet50":
        specs = synth.resnet50_quant_workload(batch, seed)
        if w["mode"] == "prune":
            import numpy as np
            rs = np.random.RandomState(seed + 1)
            for s in specs:
                s.sparsity = float(rs.choice([0.5, 0.7, 0.85, 0.9]))
    else:
        specs = [synth.LayerSpec("flat", 1 << w["log2n"], -12.0, 2.0, 0.5, 0.85, seed * 1000)]
    return w, specs


def read_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """SM clock and throttle reasons of one GPU, sampled while work runs: NVML polled from a
    thread every few milliseconds (a timed region of 20 ms still gets samples), or
    `nvidia-smi -lms` when NVML's Python module is missing.  Reads settings only."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int, period_s: float = 0.004):
        self.samples = []                # (time, sm_mhz, set of reasons)
        self.max_mhz = None
        self.marks = {}
        self.p = self.f = self.thread = None
        self.how = "nvml"
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            # NVML orders devices by PCI bus id; CUDA_VISIBLE_DEVICES may renumber them
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = index
            if vis:
                ent = [v.strip() for v in vis.split(",") if v.strip()]
                if index < len(ent) and ent[index].isdigit():
                    phys = int(ent[index])
            self.h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.stop_flag = False
            import threading
            self.period = period_s
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
        except Exception:
            self.how = "nvidia-smi"
            self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            try:
                self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                           "-lms", "20", "-i", str(index)], stdout=self.f, stderr=subprocess.DEVNULL)
            except Exception:
                self.p = None

    def _poll(self):
        nv = self.nv
        bits = {"hw_slowdown": nv.nvmlClocksThrottleReasonHwSlowdown,
                "hw_thermal_slowdown": nv.nvmlClocksThrottleReasonHwThermalSlowdown,
                "sw_thermal_slowdown": nv.nvmlClocksThrottleReasonSwThermalSlowdown,
                "sw_power_cap": nv.nvmlClocksThrottleReasonSwPowerCap}
        while not self.stop_flag:
            try:
                mhz = float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                self.samples.append((time.perf_counter(), mhz, {k for k, b in bits.items() if mask & b}))
            except Exception:
                pass
            time.sleep(self.period)

    def mark(self, name: str):
        self.marks[name] = time.perf_counter()

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "how": self.how}
        if self.thread is not None:
            self.stop_flag = True
            self.thread.join(timeout=2)
            t0, t1 = self.marks.get("timed_begin"), self.marks.get("timed_end")
            load = [x for x in self.samples if self.marks.get("load_begin", 0) <= x[0] <= self.marks.get("load_end", 1e300)]
            timed = [x for x in load if t0 is not None and t1 is not None and t0 <= x[0] <= t1]
            if load:
                reasons = set()
                for x in load:
                    reasons |= x[2]
                out.update(sm_mhz=statistics.median(x[1] for x in load), sm_max_mhz=self.max_mhz, samples=len(load),
                           samples_in_timed_region=len(timed), reasons=sorted(reasons))
                if timed:
                    out["sm_mhz_timed_region"] = statistics.median(x[1] for x in timed)
            return out
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
            except ValueError:
                continue
            for nm, v in zip(self.NAMES, parts[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        os.unlink(self.f.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


def dist_setup(n_gpus: int):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl" if torch.cuda.is_available() else "gloo")
    return world, rank, local


def max_over_ranks(x: float, world: int, device) -> float:
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


# --------------------------------------------------------------------------- reference arm = the oracle
def oracle_sample(specs, w, budget_elems: int):
    """The trailing layers of the workload, up to about budget_elems elements."""
    chosen, total = [], 0
    for s in reversed(specs):
        if chosen and total + s.numel > budget_elems:
            break
        chosen.append(s)
        total += s.numel
    return list(reversed(chosen)), total


def oracle_step(orc, arrays, specs, w):
    """One pass of the whole path (statistics, closed form, apply) in the oracle."""
    for g, s in zip(arrays, specs):
        st = orc.stats(g)
        dt = orc.BF16 if g.dtype.itemsize == 2 else orc.F32
        if w["mode"] == "prune":
            tau = orc.snap_tau(orc.threshold(st["mu"], st["sigma"], st["zero_frac"], s.sparsity), dt) if st["nnz"] else 0.0
            orc.prune(g, tau, 1)
        else:
            f = orc.fp_format(st["mu"], st["sigma"], st["nnz"], w["nbits"])
            codes = orc.quantize(g, f["exp_bits"], f["man_bits"], f["scale_exp"], w["rounding"], 1)
            orc.pack(codes, w["nbits"])


def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:      # under torchrun only rank 0 works; no process group
        return
    import oracle as orc
    orc.build()
    w, specs = workload_specs(args.workload, args.batch, 0)
    dtype = torch.float32 if w["dtype"] == "f32" else torch.bfloat16
    sample, total = oracle_sample(specs, w, args.ref_sample_elems)
    arrays = [synth.as_numpy_bits(synth.lognormal_tensor(s.numel, s.mu, s.sigma, s.zero_frac, s.data_seed, dtype, "cpu"))
              for s in sample]
    bpe = bytes_per_elem(2 if w["dtype"] == "bf16" else 4, w["mode"], w.get("nbits", 6))
    for _ in range(args.warmup):
        oracle_step(orc, arrays, sample, w)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(orc, arrays, sample, w)
    dt = (time.perf_counter() - t0) / args.steps
    gbs = total * bpe / dt / 1e9
    what = f"last {len(sample)} of {len(specs)} layers of {args.workload} ({total} elements) per step"
    print(json.dumps({
        "impl": "reference", "metric": "fused_stats_apply_algorithmic_GBps", "value": gbs, "unit": "GB/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": w["dtype"], "data": "synthetic",
        "config": {"workload": args.workload, "elements_per_step": total, "sample": what},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": what},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# --------------------------------------------------------------------------- our arm
def build_layers(lgn, w, specs, tensors, outs):
    layers = []
    for k, (g, o, s) in enumerate(zip(tensors, outs, specs)):
        if w["mode"] == "prune":
            layers.append(lgn.make_layer(g, o, lgn.MODE_PRUNE, S=s.sparsity, seed=1000 + k))
        else:
            layers.append(lgn.make_layer(g, o, lgn.MODE_QUANTIZE, nbits=w["nbits"], rounding=w["rounding"], seed=1000 + k))
    return layers


class Prepared:
    """One workload, resident on the device and ready to step."""

    def __init__(self, lgn, name, batch, seed, dev, tensors=None):
        self.name = name
        self.w, self.specs = workload_specs(name, batch, seed)
        w = self.w
        self.dtype = torch.float32 if w["dtype"] == "f32" else torch.bfloat16
        self.esize = 4 if w["dtype"] == "f32" else 2
        self.tensors = tensors if tensors is not None else synth.make_layers(self.specs, self.dtype, str(dev))
        if w["mode"] == "prune":
            self.outs = [torch.empty_like(g) for g in self.tensors]
        else:
            self.outs = [torch.empty(max(16, lgn.lgn_codes_bytes(g.numel(), w["nbits"])), dtype=torch.uint8, device=dev)
                         for g in self.tensors]
        self.layers = build_layers(lgn, w, self.specs, self.tensors, self.outs)
        self.ws = lgn.new_workspace([g.numel() for g in self.tensors], dev)
        self.res = lgn.new_results(len(self.tensors), dev)
        self.total_elems = sum(g.numel() for g in self.tensors)
        self.bpe = bytes_per_elem(self.esize, w["mode"], w.get("nbits", 6))
        self.alg_bytes = self.total_elems * self.bpe
        l2_bytes = torch.cuda.get_device_properties(dev).L2_cache_size
        self.flush = None
        if self.total_elems * self.esize <= 2 * l2_bytes:      # small inputs: flush L2 between timed steps
            self.flush = torch.empty(max(2 * l2_bytes, 256 << 20), dtype=torch.uint8, device=dev)
        self.lgn = lgn

    def step(self):
        self.lgn.lgn_compress_layers(self.layers, self.res, self.ws)

    def warm(self, n):
        for _ in range(n):
            if self.flush is not None:
                self.flush.fill_(1)
            self.step()
        torch.cuda.synchronize()
        status = [r["status"] for r in self.lgn.read_results(self.res, len(self.tensors))]
        if any(status):
            raise SystemExit(f"{self.name}: per-layer status not ok: {status}")

    def timed(self, steps):
        """CUDA-event times of `steps` back-to-back steps on the current stream:
        (device ms of the whole block, per-step ms list)."""
        stream = torch.cuda.current_stream()
        starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        ends = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        for i in range(steps):
            if self.flush is not None:
                self.flush.fill_(1)
            starts[i].record(stream)
            self.step()
            ends[i].record(stream)
        torch.cuda.synchronize()
        per = [a.elapsed_time(b) for a, b in zip(starts, ends)]
        # inputs above L2: the device time of exactly K back-to-back steps; else the flushes
        # between steps are not part of the path
        total = starts[0].elapsed_time(ends[-1]) if self.flush is None else sum(per)
        return total, per


# Roofs of one workload.  HBM: the measured copy rate.  The two instruction roofs come from one ncu
# capture per kind of workload (profiles/issue_ceilings.json: instructions and integer-ALU
# instructions per element): every issue slot used (148 SMs x 4 schedulers x 32 lanes per clock),
# or every lane of the integer ALU pipe used (148 x 64 per clock), at the SM clock sampled during
# the run.  `bound` names the lowest roof: "hbm", or "alu" where the ALU pipe's lies below it
# (bf16 FP6), and `frac` is measured against that roof; `frac_hbm` is always against the copy rate.
SMS, ISSUE_LANES, ALU_LANES = 148, 128, 64


def roofline_of(name, alg_bytes, per_step_ms, sm_mhz=None):
    peak, peak_kind = read_peak()
    kern_ms = statistics.mean(per_step_ms)
    achieved = alg_bytes / (kern_ms * 1e-3) / 1e9
    r = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
         "traffic": None, "peak_kind": f"of {peak_kind}", "frac_hbm": achieved / peak,
         "frac_of_nominal_8TBps": achieved / NOMINAL_HBM_GBS,
         "kernel": "compress_kernel", "algorithmic_bytes_per_launch": alg_bytes,
         "best_ms": min(per_step_ms), "median_ms": statistics.median(per_step_ms)}
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            tr = json.load(f).get(name)
        if tr and tr.get("library_sha") == lib_sha():
            r["traffic"] = tr["dram_bytes_per_launch"]
    except Exception:
        pass
    try:
        w = WORKLOADS[name]
        fam = f"{w['dtype']}_{'prune' if w['mode'] == 'prune' else 'quant' + str(w.get('nbits', 6))}"
        with open(os.path.join(ROOT, "profiles", "issue_ceilings.json")) as f:
            ic = json.load(f)
        c = ic.get(fam)
        if c and ic.get("library_sha") == lib_sha():
            bpe = bytes_per_elem(2 if w["dtype"] == "bf16" else 4, w["mode"], w.get("nbits", 6))
            hz = (sm_mhz or 1965.0) * 1e6
            issue = SMS * ISSUE_LANES * hz / c["instr_per_elem"] * bpe / 1e9
            alu = SMS * ALU_LANES * hz / c["alu_per_elem"] * bpe / 1e9
            r["instruction_roofs"] = {"issue_GBps": issue, "alu_GBps": alu, "instr_per_elem": c["instr_per_elem"],
                                      "alu_instr_per_elem": c["alu_per_elem"], "sm_mhz": hz / 1e6}
            if alu < peak:
                r.update(bound="alu", peak=alu, frac=achieved / alu, peak_kind="ALU-pipe lanes x SM clock / ALU instructions per element")
    except Exception:
        pass
    return r


ALSO_DEFAULT = ["resnet18_bs256_fp32_fp6", "resnet50_bs256_bf16_fp6", "resnet50_bs256_bf16_prune",
                "flat_2p26_fp32_prune", "flat_2p26_fp32_fp6", "flat_2p26_bf16_prune", "flat_2p26_bf16_fp6",
                "flat_2p30_fp32_prune", "flat_2p30_fp32_fp6", "flat_2p30_bf16_prune", "flat_2p30_bf16_fp6"]


def tensor_key(name):
    w = WORKLOADS[name]
    return (w["net"], w.get("log2n"), w["dtype"])


def run_also(lgn, args, dev, first: "Prepared"):
    """The other halves of the metric and the other configurations, a few steps each, on the
    same GPU right after the headline workload: rows of {workload, ms_per_step, value, roofline}."""
    rows = []
    names = [n for n in args.also.split(",") if n and n != args.workload]
    cache_key, cache_tensors = tensor_key(first.name), first.tensors
    for name in sorted(names, key=lambda n: (tensor_key(n) != cache_key, names.index(n))):
        if WORKLOADS[name]["net"] == "aux":
            continue
        if tensor_key(name) != cache_key:
            cache_tensors = None
            torch.cuda.empty_cache()
        p = Prepared(lgn, name, args.batch, 0, dev, tensors=cache_tensors)
        cache_key, cache_tensors = tensor_key(name), p.tensors
        p.warm(3)
        total_ms, per = p.timed(args.also_steps)
        ms = total_ms / args.also_steps
        rows.append({"workload": name, "dtype": p.w["dtype"], "mode": p.w["mode"], "elements": p.total_elems,
                     "steps": args.also_steps, "ms_per_step": ms, "value": p.alg_bytes / (ms * 1e-3) / 1e9,
                     "unit": "GB/s", "elements_per_s": p.total_elems / (ms * 1e-3),
                     "l2": "inputs larger than L2" if p.flush is None else "L2 flushed between timed steps",
                     "roofline": roofline_of(name, p.alg_bytes, per)})
        del p
    return rows


def run_ours(args):
    world, rank, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    from paper_2006_08173_b200 import binding as lgn      # raises if liblgn.so is missing
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    P = Prepared(lgn, args.workload, args.batch, rank, dev)
    w, specs, tensors = P.w, P.specs, P.tensors

    sampler = ClockSampler(local) if rank == 0 else None   # runs from before the warm-up to after the load
    if sampler:
        sampler.mark("load_begin")
    P.warm(args.warmup)
    barrier(world)
    torch.cuda.synchronize()
    if sampler:
        sampler.mark("timed_begin")
    wall0 = time.perf_counter()
    total_ms, per_step_ms = P.timed(args.steps)            # exactly K steps, CUDA events
    wall = time.perf_counter() - wall0
    if sampler:
        sampler.mark("timed_end")
    barrier(world)
    # The timed block can be as short as 20 ms.  The same steps keep running (untimed) until the
    # GPU has been under this load for half a second, so that the clock record has samples.
    if sampler:
        t_hold = time.perf_counter()
        while time.perf_counter() - sampler.marks["load_begin"] < 0.6 and time.perf_counter() - t_hold < 2.0:
            P.timed(max(1, min(args.steps, 20)))
        sampler.mark("load_end")
    clocks = sampler.stop() if sampler else None
    total_ms = max_over_ranks(total_ms, world, dev)
    ms_per_step = total_ms / args.steps
    value = world * P.alg_bytes / (ms_per_step * 1e-3) / 1e9

    line = {
        "metric": "fused_stats_apply_algorithmic_GBps", "value": value, "unit": "GB/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": w["dtype"], "data": "synthetic",
        "config": {"workload": args.workload, "layers": len(tensors), "elements_per_step_per_gpu": P.total_elems,
                   "mode": w["mode"], "nbits": w.get("nbits"), "batch": args.batch,
                   "l2": "inputs larger than L2" if P.flush is None else "L2 flushed between timed steps",
                   "parallelism": f"replicas x{world}"},
        "elements_per_s": world * P.total_elems / (ms_per_step * 1e-3),
        "gpu_launches": args.steps * lgn.lgn_launches_per_call(len(tensors)),
        "roofline": roofline_of(args.workload, P.alg_bytes, per_step_ms, clocks.get("sm_mhz") if clocks else None),
        "clocks": clocks,
        "wall_s": wall,
    }

    if rank == 0 and not args.no_e2e:
        line["e2e"] = measure_e2e(lgn, args, w, specs, tensors, dev, P.alg_bytes)
    barrier(world)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = measure_cpu_baseline(args, w, specs, tensors, P.bpe)
        line["cpu_baseline_all_cores"] = measure_cpu_baseline(args, w, specs, tensors, P.bpe, all_cores=True)
    if rank == 0 and world == 1 and args.also:
        line["also"] = run_also(lgn, args, dev, P)
    if rank == 0:
        print(json.dumps(line))


def run_aux(args):
    """Times one of the steps next to the path on a flat tensor (one GPU, no e2e / CPU legs)."""
    from paper_2006_08173_b200 import binding as lgn
    w = WORKLOADS[args.workload]
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    n = 1 << w["log2n"]
    dtype = torch.float32 if w["dtype"] == "f32" else torch.bfloat16
    esize = 4 if w["dtype"] == "f32" else 2
    launches = 1
    if w["kind"] == "dequant":
        g = synth.lognormal_tensor(n, -12.0, 2.0, 0.5, 0, torch.bfloat16, str(dev))
        st = lgn.lgn_stats(g)
        fmt = lgn.lgn_fp_format(st["mu"], st["sigma"], w["nbits"])
        codes = lgn.lgn_quantize(g, fmt, lgn.ROUND_STOCHASTIC, 1)
        del g
        out = torch.empty(n, dtype=dtype, device=dev)
        alg_bytes = n * (w["nbits"] / 8.0 + esize)
        call = lambda: lgn.lgn_dequantize(codes, n, fmt, out)
        kernel = "dequantize_kernel"
    elif w["kind"] in ("stats", "apply_prune", "apply_fp6"):
        # one entry point alone: the statistics pass, or an apply pass with a cached threshold / format
        g = synth.lognormal_tensor(n, -12.0, 2.0, 0.5, 0, dtype, str(dev))
        st = lgn.lgn_stats(g)
        if w["kind"] == "stats":
            ws = lgn.new_workspace([n], dev)
            out = torch.empty(64, dtype=torch.uint8, device=dev)
            call = lambda: lgn.lgn_stats_async(g, out, ws)
            alg_bytes = float(n * esize)
            kernel = "compress_kernel (statistics only)"
            launches = lgn.lgn_launches_per_call(1)
        elif w["kind"] == "apply_prune":
            tau = lgn.lgn_threshold(st["mu"], st["sigma"], 1.0 - st["nnz"] / st["n"], 0.85)
            out = torch.empty_like(g)
            call = lambda: lgn.lgn_prune(g, tau, 1, out)
            alg_bytes = 2.0 * n * esize
            kernel = "prune_kernel"
        else:
            fmt = lgn.lgn_fp_format(st["mu"], st["sigma"], w["nbits"])
            out = torch.empty(lgn.lgn_codes_bytes(n, w["nbits"]), dtype=torch.uint8, device=dev)
            call = lambda: lgn.lgn_quantize(g, fmt, lgn.ROUND_STOCHASTIC, 1, out)
            alg_bytes = n * (esize + w["nbits"] / 8.0)
            kernel = "quantize_kernel"
    elif w["kind"] == "quantile":
        g = synth.lognormal_tensor(n, -12.0, 2.0, 0.5, 0, dtype, str(dev))
        ws = torch.empty(lgn.lgn_quantile_workspace_bytes(), dtype=torch.uint8, device=dev)
        out = torch.empty(16, dtype=torch.uint8, device=dev)
        raw, gp, code, st_ = lgn.raw(), g.data_ptr(), lgn.dtype_code(g), torch.cuda.current_stream().cuda_stream
        call = lambda: raw.lgn_quantile(gp, n, code, 0.997, out.data_ptr(), ws.data_ptr(), ws.numel(), st_)
        alg_bytes = float(n * esize)                    # one read of the tensor
        kernel = "quantile_count_kernel (behind quantile_sample_kernel; the histogram kernels return at once)"
        launches = (4 if esize == 4 else 3) if n >= 2 ** 24 else (2 if esize == 4 else 1)
    elif w["kind"] in ("bimodal", "maxscale"):
        # one layer of the grouped call with the variant switched on
        if w["kind"] == "bimodal":
            g, mask = synth.bimodal_tensor(n, -9.0, 1.5, -17.0, 1.0, 0.5, 0, dtype, str(dev))
            out = torch.empty_like(g)
            layer = lgn.make_layer(g, out, lgn.MODE_PRUNE, S=0.85, seed=1, right_mode=mask)
            alg_bytes = n * (3.0 * esize + 1.0)          # statistics read + mask, apply read, write
        else:
            g = synth.lognormal_tensor(n, -12.0, 2.0, 0.5, 0, dtype, str(dev))
            out = torch.empty(lgn.lgn_codes_bytes(n, w["nbits"]), dtype=torch.uint8, device=dev)
            layer = lgn.make_layer(g, out, lgn.MODE_QUANTIZE, nbits=w["nbits"], rounding=lgn.ROUND_STOCHASTIC, seed=1,
                                   scale_mode=lgn.SCALE_FROM_MAX)
            alg_bytes = n * (2.0 * esize + w["nbits"] / 8.0)
        ws = lgn.new_workspace([n], dev)
        res = lgn.new_results(1, dev)
        call = lambda: lgn.lgn_compress_layers([layer], res, ws)
        kernel = "compress_kernel"
        launches = lgn.lgn_launches_per_call(1)
    else:
        g = synth.lognormal_tensor(n, -12.0, 2.0, 0.5, 0, dtype, str(dev))
        st = lgn.lgn_stats(g)
        tau = lgn.lgn_threshold(st["mu"], st["sigma"], 1.0 - st["nnz"] / st["n"], 0.8)
        stream_dev = torch.empty(lgn.lgn_prefix_bound_words(n, lgn.dtype_code(g)), dtype=torch.int32, device=dev)
        off_dev = torch.empty(lgn.lgn_prefix_blocks(n) + 1, dtype=torch.int64, device=dev)
        ws = torch.empty(max(16, lgn.lgn_prefix_workspace_bytes(n)), dtype=torch.uint8, device=dev)
        call = lambda: lgn.lgn_prefix_encode(g, tau, 1, True, stream_dev, off_dev, ws)
        call()
        torch.cuda.synchronize()
        words = int(off_dev[-1].item())
        alg_bytes = n * esize + 4.0 * words          # one read of the tensor + the stream written
        kernel = "prefix_encode_kernel"
        launches = 1
        if w.get("decode"):                          # the inverse: the stream read + the tensor written
            dec_out = torch.empty_like(g)
            sd = stream_dev[:words]
            call = lambda: lgn.lgn_prefix_decode(sd, off_dev, dec_out, tau)
            kernel = "prefix_decode_kernel"
    for _ in range(args.warmup):
        call()
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    sampler = ClockSampler(0)
    for i in range(args.steps):
        starts[i].record(stream)
        call()
        ends[i].record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    per_step_ms = [a.elapsed_time(b) for a, b in zip(starts, ends)]
    ms = statistics.mean(per_step_ms)
    peak, peak_kind = read_peak()
    achieved = alg_bytes / (ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": f"{w['kind']}_algorithmic_GBps", "value": achieved, "unit": "GB/s", "n_gpus": 1,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": w["dtype"], "data": "synthetic",
        "config": {"workload": args.workload, "elements": n, "l2": "inputs and outputs larger than L2"},
        "elements_per_s": n / (ms * 1e-3), "gpu_launches": args.steps * launches,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": None, "peak_kind": f"of {peak_kind}", "kernel": kernel,
                     "algorithmic_bytes_per_launch": alg_bytes, "best_ms": min(per_step_ms),
                     "median_ms": statistics.median(per_step_ms)},
        "clocks": clocks}))


def lib_sha():
    import hashlib
    h = hashlib.sha1()
    for rel in ("paper_2006_08173_b200/csrc/lgn.cu", "paper_2006_08173_b200/csrc/lgn_kernels.cuh", "paper_2006_08173_b200/csrc/lgn_device.cuh",
                "paper_2006_08173_b200/csrc/lgn_closed_form.cuh"):
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:12]


def measure_e2e(lgn, args, w, specs, tensors, dev, alg_bytes):
    """Same metric through lgn_compress_layers_host: inputs start in pinned host
    memory, outputs and per-layer results end there; copies are inside the
    timed region."""
    host_in = [torch.empty(g.shape, dtype=g.dtype).pin_memory() for g in tensors]
    for h, g in zip(host_in, tensors):
        h.copy_(g)
    if w["mode"] == "prune":
        host_out = [torch.empty(g.shape, dtype=g.dtype).pin_memory() for g in tensors]
    else:
        host_out = [torch.empty(max(16, lgn.lgn_codes_bytes(g.numel(), w["nbits"])), dtype=torch.uint8).pin_memory()
                    for g in tensors]
    layers = []
    for k, (hi, ho, s) in enumerate(zip(host_in, host_out, specs)):
        if w["mode"] == "prune":
            layers.append(lgn.make_host_layer(hi, ho, lgn.MODE_PRUNE, S=s.sparsity, seed=1000 + k))
        else:
            layers.append(lgn.make_host_layer(hi, ho, lgn.MODE_QUANTIZE, nbits=w["nbits"], rounding=w["rounding"],
                                              seed=1000 + k))
    dev_buf = torch.empty(lgn.lgn_host_staging_bytes(layers) + 256, dtype=torch.uint8, device=dev)
    off = (-dev_buf.data_ptr()) % 256
    dev_buf = dev_buf[off:]
    lgn.lgn_compress_layers_host(layers, dev_buf)          # warm-up
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(args.e2e_steps):
        lgn.lgn_compress_layers_host(layers, dev_buf)      # returns after the stream has drained
    dt = (time.perf_counter() - t0) / args.e2e_steps
    h2d = sum(h.numel() * h.element_size() for h in host_in)
    d2h = sum(h.numel() * h.element_size() for h in host_out) + 120 * len(layers)
    return {"value": alg_bytes / dt / 1e9, "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "ms_per_step": dt * 1e3, "steps": args.e2e_steps,
            "pcie_GBps": (h2d + d2h) / dt / 1e9}


def cpu_model():
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def measure_cpu_baseline(args, w, specs, tensors, bpe, all_cores=False):
    """The oracle as it stands on a bounded sample of the workload (its trailing layers): on
    one thread, or with the layers spread over every core the process may use (threads: the
    oracle's C functions release the interpreter lock; each layer still runs on one thread)."""
    import oracle as orc
    orc.build()
    cores = len(os.sched_getaffinity(0))
    budget = args.cpu_sample_elems * (min(cores, 8) if all_cores else 1) // (2 if all_cores else 1)
    sample, total = oracle_sample(specs, w, budget)
    arrays = [synth.as_numpy_bits(tensors[len(specs) - len(sample) + k]) for k in range(len(sample))]
    used = 1
    t0 = time.perf_counter()
    if all_cores:
        from concurrent.futures import ThreadPoolExecutor
        used = min(cores, len(sample))
        order = sorted(range(len(sample)), key=lambda k: -sample[k].numel)     # longest first
        with ThreadPoolExecutor(used) as ex:
            list(ex.map(lambda k: oracle_step(orc, [arrays[k]], [sample[k]], w), order))
    else:
        oracle_step(orc, arrays, sample, w)
    dt = time.perf_counter() - t0
    return {"value": total * bpe / dt / 1e9, "unit": "GB/s", "cores": used, "kind": "oracle",
            "sample": f"last {len(sample)} of {len(specs)} layers ({total} elements), one pass, {dt:.1f} s",
            "host_cores_available": cores, "cpu_model": cpu_model()}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet18_bs256_fp32_prune", choices=sorted(WORKLOADS))
    ap.add_argument("--batch", type=int, default=256)
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-sample-elems", type=int, default=300_000_000)
    ap.add_argument("--also", default=",".join(ALSO_DEFAULT),
                    help="comma-separated workloads timed after the headline one and reported in the line's `also` list")
    ap.add_argument("--no-also", action="store_const", const="", dest="also")
    ap.add_argument("--also-steps", type=int, default=10)
    ap.add_argument("--ref-sample-elems", type=int, default=33_000_000)
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if WORKLOADS[args.workload]["net"] == "aux":
        if args.impl == "reference" or args.gpus != 1:
            raise SystemExit("the auxiliary workloads are timed on one GPU by our arm only")
        run_aux(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
