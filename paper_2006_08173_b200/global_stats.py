"""Globally consistent per-layer statistics for data-parallel ranks.

Each rank holds its own micro-batch slice of every neural-gradient tensor, and the
path (statistics -> closed form -> apply) is per tensor and per rank: it needs no
exchange.  A caller that wants the SAME threshold or format on every rank for a
layer inserts one step between the statistics pass and the closed form: an
all-reduce (sum) of four numbers per layer -- n, nnz, sum ln|g|, sum ln^2|g| -- over
the process group (NCCL over NVLink on GPUs; any torch.distributed backend works,
the payload is 32 bytes per layer).  This module is that step; the sums come from
``lgn_stats`` / ``lgn_compress_layers`` results and the combined record goes to
``lgn_threshold`` / ``lgn_fp_format`` and the cached-parameter calls ``lgn_prune``
/ ``lgn_quantize``.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import torch
import torch.distributed as dist

from . import binding as lgn


def pack_stats(stats: Sequence[Dict[str, float]], device=None) -> torch.Tensor:
    """[L, 4] fp64: n, nnz, sum_ln, sum_ln2 per layer (counts are exact in fp64 up to 2^53)."""
    rows = [[float(s["n"]), float(s["nnz"]), float(s["sum_ln"]), float(s["sum_ln2"])] for s in stats]
    return torch.tensor(rows, dtype=torch.float64, device=device).reshape(len(rows), 4)


def unpack_stats(t: torch.Tensor) -> List[Dict[str, float]]:
    out = []
    for n, nnz, s1, s2 in t.detach().cpu().tolist():
        out.append(lgn.lgn_combine_stats([{"n": int(round(n)), "nnz": int(round(nnz)), "sum_ln": s1, "sum_ln2": s2}]))
    return out


def allreduce_stats(stats: Sequence[Dict[str, float]], group: Optional[dist.ProcessGroup] = None,
                    device=None) -> List[Dict[str, float]]:
    """Per-layer statistics of the union of all ranks' tensors.  ``stats``: this rank's
    per-layer records (as returned by ``lgn_stats`` or ``read_results``), the same
    layers in the same order on every rank.  One all-reduce of [L, 4] fp64."""
    t = pack_stats(stats, device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return unpack_stats(t)


def rank_seed(seed: int, rank: int) -> int:
    """A per-rank seed, so that the ranks' random bits differ although their element
    indices coincide: the rank goes into the upper half of the 64-bit key."""
    return (int(seed) & 0xFFFFFFFF) | ((int(rank) & 0xFFFFFFFF) << 32)
