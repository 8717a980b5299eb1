"""lgn_stats_static_scratch: the statistics pass for callers that cannot give
the library a workspace because they cannot allocate device memory where they
call it (inside a training step, after handing all memory to their own pool,
from a plug-in without the framework's allocator).  Its scratch is an array
inside the library, so the checks here are the ones that matter for such a
caller: same answer as lgn_stats, again on a second call that finds the first
call's leftovers in the array, and a clear refusal beyond the array's capacity.

Collected last on purpose (file name): a failure here cannot hide another test.
"""
import numpy as np
import pytest
import torch

from gpu_helpers import assert_stats_close, np_bits
from paper_2006_08173_b200 import synth

pytestmark = pytest.mark.gpu


def stats_both_ways(lgn, g):
    out = torch.full((64,), 0xEE, dtype=torch.uint8, device=g.device)
    lgn.lgn_stats_static_scratch_async(g, out)          # through the C ABI, no workspace argument
    got = lgn.read_stats(out)                           # synchronises
    return got, lgn.lgn_stats(g)


def test_two_calls_in_a_row_match_the_workspace_entry_point(lgn, oracle):
    big = synth.lognormal_tensor(3_000_001, -12.0, 2.0, 0.4, seed=21, device="cuda")
    small = synth.lognormal_tensor(70_003, -9.0, 3.0, 0.1, seed=22, dtype=torch.bfloat16, device="cuda")
    for g in (big, small, big):                         # the later calls start from a used array
        got, ref = stats_both_ways(lgn, g)
        assert got == ref                               # same kernel, same order of additions
        assert_stats_close(got, oracle.stats(np_bits(g)))
    empty = torch.zeros(0, device="cuda")
    got, ref = stats_both_ways(lgn, empty)
    assert got == ref and got["n"] == 0


def test_the_call_leaves_free_device_memory_as_it_found_it(lgn):
    """The one promise of this entry point: nothing is allocated.  Everything the test
    itself needs exists before the first reading of cudaMemGetInfo; the first call (which
    looks the array's address up) has been made; the second call must leave the free
    byte count where it was."""
    g = synth.lognormal_tensor(2_000_003, -11.0, 2.0, 0.3, seed=25, device="cuda")
    out = torch.zeros(64, dtype=torch.uint8, device="cuda")
    lgn.lgn_stats_static_scratch_async(g, out)
    torch.cuda.synchronize()
    first = lgn.read_stats(out)
    out.zero_()
    torch.cuda.synchronize()
    free_before, total = torch.cuda.mem_get_info()
    lgn.lgn_stats_static_scratch_async(g, out)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert lgn.read_stats(out) == first


def test_back_to_back_without_a_sync_between_them(lgn):
    a = synth.lognormal_tensor(1_000_000, -12.0, 2.0, 0.5, seed=23, device="cuda")
    b = synth.lognormal_tensor(500_000, -6.0, 1.5, 0.0, seed=24, device="cuda")
    oa = torch.zeros(64, dtype=torch.uint8, device="cuda")
    ob = torch.zeros(64, dtype=torch.uint8, device="cuda")
    lgn.lgn_stats_static_scratch_async(a, oa)           # same stream: ordered, so sharing the array is safe
    lgn.lgn_stats_static_scratch_async(b, ob)
    assert lgn.read_stats(oa) == lgn.lgn_stats(a)
    assert lgn.read_stats(ob) == lgn.lgn_stats(b)


def test_sizes_beyond_the_array_are_refused(lgn):
    n = lgn.STATS_STATIC_MAX_ELEMS + 16384
    g = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(64, dtype=torch.uint8, device="cuda")
    with pytest.raises(lgn.LgnError) as e:
        lgn.lgn_stats_static_scratch_async(g, out)
    assert e.value.code == 2                            # LGN_ERR_UNSUPPORTED, nothing enqueued
    at_limit = g[:lgn.STATS_STATIC_MAX_ELEMS]
    got, ref = stats_both_ways(lgn, at_limit)           # exactly the maximum still works
    assert got == ref and got["nnz"] == 0
