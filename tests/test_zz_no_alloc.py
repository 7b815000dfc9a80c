"""The entry point that allocates nothing (opt_gqa_paged_attention_decode_no_alloc).

It exists for callers that cannot give the library a workspace -- code embedded in an engine that has
already handed all device memory to its cache pool, or running where cudaMalloc is not allowed -- and keeps
the partitions' partial results in an 8 MiB array built into the library.  Checked here through the C ABI
against the ordinary decode + reduce pair on the same inputs, on several calls in a row (each later call
finds the earlier ones' leftovers in the shared array).  This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from paper_2505_02351_b200 import binding
from paper_2505_02351_b200 import workloads as W
from tests import util

pytestmark = pytest.mark.gpu


def _pair(wl, P):
    """out of (append, decode with partition_size P, reduce) through the workspace-taking entry points."""
    got, _ = util.gpu_decode(wl, partition_size=P)
    return got


def _no_alloc(wl, P):
    d = util.DeviceWorkload(wl)
    maxP = max(1, (int(wl.context_lens.max()) + P - 1) // P)
    binding.cache_append(d.k_new, d.v_new, d.k_cache, d.v_cache, d.slot_mapping)
    binding.paged_attention_decode_no_alloc(d.out, d.q, d.k_cache, d.v_cache, d.block_tables, d.context_lens,
                                            d.alibi_slopes, wl.scale, P, maxP)
    torch.cuda.synchronize()
    assert binding.device_status() == 0
    return d.out.double().cpu().numpy()


def test_calls_in_a_row_match_the_workspace_entry_points():
    first = W.make_custom("na1", "bf16", 32, 4, 128, 16, [3000, 700, 0, 45], seed=41, poison=True)
    second = W.make_custom("na2", "fp32", 4, 2, 64, 16, [100, 37, 513], seed=42, poison=True)
    third = W.make_custom("na3", "bf16", 8, 2, 128, 32, [260, 1200], seed=43)
    for wl, P in ((first, 512), (second, 32), (third, 64), (first, 256)):
        want = _pair(wl, P)
        got = _no_alloc(wl, P)
        assert np.isfinite(got).all()
        assert np.max(np.abs(got - want)) <= util.TOL[wl.dtype], wl.name
        # and against the oracle, so that the comparison above cannot pass on two equal mistakes
        assert np.max(np.abs(got - util.oracle_attention(wl))) <= util.TOL[wl.dtype], wl.name


def test_sizes_beyond_the_built_in_array_are_refused():
    wl = W.make_custom("na4", "bf16", 32, 4, 128, 16, [64, 64], seed=44)
    d = util.DeviceWorkload(wl)
    binding.cache_append(d.k_new, d.v_new, d.k_cache, d.v_cache, d.slot_mapping)
    d.out.fill_(7.0)
    too_many = (8 << 20) // (wl.B * wl.Hq * (wl.D + 1) * 4) + 1      # partitions that no longer fit in 8 MiB
    with pytest.raises(binding.OptGqaError) as e:
        binding.paged_attention_decode_no_alloc(d.out, d.q, d.k_cache, d.v_cache, d.block_tables, d.context_lens,
                                                d.alibi_slopes, wl.scale, 16, too_many)
    assert e.value.code == -7 and "scratch" in str(e.value)
    torch.cuda.synchronize()
    assert bool((d.out == 7.0).all())            # nothing was enqueued
    binding.paged_attention_decode_no_alloc(d.out, d.q, d.k_cache, d.v_cache, d.block_tables, d.context_lens,
                                            d.alibi_slopes, wl.scale, 16, too_many - 1)
    torch.cuda.synchronize()
    assert np.max(np.abs(d.out.double().cpu().numpy() - util.oracle_attention(wl))) <= util.TOL["bf16"]
