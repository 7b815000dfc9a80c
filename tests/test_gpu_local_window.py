"""Local (sliding-window) mask through the C ABI against the oracle's window mode (Algorithm 1, "Create causal
and local attention masks")."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_02351_b200 import binding
from paper_2505_02351_b200 import workloads as W
from tests import util

pytestmark = pytest.mark.gpu
TOL = util.TOL["bf16"]


def _oracle(wl, window, slopes):
    a = util.oracle_inputs(wl)
    return oracle.paged_attention(a["q"], a["k"], a["v"], a["bt"], a["n"], a["slopes"] if slopes else None, wl.scale,
                                  wl.dtype, q_start_loc=a["qsl"], window=window)


@pytest.mark.parametrize("window", [1, 16, 17, 100, 512, 5000])
@pytest.mark.parametrize("slopes", [False, True])
def test_decode_local_window(window, slopes):
    wl = W.make_custom("win", "bf16", 8, 2, 128, 16, [1, 15, 16, 17, 33, 100, 257, 0, 640, 3000], seed=80, poison=True)
    d = util.DeviceWorkload(wl)
    binding.cache_append(d.k_new, d.v_new, d.k_cache, d.v_cache, d.slot_mapping)
    for P in (64, 512):
        maxP = (int(wl.context_lens.max()) + P - 1) // P
        ws = torch.full((binding.workspace_bytes(wl.B, wl.Hq, wl.D, maxP) // 4,), float("nan"), device="cuda:0")
        d.out.fill_(float("nan"))
        binding.paged_attention_decode_local(d.out, d.q, d.k_cache, d.v_cache, d.block_tables, d.context_lens,
                                             d.alibi_slopes if slopes else None, wl.scale, P, ws, maxP, window)
        torch.cuda.synchronize()
        assert binding.device_status() == 0
        got = d.out.double().cpu().numpy()
        want = _oracle(wl, window, slopes)
        assert np.isfinite(got).all()
        assert np.max(np.abs(got - want)) <= TOL, (window, P)


def test_decode_window_longer_than_every_sequence_is_plain_decode():
    wl = W.make_config(2)
    d = util.DeviceWorkload(wl)
    binding.cache_append(d.k_new, d.v_new, d.k_cache, d.v_cache, d.slot_mapping)
    P, maxP = 256, 8
    ws = torch.empty(binding.workspace_bytes(wl.B, wl.Hq, wl.D, maxP), dtype=torch.uint8, device="cuda:0")
    binding.paged_attention_decode_local(d.out, d.q, d.k_cache, d.v_cache, d.block_tables, d.context_lens,
                                         d.alibi_slopes, wl.scale, P, ws, maxP, 1 << 20)
    torch.cuda.synchronize()
    plain, _ = util.gpu_decode(wl, partition_size=P, balanced=True)
    assert np.array_equal(d.out.double().cpu().numpy(), plain)


@pytest.mark.parametrize("window", [1, 33, 64, 200, 4096])
@pytest.mark.parametrize("Hq,Hkv", [(8, 2), (8, 1), (2, 2)])
def test_prefill_local_window(window, Hq, Hkv):
    lens = [700, 77, 130, 1, 300]
    qls = [300, 77, 129, 1, 17]
    wl = W.make_custom("winpf", "bf16", Hq, Hkv, 128, 16, lens, q_lens=qls, seed=81, poison=True)
    d = util.DeviceWorkload(wl)
    binding.cache_append(d.k_new, d.v_new, d.k_cache, d.v_cache, d.slot_mapping)
    for slopes in (False, True):
        d.out.fill_(float("nan"))
        binding.paged_attention_prefill_local(d.out, d.q, d.q_start_loc, max(qls), d.k_cache, d.v_cache, d.block_tables,
                                              d.context_lens, d.alibi_slopes if slopes else None, wl.scale, window)
        torch.cuda.synchronize()
        assert binding.device_status() == 0
        got = d.out.double().cpu().numpy()
        assert np.isfinite(got).all()
        assert np.max(np.abs(got - _oracle(wl, window, slopes))) <= TOL, (window, slopes)


@pytest.mark.parametrize("window", [1, 16, 17, 100, 5000])
@pytest.mark.parametrize("D", [64, 128])
def test_decode_local_window_on_fp32_caches(window, D):
    """fp32 caches: one partial per partition on the CUDA-core kernel, merge over the partitions inside the window."""
    wl = W.make_custom("win32", "fp32", 8, 2, D, 16, [1, 15, 16, 17, 33, 100, 257, 0, 640], seed=83, poison=True)
    d = util.DeviceWorkload(wl)
    binding.cache_append(d.k_new, d.v_new, d.k_cache, d.v_cache, d.slot_mapping)
    for P in (32, 512):
        maxP = (int(wl.context_lens.max()) + P - 1) // P
        ws = torch.full((wl.B * wl.Hq * maxP * (wl.D + 1),), float("nan"), device="cuda:0")
        for slopes in (False, True):
            d.out.fill_(float("nan"))
            binding.paged_attention_decode_local(d.out, d.q, d.k_cache, d.v_cache, d.block_tables, d.context_lens,
                                                 d.alibi_slopes if slopes else None, wl.scale, P, ws, maxP, window)
            torch.cuda.synchronize()
            assert binding.device_status() == 0
            got = d.out.double().cpu().numpy()
            assert np.isfinite(got).all()
            assert np.max(np.abs(got - _oracle(wl, window, slopes))) <= util.TOL["fp32"], (window, P, slopes)


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("scale", [0.0, -0.07, 0.2])
def test_prefill_local_window_head_dims_and_scales(D, scale):
    """The windowed chunked prefill on tcgen05 for head dimension 64 and for scales that are zero or negative."""
    lens = [700, 77, 130, 1, 300]
    qls = [300, 77, 129, 1, 17]
    wl = W.make_custom("winpf2", "bf16", 8, 2, D, 32, lens, q_lens=qls, seed=84, poison=True, scale=scale)
    d = util.DeviceWorkload(wl)
    binding.cache_append(d.k_new, d.v_new, d.k_cache, d.v_cache, d.slot_mapping)
    for window, slopes in ((40, True), (200, False), (64, True)):
        d.out.fill_(float("nan"))
        binding.paged_attention_prefill_local(d.out, d.q, d.q_start_loc, max(qls), d.k_cache, d.v_cache, d.block_tables,
                                              d.context_lens, d.alibi_slopes if slopes else None, wl.scale, window)
        torch.cuda.synchronize()
        assert binding.device_status() == 0
        got = d.out.double().cpu().numpy()
        assert np.isfinite(got).all()
        assert np.max(np.abs(got - _oracle(wl, window, slopes))) <= TOL, (window, slopes)


def test_window_entry_points_reject_what_they_do_not_support():
    wl = W.make_custom("w0", "bf16", 8, 2, 128, 16, [64], seed=82)
    d = util.DeviceWorkload(wl)
    ws = torch.empty(binding.workspace_bytes(wl.B, wl.Hq, wl.D, 8), dtype=torch.uint8, device="cuda:0")
    with pytest.raises(binding.OptGqaError) as e:
        binding.paged_attention_decode_local(d.out, d.q, d.k_cache, d.v_cache, d.block_tables, d.context_lens, None,
                                             wl.scale, 16, ws, 8, 0)
    assert e.value.code == -2          # window must be positive
    with pytest.raises(binding.OptGqaError) as e:
        binding.paged_attention_prefill_local(d.out, d.q, torch.zeros(2, dtype=torch.int32, device="cuda:0"), 1,
                                              d.k_cache, d.v_cache, d.block_tables, d.context_lens, None, wl.scale, 0)
    assert e.value.code == -2
