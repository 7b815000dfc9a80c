"""Helpers shared by the parity tests: run a workload through the CUDA library and through the oracle."""
import os

import numpy as np
import torch

import oracle
from paper_2505_02351_b200 import binding
from paper_2505_02351_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))   # the repository root (for child processes)
TOL = {"fp32": 1e-5, "bf16": 2e-2}   # max-abs tolerance on attention outputs (fp32 accumulation)


class DeviceWorkload:
    """Device copies of a workload's tensors."""

    def __init__(self, wl: W.Workload, device="cuda:0"):
        self.wl = wl
        dev = torch.device(device)
        for name in ("q", "k_cache", "v_cache", "block_tables", "context_lens", "alibi_slopes", "k_new", "v_new",
                     "slot_mapping"):
            setattr(self, name, getattr(wl, name).to(dev))
        self.q_start_loc = None if wl.q_start_loc is None else wl.q_start_loc.to(dev)
        self.out = torch.full_like(self.q, float("nan"))


def gpu_decode(wl: W.Workload, partition_size=None, append=True, slopes=True, simt=False, balanced=False):
    """append + decode (+ reduce) through the C ABI; returns (out float64 numpy, DeviceWorkload).

    balanced=True takes the load-balanced split (decode_balanced + reduce_balanced, bf16, partition_size > 0)."""
    d = DeviceWorkload(wl)
    P = wl.partition_size if partition_size is None else partition_size
    if append:
        binding.cache_append(d.k_new, d.v_new, d.k_cache, d.v_cache, d.slot_mapping)
    sl = d.alibi_slopes if slopes else None
    if balanced:
        assert P > 0 and wl.dtype == "bf16"
        maxP = max(1, (int(wl.context_lens.max()) + P - 1) // P) if wl.B else 1
        ws = torch.full((binding.workspace_bytes(max(wl.B, 1), wl.Hq, wl.D, maxP) // 4,), float("nan"), device="cuda:0",
                        dtype=torch.float32)
        binding.paged_attention_decode_balanced(d.q, d.k_cache, d.v_cache, d.block_tables, d.context_lens, sl, wl.scale,
                                                P, ws, maxP)
        binding.paged_attention_reduce_balanced(d.out, ws, d.context_lens, wl.Hkv, P, maxP)
        torch.cuda.synchronize()
        assert binding.device_status() == 0
        return d.out.double().cpu().numpy(), d
    decode = binding.paged_attention_decode_simt if simt else binding.paged_attention_decode
    if P > 0:
        maxP = max(1, (int(wl.context_lens.max()) + P - 1) // P) if wl.B else 1
        po = torch.full((wl.B, wl.Hq, maxP, wl.D), float("nan"), device="cuda:0", dtype=torch.float32)
        pl = torch.full((wl.B, wl.Hq, maxP), float("nan"), device="cuda:0", dtype=torch.float32)
        decode(None, d.q, d.k_cache, d.v_cache, d.block_tables, d.context_lens, sl, wl.scale,
                                       partition_size=P, partial_out=po, partial_lse=pl, max_partitions=maxP)
        binding.paged_attention_reduce(d.out, po, pl, d.context_lens, P)
        d.partial_out, d.partial_lse = po, pl
    else:
        decode(d.out, d.q, d.k_cache, d.v_cache, d.block_tables, d.context_lens, sl, wl.scale)
    torch.cuda.synchronize()
    assert binding.device_status() == 0
    return d.out.double().cpu().numpy(), d


def oracle_inputs(wl: W.Workload, append=True):
    k = W.storage_numpy(wl.k_cache)
    v = W.storage_numpy(wl.v_cache)
    if append:
        oracle.cache_append(W.storage_numpy(wl.k_new), W.storage_numpy(wl.v_new), k, v, wl.slot_mapping.numpy(),
                            wl.dtype)
    return dict(q=W.storage_numpy(wl.q), k=k, v=v, bt=wl.block_tables.numpy(), n=wl.context_lens.numpy(),
                slopes=wl.alibi_slopes.numpy().astype(np.float64),
                qsl=None if wl.q_start_loc is None else wl.q_start_loc.numpy())


def oracle_attention(wl: W.Workload, append=True, slopes=True, simt=False, balanced=False, mma=False):
    a = oracle_inputs(wl, append)
    return oracle.paged_attention(a["q"], a["k"], a["v"], a["bt"], a["n"], a["slopes"] if slopes else None, wl.scale,
                                  wl.dtype, q_start_loc=a["qsl"])


def gpu_prefill(wl: W.Workload, append=True, slopes=True, mma=False):
    """append + chunked prefill through the C ABI; returns (out float64 numpy, DeviceWorkload).

    mma=True forces the warp-level kernel (the default entry point runs D = 128 on tcgen05)."""
    d = DeviceWorkload(wl)
    if append:
        binding.cache_append(d.k_new, d.v_new, d.k_cache, d.v_cache, d.slot_mapping)
    qsl = wl.q_start_loc.numpy()
    max_q_len = int((qsl[1:] - qsl[:-1]).max()) if wl.B else 0
    fn = binding.paged_attention_prefill_mma if mma else binding.paged_attention_prefill
    fn(d.out, d.q, d.q_start_loc, max_q_len, d.k_cache, d.v_cache, d.block_tables, d.context_lens,
       d.alibi_slopes if slopes else None, wl.scale)
    torch.cuda.synchronize()
    assert binding.device_status() == 0
    return d.out.double().cpu().numpy(), d


def oracle_prefill_rows(wl: W.Workload, rows, append=True, slopes=True):
    """Oracle output for selected new-token rows only: row t of sequence s is a decode query at
    position pos_t over the context truncated to pos_t + 1 tokens (the oracle's decode mode)."""
    a = oracle_inputs(wl, append)
    qsl = a["qsl"]
    seq = np.searchsorted(qsl, rows, side="right") - 1
    qlen = qsl[seq + 1] - qsl[seq]
    pos = a["n"][seq] - qlen + (np.asarray(rows) - qsl[seq])
    return oracle.paged_attention(np.ascontiguousarray(a["q"][rows]), a["k"], a["v"],
                                  np.ascontiguousarray(a["bt"][seq]), (pos + 1).astype(np.int32),
                                  a["slopes"] if slopes else None, wl.scale, wl.dtype)
