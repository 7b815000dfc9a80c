#!/usr/bin/env python
"""Benchmark of the Opt-GQA decode hot path on B200.

One "step" is one pass of the whole path over one batch of synthetic input:
cache_append of the step's new tokens -> paged GQA-ALiBi decode over context
partitions -> log-sum-exp reduce.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config 3] [--impl ours|reference]
                  [--only step|prefill|projection]

--steps / --warmup size the timed region behind `value`.  The legs that explain it have sample counts of their
own, whatever --steps says: the decode kernel's launch duration comes from KERNEL_TIMING_STEPS further steps
(event brackets around back-to-back launches), the end-to-end number from E2E_STEPS steps through host buffers,
the read-only ceiling of the data path from a streaming probe over 1 GiB.

N > 1 is launched with torch.distributed.run; the path shards by sequence with no
data-path collective (every rank runs its own batch of the same shape), so the
line reports weak scaling and the only communication is the timing reduction.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "paged GQA-ALiBi decode: achieved HBM TB/s vs peak; tokens/s per step"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0
# Partition size used for workloads that do not fix one (the caller's choice under the C ABI).
DEFAULT_PARTITION = {2: 256, 3: 512, 4: 512}
# dram__bytes_read.sum + dram__bytes_write.sum of one decode launch, from the ncu capture summarised
# under profiles/ (None until a capture of that workload exists).
NCU_TRAFFIC_BYTES = {3: 378_703_104 + 3_860_992}   # profiles/decode_stream_cfg3.md
KERNEL_TIMING_STEPS = 512   # steps of the kernel-timing region (a bracket every EVENT_EVERY-th step)
E2E_STEPS = 200             # steps of the end-to-end leg
READ_PROBE_BYTES = 1 << 30  # bytes streamed by the read-only ceiling probe per launch
DTYPE = "bf16 operands, f32 accumulate"
KERNEL_FAMILY = ("tensor-core tile kernels: 2-D TMA tiles into per-warp rings, mma.sync m16n8k16 with the query group "
                 "as one tile side, fp32 online softmax")


# ----------------------------------------------------------------------------- distributed plumbing
def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def max_over_ranks(value: float, backend_device: str) -> float:
    """MAX all-reduce of one float over the process group (identity when not initialised)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()):
        return value
    t = torch.tensor([value], dtype=torch.float64, device=backend_device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, backend_device: str) -> float:
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()):
        return value
    t = torch.tensor([value], dtype=torch.float64, device=backend_device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def barrier():
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized():
        dist.barrier()


# ----------------------------------------------------------------------------- clocks
_REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
            0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost"}


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons of one GPU while the timed region runs (read-only NVML)."""

    def __init__(self, device_index: int, period_s: float = 0.002):
        super().__init__(daemon=True)
        self.device_index = device_index
        self.period = period_s
        self.samples, self.reasons, self.sm_max = [], set(), None
        self._halt = threading.Event()
        self._h = None
        try:
            import pynvml
            import torch

            pynvml.nvmlInit()
            self._nv = pynvml
            try:
                uuid = str(torch.cuda.get_device_properties(device_index).uuid)
                uuid = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.sm_max = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _one(self):
        nv = self._nv
        self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
        try:
            mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
        except Exception:
            mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
        for bit, name in _REASONS.items():
            if mask & bit:
                self.reasons.add(name)

    def run(self):
        if self._h is None:
            # no NVML binding: read-only nvidia-smi queries while the timed legs run
            while not self._halt.is_set():
                one = self._smi_query()
                if one is not None:
                    self.samples.append(one[0])
                    self.sm_max = one[1]
                    self.reasons.update(one[2])
                self._halt.wait(0.05)
            return
        while not self._halt.is_set():
            try:
                self._one()
            except Exception:
                pass
            self._halt.wait(self.period)

    def stop(self) -> dict:
        self._halt.set()
        self.join(timeout=2.0)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_min_mhz": s[0], "sm_max_mhz": self.sm_max, "reasons": sorted(self.reasons),
                "samples": len(s), "source": "nvml" if self._h is not None else "nvidia-smi"}

    def _smi_query(self):
        fields = ["clocks.sm", "clocks.max.sm", "clocks_event_reasons.hw_slowdown",
                  "clocks_event_reasons.hw_thermal_slowdown", "clocks_event_reasons.sw_thermal_slowdown",
                  "clocks_event_reasons.sw_power_cap"]
        try:
            out = subprocess.run(["nvidia-smi", "-i", str(self.device_index), "--query-gpu=" + ",".join(fields),
                                  "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=10)
            cells = [c.strip() for c in out.stdout.strip().splitlines()[0].split(",")]
            reasons = [f.split(".")[1] for f, c in zip(fields[2:], cells[2:]) if c.lower().startswith("active")]
            return int(cells[0]), int(cells[1]), reasons
        except Exception:
            return None


# ----------------------------------------------------------------------------- workload on the device
class DeviceBatch:
    """A workload resident in HBM, with `copies` distinct copies of the KV pool to rotate through."""

    def __init__(self, wl, partition_size: int, copies: int, device):
        import torch

        from paper_2505_02351_b200 import binding

        self.wl, self.P = wl, partition_size
        self.dev = device
        to = lambda t: t.to(device)
        self.q, self.k_new, self.v_new = to(wl.q), to(wl.k_new), to(wl.v_new)
        self.slots, self.tables, self.lens = to(wl.slot_mapping), to(wl.block_tables), to(wl.context_lens)
        self.slopes = to(wl.alibi_slopes)
        self.out = torch.zeros_like(self.q)
        self.k_pools = [to(wl.k_cache)]
        self.v_pools = [to(wl.v_cache)]
        for _ in range(copies - 1):
            self.k_pools.append(self.k_pools[0].clone())
            self.v_pools.append(self.v_pools[0].clone())
        self.maxP = max(1, (int(wl.context_lens.max()) + partition_size - 1) // partition_size) if partition_size else 1
        ws = binding.workspace_bytes(wl.B, wl.Hq, wl.D, self.maxP) if partition_size else 0
        self.workspace = torch.empty(max(ws, 16), dtype=torch.uint8, device=device)
        self.ws_bytes = int(self.workspace.numel())
        npart = wl.B * wl.Hq * self.maxP
        self.partial_out = self.workspace[: npart * wl.D * 4].view(torch.float32)
        self.partial_lse = self.workspace[npart * wl.D * 4: npart * (wl.D + 1) * 4].view(torch.float32) if ws else None
        self.lib = binding.load()
        self.dt = binding.BF16 if wl.dtype == "bf16" else binding.FP32

    # Pre-marshalled argument tuples: the timed loop then costs one foreign call per kernel.
    def args_append(self, i, stream):
        wl = self.wl
        return (self.k_new.data_ptr(), self.v_new.data_ptr(), self.k_pools[i].data_ptr(), self.v_pools[i].data_ptr(),
                self.slots.data_ptr(), wl.B, wl.Hkv, wl.D, wl.bs, wl.num_blocks, self.dt, stream)

    @property
    def balanced(self) -> bool:
        """bf16 partitioned steps take the load-balanced split (what opt_gqa_decode_step runs)."""
        return self.P > 0 and self.wl.dtype == "bf16"

    def args_decode(self, i, stream):
        wl = self.wl
        if self.balanced:
            return (self.q.data_ptr(), self.k_pools[i].data_ptr(), self.v_pools[i].data_ptr(), self.tables.data_ptr(),
                    wl.max_blocks, self.lens.data_ptr(), self.slopes.data_ptr(), wl.scale, wl.B, wl.Hq, wl.Hkv, wl.D,
                    wl.bs, wl.num_blocks, self.P, self.workspace.data_ptr(), self.ws_bytes, self.maxP, self.dt, stream)
        return self.args_decode_plain(i, stream)

    def args_decode_plain(self, i, stream):
        """opt_gqa_paged_attention_decode: single pass (P = 0) or one partial per partition."""
        wl = self.wl
        return (self.out.data_ptr(), self.q.data_ptr(), self.k_pools[i].data_ptr(), self.v_pools[i].data_ptr(),
                self.tables.data_ptr(), wl.max_blocks, self.lens.data_ptr(), self.slopes.data_ptr(), wl.scale, wl.B,
                wl.Hq, wl.Hkv, wl.D, wl.bs, wl.num_blocks, self.P,
                self.partial_out.data_ptr() if self.P else None, self.partial_lse.data_ptr() if self.P else None,
                self.maxP, self.dt, stream)

    def args_decode_single(self, i, stream):
        """opt_gqa_paged_attention_decode as a single pass (what a one-launch step runs, minus the token store)."""
        wl = self.wl
        return (self.out.data_ptr(), self.q.data_ptr(), self.k_pools[i].data_ptr(), self.v_pools[i].data_ptr(),
                self.tables.data_ptr(), wl.max_blocks, self.lens.data_ptr(), self.slopes.data_ptr(), wl.scale, wl.B,
                wl.Hq, wl.Hkv, wl.D, wl.bs, wl.num_blocks, 0, None, None, 1, self.dt, stream)

    def args_reduce(self, stream):
        wl = self.wl
        if self.balanced:
            return (self.out.data_ptr(), self.workspace.data_ptr(), self.ws_bytes, self.lens.data_ptr(), wl.B, wl.Hq,
                    wl.Hkv, wl.D, self.P, self.maxP, self.dt, stream)
        return (self.out.data_ptr(), self.partial_out.data_ptr(), self.partial_lse.data_ptr(), self.lens.data_ptr(),
                wl.B, wl.Hq, wl.D, self.P, self.maxP, self.dt, stream)

    def args_step(self, i, stream):
        wl = self.wl
        return (self.out.data_ptr(), self.q.data_ptr(), self.k_new.data_ptr(), self.v_new.data_ptr(),
                self.slots.data_ptr(), self.k_pools[i].data_ptr(), self.v_pools[i].data_ptr(), self.tables.data_ptr(),
                wl.max_blocks, self.lens.data_ptr(), self.slopes.data_ptr(), wl.scale, wl.B, wl.Hq, wl.Hkv, wl.D,
                wl.bs, wl.num_blocks, self.P, self.workspace.data_ptr() if self.P else None,
                self.ws_bytes if self.P else 0, self.maxP, self.dt, stream)

    def algorithmic_bytes(self) -> int:
        """Bytes one decode launch must move: every K and V element of every context once, q, out, table entries."""
        wl = self.wl
        es = 2 if wl.dtype == "bf16" else 4
        n = wl.context_lens.long()
        tables = int(((n + wl.bs - 1) // wl.bs).sum()) * 4
        return wl.kv_bytes() + 2 * wl.B * wl.Hq * wl.D * es + tables


class PrefillBatch:
    """The chunked-prefill workload resident in HBM: a step appends every sequence's new tokens, then attends."""

    def __init__(self, wl, device):
        import torch

        from paper_2505_02351_b200 import binding

        self.wl, self.dev = wl, device
        to = lambda t: t.to(device)
        self.q, self.k_new, self.v_new = to(wl.q), to(wl.k_new), to(wl.v_new)
        self.slots, self.tables, self.lens = to(wl.slot_mapping), to(wl.block_tables), to(wl.context_lens)
        self.slopes, self.qsl = to(wl.alibi_slopes), to(wl.q_start_loc)
        self.k_pool, self.v_pool = to(wl.k_cache), to(wl.v_cache)
        self.out = torch.zeros_like(self.q)
        qsl = wl.q_start_loc.numpy()
        self.max_q_len = int((qsl[1:] - qsl[:-1]).max())
        self.lib = binding.load()

    def flops(self) -> float:
        """4*D flop (q.k and p.v) per unmasked (new token, key) pair per query head."""
        wl = self.wl
        qsl = wl.q_start_loc.numpy().astype("int64")
        n = wl.context_lens.numpy().astype("int64")
        pairs = 0
        for s in range(wl.B):
            ql = int(qsl[s + 1] - qsl[s])
            first = int(n[s]) - ql + 1                       # keys seen by the first new token
            pairs += ql * first + ql * (ql - 1) // 2
        return 4.0 * wl.D * wl.Hq * pairs

    def run(self, steps: int, warmup: int):
        """Returns (ms per step, ms per prefill launch)."""
        import torch

        wl = self.wl
        stream = torch.cuda.current_stream()
        sh = stream.cuda_stream
        a_app = (self.k_new.data_ptr(), self.v_new.data_ptr(), self.k_pool.data_ptr(), self.v_pool.data_ptr(),
                 self.slots.data_ptr(), wl.T, wl.Hkv, wl.D, wl.bs, wl.num_blocks, 1, sh)
        a_pf = (self.out.data_ptr(), self.q.data_ptr(), self.qsl.data_ptr(), wl.T, self.max_q_len, self.k_pool.data_ptr(),
                self.v_pool.data_ptr(), self.tables.data_ptr(), wl.max_blocks, self.lens.data_ptr(),
                self.slopes.data_ptr(), wl.scale, wl.B, wl.Hq, wl.Hkv, wl.D, wl.bs, wl.num_blocks, 1, sh)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for i in range(warmup + steps):
            if i == warmup:
                torch.cuda.synchronize()
                start.record(stream)
            check(self.lib.opt_gqa_cache_append(*a_app), "cache_append")
            if i >= warmup:
                evs[i - warmup][0].record(stream)
            check(self.lib.opt_gqa_paged_attention_prefill(*a_pf), "prefill")
            if i >= warmup:
                evs[i - warmup][1].record(stream)
        end.record(stream)
        torch.cuda.synchronize()
        return start.elapsed_time(end) / steps, sum(a.elapsed_time(b) for a, b in evs) / steps


def measured_tensor_peak():
    """(sustained, burst, kind) dense bf16 TFLOP/s: the measured cuBLAS figures, else the earlier pool measurement."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return float(d["bf16_tflops_sustained"]), float(d["bf16_tflops"]), "measured"
    except Exception:
        return 1400.0, 1590.0, "fallback"


def prefill_report(dev, steps: int, warmup: int) -> dict:
    """Side measurement of the chunked-prefill workload: append of the new tokens + tensor-core prefill."""
    from paper_2505_02351_b200 import workloads as W

    wl = W.make_config(5)
    pb = PrefillBatch(wl, dev)
    step_ms, pf_ms = pb.run(steps, warmup)
    sustained, burst, kind = measured_tensor_peak()
    tf = pb.flops() / (pf_ms * 1e-3) / 1e12
    return {"new_tokens_per_s": wl.T / (step_ms * 1e-3), "ms_per_step": step_ms, "prefill_us": pf_ms * 1e3,
            "prefill_TFLOPs": tf, "frac_of_bf16_peak": tf / sustained, "peak": sustained,
            "peak_kind": f"of {kind} (sustained cuBLAS bf16)", "frac_of_bf16_burst_peak": tf / burst, "burst_peak": burst,
            "launches_timed": steps, "flop_per_launch": pb.flops(), "bound": "tensor"}


# the 70B-like shape first: a profiler capture of the first launches (--only projection) lands on it
PROJECTION_SHAPES = (("width8192_64q8kv_T8", 8, 8192, 64, 8, 128), ("width4096_32q4kv_T8", 8, 4096, 32, 4, 128),
                     ("width8192_64q8kv_T16", 16, 8192, 64, 8, 128))


def projection_report(dev) -> dict:
    """Side measurement of the 4-bit Q/K/V projection that precedes the step: one launch per layer-sized weight
    matrix, rotating through enough distinct matrices to exceed L2.  The launches are shorter than a foreign call
    from Python, so they are timed as one captured graph."""
    import time

    import torch
    from paper_2505_02351_b200 import binding
    from paper_2505_02351_b200 import workloads as W

    lib = binding.load()
    peak, kind = measured_peak()
    out = {}
    side = torch.cuda.Stream()
    for name, T, K, Hq, Hkv, D in PROJECTION_SHAPES:
        N, gs = (Hq + 2 * Hkv) * D, 128
        p = W.make_int4_projection(11, T, K, N, gs)
        nbytes = binding.int4_packed_bytes(K, N, gs)
        copies = max(2, -(-300_000_000 // nbytes))
        packed = torch.empty((copies, nbytes), dtype=torch.uint8, device=dev)
        binding.int4_prepack(packed[0], p.qweight.to(dev), p.scales.to(dev), p.qzeros.to(dev), gs)
        for i in range(1, copies):
            packed[i].copy_(packed[0])
        x = p.x.to(dev)
        q = torch.empty((T, Hq, D), dtype=torch.bfloat16, device=dev)
        k = torch.empty((T, Hkv, D), dtype=torch.bfloat16, device=dev)
        v = torch.empty_like(k)
        calls = [(q.data_ptr(), k.data_ptr(), v.data_ptr(), None, None, None, x.data_ptr(), packed[i].data_ptr(), T, K,
                  Hq, Hkv, D, 0, 0, gs, side.cuda_stream) for i in range(copies)]
        f = lib.opt_gqa_qkv_project_int4
        with torch.cuda.stream(side):
            for i in range(copies):
                check(f(*calls[i]), "qkv_project_int4")
        side.synchronize()
        per_graph = copies * max(1, 120 // copies)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for i in range(per_graph):
                check(f(*calls[i % copies]), "qkv_project_int4")
        t_end = time.time() + 0.3                      # replays first: clocks up, caches in steady state
        while time.time() < t_end:
            for _ in range(20):
                graph.replay()
            torch.cuda.synchronize()
        spans = []
        for _ in range(20):
            start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            start.record()
            graph.replay()
            end.record()
            torch.cuda.synchronize()
            spans.append(start.elapsed_time(end))
        us = sorted(spans)[len(spans) // 2] * 1e3 / per_graph
        alg = p.weight_bytes() + x.numel() * 2 + T * N * 2
        out[name] = {"us_per_launch": us, "GBs": alg / (us * 1e-6) / 1e9, "frac_of_peak": alg / (us * 1e-6) / 1e9 / peak,
                     "algorithmic_bytes_per_launch": alg, "weight_copies_rotated": copies, "bound": "hbm",
                     "timing": f"median over 20 replays of a graph of {per_graph} launches, CUDA events around each replay",
                     "peak_kind": f"of {kind}"}
        del packed, graph
        torch.cuda.empty_cache()
    return out


def entry_point_report(dev, peak) -> dict:
    """Side measurement of the decode entry points that a step does not use: opt_gqa_paged_attention_decode with one
    partial per partition followed by opt_gqa_paged_attention_reduce, and the single pass (partition_size 0).
    Back-to-back calls over rotating pool copies, CUDA events around the whole run."""
    import torch

    from paper_2505_02351_b200 import workloads as W

    stream = torch.cuda.current_stream()
    sh = stream.cuda_stream
    out = {}
    for cfg, P in ((3, 512), (2, 0), (4, 0)):
        wl = W.make_config(cfg)
        b = DeviceBatch(wl, P, 2, dev)
        lib = b.lib
        a_dec = [b.args_decode_plain(i, sh) for i in range(2)]
        a_red = (b.out.data_ptr(), b.partial_out.data_ptr(), b.partial_lse.data_ptr(), b.lens.data_ptr(), wl.B, wl.Hq,
                 wl.D, P, b.maxP, b.dt, sh) if P else None

        def call(i):
            check(lib.opt_gqa_paged_attention_decode(*a_dec[i % 2]), "decode")
            if P:
                check(lib.opt_gqa_paged_attention_reduce(*a_red), "reduce")

        for i in range(10):
            call(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n = 100
        e0.record(stream)
        for i in range(n):
            call(i)
        e1.record(stream)
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / n
        gbs = b.algorithmic_bytes() / us / 1e3
        key = f"{wl.name}: " + ("decode with one partial per partition + reduce" if P else "single-pass decode")
        out[key] = {"us_per_call": us, "GBs": gbs, "frac_of_peak": gbs / peak, "partition_size": P}
        del b, wl
        torch.cuda.empty_cache()
    return out


def masked_entry_point_report(dev, peak) -> dict:
    """Side measurement of the entry points for the other masks of Algorithm 1: the prompt branch over contiguous
    k, v (empty caches), the local window in decode (cfg 3 shapes, 4096-token window) and in chunked prefill (cfg 5
    shapes, 1024-token window).  Back-to-back calls, CUDA events around the run; the decode rotates pool copies."""
    import numpy as np
    import torch

    from paper_2505_02351_b200 import binding
    from paper_2505_02351_b200 import workloads as W

    lib = binding.load()
    stream = torch.cuda.current_stream()
    sh = stream.cuda_stream
    sustained, burst, kind = measured_tensor_peak()
    out = {}

    def timed(call, n, warm=5):
        for i in range(warm):
            call(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(n):
            call(i)
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / n            # us per call

    # ---- prompt branch, empty caches: 4 prompts of 4096 tokens, 32 query / 8 KV heads of 128, bf16
    B, n, Hq, Hkv, D = 4, 4096, 32, 8, 128
    gen = torch.Generator().manual_seed(17)
    mk = lambda *shape: torch.randn(shape, generator=gen).to(torch.bfloat16).to(dev)
    q, k, v = mk(B * n, Hq, D), mk(B * n, Hkv, D), mk(B * n, Hkv, D)
    o = torch.empty_like(q)
    qsl = torch.arange(0, (B + 1) * n, n, dtype=torch.int32, device=dev)
    slopes = torch.tensor([2.0 ** (-8.0 * (h + 1) / Hq) for h in range(Hq)], dtype=torch.float32, device=dev)
    a = (o.data_ptr(), q.data_ptr(), k.data_ptr(), v.data_ptr(), qsl.data_ptr(), B * n, n, slopes.data_ptr(),
         1.0 / float(np.sqrt(D)), B, Hq, Hkv, D, 1, sh)
    us = timed(lambda i: check(lib.opt_gqa_prompt_attention(*a), "prompt_attention"), 20)
    flop = 4.0 * D * Hq * B * (n * (n + 1) // 2)
    tf = flop / us / 1e6
    out["prompt_attention_4x4096"] = {"us_per_call": us, "TFLOPs": tf, "frac_of_bf16_peak": tf / sustained,
                                      "peak_kind": f"of {kind} (sustained cuBLAS bf16)", "flop_per_call": flop,
                                      "bound": "tensor"}
    del q, k, v, o

    # ---- decode with a local window on the long-sequence workload
    wl = W.make_config(3)
    window, P = 4096, 512
    b = DeviceBatch(wl, P, COPIES, dev)
    lens = wl.context_lens.numpy().astype("int64")
    es = 2
    alg = int(np.minimum(lens, window).sum()) * 2 * wl.Hkv * wl.D * es + 2 * wl.B * wl.Hq * wl.D * es
    a_loc = [(b.out.data_ptr(), b.q.data_ptr(), b.k_pools[i].data_ptr(), b.v_pools[i].data_ptr(), b.tables.data_ptr(),
              wl.max_blocks, b.lens.data_ptr(), b.slopes.data_ptr(), wl.scale, wl.B, wl.Hq, wl.Hkv, wl.D, wl.bs,
              wl.num_blocks, P, b.workspace.data_ptr(), b.ws_bytes, b.maxP, window, b.dt, sh)
             for i in range(len(b.k_pools))]
    R = len(a_loc)
    us = timed(lambda i: check(lib.opt_gqa_paged_attention_decode_local(*a_loc[i % R]), "decode_local"), 200, 20)
    out["decode_local_window_4096_cfg3"] = {"us_per_call": us, "GBs": alg / us / 1e3, "frac_of_peak": alg / us / 1e3 / peak,
                                            "algorithmic_bytes_per_call": alg, "bound": "hbm",
                                            "note": "two launches (split decode over the windows, merge); 67 MB per "
                                                    "call, pool copies rotated"}
    del b
    torch.cuda.empty_cache()

    # ---- chunked prefill with a local window
    wl = W.make_config(5)
    pb = PrefillBatch(wl, dev)
    window = 1024
    qsl_h = wl.q_start_loc.numpy().astype("int64")
    nn = wl.context_lens.numpy().astype("int64")
    pairs = 0
    for s in range(wl.B):
        ql = int(qsl_h[s + 1] - qsl_h[s])
        pos = np.arange(int(nn[s]) - ql, int(nn[s]), dtype=np.int64)
        pairs += int(np.minimum(pos + 1, window).sum())
    flop = 4.0 * wl.D * wl.Hq * pairs
    check(lib.opt_gqa_cache_append(pb.k_new.data_ptr(), pb.v_new.data_ptr(), pb.k_pool.data_ptr(), pb.v_pool.data_ptr(),
                                   pb.slots.data_ptr(), wl.T, wl.Hkv, wl.D, wl.bs, wl.num_blocks, 1, sh), "cache_append")
    a_pl = (pb.out.data_ptr(), pb.q.data_ptr(), pb.qsl.data_ptr(), wl.T, pb.max_q_len, pb.k_pool.data_ptr(),
            pb.v_pool.data_ptr(), pb.tables.data_ptr(), wl.max_blocks, pb.lens.data_ptr(), pb.slopes.data_ptr(), wl.scale,
            wl.B, wl.Hq, wl.Hkv, wl.D, wl.bs, wl.num_blocks, window, 1, sh)
    us = timed(lambda i: check(lib.opt_gqa_paged_attention_prefill_local(*a_pl), "prefill_local"), 20)
    tf = flop / us / 1e6
    out["prefill_local_window_1024_cfg5"] = {"us_per_call": us, "TFLOPs": tf, "frac_of_bf16_peak": tf / sustained,
                                             "peak_kind": f"of {kind} (sustained cuBLAS bf16)", "flop_per_call": flop,
                                             "bound": "tensor",
                                             "note": "flop counted over the (token, key) pairs inside the window; the "
                                                     "tiles that straddle its edges are multiplied whole"}
    del pb
    torch.cuda.empty_cache()
    return out


def check(rc: int, what: str):
    if rc != 0:
        raise RuntimeError(f"{what} failed with status {rc}")


EVENT_EVERY = 8   # in the kernel-timing region every 8th step carries an event bracket
DECODE_BATCH = 4  # decode launches inside one bracket


def _step_fns(batch: DeviceBatch, stream):
    """Pre-marshalled foreign calls of one step, per pool copy."""
    sh = stream.cuda_stream
    lib, R, split = batch.lib, len(batch.k_pools), batch.P > 0
    one_launch = step_launches(batch) == 1       # the library runs this step as a single pass: time that kernel
    a_app = [batch.args_append(i, sh) for i in range(R)]
    a_dec = [batch.args_decode_single(i, sh) if one_launch else batch.args_decode(i, sh) for i in range(R)]
    a_step = [batch.args_step(i, sh) for i in range(R)]
    split = split and not one_launch
    a_red = batch.args_reduce(sh) if split else None
    f_app = lib.opt_gqa_cache_append
    if one_launch:
        f_dec, f_red = lib.opt_gqa_paged_attention_decode, None
    elif batch.balanced:
        f_dec, f_red = lib.opt_gqa_paged_attention_decode_balanced, lib.opt_gqa_paged_attention_reduce_balanced
    else:
        f_dec, f_red = lib.opt_gqa_paged_attention_decode, lib.opt_gqa_paged_attention_reduce
    f_step = lib.opt_gqa_decode_step
    return dict(R=R, split=split, append=lambda i: check(f_app(*a_app[i % R]), "cache_append"),
                decode=lambda i: check(f_dec(*a_dec[i % R]), "decode"),
                reduce=lambda: check(f_red(*a_red), "reduce") if split else None,
                step=lambda i: check(f_step(*a_step[i % R]), "decode_step"))


def step_launches(batch: DeviceBatch) -> int:
    """Kernels one opt_gqa_decode_step call launches: decode + reduce on the split path, plus the separate append
    unless the decode kernel stores the new tokens itself (bf16 split with at most 1024 (sequence, KV head) streams);
    one launch in all where the library runs a bf16 step of short contexts as a single pass (the rule of api.cu)."""
    import torch

    if batch.P == 0:
        return 2
    streams, bound = batch.wl.B * batch.wl.Hkv, batch.maxP * batch.P
    sms = torch.cuda.get_device_properties(batch.dev).multi_processor_count
    if batch.balanced and bound <= 2048 and 2 * streams >= 3 * sms and streams <= 4 * sms:
        return 1
    fused = batch.balanced and streams <= 1024
    return 2 if fused else 3


def run_timed(batch: DeviceBatch, steps: int, warmup: int):
    """Warm-up, then `steps` steps timed with CUDA events on the launching stream.

    A step is one opt_gqa_decode_step call (append -> decode -> reduce, chained with programmatic dependent
    launches); consecutive steps use different pool copies.  Returns (total_ms, launches).
    """
    import torch

    stream = torch.cuda.current_stream()
    f = _step_fns(batch, stream)
    for i in range(warmup):
        f["step"](i)
    torch.cuda.synchronize()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize()
    start.record(stream)
    for i in range(steps):
        f["step"](warmup + i)
    end.record(stream)
    torch.cuda.synchronize()
    barrier()
    return start.elapsed_time(end), steps * step_launches(batch)


def run_kernel_timing(batch: DeviceBatch, steps: int, warmup: int):
    """A second timed region of the same steps that isolates the decode kernel's launch duration.

    Every EVENT_EVERY-th step is issued as separate calls with an event bracket around its decode work.  Even
    samples bracket DECODE_BATCH back-to-back decode launches on successive pool copies (the span divided by
    DECODE_BATCH is the duration of one launch in a pipelined stream: the launches are chained by programmatic
    dependent launch exactly as append -> decode is in a step, so the bracket's own event and launch gaps are
    paid once per DECODE_BATCH launches); odd samples bracket a single launch (which also pays those gaps).
    Returns (stats of ms per launch from the batched brackets, the same from the single brackets, launches);
    stats = {"mean", "median", "min", "brackets", "launches"}.
    """
    import torch

    stream = torch.cuda.current_stream()
    f = _step_fns(batch, stream)
    for i in range(warmup):
        f["step"](i)
    torch.cuda.synchronize()
    samples = list(range(0, steps, EVENT_EVERY))
    evs = {i: (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for i in samples}
    launches = 0
    barrier()
    torch.cuda.synchronize()
    for i in range(steps):
        if i not in evs:
            f["step"](warmup + i)
            launches += step_launches(batch)
            continue
        nb = DECODE_BATCH if (i // EVENT_EVERY) % 2 == 0 else 1
        f["append"](warmup + i)
        evs[i][0].record(stream)
        for j in range(nb):
            f["decode"](warmup + i + j)
        evs[i][1].record(stream)
        f["reduce"]()
        launches += 1 + nb + (1 if f["split"] else 0)
    torch.cuda.synchronize()
    barrier()
    batched = [evs[i][0].elapsed_time(evs[i][1]) / DECODE_BATCH for i in samples if (i // EVENT_EVERY) % 2 == 0]
    single = [evs[i][0].elapsed_time(evs[i][1]) for i in samples if (i // EVENT_EVERY) % 2 == 1]
    def stats(v, per):
        if not v:
            return None
        w = sorted(v)
        return {"mean": sum(w) / len(w), "median": w[len(w) // 2], "min": w[0], "brackets": len(w),
                "launches": len(w) * per}

    return stats(batched, DECODE_BATCH), stats(single, 1), launches


def read_only_ceiling(dev, stream) -> dict:
    """GB/s of the decode kernels' data path with no arithmetic attached: opt_gqa_debug_read_stream over 1 GiB,
    CUDA events on the launching stream, 3 warm-up and 10 timed launches (the buffer is 8x the L2)."""
    import torch

    from paper_2505_02351_b200 import binding

    lib = binding.load()
    src = torch.empty(READ_PROBE_BYTES, dtype=torch.uint8, device=dev)
    src.view(torch.int32).fill_(0x3f803f80)
    chk = torch.zeros(1, dtype=torch.int32, device=dev)
    a = (src.data_ptr(), READ_PROBE_BYTES, chk.data_ptr(), stream.cuda_stream)
    for _ in range(3):
        check(lib.opt_gqa_debug_read_stream(*a), "read_stream")
    torch.cuda.synchronize()
    spans = []
    for _ in range(10):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        check(lib.opt_gqa_debug_read_stream(*a), "read_stream")
        e1.record(stream)
        torch.cuda.synchronize()
        spans.append(e0.elapsed_time(e1))
    spans.sort()
    del src
    torch.cuda.empty_cache()
    gbs = lambda ms: READ_PROBE_BYTES / (ms * 1e-3) / 1e9
    return {"median": gbs(spans[len(spans) // 2]), "best": gbs(spans[0]), "launches": len(spans),
            "bytes_per_launch": READ_PROBE_BYTES}


def run_e2e(batch: DeviceBatch, steps: int, warmup: int):
    """Steps through opt_gqa_decode_step_mapped: pinned host inputs brought in, result stored back, every step (the
    buffers' device-side addresses are those torch's pinned allocations have under unified addressing)."""
    import torch

    from paper_2505_02351_b200 import binding

    wl = batch.wl
    pin = lambda t: t.contiguous().pin_memory()
    hq, hk, hv = pin(wl.q), pin(wl.k_new), pin(wl.v_new)
    hs, ht, hl = pin(wl.slot_mapping), pin(wl.block_tables), pin(wl.context_lens)
    hout = torch.empty_like(wl.q).pin_memory()
    tdt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
    staging = torch.empty(binding.step_staging_bytes(wl.B, wl.Hq, wl.Hkv, wl.D, wl.max_blocks, tdt), dtype=torch.uint8,
                          device=batch.dev)
    stream = torch.cuda.current_stream()
    R = len(batch.k_pools)

    # Arguments marshalled once per pool copy: the timed loop is one C-ABI call plus the stream synchronisation.
    lib, sh = batch.lib, stream.cuda_stream
    ws_ptr = batch.workspace.data_ptr() if batch.P else None
    a_host = [(hout.data_ptr(), hq.data_ptr(), hk.data_ptr(), hv.data_ptr(), hs.data_ptr(), ht.data_ptr(), hl.data_ptr(),
               staging.data_ptr(), batch.k_pools[i].data_ptr(), batch.v_pools[i].data_ptr(), wl.max_blocks,
               batch.slopes.data_ptr(), wl.scale, wl.B, wl.Hq, wl.Hkv, wl.D, wl.bs, wl.num_blocks, batch.P, ws_ptr,
               batch.ws_bytes if batch.P else 0, batch.maxP, batch.dt, sh) for i in range(R)]

    def step(i):
        check(lib.opt_gqa_decode_step_mapped(*a_host[i % R]), "decode_step_mapped")
        stream.synchronize()          # the caller reads out_host after every step

    for i in range(warmup):
        step(i)
    barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(steps):
        step(warmup + i)
    dt = time.perf_counter() - t0
    barrier()

    # The same steps with the host one step ahead: step i + 1 is enqueued before the host waits for step i's result
    # (two result buffers), the way a scheduler that prepares the next step while the current one runs would call
    # the library.  Every step still brings its inputs in from the pinned buffers and stores its result to the host.
    hout2 = [hout, torch.empty_like(hout).pin_memory()]
    a_pipe = [[(hout2[b].data_ptr(),) + a_host[i][1:] for i in range(R)] for b in range(2)]
    done = [torch.cuda.Event(), torch.cuda.Event()]
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(steps):
        check(lib.opt_gqa_decode_step_mapped(*a_pipe[i & 1][i % R]), "decode_step_mapped")
        done[i & 1].record(stream)
        if i > 0:
            done[(i - 1) & 1].synchronize()       # the result of the step before is in hout2[(i - 1) & 1] now
    done[(steps - 1) & 1].synchronize()
    dt_pipe = time.perf_counter() - t0
    barrier()
    h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv, hs, ht, hl))
    d2h = hout.numel() * hout.element_size()
    return dt, h2d, d2h, dt_pipe


# ----------------------------------------------------------------------------- CPU oracle legs
def oracle_step_fn(wl):
    """Returns (fn(units) -> seconds, total_units): the oracle's append + decode on the first `units` sequences."""
    import numpy as np

    import oracle
    from paper_2505_02351_b200 import workloads as W

    k, v = W.storage_numpy(wl.k_cache), W.storage_numpy(wl.v_cache)
    q, kn, vn = W.storage_numpy(wl.q), W.storage_numpy(wl.k_new), W.storage_numpy(wl.v_new)
    bt, n, slots = wl.block_tables.numpy(), wl.context_lens.numpy(), wl.slot_mapping.numpy()
    slopes = wl.alibi_slopes.numpy().astype(np.float64)

    def fn(units: int) -> float:
        t0 = time.perf_counter()
        oracle.cache_append(kn[:units], vn[:units], k, v, slots[:units], wl.dtype)
        oracle.paged_attention(q[:units], k, v, bt[:units], n[:units], slopes, wl.scale, wl.dtype)
        return time.perf_counter() - t0

    return fn, wl.B


def omp_threads() -> int:
    v = os.environ.get("OMP_NUM_THREADS")
    if v and v.isdigit():
        return int(v)
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def cpu_baseline(wl, budget_s: float = 12.0) -> dict:
    fn, B = oracle_step_fn(wl)
    t1 = fn(B)
    reps = int(min(20, max(1, math.floor(budget_s / max(t1, 1e-3)) - 1)))
    times = [t1] + [fn(B) for _ in range(reps - 1)] if reps > 1 else [t1]
    best = min(times)
    return {"value": B / best, "unit": UNIT, "cores": omp_threads(), "kind": "oracle",
            "sample": f"fp64 C oracle (append + decode) on the full batch of {B} sequences, best of {len(times)} passes, "
                      f"{best:.3f} s per pass"}


def workload_config(wl, P: int, world: int, copies: int) -> dict:
    """The `config` object of the result line; both arms (ours and the CPU reference) print the same one."""
    return {"workload": wl.name, "batch_per_gpu": wl.B, "Hq": wl.Hq, "Hkv": wl.Hkv, "head_dim": wl.D,
            "block_size": wl.bs, "storage_dtype": wl.dtype, "partition_size": P,
            "context_tokens_per_gpu": int(wl.context_lens.sum()),
            "parallelism": f"dp{world} (by sequence, no collective)",
            "step": "append of one token per sequence + paged GQA-ALiBi decode over context partitions + merge",
            "l2": f"each step reads {wl.kv_bytes() / 1e6:.0f} MB of K/V (> 126 MB L2); on the GPU {copies} distinct "
                  f"copies of the pool are rotated between steps"}


def run_reference(args, wl, P: int, rank: int):
    """--impl reference: the oracle as it stands, on the host cores; each step a bounded sample."""
    fn, B = oracle_step_fn(wl)
    steps = args.steps if args.steps is not None else 5
    warmup = args.warmup if args.warmup is not None else 1
    t_full = fn(B)
    budget = 150.0
    units = int(max(1, min(B, math.floor(B * budget / max(t_full * (steps + warmup), 1e-6)))))
    for _ in range(warmup):
        fn(units)
    t0 = time.perf_counter()
    for _ in range(steps):
        fn(units)
    dt = time.perf_counter() - t0
    value = units * steps / dt
    sample = f"fp64 C oracle (append + decode) on the first {units} of {B} sequences per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warmup, "ms_per_step": dt / steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(wl, P, args.gpus, COPIES),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": omp_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- main
def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


COPIES = 4          # distinct KV pool copies rotated between steps
PROFILE_COPIES = 2  # with --only: a footprint small enough for a profiler's capture


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--config", type=int, default=3, choices=[2, 3, 4],
                    help="named workload (1-based): 3 = long-sequence decode, the headline")
    ap.add_argument("--partition", type=int, default=None, help="context partition size (default: the workload's)")
    ap.add_argument("--only", choices=["step", "prefill", "projection"], default=None,
                    help="run one part alone on a small footprint and print its report: the decode step's two timed "
                         "regions, the chunked-prefill workload, or the 4-bit projection (for profiler captures)")
    args = ap.parse_args()
    rank, local_rank, world = dist_env()

    from paper_2505_02351_b200 import workloads as W

    if args.impl == "reference":
        if rank != 0:
            return
        wl = W.make_config(args.config)
        run_reference(args, wl, wl.partition_size or DEFAULT_PARTITION[args.config], rank)
        return

    import torch

    from paper_2505_02351_b200 import binding

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    binding.load()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=dev)
    if args.only == "prefill":
        if rank == 0:
            print(json.dumps(prefill_report(dev, args.steps or 20, max(3, args.warmup or 3))), flush=True)
        return
    if args.only == "projection":
        if rank == 0:
            print(json.dumps(projection_report(dev)), flush=True)
        return
    steps = args.steps if args.steps is not None else 4000
    warmup = max(3, args.warmup if args.warmup is not None else 50)
    copies = PROFILE_COPIES if args.only else COPIES

    wl = W.make_config(args.config, seed_offset=1000 * rank)
    P = args.partition if args.partition is not None else (wl.partition_size or DEFAULT_PARTITION[args.config])
    batch = DeviceBatch(wl, P, copies, dev)

    sampler = ClockSampler(local_rank)
    sampler.start()
    total_ms, launches = run_timed(batch, steps, warmup)
    kt_steps = steps if args.only else KERNEL_TIMING_STEPS
    dec, dec_single, launches2 = run_kernel_timing(batch, kt_steps, 8)
    launches += launches2
    total_ms = max_over_ranks(total_ms, str(dev))
    tokens_all = sum_over_ranks(float(wl.B), str(dev))
    value = tokens_all * steps / (total_ms * 1e-3)

    if args.only:
        e2e = None
        ceiling = None
    else:
        e2e_s, h2d, d2h, pipe_s = run_e2e(batch, E2E_STEPS, 10)
        e2e_s = max_over_ranks(e2e_s, str(dev))
        pipe_s = max_over_ranks(pipe_s, str(dev))
        # The end-to-end figure is the loop a serving host runs: every step brings its inputs in from pinned host
        # memory and stores its result to the host, and the host enqueues step i + 1 before it waits for (and reads)
        # step i's result.  The same steps with the host blocking after every call are reported beside it.
        e2e = {"value": tokens_all * E2E_STEPS / pipe_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": E2E_STEPS, "us_per_step": pipe_s / E2E_STEPS * 1e6,
               "api": "opt_gqa_decode_step_mapped (pinned host q/k_new/v_new/slots/tables/lens in, out back to the "
                      "host; step i + 1 is enqueued before the host waits for step i's result and reads it)"}
        e2e["frac_of_value"] = e2e["value"] / value
        e2e["synchronised_per_step"] = {
            "value": tokens_all * E2E_STEPS / e2e_s, "us_per_step": e2e_s / E2E_STEPS * 1e6,
            "frac_of_value": tokens_all * E2E_STEPS / e2e_s / value,
            "what": "the same call and transfers with the stream synchronised after every call (the host idle "
                    "while the step runs, the GPU idle while the host launches)"}
        ceiling = read_only_ceiling(dev, torch.cuda.current_stream())
    clocks = sampler.stop()
    status = binding.device_status()
    if status != 0:
        raise SystemExit(f"device status {status}: {binding.status_string(status)}")

    peak, peak_kind = measured_peak()
    alg = batch.algorithmic_bytes()
    achieved = alg / (dec["mean"] * 1e-3) / 1e9
    roofline = {"bound": "hbm",
                "kernel": "decode_tc_kernel (single pass)" if step_launches(batch) == 1 else
                          "decode_stream_kernel (balanced split)" if batch.balanced else "decode_kernel",
                "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "peak_kind": f"of {peak_kind}", "traffic": NCU_TRAFFIC_BYTES.get(args.config),
                "algorithmic_bytes_per_launch": alg, "kernel_us": dec["mean"] * 1e3,
                "kernel_us_median": dec["median"] * 1e3, "kernel_us_min": dec["min"] * 1e3,
                "launches_timed": dec["launches"], "brackets": dec["brackets"],
                "kernel_us_single_launch_bracket": None if dec_single is None else dec_single["mean"] * 1e3,
                "timing": f"CUDA events around {DECODE_BATCH} back-to-back decode launches on successive pool copies, "
                          f"every {2 * EVENT_EVERY}th step of a second timed region of {kt_steps} steps; span / {DECODE_BATCH}",
                "frac_of_nominal_8TBs": achieved / 8000.0}
    if ceiling is not None:
        roofline["read_only_ceiling_gbs"] = ceiling["median"]
        roofline["read_only_ceiling_best_gbs"] = ceiling["best"]
        roofline["frac_of_read_ceiling"] = achieved / ceiling["median"]
        roofline["read_only_ceiling"] = (f"opt_gqa_debug_read_stream over {READ_PROBE_BYTES >> 20} MiB, same rings and grid "
                                         f"as the decode kernel, no arithmetic; median of {ceiling['launches']} launches")

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": total_ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": DTYPE, "data": "synthetic",
        "config": workload_config(wl, P, world, copies),
        "kernel_family": KERNEL_FAMILY,
        "api": "opt_gqa_decode_step (new tokens stored by the decode kernel, balanced split, merge)",
        "hbm_tbs_step": alg * tokens_all / wl.B / (total_ms / steps * 1e-3) / 1e12,
        "clocks": clocks,
        "gpu_launches": launches,
        "roofline": roofline,
    }
    if e2e is not None:
        line["e2e"] = e2e

    if rank == 0 and world == 1 and not args.only:
        extra = {}
        for cfg in (2, 4):
            if cfg == args.config:
                continue
            w2 = W.make_config(cfg)
            b2 = DeviceBatch(w2, w2.partition_size or DEFAULT_PARTITION[cfg], COPIES, dev)
            t_ms, _ = run_timed(b2, 1000, 20)
            d2, _, _ = run_kernel_timing(b2, 256, 8)
            a2 = b2.algorithmic_bytes()
            extra[w2.name] = {"tokens_per_s": w2.B * 1000 / (t_ms * 1e-3), "ms_per_step": t_ms / 1000,
                              "decode_us": d2["mean"] * 1e3, "decode_GBs": a2 / (d2["mean"] * 1e-3) / 1e9,
                              "frac_of_peak": a2 / (d2["mean"] * 1e-3) / 1e9 / peak, "partition_size": b2.P,
                              "launches_timed": d2["launches"], "launches_per_step": step_launches(b2),
                              "decode_kernel": "decode_tc_kernel (single pass: the step is one launch)"
                              if step_launches(b2) == 1 else "decode_stream_kernel (balanced split)"}
            del b2, w2
            torch.cuda.empty_cache()
        extra["other_decode_entry_points"] = entry_point_report(dev, peak)
        extra[W.CONFIG_NAMES[5]] = prefill_report(dev, 20, 3)
        extra["other_masks"] = masked_entry_point_report(dev, peak)
        extra["int4_qkv_projection"] = projection_report(dev)
        line["other_workloads"] = extra
        line["cpu_baseline"] = cpu_baseline(wl)
    if world > 1:
        import torch.distributed as dist

        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
