"""Seeded synthetic inputs for the Opt-GQA path.

This module only draws numbers and lays them out; it holds none of the
attention arithmetic.  It serves the CUDA path, the CPU checker and the
benchmark alike, so that all of them see the same bits.

Every workload is a paged KV pool ``[num_blocks, Hkv, bs, D]`` whose pages are
handed out from a random permutation (the pool holds 1.2x the pages needed),
a block table per sequence (unused entries are -1), the context lengths
(counting the tokens that the step appends), the new tokens' K/V with their
slot mapping, the queries and the ALiBi slopes.  Values are N(0,1) drawn in
fp32 with ``torch.Generator().manual_seed(seed)`` and rounded once to the
storage type; lengths and permutations come from
``numpy.random.default_rng(seed)``.

The five named workloads stand in for long-sequence LLM serving traffic
(Llama-7B-like and 70B-like head shapes); no real model or dataset is used.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Optional

import numpy as np
import torch

TORCH_DTYPES = {"fp32": torch.float32, "bf16": torch.bfloat16}


@dataclass
class Workload:
    name: str
    dtype: str                      # "fp32" | "bf16"
    B: int
    Hq: int
    Hkv: int
    D: int
    bs: int
    num_blocks: int
    max_blocks: int
    scale: float
    partition_size: int             # 0 = single pass
    q: torch.Tensor                 # [T, Hq, D]
    k_cache: torch.Tensor           # [num_blocks, Hkv, bs, D]  state BEFORE the step's append
    v_cache: torch.Tensor
    block_tables: torch.Tensor      # [B, max_blocks] int32
    context_lens: torch.Tensor      # [B] int32, counts the appended tokens
    alibi_slopes: torch.Tensor      # [Hq] fp32
    k_new: torch.Tensor             # [T, Hkv, D]
    v_new: torch.Tensor
    slot_mapping: torch.Tensor      # [T] int64
    q_start_loc: Optional[torch.Tensor] = None   # [B+1] int32 (prefill only)
    meta: dict = field(default_factory=dict)

    @property
    def T(self) -> int:
        return int(self.q.shape[0])

    @property
    def max_partitions(self) -> int:
        if self.partition_size <= 0:
            return 1
        return max(1, int((int(self.context_lens.max()) + self.partition_size - 1) // self.partition_size))

    def kv_bytes(self) -> int:
        """Bytes of K and V that one decode step must read: sum_s n_s * 2 * Hkv * D * es."""
        es = 4 if self.dtype == "fp32" else 2
        return int(self.context_lens.to(torch.int64).sum()) * 2 * self.Hkv * self.D * es


def storage_numpy(t: torch.Tensor) -> np.ndarray:
    """fp32 tensor -> float32 array; bf16 tensor -> uint16 bit patterns (a copy)."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16).copy()
    return t.numpy().copy()


def alibi_slopes_input(Hq: int) -> torch.Tensor:
    """The slope vector handed to the library: 2^(-8(h+1)/Hq) rounded to fp32."""
    h = np.arange(1, Hq + 1, dtype=np.float64)
    return torch.from_numpy(np.exp2(-8.0 * h / Hq).astype(np.float32))


def _randn(shape, gen: torch.Generator, dtype: str) -> torch.Tensor:
    return torch.randn(shape, generator=gen, dtype=torch.float32).to(TORCH_DTYPES[dtype])


def make_custom(name: str, dtype: str, Hq: int, Hkv: int, D: int, bs: int, context_lens, q_lens=None,
                seed: int = 0, partition_size: int = 0, pool_factor: float = 1.2, poison: bool = False,
                shuffle_pages: bool = True, slopes: Optional[torch.Tensor] = None,
                scale: Optional[float] = None) -> Workload:
    """Build a workload from explicit lengths.

    ``context_lens[s]`` counts the ``q_lens[s]`` new tokens (default one per
    sequence: decode).  ``poison=True`` writes NaN bit patterns into every
    slot that no valid token occupies (spare pages, the tail of each last
    page) and into the slots the append must fill.
    """
    gen = torch.Generator(device="cpu").manual_seed(seed)
    rng = np.random.default_rng(seed)
    n = np.asarray(context_lens, dtype=np.int64)
    B = int(n.shape[0])
    decode = q_lens is None
    ql = np.ones(B, dtype=np.int64) if decode else np.asarray(q_lens, dtype=np.int64)
    assert decode or np.all(ql <= n)
    pages_per_seq = (n + bs - 1) // bs
    needed = int(pages_per_seq.sum())
    num_blocks = max(1, int(math.ceil(pool_factor * needed)))
    max_blocks = max(1, int(pages_per_seq.max()) if B else 1)
    perm = rng.permutation(num_blocks) if shuffle_pages else np.arange(num_blocks)
    bt = np.full((B, max_blocks), -1, dtype=np.int32)
    cur = 0
    for s in range(B):
        c = int(pages_per_seq[s])
        bt[s, :c] = perm[cur:cur + c]
        cur += c

    T = int(ql.sum())          # decode: one query row per sequence, even for an empty one (slot -1)
    k_cache = _randn((num_blocks, Hkv, bs, D), gen, dtype)
    v_cache = _randn((num_blocks, Hkv, bs, D), gen, dtype)
    q = _randn((T, Hq, D), gen, dtype)
    k_new = _randn((T, Hkv, D), gen, dtype)
    v_new = _randn((T, Hkv, D), gen, dtype)

    slot = np.empty(T, dtype=np.int64)
    qsl = np.zeros(B + 1, dtype=np.int32)
    t = 0
    for s in range(B):
        for i in range(int(ql[s])):
            pos = int(n[s] - ql[s] + i)
            slot[t] = int(bt[s, pos // bs]) * bs + pos % bs if pos >= 0 else -1
            t += 1
        qsl[s + 1] = t

    if poison:
        valid = np.zeros((num_blocks, bs), dtype=bool)
        for s in range(B):
            old = max(0, int(n[s] - ql[s]))  # tokens present before the append
            for i in range(int(pages_per_seq[s])):
                lo = i * bs
                cnt = min(bs, max(0, old - lo))
                valid[bt[s, i], :cnt] = True
        mask = torch.from_numpy(~valid)[:, None, :, None].expand(num_blocks, Hkv, bs, D)
        k_cache = torch.where(mask, torch.full_like(k_cache, float("nan")), k_cache)
        v_cache = torch.where(mask, torch.full_like(v_cache, float("nan")), v_cache)

    return Workload(
        name=name, dtype=dtype, B=B, Hq=Hq, Hkv=Hkv, D=D, bs=bs, num_blocks=num_blocks,
        max_blocks=max_blocks, scale=float(scale if scale is not None else 1.0 / math.sqrt(D)),
        partition_size=partition_size, q=q, k_cache=k_cache, v_cache=v_cache,
        block_tables=torch.from_numpy(bt), context_lens=torch.from_numpy(n.astype(np.int32)),
        alibi_slopes=alibi_slopes_input(Hq) if slopes is None else slopes.to(torch.float32),
        k_new=k_new, v_new=v_new, slot_mapping=torch.from_numpy(slot),
        q_start_loc=None if decode else torch.from_numpy(qsl),
        meta={"seed": seed, "poison": poison, "pages_needed": needed},
    )


CONFIG_NAMES = {
    1: "cfg1_tiny_fp32_decode",
    2: "cfg2_bf16_decode_llama7b_like",
    3: "cfg3_bf16_long_sequence_decode_p512",
    4: "cfg4_bf16_ragged_large_batch_decode_70b_like",
    5: "cfg5_bf16_chunked_prefill",
}


def config_lengths(cfg: int, shrink: int = 1):
    """Context lengths (and new-token counts) of the named workloads; seed = cfg - 1.

    ``shrink`` divides the sequence lengths (parity tests use reduced sizes
    where the checker would otherwise take minutes); 1 = the full workload.
    """
    rng = np.random.default_rng(cfg - 1)
    if cfg == 1:
        return np.array([37, 100]), None
    if cfg == 2:
        return rng.integers(512 // shrink, 2048 // shrink + 1, size=32), None
    if cfg == 3:
        return rng.integers(16384 // shrink, 32768 // shrink + 1, size=8), None
    if cfg == 4:
        n = np.clip(np.rint(np.exp2(rng.uniform(4.0, 13.0, size=256))), 16, 8192).astype(np.int64)
        return np.maximum(16 // min(shrink, 16), n // shrink), None
    if cfg == 5:
        return np.full(4, (4096 + 2048) // shrink), np.full(4, 2048 // shrink)
    raise ValueError(cfg)


def make_config(cfg: int, poison: bool = False, shrink: int = 1, seed_offset: int = 0) -> Workload:
    """The five named workloads (1-based), seeds 0..4 (``seed_offset`` gives other ranks their own values)."""
    n, ql = config_lengths(cfg, shrink)
    seed = cfg - 1 + seed_offset
    shape = {
        1: dict(dtype="fp32", Hq=4, Hkv=2, D=64, bs=16, partition_size=0),
        2: dict(dtype="bf16", Hq=32, Hkv=8, D=128, bs=16, partition_size=0),
        3: dict(dtype="bf16", Hq=32, Hkv=4, D=128, bs=16, partition_size=512),
        4: dict(dtype="bf16", Hq=64, Hkv=8, D=128, bs=32, partition_size=0),
        5: dict(dtype="bf16", Hq=32, Hkv=8, D=128, bs=16, partition_size=0),
    }[cfg]
    return make_custom(CONFIG_NAMES[cfg], context_lens=n, q_lens=ql, seed=seed, poison=poison, **shape)


@dataclass
class Int4Projection:
    """Inputs of the 4-bit Q/K/V projection: activations and one group-quantised weight matrix [K, N]."""
    x: torch.Tensor        # [T, K] bf16
    qweight: torch.Tensor  # [K/8, N] int32, eight 4-bit codes of consecutive rows per word
    scales: torch.Tensor   # [K/gs, N] bf16
    qzeros: torch.Tensor   # [K/gs, N/8] int32, eight 4-bit zero points of consecutive columns per word
    gs: int

    @property
    def K(self) -> int:
        return self.x.shape[1]

    @property
    def N(self) -> int:
        return self.qweight.shape[1]

    def weight_bytes(self) -> int:
        """Bytes of codes, scales and zero points in the interchange layout (read once per projection)."""
        return self.qweight.numel() * 4 + self.scales.numel() * 2 + self.qzeros.numel() * 4


def make_int4_projection(seed: int, T: int, K: int, N: int, gs: int = 128) -> Int4Projection:
    """Random codes and zero points (uniform words), scales near 0.008 (the step of a 4-bit grid over
    weights of standard deviation ~0.02), activations N(0,1) rounded to bf16."""
    rng = np.random.default_rng(seed)
    gen = torch.Generator(device="cpu").manual_seed(seed)
    qweight = torch.from_numpy(rng.integers(0, 2**32, size=(K // 8, N), dtype=np.uint32).view(np.int32))
    qzeros = torch.from_numpy(rng.integers(0, 2**32, size=(K // gs, N // 8), dtype=np.uint32).view(np.int32))
    scales = (0.006 + 0.004 * torch.rand((K // gs, N), generator=gen, dtype=torch.float32)).to(torch.bfloat16)
    x = torch.randn((T, K), generator=gen, dtype=torch.float32).to(torch.bfloat16)
    return Int4Projection(x=x, qweight=qweight, scales=scales, qzeros=qzeros, gs=gs)
