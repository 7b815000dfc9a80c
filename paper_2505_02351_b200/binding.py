"""ctypes binding of ``libopt_gqa.so``: argument marshalling only.

Each function has the name of the C entry point it calls (without the
``opt_gqa_`` prefix), takes CUDA torch tensors, passes their ``data_ptr()``
and sizes straight through, and raises :class:`OptGqaError` on a non-zero
status.  There is no fallback of any kind: if the shared library is missing
or a tensor is not on a CUDA device the call fails.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libopt_gqa.so")

FP32, BF16 = 0, 1
_DTYPE_CODE = {torch.float32: FP32, torch.bfloat16: BF16}

_c = ctypes
_vp, _i, _i64, _f, _sz = _c.c_void_p, _c.c_int, _c.c_int64, _c.c_float, _c.c_size_t

SIGNATURES = {
    "opt_gqa_int4_packed_bytes": (ctypes.c_size_t, [_i, _i, _i]),
    "opt_gqa_int4_prepack": (_i, [_vp, _vp, _vp, _vp, _i, _i, _i, _vp]),
    "opt_gqa_qkv_project_int4": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _i64, _i, _vp]),
    "opt_gqa_cache_append": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i64, _i, _vp]),
    "opt_gqa_paged_attention_decode": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _vp, _vp, _f, _i, _i, _i, _i, _i, _i64,
                                            _i, _vp, _vp, _i, _i, _vp]),
    "opt_gqa_paged_attention_decode_simt": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _vp, _vp, _f, _i, _i, _i, _i, _i, _i64,
                                                 _i, _vp, _vp, _i, _i, _vp]),
    "opt_gqa_paged_attention_decode_balanced": (_i, [_vp, _vp, _vp, _vp, _i, _vp, _vp, _f, _i, _i, _i, _i, _i, _i64,
                                                     _i, _vp, _sz, _i, _i, _vp]),
    "opt_gqa_paged_attention_reduce_balanced": (_i, [_vp, _vp, _sz, _vp, _i, _i, _i, _i, _i, _i, _i, _vp]),
    "opt_gqa_paged_attention_decode_no_alloc": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _vp, _vp, _f, _i, _i, _i, _i, _i,
                                                     _i64, _i, _i, _i, _vp]),
    "opt_gqa_paged_attention_reduce": (_i, [_vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _vp]),
    "opt_gqa_paged_attention_prefill": (_i, [_vp, _vp, _vp, _i, _i, _vp, _vp, _vp, _i, _vp, _vp, _f, _i, _i, _i, _i,
                                             _i, _i64, _i, _vp]),
    "opt_gqa_paged_attention_prefill_mma": (_i, [_vp, _vp, _vp, _i, _i, _vp, _vp, _vp, _i, _vp, _vp, _f, _i, _i, _i,
                                                 _i, _i, _i64, _i, _vp]),
    "opt_gqa_paged_attention_decode_local": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _vp, _vp, _f, _i, _i, _i, _i, _i, _i64,
                                                  _i, _vp, _sz, _i, _i, _i, _vp]),
    "opt_gqa_paged_attention_prefill_local": (_i, [_vp, _vp, _vp, _i, _i, _vp, _vp, _vp, _i, _vp, _vp, _f, _i, _i, _i,
                                                   _i, _i, _i64, _i, _i, _vp]),
    "opt_gqa_prompt_attention": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _vp, _f, _i, _i, _i, _i, _i, _vp]),
    "opt_gqa_decode_step": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _vp, _vp, _f, _i, _i, _i, _i, _i, _i64,
                                 _i, _vp, _sz, _i, _i, _vp]),
    "opt_gqa_decode_step_host": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _vp, _f, _i, _i, _i, _i,
                                      _i, _i64, _i, _vp, _sz, _i, _i, _vp]),
    "opt_gqa_decode_step_mapped": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _vp, _f, _i, _i, _i, _i,
                                        _i, _i64, _i, _vp, _sz, _i, _i, _vp]),
    "opt_gqa_step_staging_bytes": (_c.c_size_t, [_i, _i, _i, _i, _i, _i]),
    "opt_gqa_workspace_bytes": (_c.c_size_t, [_i, _i, _i, _i]),
    "opt_gqa_debug_wait_timeout": (_i, [_c.c_longlong, _vp]),
    "opt_gqa_debug_read_stream": (_i, [_vp, _sz, _vp, _vp]),
    "opt_gqa_device_status": (_i, []),
    "opt_gqa_status_string": (_c.c_char_p, [_i]),
}

_lib: Optional[ctypes.CDLL] = None


class OptGqaError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


def load() -> ctypes.CDLL:
    """Loads the shared library (built in-tree by ``paper_2505_02351_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2505_02351_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    return t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream if stream is not None else torch.cuda.current_stream()).cuda_stream


def _check(code: int, where: str) -> None:
    if code != 0:
        raise OptGqaError(code, where)


def status_string(code: int) -> str:
    return load().opt_gqa_status_string(code).decode()


def workspace_bytes(B: int, Hq: int, D: int, max_partitions: int) -> int:
    return int(load().opt_gqa_workspace_bytes(B, Hq, D, max_partitions))


def device_status() -> int:
    return int(load().opt_gqa_device_status())


def debug_wait_timeout(limit_cycles: int, stream=None) -> None:
    """Launches one warp whose bounded wait runs out after `limit_cycles` SM clocks (sets the device status)."""
    _check(load().opt_gqa_debug_wait_timeout(limit_cycles, _stream(stream)), "opt_gqa_debug_wait_timeout")


def debug_read_stream(src, checksum, stream=None) -> None:
    """Streams all of `src` through the decode kernels' data path with no arithmetic (read-bandwidth ceiling)."""
    assert checksum.dtype == torch.int32 and checksum.numel() >= 1
    _check(load().opt_gqa_debug_read_stream(_ptr(src), src.numel() * src.element_size(), _ptr(checksum),
                                            _stream(stream)), "opt_gqa_debug_read_stream")


def _nbytes(t: Optional[torch.Tensor]) -> int:
    return 0 if t is None else t.numel() * t.element_size()


def cache_append(k_new, v_new, k_cache, v_cache, slot_mapping, stream=None) -> None:
    T, Hkv, D = k_new.shape
    num_blocks, _, bs, _ = k_cache.shape
    assert slot_mapping.dtype == torch.int64
    _check(load().opt_gqa_cache_append(_ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), _ptr(slot_mapping),
                                       T, Hkv, D, bs, num_blocks, _DTYPE_CODE[k_cache.dtype], _stream(stream)),
           "opt_gqa_cache_append")


def _decode(entry: str, out, q, k_cache, v_cache, block_tables, context_lens, alibi_slopes, scale, partition_size,
            partial_out, partial_lse, max_partitions, stream) -> None:
    B, Hq, D = q.shape
    num_blocks, Hkv, bs, _ = k_cache.shape
    assert block_tables.dtype == torch.int32 and context_lens.dtype == torch.int32
    assert alibi_slopes is None or alibi_slopes.dtype == torch.float32
    _check(getattr(load(), entry)(
        _ptr(out), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(block_tables), block_tables.shape[1],
        _ptr(context_lens), _ptr(alibi_slopes), scale, B, Hq, Hkv, D, bs, num_blocks, partition_size,
        _ptr(partial_out), _ptr(partial_lse), max_partitions, _DTYPE_CODE[q.dtype], _stream(stream)), entry)


def paged_attention_decode(out, q, k_cache, v_cache, block_tables, context_lens, alibi_slopes, scale: float,
                           partition_size: int = 0, partial_out=None, partial_lse=None, max_partitions: int = 0,
                           stream=None) -> None:
    _decode("opt_gqa_paged_attention_decode", out, q, k_cache, v_cache, block_tables, context_lens, alibi_slopes,
            scale, partition_size, partial_out, partial_lse, max_partitions, stream)


def paged_attention_decode_simt(out, q, k_cache, v_cache, block_tables, context_lens, alibi_slopes, scale: float,
                                partition_size: int = 0, partial_out=None, partial_lse=None,
                                max_partitions: int = 0, stream=None) -> None:
    _decode("opt_gqa_paged_attention_decode_simt", out, q, k_cache, v_cache, block_tables, context_lens,
            alibi_slopes, scale, partition_size, partial_out, partial_lse, max_partitions, stream)


def paged_attention_decode_balanced(q, k_cache, v_cache, block_tables, context_lens, alibi_slopes, scale: float,
                                    partition_size: int, workspace, max_partitions: int, stream=None) -> None:
    B, Hq, D = q.shape
    num_blocks, Hkv, bs, _ = k_cache.shape
    assert block_tables.dtype == torch.int32 and context_lens.dtype == torch.int32
    assert alibi_slopes is None or alibi_slopes.dtype == torch.float32
    _check(load().opt_gqa_paged_attention_decode_balanced(
        _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(block_tables), block_tables.shape[1], _ptr(context_lens),
        _ptr(alibi_slopes), scale, B, Hq, Hkv, D, bs, num_blocks, partition_size, _ptr(workspace), _nbytes(workspace),
        max_partitions, _DTYPE_CODE[q.dtype], _stream(stream)), "opt_gqa_paged_attention_decode_balanced")


def paged_attention_reduce_balanced(out, workspace, context_lens, Hkv: int, partition_size: int, max_partitions: int,
                                    stream=None) -> None:
    B, Hq, D = out.shape
    _check(load().opt_gqa_paged_attention_reduce_balanced(
        _ptr(out), _ptr(workspace), _nbytes(workspace), _ptr(context_lens), B, Hq, Hkv, D, partition_size,
        max_partitions, _DTYPE_CODE[out.dtype], _stream(stream)), "opt_gqa_paged_attention_reduce_balanced")


def paged_attention_decode_no_alloc(out, q, k_cache, v_cache, block_tables, context_lens, alibi_slopes, scale: float,
                                    partition_size: int, max_partitions: int, stream=None) -> None:
    """Partitioned decode + merge with the library's built-in scratch array (nothing is allocated)."""
    B, Hq, D = q.shape
    num_blocks, Hkv, bs, _ = k_cache.shape
    assert block_tables.dtype == torch.int32 and context_lens.dtype == torch.int32
    assert alibi_slopes is None or alibi_slopes.dtype == torch.float32
    _check(load().opt_gqa_paged_attention_decode_no_alloc(
        _ptr(out), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(block_tables), block_tables.shape[1],
        _ptr(context_lens), _ptr(alibi_slopes), scale, B, Hq, Hkv, D, bs, num_blocks, partition_size,
        max_partitions, _DTYPE_CODE[q.dtype], _stream(stream)), "opt_gqa_paged_attention_decode_no_alloc")


def paged_attention_reduce(out, partial_out, partial_lse, context_lens, partition_size: int, stream=None) -> None:
    B, Hq, max_partitions, D = partial_out.shape
    assert partial_out.dtype == torch.float32 and partial_lse.dtype == torch.float32
    _check(load().opt_gqa_paged_attention_reduce(
        _ptr(out), _ptr(partial_out), _ptr(partial_lse), _ptr(context_lens), B, Hq, D, partition_size,
        max_partitions, _DTYPE_CODE[out.dtype], _stream(stream)), "opt_gqa_paged_attention_reduce")


def _prefill(entry: str, out, q, q_start_loc, max_q_len, k_cache, v_cache, block_tables, context_lens, alibi_slopes,
             scale, stream) -> None:
    T, Hq, D = q.shape
    num_blocks, Hkv, bs, _ = k_cache.shape
    B = context_lens.shape[0]
    assert q_start_loc.dtype == torch.int32
    _check(getattr(load(), entry)(
        _ptr(out), _ptr(q), _ptr(q_start_loc), T, max_q_len, _ptr(k_cache), _ptr(v_cache), _ptr(block_tables),
        block_tables.shape[1], _ptr(context_lens), _ptr(alibi_slopes), scale, B, Hq, Hkv, D, bs, num_blocks,
        _DTYPE_CODE[q.dtype], _stream(stream)), entry)


def paged_attention_prefill(out, q, q_start_loc, max_q_len: int, k_cache, v_cache, block_tables, context_lens,
                            alibi_slopes, scale: float, stream=None) -> None:
    _prefill("opt_gqa_paged_attention_prefill", out, q, q_start_loc, max_q_len, k_cache, v_cache, block_tables,
             context_lens, alibi_slopes, scale, stream)


def paged_attention_prefill_mma(out, q, q_start_loc, max_q_len: int, k_cache, v_cache, block_tables, context_lens,
                                alibi_slopes, scale: float, stream=None) -> None:
    _prefill("opt_gqa_paged_attention_prefill_mma", out, q, q_start_loc, max_q_len, k_cache, v_cache, block_tables,
             context_lens, alibi_slopes, scale, stream)


def paged_attention_decode_local(out, q, k_cache, v_cache, block_tables, context_lens, alibi_slopes, scale: float,
                                 partition_size: int, workspace, max_partitions: int, window: int, stream=None) -> None:
    """Balanced decode + merge where every query sees only the last `window` keys of its sequence."""
    B, Hq, D = q.shape
    num_blocks, Hkv, bs, _ = k_cache.shape
    _check(load().opt_gqa_paged_attention_decode_local(
        _ptr(out), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(block_tables), block_tables.shape[1],
        _ptr(context_lens), _ptr(alibi_slopes), scale, B, Hq, Hkv, D, bs, num_blocks, partition_size, _ptr(workspace),
        _nbytes(workspace), max_partitions, window, _DTYPE_CODE[q.dtype], _stream(stream)),
        "opt_gqa_paged_attention_decode_local")


def paged_attention_prefill_local(out, q, q_start_loc, max_q_len: int, k_cache, v_cache, block_tables, context_lens,
                                  alibi_slopes, scale: float, window: int, stream=None) -> None:
    """Chunked prefill where the token at pos sees keys pos - window < j <= pos."""
    T, Hq, D = q.shape
    num_blocks, Hkv, bs, _ = k_cache.shape
    B = context_lens.shape[0]
    _check(load().opt_gqa_paged_attention_prefill_local(
        _ptr(out), _ptr(q), _ptr(q_start_loc), T, max_q_len, _ptr(k_cache), _ptr(v_cache), _ptr(block_tables),
        block_tables.shape[1], _ptr(context_lens), _ptr(alibi_slopes), scale, B, Hq, Hkv, D, bs, num_blocks, window,
        _DTYPE_CODE[q.dtype], _stream(stream)), "opt_gqa_paged_attention_prefill_local")


def prompt_attention(out, q, k, v, q_start_loc, max_q_len: int, alibi_slopes, scale: float, stream=None) -> None:
    """Causal GQA-ALiBi attention of each sequence over its own new tokens (contiguous k, v; empty caches)."""
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    B = q_start_loc.shape[0] - 1
    assert q_start_loc.dtype == torch.int32 and k.shape == v.shape and k.shape[0] == T
    _check(load().opt_gqa_prompt_attention(
        _ptr(out), _ptr(q), _ptr(k), _ptr(v), _ptr(q_start_loc), T, max_q_len, _ptr(alibi_slopes), scale, B, Hq, Hkv,
        D, _DTYPE_CODE[q.dtype], _stream(stream)), "opt_gqa_prompt_attention")


def int4_packed_bytes(K: int, N: int, gs: int) -> int:
    return int(load().opt_gqa_int4_packed_bytes(K, N, gs))


def int4_prepack(packed, qweight, scales, qzeros, gs: int, stream=None) -> None:
    """Rewrite qweight [K/8, N] int32, scales [K/gs, N] bf16, qzeros [K/gs, N/8] int32 into the kernel's layout."""
    K, N = qweight.shape[0] * 8, qweight.shape[1]
    assert scales.dtype == torch.bfloat16 and qweight.dtype == torch.int32 and qzeros.dtype == torch.int32
    assert packed.numel() * packed.element_size() >= int4_packed_bytes(K, N, gs) > 0
    _check(load().opt_gqa_int4_prepack(_ptr(packed), _ptr(qweight), _ptr(scales), _ptr(qzeros), K, N, gs,
                                       _stream(stream)), "opt_gqa_int4_prepack")


def qkv_project_int4(q_out, x, packed, Hq: int, Hkv: int, D: int, gs: int, k_out=None, v_out=None, k_cache=None,
                     v_cache=None, slot_mapping=None, stream=None) -> None:
    """q, k, v = x W (Eq. 1) from 4-bit weights; k, v go to k_out/v_out and/or into the paged cache."""
    T, K = x.shape
    assert x.dtype == torch.bfloat16 and q_out.dtype == torch.bfloat16
    num_blocks, bs = (k_cache.shape[0], k_cache.shape[2]) if k_cache is not None else (0, 0)
    _check(load().opt_gqa_qkv_project_int4(
        _ptr(q_out), _ptr(k_out), _ptr(v_out), _ptr(k_cache), _ptr(v_cache), _ptr(slot_mapping), _ptr(x),
        _ptr(packed), T, K, Hq, Hkv, D, bs, num_blocks, gs, _stream(stream)), "opt_gqa_qkv_project_int4")


def step_staging_bytes(B: int, Hq: int, Hkv: int, D: int, max_blocks_per_seq: int, dtype: torch.dtype) -> int:
    return int(load().opt_gqa_step_staging_bytes(B, Hq, Hkv, D, max_blocks_per_seq, _DTYPE_CODE[dtype]))


def decode_step(out, q, k_new, v_new, slot_mapping, k_cache, v_cache, block_tables, context_lens, alibi_slopes,
                scale: float, partition_size: int = 0, workspace=None, max_partitions: int = 0, stream=None) -> None:
    B, Hq, D = q.shape
    num_blocks, Hkv, bs, _ = k_cache.shape
    _check(load().opt_gqa_decode_step(
        _ptr(out), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(slot_mapping), _ptr(k_cache), _ptr(v_cache),
        _ptr(block_tables), block_tables.shape[1], _ptr(context_lens), _ptr(alibi_slopes), scale, B, Hq, Hkv, D, bs,
        num_blocks, partition_size, _ptr(workspace), _nbytes(workspace), max_partitions, _DTYPE_CODE[q.dtype],
        _stream(stream)), "opt_gqa_decode_step")


def _host_ptr(t: torch.Tensor) -> int:
    if t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous host tensor")
    return t.data_ptr()


def decode_step_host(out_host, q_host, k_new_host, v_new_host, slot_mapping_host, block_tables_host,
                     context_lens_host, staging, k_cache, v_cache, alibi_slopes, scale: float,
                     partition_size: int = 0, workspace=None, max_partitions: int = 0, stream=None) -> None:
    """Host tensors (pinned) in and out; cache, slopes, staging and workspace on the device.  Does not synchronise."""
    B, Hq, D = q_host.shape
    num_blocks, Hkv, bs, _ = k_cache.shape
    _check(load().opt_gqa_decode_step_host(
        _host_ptr(out_host), _host_ptr(q_host), _host_ptr(k_new_host), _host_ptr(v_new_host),
        _host_ptr(slot_mapping_host), _host_ptr(block_tables_host), _host_ptr(context_lens_host), _ptr(staging),
        _ptr(k_cache), _ptr(v_cache), block_tables_host.shape[1], _ptr(alibi_slopes), scale, B, Hq, Hkv, D, bs,
        num_blocks, partition_size, _ptr(workspace), _nbytes(workspace), max_partitions, _DTYPE_CODE[q_host.dtype],
        _stream(stream)), "opt_gqa_decode_step_host")


def _pinned_view(t: torch.Tensor) -> int:
    """Device-side address of a page-locked host tensor.  torch allocates pinned memory with cudaHostAlloc, whose
    device-side address under unified addressing is the host address itself."""
    if t.is_cuda or not t.is_contiguous() or not t.is_pinned():
        raise ValueError("expected a contiguous page-locked (pinned) host tensor")
    return t.data_ptr()


def decode_step_mapped(out_host, q_host, k_new_host, v_new_host, slot_mapping_host, block_tables_host,
                       context_lens_host, staging, k_cache, v_cache, alibi_slopes, scale: float,
                       partition_size: int = 0, workspace=None, max_partitions: int = 0, stream=None) -> None:
    """decode_step_host for pinned tensors whose device-side addresses are passed as they are (no pointer queries)."""
    B, Hq, D = q_host.shape
    num_blocks, Hkv, bs, _ = k_cache.shape
    _check(load().opt_gqa_decode_step_mapped(
        _pinned_view(out_host), _pinned_view(q_host), _pinned_view(k_new_host), _pinned_view(v_new_host),
        _pinned_view(slot_mapping_host), _pinned_view(block_tables_host), _pinned_view(context_lens_host), _ptr(staging),
        _ptr(k_cache), _ptr(v_cache), block_tables_host.shape[1], _ptr(alibi_slopes), scale, B, Hq, Hkv, D, bs,
        num_blocks, partition_size, _ptr(workspace), _nbytes(workspace), max_partitions, _DTYPE_CODE[q_host.dtype],
        _stream(stream)), "opt_gqa_decode_step_mapped")
