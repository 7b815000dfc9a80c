"""Opt-GQA CPU oracle: TEST INFRASTRUCTURE, not product code.

ctypes front end of ``opt_gqa_oracle.c`` (plain C, fp64).  Only the tests, the
smoke check and the benchmark's CPU-baseline leg import this package; the CUDA
library and its Python binding never do, and nothing here imports them.

Arrays are numpy.  bf16 tensors are passed as ``uint16`` bit patterns
(``dtype="bf16"``), fp32 tensors as ``float32`` (``dtype="fp32"``); the C code
widens them exactly to double.  Outputs are ``float64``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "opt_gqa_oracle.c")
_LIB = os.path.join(_HERE, "liboptgqa_oracle.so")
_lib = None

DTYPES = {"fp32": 0, "bf16": 1}


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP over (sequence, head))."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_cache_append.restype = ctypes.c_int
        _lib.oracle_paged_attention.restype = ctypes.c_int
        _lib.oracle_partition_partials.restype = ctypes.c_int
        _lib.oracle_reduce.restype = ctypes.c_int
        _lib.oracle_prompt_attention.restype = ctypes.c_int
        _lib.oracle_qkv_project_int4.restype = ctypes.c_int
        _lib.oracle_alibi_slopes.restype = None
        _lib.oracle_unpage.restype = None
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check_store(a: np.ndarray, dtype: str) -> np.ndarray:
    want = np.float32 if dtype == "fp32" else np.uint16
    if a.dtype != want:
        raise TypeError(f"{dtype} storage must be {want}, got {a.dtype}")
    return np.ascontiguousarray(a)


def alibi_slopes(Hq: int) -> np.ndarray:
    """slope_h = 2^(-8(h+1)/Hq), h = 0..Hq-1."""
    out = np.empty(Hq, dtype=np.float64)
    lib().oracle_alibi_slopes(ctypes.c_int(Hq), _p(out))
    return out


def cache_append(k_new, v_new, k_cache, v_cache, slot_mapping, dtype: str) -> None:
    """In-place slot-mapped write of new K/V rows into the paged pool."""
    k_new, v_new = _check_store(k_new, dtype), _check_store(v_new, dtype)
    assert k_cache.flags.c_contiguous and v_cache.flags.c_contiguous
    _check_store(k_cache, dtype), _check_store(v_cache, dtype)
    slot_mapping = np.ascontiguousarray(slot_mapping, dtype=np.int64)
    T, Hkv, D = k_new.shape
    num_blocks, Hkv2, bs, D2 = k_cache.shape
    assert (Hkv, D) == (Hkv2, D2) and slot_mapping.shape == (T,)
    rc = lib().oracle_cache_append(
        _p(k_new), _p(v_new), _p(k_cache), _p(v_cache), _p(slot_mapping),
        ctypes.c_int(T), ctypes.c_int(Hkv), ctypes.c_int(D), ctypes.c_int(bs),
        ctypes.c_int64(num_blocks), ctypes.c_int(DTYPES[dtype]),
    )
    if rc != 0:
        raise ValueError("slot outside the pool")


def paged_attention(q, k_cache, v_cache, block_tables, context_lens, slopes, scale, dtype: str,
                    q_start_loc=None, window: int = 0) -> np.ndarray:
    """Decode (q_start_loc None: one query token per sequence) or causal prefill over the paged cache."""
    q = _check_store(q, dtype)
    k_cache, v_cache = _check_store(k_cache, dtype), _check_store(v_cache, dtype)
    block_tables = np.ascontiguousarray(block_tables, dtype=np.int32)
    context_lens = np.ascontiguousarray(context_lens, dtype=np.int32)
    T, Hq, D = q.shape
    num_blocks, Hkv, bs, D2 = k_cache.shape
    B, max_blocks = block_tables.shape
    assert D == D2 and context_lens.shape == (B,)
    if q_start_loc is not None:
        q_start_loc = np.ascontiguousarray(q_start_loc, dtype=np.int32)
        assert q_start_loc.shape == (B + 1,) and q_start_loc[-1] == T
    else:
        assert T == B
    if slopes is not None:
        slopes = np.ascontiguousarray(slopes, dtype=np.float64)
        assert slopes.shape == (Hq,)
    out = np.empty((T, Hq, D), dtype=np.float64)
    rc = lib().oracle_paged_attention(
        _p(out), _p(q), _p(k_cache), _p(v_cache), _p(block_tables), ctypes.c_int(max_blocks),
        _p(context_lens), _p(q_start_loc), _p(slopes), ctypes.c_double(scale),
        ctypes.c_int(B), ctypes.c_int(Hq), ctypes.c_int(Hkv), ctypes.c_int(D), ctypes.c_int(bs),
        ctypes.c_int(DTYPES[dtype]), ctypes.c_int(window),
    )
    if rc != 0:
        raise ValueError("bad shapes")
    return out


def partition_partials(q, k_cache, v_cache, block_tables, context_lens, slopes, scale, dtype: str,
                       P: int, max_partitions: int):
    """Per-partition normalised outputs and log-sum-exps of decode attention."""
    q = _check_store(q, dtype)
    k_cache, v_cache = _check_store(k_cache, dtype), _check_store(v_cache, dtype)
    block_tables = np.ascontiguousarray(block_tables, dtype=np.int32)
    context_lens = np.ascontiguousarray(context_lens, dtype=np.int32)
    B, Hq, D = q.shape
    num_blocks, Hkv, bs, _ = k_cache.shape
    max_blocks = block_tables.shape[1]
    if slopes is not None:
        slopes = np.ascontiguousarray(slopes, dtype=np.float64)
    po = np.empty((B, Hq, max_partitions, D), dtype=np.float64)
    pl = np.empty((B, Hq, max_partitions), dtype=np.float64)
    rc = lib().oracle_partition_partials(
        _p(po), _p(pl), _p(q), _p(k_cache), _p(v_cache), _p(block_tables), ctypes.c_int(max_blocks),
        _p(context_lens), _p(slopes), ctypes.c_double(scale), ctypes.c_int(B), ctypes.c_int(Hq),
        ctypes.c_int(Hkv), ctypes.c_int(D), ctypes.c_int(bs), ctypes.c_int(DTYPES[dtype]),
        ctypes.c_int(P), ctypes.c_int(max_partitions),
    )
    if rc != 0:
        raise ValueError("bad shapes")
    return po, pl


def reduce(partial_out, partial_lse, context_lens, P: int) -> np.ndarray:
    """Log-sum-exp merge of the partitions."""
    partial_out = np.ascontiguousarray(partial_out, dtype=np.float64)
    partial_lse = np.ascontiguousarray(partial_lse, dtype=np.float64)
    context_lens = np.ascontiguousarray(context_lens, dtype=np.int32)
    B, Hq, maxP, D = partial_out.shape
    out = np.empty((B, Hq, D), dtype=np.float64)
    rc = lib().oracle_reduce(
        _p(out), _p(partial_out), _p(partial_lse), _p(context_lens), ctypes.c_int(B), ctypes.c_int(Hq),
        ctypes.c_int(D), ctypes.c_int(P), ctypes.c_int(maxP),
    )
    if rc != 0:
        raise ValueError("max_partitions too small")
    return out


def prompt_attention(q, k, v, q_start_loc, slopes, scale, dtype: str) -> np.ndarray:
    """Causal attention of every sequence over its own tokens, contiguous q [T,Hq,D], k, v [T,Hkv,D] (empty caches)."""
    q, k, v = _check_store(q, dtype), _check_store(k, dtype), _check_store(v, dtype)
    q_start_loc = np.ascontiguousarray(q_start_loc, dtype=np.int32)
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    assert k.shape == v.shape == (T, Hkv, D) and q_start_loc[-1] == T
    if slopes is not None:
        slopes = np.ascontiguousarray(slopes, dtype=np.float64)
    out = np.zeros((T, Hq, D), dtype=np.float64)
    rc = lib().oracle_prompt_attention(_p(out), _p(q), _p(k), _p(v), _p(q_start_loc), _p(slopes),
                                       ctypes.c_double(scale), ctypes.c_int(q_start_loc.shape[0] - 1),
                                       ctypes.c_int(Hq), ctypes.c_int(Hkv), ctypes.c_int(D), ctypes.c_int(DTYPES[dtype]))
    if rc != 0:
        raise ValueError("bad shapes")
    return out


def unpage(cache, table, n: int, kvh: int, dtype: str) -> np.ndarray:
    """One sequence's K or V head in logical token order, [n, D] float64."""
    cache = _check_store(cache, dtype)
    table = np.ascontiguousarray(table, dtype=np.int32)
    num_blocks, Hkv, bs, D = cache.shape
    dst = np.empty((n, D), dtype=np.float64)
    lib().oracle_unpage(_p(dst), _p(cache), _p(table), ctypes.c_int(n), ctypes.c_int(kvh),
                        ctypes.c_int(Hkv), ctypes.c_int(D), ctypes.c_int(bs), ctypes.c_int(DTYPES[dtype]))
    return dst


def qkv_project_int4(x, qweight, scales, qzeros, gs: int) -> np.ndarray:
    """y [T, N] = x [T, K] (bf16 bits) times the 4-bit group-quantised W [K, N] (Eq. 1, weights of Q, K, V side by side)."""
    x, scales = _check_store(x, "bf16"), _check_store(scales, "bf16")
    qweight = np.ascontiguousarray(qweight, dtype=np.uint32)
    qzeros = np.ascontiguousarray(qzeros, dtype=np.uint32)
    T, K = x.shape
    N = qweight.shape[1]
    assert qweight.shape == (K // 8, N) and scales.shape == (K // gs, N) and qzeros.shape == (K // gs, N // 8)
    y = np.zeros((T, N), dtype=np.float64)
    rc = lib().oracle_qkv_project_int4(_p(y), _p(x), _p(qweight), _p(scales), _p(qzeros), ctypes.c_int(T),
                                       ctypes.c_int(K), ctypes.c_int(N), ctypes.c_int(gs))
    if rc != 0:
        raise ValueError("bad shapes")
    return y
