"""The C-ABI library loads and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

from paper_2505_02351_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return binding.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "opt_gqa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(opt_gqa_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported_and_bound(lib):
    names = declared_symbols()
    assert "opt_gqa_cache_append" in names and "opt_gqa_paged_attention_decode" in names
    assert "opt_gqa_paged_attention_reduce" in names
    for name in names:
        assert hasattr(lib, name), name
        assert name in binding.SIGNATURES, f"{name} has no Python binding"
    assert sorted(binding.SIGNATURES) == names


def test_host_only_entry_points(lib):
    rows = 8 * 32 * 64
    assert binding.workspace_bytes(8, 32, 128, 64) >= rows * 129 * 4                       # one row per partition
    assert binding.workspace_bytes(8, 32, 128, 64) >= (rows + 2048 * 8) * 129 * 4 + 8 * 16   # the balanced split
    assert binding.workspace_bytes(8, 32, 128, 64) < (rows + 2048 * 8) * 129 * 4 + 4096
    assert binding.workspace_bytes(0, 32, 128, 64) == 0
    assert binding.status_string(0) == "ok"
    for code in range(-6, 0):
        assert binding.status_string(code) not in ("ok", "unknown status")
    assert binding.status_string(-99) == "unknown status"


def test_argument_checks_run_before_any_cuda_call(lib):
    f = lib.opt_gqa_paged_attention_decode
    null = None
    one = ctypes.c_void_p(16)
    # bad dtype, bad group size, bad head_dim, bad block size, bad partition size: all rejected on the host
    assert f(one, one, one, one, one, 1, one, one, 1.0, 1, 4, 2, 64, 16, 1, 0, null, null, 0, 7, null) == -3
    assert f(one, one, one, one, one, 1, one, one, 1.0, 1, 6, 2, 64, 16, 1, 0, null, null, 0, 0, null) == -2
    assert f(one, one, one, one, one, 1, one, one, 1.0, 1, 4, 2, 96, 16, 1, 0, null, null, 0, 0, null) == -2
    assert f(one, one, one, one, one, 1, one, one, 1.0, 1, 4, 2, 64, 8, 1, 0, null, null, 0, 0, null) == -2
    assert f(one, one, one, one, one, 1, one, one, 1.0, 1, 4, 2, 64, 16, 1, 24, one, one, 1, 0, null) == -2
    # B = 0 is fine and launches nothing
    assert f(null, null, null, null, null, 0, null, null, 1.0, 0, 4, 2, 64, 16, 0, 0, null, null, 0, 0, null) == 0
    # NULL and misaligned pointers
    assert f(null, one, one, one, one, 1, one, one, 1.0, 1, 4, 2, 64, 16, 1, 0, null, null, 0, 0, null) == -1
    assert f(one, ctypes.c_void_p(8), one, one, one, 1, one, one, 1.0, 1, 4, 2, 64, 16, 1, 0, null, null, 0, 0, null) == -4
    assert f(null, one, one, one, one, 1, one, one, 1.0, 1, 4, 2, 64, 16, 1, 16, null, one, 1, 0, null) == -1
    g = lib.opt_gqa_cache_append
    assert g(null, null, null, null, null, 0, 2, 64, 16, 4, 0, null) == 0
    assert g(null, one, one, one, one, 1, 2, 64, 16, 4, 0, null) == -1
    assert g(one, one, one, one, one, 1, 2, 64, 16, 4, 5, null) == -3
    assert g(one, one, one, one, one, 1, 2, 100, 16, 4, 0, null) == -2
    r = lib.opt_gqa_paged_attention_reduce
    assert r(one, one, one, one, 0, 4, 64, 16, 1, 0, null) == 0
    assert r(one, one, one, one, 1, 4, 64, 0, 1, 0, null) == -2
    assert r(null, one, one, one, 1, 4, 64, 16, 1, 0, null) == -1


def test_undersized_workspace_is_a_host_side_error(lib):
    """The calls that take a workspace take its size too and refuse one that is too small for the sizes given,
    before any CUDA call (fake pointers are enough to see it)."""
    one = ctypes.c_void_p(256)
    B, Hq, Hkv, D, P, maxP = 8, 32, 4, 128, 512, 64
    need = binding.workspace_bytes(B, Hq, D, maxP)
    f = lib.opt_gqa_paged_attention_decode_balanced
    assert f(one, one, one, one, 8, one, one, 1.0, B, Hq, Hkv, D, 16, 100, P, one, need // 2, maxP, 1, None) == -2
    assert f(one, one, one, one, 8, one, one, 1.0, B, Hq, Hkv, D, 16, 100, P, one, 0, maxP, 1, None) == -2
    r = lib.opt_gqa_paged_attention_reduce_balanced
    assert r(one, one, need // 2, one, B, Hq, Hkv, D, P, maxP, 1, None) == -2
    loc = lib.opt_gqa_paged_attention_decode_local
    assert loc(one, one, one, one, one, 8, one, one, 1.0, B, Hq, Hkv, D, 16, 100, P, one, 1024, maxP, 100, 1, None) == -2
    st = lib.opt_gqa_decode_step
    assert st(one, one, one, one, one, one, one, one, 8, one, one, 1.0, B, Hq, Hkv, D, 16, 100, P, one, need // 2, maxP, 1,
              None) == -2
    # fp32 caches: one (D + 1)-float row per (sequence, head, partition)
    assert st(one, one, one, one, one, one, one, one, 8, one, one, 1.0, B, Hq, Hkv, D, 16, 100, P, one,
              B * Hq * maxP * (D + 1) * 4 - 4, maxP, 0, None) == -2


def test_debug_entry_points_check_their_arguments(lib):
    assert lib.opt_gqa_debug_wait_timeout(0, None) == -2
    assert lib.opt_gqa_debug_wait_timeout(1 << 25, None) == -2
    assert lib.opt_gqa_debug_read_stream(None, 0, None, None) == 0
    assert lib.opt_gqa_debug_read_stream(None, 8192, None, None) == -1
    assert lib.opt_gqa_debug_read_stream(ctypes.c_void_p(256), 100, ctypes.c_void_p(256), None) == -2
    assert lib.opt_gqa_debug_read_stream(ctypes.c_void_p(8), 8192, ctypes.c_void_p(256), None) == -4
