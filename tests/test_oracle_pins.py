"""Pins for the CPU oracle: closed forms, invariants, special cases, brute force.

The paper prints no worked numerical example and no error bound, so the oracle
is pinned to what the paper's equations and the mathematics fix (Eq. 3-5, the
grouping and paging statements, the ALiBi paragraph).  None of these tests
touches the CUDA path.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2505_02351_b200 import workloads as W
from tests import brute

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _np(wl):
    """Workload -> storage arrays for the oracle, after the step's append."""
    k = W.storage_numpy(wl.k_cache)
    v = W.storage_numpy(wl.v_cache)
    oracle.cache_append(W.storage_numpy(wl.k_new), W.storage_numpy(wl.v_new), k, v,
                        wl.slot_mapping.numpy(), wl.dtype)
    return dict(
        q=W.storage_numpy(wl.q), k=k, v=v, bt=wl.block_tables.numpy(), n=wl.context_lens.numpy(),
        slopes=wl.alibi_slopes.numpy().astype(np.float64),
        qsl=None if wl.q_start_loc is None else wl.q_start_loc.numpy(),
    )


def _attn(wl, a, **kw):
    return oracle.paged_attention(a["q"], a["k"], a["v"], a["bt"], a["n"], a["slopes"], wl.scale, wl.dtype,
                                  q_start_loc=a["qsl"], **kw)


def _single(q, K, V, slope, scale, bs=4, window=0, shuffle_seed=None):
    """One sequence, one head, fp32 storage, arbitrary D: returns the oracle's [D] output."""
    n, D = K.shape
    npages = (n + bs - 1) // bs
    order = np.arange(npages)
    if shuffle_seed is not None:
        order = np.random.default_rng(shuffle_seed).permutation(npages)
    kc = np.zeros((npages, 1, bs, D), np.float32)
    vc = np.zeros((npages, 1, bs, D), np.float32)
    for j in range(n):
        kc[order[j // bs], 0, j % bs] = K[j]
        vc[order[j // bs], 0, j % bs] = V[j]
    out = oracle.paged_attention(np.asarray(q, np.float32).reshape(1, 1, D), kc, vc,
                                 order.astype(np.int32).reshape(1, -1), np.array([n], np.int32),
                                 np.array([slope], np.float64), scale, "fp32", window=window)
    return out[0, 0]


# ---------------------------------------------------------------- slopes
def test_slopes_match_closed_form_fixture():
    with open(os.path.join(GOLDEN, "alibi_slopes.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            hq, vals = line.split(":")
            want = np.array([float(x) for x in vals.split()])
            got = oracle.alibi_slopes(int(hq))
            assert np.array_equal(got, want), (hq, got, want)


def test_slopes_geometric_and_generator_agrees():
    for hq in (16, 32, 64):
        s = oracle.alibi_slopes(hq)
        ratio = s[1:] / s[:-1]
        assert np.allclose(ratio, 2.0 ** (-8.0 / hq), rtol=1e-14)
        assert s[-1] == 2.0 ** -8
        gen = W.alibi_slopes_input(hq).numpy()
        assert gen.dtype == np.float32
        assert np.array_equal(gen, s.astype(np.float32))


# ---------------------------------------------------------------- closed forms
def test_hand_example_two_keys():
    # D=1, scale=1, q=1, k=(0,0), v=(0,1), slope=ln 2: raw = (-ln2, 0) -> weights (1/3, 2/3).
    out = _single([1.0], np.zeros((2, 1)), np.array([[0.0], [1.0]]), math.log(2.0), 1.0)
    assert abs(out[0] - 2.0 / 3.0) < 1e-15


def test_scale_applies_to_dot_product_not_to_bias():
    # raw_0 = scale*q*k_0 - slope = 0.5*1*2 - ln3, raw_1 = 0  ->  w_0 = e / (e + 3).
    out = _single([1.0], np.array([[2.0], [0.0]]), np.array([[1.0], [0.0]]), math.log(3.0), 0.5)
    assert abs(out[0] - math.e / (math.e + 3.0)) < 1e-15
    # were the bias scaled too, the answer would be e / (e + sqrt(3)); were nothing scaled, e^2/(e^2+3)
    assert abs(out[0] - math.e / (math.e + math.sqrt(3.0))) > 1e-2


@pytest.mark.parametrize("n,slope", [(5, 0.25), (37, 0.0625), (100, 2.0 ** -8), (64, 0.0)])
def test_identical_keys_give_geometric_weights(n, slope):
    # identical keys: scores differ only by the bias, so w_j = r^(n-1-j) (1-r)/(1-r^n), r = e^-slope;
    # slope = 0 gives the mean of V.
    rng = np.random.default_rng(n)
    D = 8
    key = rng.standard_normal(D).astype(np.float32)
    K = np.tile(key, (n, 1))
    V = rng.standard_normal((n, D)).astype(np.float32)
    q = rng.standard_normal(D).astype(np.float32)
    out = _single(q, K, V, slope, 0.3, shuffle_seed=1)
    if slope == 0.0:
        want = V.astype(np.float64).mean(axis=0)
    else:
        r = math.exp(-slope)
        w = r ** (n - 1 - np.arange(n)) * (1 - r) / (1 - r ** n)
        assert abs(w.sum() - 1) < 1e-12
        want = w @ V.astype(np.float64)
    assert np.max(np.abs(out - want)) < 1e-13


def test_zero_query_ignores_keys():
    rng = np.random.default_rng(3)
    n, D, slope = 23, 4, 0.5
    K = rng.standard_normal((n, D)).astype(np.float32)
    V = rng.standard_normal((n, D)).astype(np.float32)
    out = _single(np.zeros(D), K, V, slope, 1.0)
    r = math.exp(-slope)
    w = r ** (n - 1 - np.arange(n)) * (1 - r) / (1 - r ** n)
    assert np.max(np.abs(out - w @ V.astype(np.float64))) < 1e-13


def test_single_token_and_constant_values_and_steep_slope():
    rng = np.random.default_rng(4)
    D = 16
    q = rng.standard_normal(D).astype(np.float32)
    v0 = rng.standard_normal((1, D)).astype(np.float32)
    out = _single(q, rng.standard_normal((1, D)).astype(np.float32), v0, 0.25, 0.7)
    assert np.array_equal(out, v0[0].astype(np.float64))                      # n = 1: out = v_0 exactly
    K = rng.standard_normal((19, D)).astype(np.float32)
    Vc = np.tile(v0, (19, 1))
    out = _single(q, K, Vc, 0.25, 0.7)
    assert np.max(np.abs(out - v0[0])) < 1e-15                                # constant V rows
    V = rng.standard_normal((19, D)).astype(np.float32)
    out = _single(q, K, V, 500.0, 0.7)
    assert np.max(np.abs(out - V[-1])) < 1e-12                                # steep slope: last token wins


def test_two_key_softmax_is_logistic():
    # n=2, D=3: w_1 = sigmoid(scale*q.(k_1-k_0) + slope)
    q = np.array([0.5, -1.0, 2.0], np.float32)
    K = np.array([[1.0, 0.0, -1.0], [0.25, 2.0, 0.5]], np.float32)
    V = np.array([[0.0, 0.0, 0.0], [1.0, 1.0, 1.0]], np.float32)
    scale, slope = 0.37, 0.8
    z = scale * float(q.astype(np.float64) @ (K[1] - K[0]).astype(np.float64)) + slope
    out = _single(q, K, V, slope, scale)
    assert np.max(np.abs(out - 1.0 / (1.0 + math.exp(-z)))) < 1e-15


# ---------------------------------------------------------------- brute force
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("Hq,Hkv", [(4, 4), (4, 2), (8, 1), (6, 3)])
def test_decode_matches_dense_numpy(dtype, Hq, Hkv):
    wl = W.make_custom("t", dtype, Hq, Hkv, 8, 4, [1, 3, 4, 5, 17, 0 + 9], seed=11 + Hq)
    a = _np(wl)
    got = _attn(wl, a)
    want = brute.dense_attention(a["q"], a["k"], a["v"], a["bt"], a["n"], a["slopes"], wl.scale)
    assert np.max(np.abs(got - want)) < 1e-12


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_prefill_matches_dense_numpy(dtype):
    wl = W.make_custom("t", dtype, 4, 2, 8, 4, [9, 12, 5, 7], q_lens=[9, 3, 1, 4], seed=5)
    a = _np(wl)
    got = _attn(wl, a)
    want = brute.dense_attention(a["q"], a["k"], a["v"], a["bt"], a["n"], a["slopes"], wl.scale,
                                 q_start_loc=a["qsl"])
    assert np.max(np.abs(got - want)) < 1e-12
    got_w = _attn(wl, a, window=3)
    want_w = brute.dense_attention(a["q"], a["k"], a["v"], a["bt"], a["n"], a["slopes"], wl.scale,
                                   q_start_loc=a["qsl"], window=3)
    assert np.max(np.abs(got_w - want_w)) < 1e-12
    assert np.max(np.abs(got_w - got)) > 1e-3


def test_config1_matches_dense_numpy():
    wl = W.make_config(1)
    a = _np(wl)
    got = _attn(wl, a)
    want = brute.dense_attention(a["q"], a["k"], a["v"], a["bt"], a["n"], a["slopes"], wl.scale)
    assert np.max(np.abs(got - want)) < 1e-12


# ---------------------------------------------------------------- grouping
def test_group_size_one_is_mha_and_gqa_is_mha_on_repeated_kv():
    wl = W.make_custom("t", "fp32", 8, 2, 16, 4, [13, 30], seed=2)
    a = _np(wl)
    got = _attn(wl, a)
    G = 4
    k_rep = np.repeat(a["k"], G, axis=1)       # KV head h -> heads 4h..4h+3: consecutive grouping
    v_rep = np.repeat(a["v"], G, axis=1)
    mha = oracle.paged_attention(a["q"], k_rep, v_rep, a["bt"], a["n"], a["slopes"], wl.scale, "fp32")
    assert np.array_equal(got, mha)
    # and every query head on its own (Hq = Hkv = 1) gives the same row
    for h in range(8):
        one = oracle.paged_attention(np.ascontiguousarray(a["q"][:, h:h + 1]),
                                     np.ascontiguousarray(a["k"][:, h // G:h // G + 1]),
                                     np.ascontiguousarray(a["v"][:, h // G:h // G + 1]),
                                     a["bt"], a["n"], a["slopes"][h:h + 1], wl.scale, "fp32")
        assert np.array_equal(one[:, 0], got[:, h])
    # heads of one group differ only through q and slope: same q, zero slopes -> identical rows
    q_same = a["q"].copy()
    q_same[:, 1] = q_same[:, 0]
    z = oracle.paged_attention(q_same, a["k"], a["v"], a["bt"], a["n"], None, wl.scale, "fp32")
    assert np.array_equal(z[:, 0], z[:, 1])
    assert not np.array_equal(z[:, 0], z[:, 4])


# ---------------------------------------------------------------- paging
def test_invariance_to_physical_page_permutation():
    wl = W.make_custom("t", "bf16", 4, 2, 16, 4, [21, 40, 7], seed=9)
    a = _np(wl)
    ref = _attn(wl, a)
    rng = np.random.default_rng(0)
    perm = rng.permutation(wl.num_blocks)            # new physical id of old page p is perm[p]
    k2 = np.empty_like(a["k"]); v2 = np.empty_like(a["v"])
    k2[perm] = a["k"]; v2[perm] = a["v"]
    bt2 = np.where(a["bt"] >= 0, perm[np.maximum(a["bt"], 0)], -1).astype(np.int32)
    got = oracle.paged_attention(a["q"], k2, v2, bt2, a["n"], a["slopes"], wl.scale, wl.dtype)
    assert np.array_equal(got, ref)                  # bitwise: paging is pure memory management


def test_unused_slots_never_matter():
    clean = W.make_custom("t", "bf16", 4, 2, 16, 4, [21, 40, 7], seed=9, poison=False)
    dirty = W.make_custom("t", "bf16", 4, 2, 16, 4, [21, 40, 7], seed=9, poison=True)
    assert torch.isnan(dirty.k_cache.float()).any()
    a, b = _np(clean), _np(dirty)
    ra, rb = _attn(clean, a), _attn(dirty, b)
    assert np.isfinite(rb).all() and np.array_equal(ra, rb)


def test_empty_sequence_gives_zero_rows():
    wl = W.make_custom("t", "fp32", 2, 1, 8, 4, [0, 6], seed=1)
    assert wl.T == 2 and wl.slot_mapping[0] == -1
    a = _np(wl)
    out = _attn(wl, a)
    assert np.array_equal(out[0], np.zeros_like(out[0])) and np.abs(out[1]).max() > 0


# ---------------------------------------------------------------- partitions
@pytest.mark.parametrize("P", [4, 16, 48, 512])
def test_partition_merge_equals_single_pass(P):
    wl = W.make_custom("t", "bf16", 4, 2, 16, 4, [1, 50, 129, 64], seed=6)
    a = _np(wl)
    ref = _attn(wl, a)
    maxP = (129 + P - 1) // P
    po, pl = oracle.partition_partials(a["q"], a["k"], a["v"], a["bt"], a["n"], a["slopes"], wl.scale,
                                       wl.dtype, P, maxP)
    got = oracle.reduce(po, pl, a["n"], P)
    assert np.max(np.abs(got - ref)) < 1e-13
    # partitions past the end are empty: lse = -inf, o = 0
    np_s = (a["n"] + P - 1) // P
    for s in range(4):
        assert np.all(np.isneginf(pl[s, :, np_s[s]:])) and np.all(po[s, :, np_s[s]:] == 0)
        assert np.all(np.isfinite(pl[s, :, :np_s[s]]))


def test_lse_is_log_of_the_softmax_denominator():
    # one partition covering everything: lse = log sum_j exp(raw_j), o = the full answer
    wl = W.make_custom("t", "fp32", 2, 2, 8, 4, [11], seed=8)
    a = _np(wl)
    po, pl = oracle.partition_partials(a["q"], a["k"], a["v"], a["bt"], a["n"], a["slopes"], wl.scale,
                                       "fp32", 64, 1)
    assert np.max(np.abs(po[:, :, 0] - _attn(wl, a))) < 1e-14
    for h in range(2):
        K = brute.logical_kv(a["k"], a["bt"][0], 11)[h]
        raw = wl.scale * K @ a["q"][0, h].astype(np.float64) - a["slopes"][h] * (10 - np.arange(11))
        assert abs(pl[0, h, 0] - math.log(np.exp(raw).sum())) < 1e-13


def test_reduce_with_hand_partials():
    # two partitions with lse = (ln 1, ln 3): weights (1/4, 3/4)
    po = np.zeros((1, 1, 2, 2)); po[0, 0, 0] = [4.0, 0.0]; po[0, 0, 1] = [0.0, 8.0]
    pl = np.array([[[0.0, math.log(3.0)]]])
    out = oracle.reduce(po, pl, np.array([6], np.int32), 4)
    assert np.max(np.abs(out[0, 0] - np.array([1.0, 6.0]))) < 1e-15
    # only ceil(n/P) partitions count
    out = oracle.reduce(po, pl, np.array([3], np.int32), 4)
    assert np.array_equal(out[0, 0], np.array([4.0, 0.0]))


# ---------------------------------------------------------------- prefill vs decode
def test_prefill_row_equals_decode_on_truncated_context():
    wl = W.make_custom("t", "bf16", 4, 2, 16, 4, [14, 9], q_lens=[6, 9], seed=12)
    a = _np(wl)
    full = _attn(wl, a)
    for s in range(2):
        ql = int(a["qsl"][s + 1] - a["qsl"][s])
        for i in range(ql):
            pos = int(a["n"][s]) - ql + i
            t = int(a["qsl"][s]) + i
            dec = oracle.paged_attention(np.ascontiguousarray(a["q"][t:t + 1]), a["k"], a["v"],
                                         a["bt"][s:s + 1], np.array([pos + 1], np.int32), a["slopes"],
                                         wl.scale, wl.dtype)
            assert np.array_equal(dec[0], full[t])


def test_prefill_with_one_new_token_is_decode():
    wl = W.make_custom("t", "fp32", 4, 2, 8, 4, [5, 12, 8], seed=13)
    a = _np(wl)
    dec = _attn(wl, a)
    pre = oracle.paged_attention(a["q"], a["k"], a["v"], a["bt"], a["n"], a["slopes"], wl.scale, "fp32",
                                 q_start_loc=np.arange(4, dtype=np.int32))
    assert np.array_equal(dec, pre)


def test_window_special_cases():
    wl = W.make_custom("t", "fp32", 2, 1, 8, 4, [13], seed=14)
    a = _np(wl)
    assert np.array_equal(_attn(wl, a, window=13), _attn(wl, a))       # window >= n: no effect
    w1 = _attn(wl, a, window=1)                                        # window 1: only the own token
    v_last = brute.logical_kv(a["v"], a["bt"][0], 13)[0, 12]
    assert np.array_equal(w1[0, 0], v_last)


# ---------------------------------------------------------------- convexity
def test_output_is_a_convex_combination():
    wl = W.make_config(1)
    a = _np(wl)
    out = _attn(wl, a)
    for s in range(wl.B):
        V = brute.logical_kv(a["v"], a["bt"][s], int(a["n"][s]))
        for h in range(wl.Hq):
            lo, hi = V[h // 2].min(axis=0), V[h // 2].max(axis=0)
            assert np.all(out[s, h] >= lo - 1e-12) and np.all(out[s, h] <= hi + 1e-12)


# ---------------------------------------------------------------- cache append
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_cache_append_is_a_slot_mapped_bit_copy(dtype):
    wl = W.make_custom("t", dtype, 4, 2, 16, 4, [9, 14, 3], q_lens=[2, 5, 3], seed=3)
    k0, v0 = W.storage_numpy(wl.k_cache), W.storage_numpy(wl.v_cache)
    k, v = k0.copy(), v0.copy()
    kn, vn = W.storage_numpy(wl.k_new), W.storage_numpy(wl.v_new)
    slots = wl.slot_mapping.numpy().copy()
    slots[1] = -1                                                    # skipped token
    oracle.cache_append(kn, vn, k, v, slots, dtype)
    touched = np.zeros(k.shape[:1] + k.shape[2:3], bool)
    for t, sl in enumerate(slots):
        if sl < 0:
            continue
        assert np.array_equal(k[sl // 4, :, sl % 4], kn[t]) and np.array_equal(v[sl // 4, :, sl % 4], vn[t])
        touched[sl // 4, sl % 4] = True
    keep = ~touched[:, None, :, None] & np.ones_like(k, bool)
    assert np.array_equal(k[keep], k0[keep]) and np.array_equal(v[keep], v0[keep])
    # un-paging afterwards equals writing the logical sequence directly (Eq. 2: old tokens, then new ones)
    n, qsl = wl.context_lens.numpy(), wl.q_start_loc.numpy()
    s = 2                                                            # all 3 tokens of seq 2 are new
    seq = oracle.unpage(k, wl.block_tables.numpy()[s], int(n[s]), 1, dtype)
    assert np.array_equal(seq, brute.widen(kn[qsl[s]:qsl[s + 1], 1]))
    with pytest.raises(ValueError):
        oracle.cache_append(kn, vn, k, v, np.full_like(slots, wl.num_blocks * 4), dtype)


def test_bf16_widening_is_exact():
    x = torch.tensor([1.0, -2.5, 3.140625, 1e-3, 65280.0], dtype=torch.float32).to(torch.bfloat16)
    got = brute.widen(W.storage_numpy(x))
    assert np.array_equal(got, x.double().numpy())
    cache = W.storage_numpy(x).reshape(1, 1, 5, 1)
    seq = oracle.unpage(cache, np.array([0], np.int32), 5, 0, "bf16")
    assert np.array_equal(seq[:, 0], x.double().numpy())


# ------------------------------------------------------------------ the prompt branch with empty caches
def _prompt_inputs(Hq, Hkv, D, lens, dtype, seed):
    wl = W.make_custom("prompt", dtype, Hq, Hkv, D, 16, lens, q_lens=lens, seed=seed)
    return wl, W.storage_numpy(wl.q), W.storage_numpy(wl.k_new), W.storage_numpy(wl.v_new), wl.q_start_loc.numpy()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_prompt_attention_matches_dense_numpy(dtype):
    """Written out with matrices in numpy, sequence by sequence: softmax(scale QK^T - slope*(i-j), j <= i) V."""
    wl, q, k, v, qsl = _prompt_inputs(4, 2, 64, [5, 33, 1, 18], dtype, 61)
    slopes = wl.alibi_slopes.numpy().astype(np.float64)
    got = oracle.prompt_attention(q, k, v, qsl, slopes, wl.scale, dtype)
    qd, kd, vd = brute.widen(q), brute.widen(k), brute.widen(v)
    for s in range(4):
        a, b = qsl[s], qsl[s + 1]
        i = np.arange(b - a)
        rel = i[:, None] - i[None, :]
        for h in range(4):
            S = wl.scale * qd[a:b, h] @ kd[a:b, h // 2].T - slopes[h] * rel
            S = np.where(rel < 0, -np.inf, S)
            Wt = np.exp(S - S.max(axis=1, keepdims=True))
            Wt /= Wt.sum(axis=1, keepdims=True)
            assert np.max(np.abs(got[a:b, h] - Wt @ vd[a:b, h // 2])) < 1e-12


def test_prompt_attention_is_prefill_over_a_cache_holding_only_the_new_tokens():
    wl, q, k, v, qsl = _prompt_inputs(8, 2, 64, [40, 7, 65], "bf16", 62)
    slopes = wl.alibi_slopes.numpy().astype(np.float64)
    kc, vc = W.storage_numpy(wl.k_cache), W.storage_numpy(wl.v_cache)
    oracle.cache_append(k, v, kc, vc, wl.slot_mapping.numpy(), "bf16")
    paged = oracle.paged_attention(q, kc, vc, wl.block_tables.numpy(), wl.context_lens.numpy(), slopes, wl.scale,
                                   "bf16", q_start_loc=qsl)
    got = oracle.prompt_attention(q, k, v, qsl, slopes, wl.scale, "bf16")
    assert np.max(np.abs(got - paged)) < 1e-12
    # the first token of every sequence sees only itself
    for s in range(3):
        assert np.allclose(got[qsl[s]], brute.widen(v)[qsl[s]].repeat(4, axis=0), atol=1e-15)


# ---- 4-bit Q/K/V projection (Eq. 1 with group-quantised weights) ----

def _bf16_bits(a):
    return W.storage_numpy(torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16))


def test_int4_projection_hand_example():
    """One 8 x 8 block typed by hand: row k of every column holds code k except row 0, which holds the
    column index; zero point of column i is 7 - i; every scale is 0.5."""
    qweight = np.array([[0x76543210 + n for n in range(8)]], dtype=np.uint32)
    qzeros = np.array([[0x01234567]], dtype=np.uint32)
    scales = _bf16_bits(np.full((1, 8), 0.5))
    e0 = _bf16_bits(np.eye(8)[0:1])
    e3 = _bf16_bits(np.eye(8)[3:4])
    y0 = oracle.qkv_project_int4(e0, qweight, scales, qzeros, 8)
    y3 = oracle.qkv_project_int4(e3, qweight, scales, qzeros, 8)
    assert y0.tolist() == [[-3.5, -2.5, -1.5, -0.5, 0.5, 1.5, 2.5, 3.5]]
    assert y3.tolist() == [[-2.0, -1.5, -1.0, -0.5, 0.0, 0.5, 1.0, 1.5]]


def test_int4_projection_is_an_integer_matmul_when_scales_are_powers_of_two():
    rng = np.random.default_rng(5)
    T, K, N, gs = 3, 64, 24, 16
    qweight = rng.integers(0, 2**32, size=(K // 8, N), dtype=np.uint32)
    qzeros = rng.integers(0, 2**32, size=(K // gs, N // 8), dtype=np.uint32)
    exps = rng.integers(-2, 3, size=(K // gs, N))
    xi = rng.integers(-8, 9, size=(T, K))
    codes = np.stack([(qweight >> np.uint32(4 * i)) & np.uint32(15) for i in range(8)], axis=1).reshape(K, N).astype(np.int64)
    zeros = np.stack([(qzeros >> np.uint32(4 * i)) & np.uint32(15) for i in range(8)], axis=2).reshape(K // gs, N).astype(np.int64)
    want = np.zeros((T, N))
    for g in range(K // gs):
        want += (xi[:, g * gs:(g + 1) * gs] @ (codes[g * gs:(g + 1) * gs] - zeros[g])) * np.exp2(exps[g])
    got = oracle.qkv_project_int4(_bf16_bits(xi), qweight, _bf16_bits(np.exp2(exps)), qzeros, gs)
    assert np.array_equal(got, want)


def test_int4_projection_group_whose_codes_equal_its_zero_points_contributes_nothing():
    p = W.make_int4_projection(9, 2, 64, 16, gs=32)
    qweight = p.qweight.numpy().view(np.uint32).copy()
    qzeros = p.qzeros.numpy().view(np.uint32)
    zeros = np.stack([(qzeros >> np.uint32(4 * i)) & np.uint32(15) for i in range(8)], axis=2).reshape(2, 16)
    qweight[4:8] = (zeros[1] * np.uint32(0x11111111))[None, :]          # rows 32..63 = group 1
    x = W.storage_numpy(p.x)
    s = W.storage_numpy(p.scales)
    y = oracle.qkv_project_int4(x, qweight, s, qzeros, 32)
    x2 = x.copy()
    x2[:, 32:] = _bf16_bits(np.full((2, 32), 3.0))
    assert np.array_equal(y, oracle.qkv_project_int4(x2, qweight, s, qzeros, 32))
    assert np.abs(y).max() > 0
