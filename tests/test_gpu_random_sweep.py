"""Seeded random shapes through every decode entry point against the CPU oracle: group size, head dimension, page
size, partition size, window and a ragged mix of lengths (empty sequences, single tokens, lengths on and next to
tile, page and partition boundaries) are drawn together, so that combinations nobody wrote a case for still get
checked."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_02351_b200 import binding
from paper_2505_02351_b200 import workloads as W
from tests import util

pytestmark = pytest.mark.gpu
TOL = util.TOL["bf16"]


def _draw(seed):
    rng = np.random.default_rng(1000 + seed)
    G = int(rng.choice([1, 2, 4, 8]))
    Hkv = int(rng.choice([1, 2, 3, 8]))
    D = int(rng.choice([64, 128]))
    bs = int(rng.choice([16, 32]))
    P = int(rng.choice([16, 48, 64, 256, 512, 1024, 2048]))
    B = int(rng.integers(1, 24))
    special = [0, 1, 15, 16, 17, 31, 32, 33, P - 1, P, P + 1, 2 * P, 2 * P + 16]
    lens = []
    for _ in range(B):
        if rng.random() < 0.4:
            lens.append(int(rng.choice(special)))
        else:
            lens.append(int(2 ** rng.uniform(0, 12.5)))
    window = int(rng.choice([0, 0, 0, 0, 1, 20, 300, 5000]))
    slopes = bool(rng.random() < 0.75)
    return G, Hkv, D, bs, P, lens, window, slopes


def _oracle(wl, window, slopes):
    a = util.oracle_inputs(wl)
    return oracle.paged_attention(a["q"], a["k"], a["v"], a["bt"], a["n"], a["slopes"] if slopes else None, wl.scale,
                                  wl.dtype, q_start_loc=a["qsl"], window=window)


@pytest.mark.parametrize("seed", range(24))
def test_random_shapes(seed):
    G, Hkv, D, bs, P, lens, window, slopes = _draw(seed)
    wl = W.make_custom(f"sweep{seed}", "bf16", G * Hkv, Hkv, D, bs, lens, seed=500 + seed, poison=True)
    d = util.DeviceWorkload(wl)
    binding.cache_append(d.k_new, d.v_new, d.k_cache, d.v_cache, d.slot_mapping)
    sl = d.alibi_slopes if slopes else None
    maxP = max(1, (max(lens) + P - 1) // P)
    ws = torch.full((binding.workspace_bytes(wl.B, wl.Hq, wl.D, maxP) // 4,), float("nan"), device="cuda:0")
    want = _oracle(wl, window, slopes)

    def check(what):
        torch.cuda.synchronize()
        assert binding.device_status() == 0, what
        got = d.out.double().cpu().numpy()
        assert np.isfinite(got).all(), (what, seed)
        assert np.max(np.abs(got - want)) <= TOL, (what, seed, G, Hkv, D, bs, P, window)
        d.out.fill_(float("nan"))

    d.out.fill_(float("nan"))
    if window:
        binding.paged_attention_decode_local(d.out, d.q, d.k_cache, d.v_cache, d.block_tables, d.context_lens, sl,
                                             wl.scale, P, ws, maxP, window)
        check("local window")
        return
    binding.paged_attention_decode_balanced(d.q, d.k_cache, d.v_cache, d.block_tables, d.context_lens, sl, wl.scale,
                                            P, ws, maxP)
    binding.paged_attention_reduce_balanced(d.out, ws, d.context_lens, wl.Hkv, P, maxP)
    check("balanced split")
    po = torch.full((wl.B, wl.Hq, maxP, wl.D), float("nan"), device="cuda:0")
    pl = torch.full((wl.B, wl.Hq, maxP), float("nan"), device="cuda:0")
    binding.paged_attention_decode(None, d.q, d.k_cache, d.v_cache, d.block_tables, d.context_lens, sl, wl.scale,
                                   partition_size=P, partial_out=po, partial_lse=pl, max_partitions=maxP)
    binding.paged_attention_reduce(d.out, po, pl, d.context_lens, P)
    check("one partial per partition")
    binding.paged_attention_decode(d.out, d.q, d.k_cache, d.v_cache, d.block_tables, d.context_lens, sl, wl.scale)
    check("single pass")


def _draw_prefill(seed):
    rng = np.random.default_rng(7000 + seed)
    G = int(rng.choice([1, 2, 4, 8]))
    Hkv = int(rng.choice([1, 2, 3]))
    D = int(rng.choice([64, 128]))
    bs = int(rng.choice([16, 32]))
    TQ = 128 // G
    B = int(rng.integers(1, 7))
    special = [0, 1, 63, 64, 65, 127, 128, 129, TQ - 1, TQ, TQ + 1, 2 * TQ, 255, 256, 257]
    lens, qls = [], []
    for _ in range(B):
        n = int(rng.choice(special)) if rng.random() < 0.4 else int(2 ** rng.uniform(0, 10.3))
        pick = rng.random()
        ql = n if pick < 0.2 else (min(n, 1) if pick < 0.3 else int(rng.integers(0, n + 1)))
        lens.append(n)
        qls.append(ql)
    window = int(rng.choice([0, 0, 0, 1, 33, 64, 200, 4096]))
    slopes = bool(rng.random() < 0.75)
    scale = float(rng.choice([1.0, 1.0, 1.0, -0.5, 0.0]))      # multiples of the usual 1 / sqrt(D)
    return G, Hkv, D, bs, lens, qls, window, slopes, scale


@pytest.mark.parametrize("seed", range(20))
def test_random_prefill_shapes(seed):
    """Chunked prefill (prompt branch of Algorithms 1 and 2: causal mask from indices, ALiBi bias, optional local
    window) on drawn shapes: new-token counts from none to the whole context, contexts on and next to the 64-key tile
    and the query-block boundaries, both head dimensions, usual, negative and zero scale."""
    G, Hkv, D, bs, lens, qls, window, slopes, scale = _draw_prefill(seed)
    wl = W.make_custom(f"pfsweep{seed}", "bf16", G * Hkv, Hkv, D, bs, lens, q_lens=qls, seed=900 + seed, poison=True,
                       scale=scale / np.sqrt(D))
    a = util.oracle_inputs(wl)
    want = oracle.paged_attention(a["q"], a["k"], a["v"], a["bt"], a["n"], a["slopes"] if slopes else None, wl.scale,
                                  wl.dtype, q_start_loc=a["qsl"], window=window)
    d = util.DeviceWorkload(wl)
    binding.cache_append(d.k_new, d.v_new, d.k_cache, d.v_cache, d.slot_mapping)
    qsl = wl.q_start_loc.numpy()
    mq = int((qsl[1:] - qsl[:-1]).max()) if wl.B else 0
    sl = d.alibi_slopes if slopes else None
    d.out.fill_(float("nan"))
    if window:
        binding.paged_attention_prefill_local(d.out, d.q, d.q_start_loc, mq, d.k_cache, d.v_cache, d.block_tables,
                                              d.context_lens, sl, wl.scale, window)
    else:
        binding.paged_attention_prefill(d.out, d.q, d.q_start_loc, mq, d.k_cache, d.v_cache, d.block_tables,
                                        d.context_lens, sl, wl.scale)
    torch.cuda.synchronize()
    assert binding.device_status() == 0
    got = d.out.double().cpu().numpy()
    what = (seed, G, Hkv, D, bs, lens, qls, window, slopes, scale)
    assert np.isfinite(got).all(), what
    assert np.max(np.abs(got - want), initial=0.0) <= TOL, what
