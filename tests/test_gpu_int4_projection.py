"""4-bit Q/K/V projection (Eq. 1 with group-quantised weights, keys and values stored into the paged cache as in
Algorithm 1, "Reshape and store K, V into C_K, C_V") through the C ABI against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_02351_b200 import binding
from paper_2505_02351_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _tol(want):
    # fp32 sums of exact products, one rounding to bf16 at the end: half an ulp of an 8-bit significand is at
    # most 2^-8 relative
    return 2.0 ** -8 * np.abs(want) * 1.01 + 1e-4


def _run(seed, T, Hq, Hkv, D, K, gs, bs=16, plain=True, cache=True):
    N = (Hq + 2 * Hkv) * D
    p = W.make_int4_projection(seed, T, K, N, gs)
    want = oracle.qkv_project_int4(W.storage_numpy(p.x), p.qweight.numpy().view(np.uint32), W.storage_numpy(p.scales),
                                   p.qzeros.numpy().view(np.uint32), gs)
    packed = torch.empty(binding.int4_packed_bytes(K, N, gs), dtype=torch.uint8, device=DEV)
    binding.int4_prepack(packed, p.qweight.to(DEV), p.scales.to(DEV), p.qzeros.to(DEV), gs)
    q_out = torch.full((T, Hq, D), float("nan"), dtype=torch.bfloat16, device=DEV)
    k_out = torch.full((T, Hkv, D), float("nan"), dtype=torch.bfloat16, device=DEV) if plain else None
    v_out = torch.full_like(k_out, float("nan")) if plain else None
    rng = np.random.default_rng(seed)
    num_blocks = (T + bs - 1) // bs + 3
    slots = rng.permutation(num_blocks * bs)[:T].astype(np.int64)
    if T > 2:
        slots[1] = -1                                   # a skipped token
    k_cache = torch.full((num_blocks, Hkv, bs, D), -7.0, dtype=torch.bfloat16, device=DEV) if cache else None
    v_cache = torch.full_like(k_cache, -9.0) if cache else None
    binding.qkv_project_int4(q_out, p.x.to(DEV), packed, Hq, Hkv, D, gs, k_out=k_out, v_out=v_out, k_cache=k_cache,
                             v_cache=v_cache, slot_mapping=torch.from_numpy(slots).to(DEV) if cache else None)
    torch.cuda.synchronize()
    qn, kvn = Hq * D, Hkv * D
    got_q = q_out.double().cpu().numpy().reshape(T, qn)
    assert np.all(np.abs(got_q - want[:, :qn]) <= _tol(want[:, :qn]))
    parts = {"k": want[:, qn:qn + kvn], "v": want[:, qn + kvn:]}
    if plain:
        for name, t in (("k", k_out), ("v", v_out)):
            got = t.double().cpu().numpy().reshape(T, kvn)
            assert np.all(np.abs(got - parts[name]) <= _tol(parts[name])), name
    if cache:
        for name, c, fill in (("k", k_cache, -7.0), ("v", v_cache, -9.0)):
            c = c.double().cpu().numpy()
            touched = np.zeros((num_blocks, bs), dtype=bool)
            for t in range(T):
                if slots[t] < 0:
                    continue
                page, off = divmod(int(slots[t]), bs)
                touched[page, off] = True
                got = c[page, :, off, :].reshape(kvn)
                assert np.all(np.abs(got - parts[name][t]) <= _tol(parts[name][t])), (name, t)
            untouched = c.transpose(0, 2, 1, 3)[~touched]
            assert np.all(untouched == fill), name
    if plain and cache:                                 # both destinations hold the same bits
        for t in range(T):
            if slots[t] >= 0:
                page, off = divmod(int(slots[t]), bs)
                assert torch.equal(k_cache[page, :, off, :], k_out[t]) and torch.equal(v_cache[page, :, off, :], v_out[t])


@pytest.mark.parametrize("T", [1, 7, 8, 9, 16, 37])
@pytest.mark.parametrize("gs", [64, 128])
def test_projection_small(T, gs):
    _run(100 + T, T, 8, 2, 64, 1024, gs)


@pytest.mark.parametrize("K", [128, 256, 2560, 4224])
def test_projection_widths_that_do_not_fill_the_warps_evenly(K):
    _run(7, 5, 4, 2, 128, K, 128, bs=32)
    _run(8, 12, 4, 4, 64, K, 64)


def test_projection_destinations():
    _run(3, 8, 8, 2, 128, 512, 128, plain=True, cache=False)
    _run(4, 8, 8, 2, 128, 512, 128, plain=False, cache=True)


def test_projection_long_sequence_decode_shape():
    """Model width 4096, 32 query / 4 KV heads of 128, the eight tokens of one step."""
    _run(2, 8, 32, 4, 128, 4096, 128)


def test_projection_70b_like_shape():
    _run(3, 8, 64, 8, 128, 8192, 128, bs=32)


@pytest.mark.parametrize("T,gs,K,Hq", [(5, 128, 1024, 64), (16, 64, 512, 64), (8, 128, 640, 64), (3, 64, 256, 80),
                                        (11, 128, 512, 96), (8, 64, 192, 64)])
def test_projection_more_tiles_than_one_wave_of_ctas(T, gs, K, Hq):
    """N / 32 = 320 tiles (Hq 64), 384 (Hq 80) or 448 (Hq 96) exceed what a B200 holds at once: the tiles past the
    last complete wave are cut into K slices whose CTAs add their sums up across a cluster, unless they are more than
    half a wave (Hq 96) or there are fewer groups than slices (K 192, gs 64: three).  K = 640 with 128-row groups gives
    slices of unequal length."""
    _run(40 + T, T, Hq, 8, 128, K, gs, bs=32)


@pytest.mark.parametrize("seed", range(12))
def test_projection_random_shapes(seed):
    """Drawn token counts (one pass of 8, of 16, several passes), group sizes, widths that are odd multiples of a
    group, head counts and destinations."""
    rng = np.random.default_rng(3000 + seed)
    T = int(rng.choice([1, 2, 7, 8, 9, 15, 16, 17, 33]))
    gs = int(rng.choice([64, 128]))
    K = gs * int(rng.integers(1, 13))
    D = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 4, 8]))
    Hq = Hkv * int(rng.choice([1, 2, 4, 8]))
    plain, cache = [(True, True), (True, False), (False, True)][int(rng.integers(0, 3))]
    _run(3100 + seed, T, Hq, Hkv, D, K, gs, bs=int(rng.choice([16, 32])), plain=plain, cache=cache)


def test_projection_rejects_bad_arguments():
    lib = binding.load()
    x = torch.zeros((8, 512), dtype=torch.bfloat16, device=DEV)
    buf = torch.zeros(1 << 20, dtype=torch.uint8, device=DEV)
    q = torch.zeros((8, 8, 64), dtype=torch.bfloat16, device=DEV)
    kv = torch.zeros((8, 2, 64), dtype=torch.bfloat16, device=DEV)
    def call(**kw):
        a = dict(q=q.data_ptr(), k=kv.data_ptr(), v=kv.data_ptr(), kc=None, vc=None, sm=None, x=x.data_ptr(),
                 pk=buf.data_ptr(), T=8, K=512, Hq=8, Hkv=2, D=64, bs=16, nb=0, gs=128)
        a.update(kw)
        return lib.opt_gqa_qkv_project_int4(a["q"], a["k"], a["v"], a["kc"], a["vc"], a["sm"], a["x"], a["pk"], a["T"],
                                            a["K"], a["Hq"], a["Hkv"], a["D"], a["bs"], a["nb"], a["gs"], None)
    assert call() == 0
    assert call(gs=32) == -2 and call(K=500) == -2 and call(D=96) == -2 and call(Hkv=3) == -2
    assert call(k=None, v=None) == -1 and call(x=None) == -1 and call(v=None) == -1
    assert call(kc=buf.data_ptr(), vc=buf.data_ptr(), nb=4) == -1          # cache without slot_mapping
    assert call(x=x.data_ptr() + 2) == -4
    assert call(T=0, x=None) == 0
    assert binding.int4_packed_bytes(512, 768, 128) == 512 * 768 // 2 + 4 * 768 * 4
    assert binding.int4_packed_bytes(512, 760, 128) == 0
    torch.cuda.synchronize()


def test_projection_then_decode_on_one_stream_without_synchronisation():
    """Eq. 1 -> "Reshape and store K, V" -> "Compute context attention with caches" as one chain on one stream: the
    projection lets its dependents start early and writes q and the new K/V rows; the balanced decode and its merge
    must see them (q is read only after the dependency wait, through L2).  Repeated with new activations into the
    same buffers, so that a stale line of the previous round's q would show."""
    from tests import util

    Hq, Hkv, D, K, gs = 32, 4, 128, 4096, 128
    wl = W.make_custom("chain", "bf16", Hq, Hkv, D, 16, [3000, 1500, 700, 2049, 16, 1, 512, 4000], seed=81)
    d = util.DeviceWorkload(wl)
    T, N = wl.B, (Hq + 2 * Hkv) * D
    p = W.make_int4_projection(82, T, K, N, gs)
    packed = torch.empty(binding.int4_packed_bytes(K, N, gs), dtype=torch.uint8, device=DEV)
    binding.int4_prepack(packed, p.qweight.to(DEV), p.scales.to(DEV), p.qzeros.to(DEV), gs)
    P, maxP = 512, 8
    ws = torch.empty(binding.workspace_bytes(wl.B, Hq, D, maxP), dtype=torch.uint8, device=DEV)
    q_buf = torch.zeros((T, Hq, D), dtype=torch.bfloat16, device=DEV)
    gen = torch.Generator().manual_seed(83)
    stream = torch.cuda.Stream()
    for rep in range(4):
        x = (0.3 * torch.randn((T, K), generator=gen)).to(torch.bfloat16).to(DEV)
        d.out.fill_(float("nan"))
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            binding.qkv_project_int4(q_buf, x, packed, Hq, Hkv, D, gs, k_cache=d.k_cache, v_cache=d.v_cache,
                                     slot_mapping=d.slot_mapping)
            binding.paged_attention_decode_balanced(q_buf, d.k_cache, d.v_cache, d.block_tables, d.context_lens,
                                                    d.alibi_slopes, wl.scale, P, ws, maxP)
            binding.paged_attention_reduce_balanced(d.out, ws, d.context_lens, Hkv, P, maxP)
        stream.synchronize()
        assert binding.device_status() == 0
        # the oracle attends with the projection's own outputs (read back after the chain has finished)
        want = oracle.paged_attention(W.storage_numpy(q_buf), W.storage_numpy(d.k_cache), W.storage_numpy(d.v_cache),
                                      wl.block_tables.numpy(), wl.context_lens.numpy(),
                                      wl.alibi_slopes.numpy().astype(np.float64), wl.scale, "bf16")
        got = d.out.double().cpu().numpy()
        assert np.isfinite(got).all()
        assert np.max(np.abs(got - want)) <= util.TOL["bf16"], rep
        # and q is what Eq. 1 gives for this round's activations
        y = oracle.qkv_project_int4(W.storage_numpy(x), p.qweight.numpy().view(np.uint32), W.storage_numpy(p.scales),
                                    p.qzeros.numpy().view(np.uint32), gs)
        got_q = q_buf.double().cpu().numpy().reshape(T, Hq * D)
        assert np.all(np.abs(got_q - y[:, :Hq * D]) <= _tol(y[:, :Hq * D]))
