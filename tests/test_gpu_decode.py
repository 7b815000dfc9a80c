"""Parity of the CUDA decode path (append -> decode -> reduce, through the C ABI) with the CPU oracle."""
import numpy as np
import pytest
import torch

from paper_2505_02351_b200 import binding
from paper_2505_02351_b200 import workloads as W
from tests import util

pytestmark = pytest.mark.gpu


def _check(wl, partition_size=None, **kw):
    got, d = util.gpu_decode(wl, partition_size=partition_size, **kw)
    want = util.oracle_attention(wl, **kw)
    assert np.isfinite(got).all()
    err = np.max(np.abs(got - want)) if got.size else 0.0
    assert err <= util.TOL[wl.dtype], f"{wl.name}: max-abs error {err}"
    return got, want, d


def test_config1_tiny_fp32():
    _check(W.make_config(1))
    _check(W.make_config(1), partition_size=16)
    _check(W.make_config(1), partition_size=48)


def test_config1_poisoned_unused_slots():
    _check(W.make_config(1, poison=True))
    _check(W.make_config(1, poison=True), partition_size=32)


def test_config2_bf16_llama7b_like():
    _check(W.make_config(2))
    _check(W.make_config(2, poison=True), partition_size=256)
    _check(W.make_config(2, poison=True), partition_size=256, simt=True)


def test_config3_long_sequence_partitioned():
    wl = W.make_config(3)
    assert wl.partition_size == 512
    _check(wl)
    _check(wl, simt=True)
    _check(wl, balanced=True)


def test_balanced_split_on_the_named_workloads():
    _check(W.make_config(2, poison=True), partition_size=256, balanced=True)
    _check(W.make_config(4, poison=True), partition_size=512, balanced=True)
    _check(W.make_config(4, poison=True), partition_size=1024, balanced=True)


def test_decode_step_one_call_matches_the_oracle():
    """opt_gqa_decode_step (append -> balanced decode -> reduce for bf16; per-partition partials for fp32)."""
    for wl, P in ((W.make_config(3, shrink=8), 512), (W.make_config(4, poison=True), 512), (W.make_config(1), 32),
                  (W.make_config(2), 0)):
        d = util.DeviceWorkload(wl)
        maxP = max(1, (int(wl.context_lens.max()) + P - 1) // P) if P else 1
        ws = torch.full((binding.workspace_bytes(wl.B, wl.Hq, wl.D, maxP),), 0xff, device="cuda:0", dtype=torch.uint8)
        binding.decode_step(d.out, d.q, d.k_new, d.v_new, d.slot_mapping, d.k_cache, d.v_cache, d.block_tables,
                            d.context_lens, d.alibi_slopes, wl.scale, partition_size=P, workspace=ws if P else None,
                            max_partitions=maxP)
        torch.cuda.synchronize()
        assert binding.device_status() == 0
        want = util.oracle_attention(wl)
        got = d.out.double().cpu().numpy()
        assert np.max(np.abs(got - want)) <= util.TOL[wl.dtype], wl.name


@pytest.mark.parametrize("B,Hkv", [(40, 2), (9, 8), (600, 2), (64, 4), (37, 8)])
def test_decode_step_leaves_the_cache_as_the_slot_mapped_write_does(B, Hkv):
    """With few streams the step's decode kernel stores the new tokens itself (B * Hkv <= 1024), with many a separate
    kernel does, and with 1.5 to 4 streams per multiprocessor and short contexts (the last two cases on a 148-SM GPU)
    the whole step is one single-pass launch that stores them: either way the pools afterwards are bit for bit what
    opt_gqa_cache_append gives, skipped tokens (slot -1, empty sequences) included."""
    rng = np.random.default_rng(B)
    lens = [int(x) for x in rng.integers(1, 700, size=B)]
    lens[1] = 0
    lens[2] = 1
    lens[3] = 16
    lens[4] = 17
    wl = W.make_custom("fused", "bf16", Hkv * 4, Hkv, 128, 16, lens, seed=90 + B, poison=True)
    d = util.DeviceWorkload(wl)
    k_ref, v_ref = d.k_cache.clone(), d.v_cache.clone()
    binding.cache_append(d.k_new, d.v_new, k_ref, v_ref, d.slot_mapping)
    P, maxP = 256, 3
    ws = torch.full((binding.workspace_bytes(wl.B, wl.Hq, wl.D, maxP),), 0xff, device="cuda:0", dtype=torch.uint8)
    binding.decode_step(d.out, d.q, d.k_new, d.v_new, d.slot_mapping, d.k_cache, d.v_cache, d.block_tables,
                        d.context_lens, d.alibi_slopes, wl.scale, partition_size=P, workspace=ws, max_partitions=maxP)
    torch.cuda.synchronize()
    assert binding.device_status() == 0
    assert torch.equal(d.k_cache.view(torch.int16), k_ref.view(torch.int16))
    assert torch.equal(d.v_cache.view(torch.int16), v_ref.view(torch.int16))
    want = util.oracle_attention(wl)
    assert np.max(np.abs(d.out.double().cpu().numpy() - want)) <= util.TOL["bf16"]


def test_config4_ragged_large_batch_with_append():
    wl = W.make_config(4, poison=True)
    got, want, d = _check(wl, partition_size=512)
    got1, _, _ = _check(wl, partition_size=0)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (4, 2), (8, 2), (8, 1)])
@pytest.mark.parametrize("bs", [16, 32])
def test_shape_matrix(dtype, D, Hq, Hkv, bs):
    lens = [1, 15, 16, 17, 33, 100, 257, 0, 640]
    wl = W.make_custom("m", dtype, Hq, Hkv, D, bs, lens, seed=D + Hq + bs, poison=True)
    _check(wl)
    _check(wl, partition_size=64)
    _check(wl, partition_size=0, slopes=False)
    if dtype == "bf16":        # the CUDA-core kernel on bf16 caches (fp32 always runs on it); the balanced split
        _check(wl, simt=True)
        _check(wl, partition_size=64, simt=True)
        _check(wl, partition_size=64, balanced=True)
        _check(wl, partition_size=16, balanced=True, slopes=False)


@pytest.mark.parametrize("P", [16, 48, 512, 4096])
def test_any_partition_size_agrees_with_single_pass(P):
    wl = W.make_custom("p", "bf16", 8, 2, 128, 16, [700, 33, 2049], seed=21)
    _check(wl, partition_size=P)
    _check(wl, partition_size=P, simt=True)
    _check(wl, partition_size=P, balanced=True)


def test_balanced_split_with_fewer_tiles_than_workers_and_empty_sequences():
    # 3 + 1 + 0 + 2 tiles per head: most workers of the persistent grid get an empty range
    wl = W.make_custom("few", "bf16", 8, 2, 128, 16, [40, 7, 0, 32], seed=25, poison=True)
    _check(wl, partition_size=16, balanced=True)
    _check(wl, partition_size=512, balanced=True)
    wl0 = W.make_custom("none", "bf16", 8, 2, 128, 16, [0, 0], seed=26)
    got, _ = util.gpu_decode(wl0, partition_size=64, balanced=True)
    assert np.array_equal(got, np.zeros_like(got))


def test_partials_match_the_oracle_partials():
    import oracle
    wl = W.make_custom("p", "fp32", 4, 2, 64, 16, [130, 40, 77], seed=22)
    got, d = util.gpu_decode(wl, partition_size=32)
    a = util.oracle_inputs(wl)
    maxP = d.partial_out.shape[2]
    po, pl = oracle.partition_partials(a["q"], a["k"], a["v"], a["bt"], a["n"], a["slopes"], wl.scale, wl.dtype, 32, maxP)
    gpo, gpl = d.partial_out.double().cpu().numpy(), d.partial_lse.double().cpu().numpy()
    for s in range(wl.B):
        np_s = (int(a["n"][s]) + 31) // 32
        assert np.max(np.abs(gpo[s, :, :np_s] - po[s, :, :np_s])) < 1e-5
        assert np.max(np.abs(gpl[s, :, :np_s] - pl[s, :, :np_s])) < 1e-5
        assert np.isnan(gpo[s, :, np_s:]).all()          # entries past the sequence are left untouched


def test_cache_append_is_bit_exact_and_touches_nothing_else():
    import oracle
    for dtype in ("fp32", "bf16"):
        wl = W.make_custom("a", dtype, 8, 4, 128, 32, [70, 5, 300], q_lens=[7, 5, 33], seed=23)
        d = util.DeviceWorkload(wl)
        slots = wl.slot_mapping.clone()
        slots[3] = -1
        binding.cache_append(d.k_new, d.v_new, d.k_cache, d.v_cache, slots.cuda())
        torch.cuda.synchronize()
        k = W.storage_numpy(wl.k_cache); v = W.storage_numpy(wl.v_cache)
        oracle.cache_append(W.storage_numpy(wl.k_new), W.storage_numpy(wl.v_new), k, v, slots.numpy(), dtype)
        assert np.array_equal(W.storage_numpy(d.k_cache), k)
        assert np.array_equal(W.storage_numpy(d.v_cache), v)


def test_page_permutation_leaves_the_result_bitwise_unchanged():
    wl = W.make_custom("perm", "bf16", 8, 2, 128, 16, [300, 41], seed=24)
    got, _ = util.gpu_decode(wl)
    perm = torch.from_numpy(np.random.default_rng(1).permutation(wl.num_blocks))
    k2 = torch.empty_like(wl.k_cache); v2 = torch.empty_like(wl.v_cache)
    k2[perm] = wl.k_cache; v2[perm] = wl.v_cache
    bt = wl.block_tables.long()
    bt2 = torch.where(bt >= 0, perm[bt.clamp(min=0)], torch.full_like(bt, -1)).int()
    slot2 = perm[wl.slot_mapping // wl.bs] * wl.bs + wl.slot_mapping % wl.bs
    wl2 = W.Workload(**{**wl.__dict__, "k_cache": k2, "v_cache": v2, "block_tables": bt2, "slot_mapping": slot2})
    got2, _ = util.gpu_decode(wl2)
    assert np.array_equal(got, got2)


def test_empty_batch_and_error_codes_on_device_pointers():
    wl = W.make_config(1)
    d = util.DeviceWorkload(wl)
    empty = torch.empty((0, 4, 64), device="cuda")
    binding.paged_attention_decode(empty, empty, d.k_cache, d.v_cache, d.block_tables[:0], d.context_lens[:0],
                                   d.alibi_slopes, wl.scale)
    with pytest.raises(binding.OptGqaError) as e:
        binding.paged_attention_decode(d.out, d.q, d.k_cache, d.v_cache, d.block_tables, d.context_lens,
                                       d.alibi_slopes, wl.scale, partition_size=20)
    assert e.value.code == -2


def test_decode_step_replayed_from_a_cuda_graph():
    """One step (append -> balanced decode -> reduce, chained by programmatic dependent launches) captured once
    and replayed on new inputs written into the same buffers."""
    wl = W.make_custom("graph", "bf16", 32, 4, 128, 16, [1500, 700, 40], seed=27)
    d = util.DeviceWorkload(wl)
    P, maxP = 512, 3
    ws = torch.empty(binding.workspace_bytes(wl.B, wl.Hq, wl.D, maxP), device="cuda:0", dtype=torch.uint8)
    k0, v0 = d.k_cache.clone(), d.v_cache.clone()

    def step():
        binding.decode_step(d.out, d.q, d.k_new, d.v_new, d.slot_mapping, d.k_cache, d.v_cache, d.block_tables,
                            d.context_lens, d.alibi_slopes, wl.scale, partition_size=P, workspace=ws,
                            max_partitions=maxP, stream=stream)

    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        step()                                   # first call outside capture: one-time per-device set-up
    stream.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        step()
    # new values in the same buffers, then replay
    wl2 = W.make_custom("graph2", "bf16", 32, 4, 128, 16, [1500, 700, 40], seed=28)
    for name in ("q", "k_new", "v_new", "k_cache", "v_cache", "block_tables", "slot_mapping"):
        getattr(d, name).copy_(getattr(wl2, name).cuda())
    d.out.fill_(float("nan"))
    torch.cuda.synchronize()
    graph.replay()
    torch.cuda.synchronize()
    assert binding.device_status() == 0
    want = util.oracle_attention(wl2)
    got = d.out.double().cpu().numpy()
    assert np.max(np.abs(got - want)) <= util.TOL["bf16"]
    del k0, v0


def test_one_very_long_sequence():
    """200k tokens in one sequence (12.5k pages): the stream is cut across all workers, partitions of 512 and 4096."""
    wl = W.make_custom("long", "bf16", 8, 1, 128, 16, [200_003], seed=29)
    _check(wl, partition_size=512, balanced=True)
    _check(wl, partition_size=4096)
    _check(wl, partition_size=4096, balanced=True)


def test_many_short_sequences():
    """2048 sequences of 0..64 tokens: more sequences than one 32-lane scan step, single-tile pieces, empty rows."""
    rng = np.random.default_rng(30)
    lens = rng.integers(0, 65, size=2048)
    wl = W.make_custom("short", "bf16", 8, 1, 128, 16, lens, seed=30, poison=True)
    _check(wl, partition_size=512, balanced=True)
    _check(wl, partition_size=16)
    _check(wl)


def test_largest_group_and_smallest_head_dim():
    wl = W.make_custom("g8d64", "bf16", 64, 8, 64, 32, [3000, 17, 4100], seed=31, poison=True)
    _check(wl, partition_size=512, balanced=True)
    _check(wl, partition_size=256)
    wl32 = W.make_custom("g8d64f", "fp32", 16, 2, 64, 32, [700, 17], seed=32, poison=True)
    _check(wl32, partition_size=128)


@pytest.mark.parametrize("pinned", [True, False, "mapped"])
def test_decode_step_from_host_buffers(pinned):
    """opt_gqa_decode_step_host: pinned buffers are read and written by the kernels directly, pageable ones are copied;
    opt_gqa_decode_step_mapped takes the pinned buffers' device-side addresses without looking them up."""
    for wl, P in ((W.make_config(3, shrink=8), 512), (W.make_config(1), 0)):
        d = util.DeviceWorkload(wl)
        pin = (lambda t: t.contiguous().pin_memory()) if pinned else (lambda t: t.contiguous().clone())
        hq, hk, hv = pin(wl.q), pin(wl.k_new), pin(wl.v_new)
        hs, ht, hl = pin(wl.slot_mapping), pin(wl.block_tables), pin(wl.context_lens)
        hout = pin(torch.full_like(wl.q, float("nan")))
        tdt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
        maxP = max(1, (int(wl.context_lens.max()) + P - 1) // P) if P else 1
        staging = torch.empty(binding.step_staging_bytes(wl.B, wl.Hq, wl.Hkv, wl.D, wl.max_blocks, tdt), dtype=torch.uint8,
                              device="cuda:0")
        ws = torch.empty(max(16, binding.workspace_bytes(wl.B, wl.Hq, wl.D, maxP)), dtype=torch.uint8, device="cuda:0")
        step = binding.decode_step_mapped if pinned == "mapped" else binding.decode_step_host
        step(hout, hq, hk, hv, hs, ht, hl, staging, d.k_cache, d.v_cache, d.alibi_slopes, wl.scale,
             partition_size=P, workspace=ws if P else None, max_partitions=maxP)
        torch.cuda.synchronize()
        assert binding.device_status() == 0
        want = util.oracle_attention(wl)
        assert np.max(np.abs(hout.double().numpy() - want)) <= util.TOL[wl.dtype], (wl.name, pinned)


@pytest.mark.parametrize("scale", [0.0, 0.02, 1.0, 6.0])
@pytest.mark.parametrize("slope", ["usual", "zero", "steep", "negative"])
def test_reference_maximum_that_moves_inside_a_piece(scale, slope):
    """The streaming kernel walks a piece from its last tile backwards and moves its reference maximum only when a
    score exceeds it by 2^8.  Large scales make the maximum jump at arbitrary tiles, steep or negative slopes make it
    move at every tile or never: the result must be the oracle's in every case."""
    Hq = 8
    slopes = {"usual": None, "zero": torch.zeros(Hq), "steep": torch.full((Hq,), 3.0),
              "negative": -torch.logspace(-3, -1, Hq)}[slope]
    wl = W.make_custom("maxmove", "bf16", Hq, 2, 128, 16, [2100, 515, 16, 1, 700], seed=29, poison=True,
                       slopes=slopes, scale=scale)
    for P in (512, 64):
        _check(wl, partition_size=P, balanced=True)
    _check(wl, partition_size=128)


def test_host_step_called_repeatedly_reads_the_buffers_anew():
    """Repeated calls of opt_gqa_decode_step_host with the same buffers, on a stream of the caller's: every call
    reads what the pinned buffers hold at that moment and leaves its result in out_host."""
    wl = W.make_custom("hoststeps", "bf16", 32, 4, 128, 16, [1500, 700, 40, 1], seed=31)
    d = util.DeviceWorkload(wl)
    pin = lambda t: t.contiguous().pin_memory()
    hq, hk, hv = pin(wl.q), pin(wl.k_new), pin(wl.v_new)
    hs, ht, hl = pin(wl.slot_mapping), pin(wl.block_tables), pin(wl.context_lens)
    hout = pin(torch.full_like(wl.q, float("nan")))
    P, maxP = 512, 3
    staging = torch.empty(binding.step_staging_bytes(wl.B, wl.Hq, wl.Hkv, wl.D, wl.max_blocks, torch.bfloat16),
                          dtype=torch.uint8, device="cuda:0")
    ws = torch.empty(binding.workspace_bytes(wl.B, wl.Hq, wl.D, maxP), dtype=torch.uint8, device="cuda:0")
    stream = torch.cuda.Stream()
    gen = torch.Generator().manual_seed(5)
    for call in range(5):
        q = torch.randn(wl.q.shape, generator=gen).to(torch.bfloat16)
        hq.copy_(q)
        hout.fill_(float("nan"))
        with torch.cuda.stream(stream):
            binding.decode_step_host(hout, hq, hk, hv, hs, ht, hl, staging, d.k_cache, d.v_cache, d.alibi_slopes,
                                     wl.scale, partition_size=P, workspace=ws, max_partitions=maxP)
        stream.synchronize()
        assert binding.device_status() == 0
        want = util.oracle_attention(W.Workload(**{**wl.__dict__, "q": q}))
        assert np.max(np.abs(hout.double().numpy() - want)) <= util.TOL["bf16"], call


@pytest.mark.parametrize("shape", [(32, 4, 128, 16), (8, 2, 64, 32), (4, 4, 128, 32)])
def test_bf16_partials_of_the_tile_kernel_match_the_oracle_partials(shape):
    """opt_gqa_paged_attention_decode on bf16 caches (the tensor-core tile kernel, one CTA per partition): every
    partition's normalised result and log-sum-exp on their own, not only the merged output."""
    import oracle
    Hq, Hkv, D, bs = shape
    P = 64
    wl = W.make_custom("pbf16", "bf16", Hq, Hkv, D, bs, [130, 40, 77, 1, 0, 1029], seed=61, poison=True)
    _, d = util.gpu_decode(wl, partition_size=P)
    a = util.oracle_inputs(wl)
    maxP = d.partial_out.shape[2]
    po, pl = oracle.partition_partials(a["q"], a["k"], a["v"], a["bt"], a["n"], a["slopes"], wl.scale, wl.dtype, P, maxP)
    gpo, gpl = d.partial_out.double().cpu().numpy(), d.partial_lse.double().cpu().numpy()
    for s in range(wl.B):
        np_s = (int(a["n"][s]) + P - 1) // P
        # p enters the tensor core rounded to bf16 (relative 2^-9 per term, averaged by the normalised sum)
        assert np.max(np.abs(gpo[s, :, :np_s] - po[s, :, :np_s]), initial=0.0) <= util.TOL["bf16"]
        assert np.max(np.abs(gpl[s, :, :np_s] - pl[s, :, :np_s]), initial=0.0) <= 5e-3
        assert np.isnan(gpo[s, :, np_s:]).all() and np.isnan(gpl[s, :, np_s:]).all()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("D", [64, 128])
def test_reduce_kernel_alone_on_the_oracle_partials(dtype, D):
    """opt_gqa_paged_attention_reduce fed with the ORACLE's partials (rounded to fp32) against the oracle's merge:
    the merge kernel on its own, with no decode kernel of the library in the loop."""
    import oracle
    P = 32
    wl = W.make_custom("ronly", dtype, 8, 2, D, 16, [700, 33, 0, 31, 32, 2049], seed=62)
    a = util.oracle_inputs(wl)
    maxP = (2049 + P - 1) // P
    po, pl = oracle.partition_partials(a["q"], a["k"], a["v"], a["bt"], a["n"], a["slopes"], wl.scale, wl.dtype, P, maxP)
    po32, pl32 = po.astype(np.float32), pl.astype(np.float32)
    for s in range(wl.B):                   # entries past a sequence's partitions must never be read
        np_s = (int(a["n"][s]) + P - 1) // P
        po32[s, :, np_s:] = np.nan
        pl32[s, :, np_s:] = np.nan
    want = oracle.reduce(po32.astype(np.float64), pl32.astype(np.float64), a["n"], P)
    out = torch.full((wl.B, wl.Hq, D), float("nan"), device="cuda:0", dtype=W.TORCH_DTYPES[dtype])
    binding.paged_attention_reduce(out, torch.from_numpy(po32).cuda(), torch.from_numpy(pl32).cuda(),
                                   wl.context_lens.cuda(), P)
    torch.cuda.synchronize()
    got = out.double().cpu().numpy()
    assert np.isfinite(got).all()
    assert np.max(np.abs(got - want)) <= (1e-6 if dtype == "fp32" else 2.0 ** -8 * 4.5)   # fp32 sums; one bf16 rounding
    assert np.array_equal(got[2], np.zeros_like(got[2]))                                    # the empty sequence


@pytest.mark.parametrize("dtype,simt", [("fp32", False), ("bf16", False), ("bf16", True)])
def test_context_lengths_beyond_the_promised_sizes_stay_inside_the_buffers(dtype, simt):
    """A length that breaks the caller's promises (n_s > max_partitions * P, n_s > max_blocks * bs) must give a wrong
    row for that sequence, never an access outside the page table, the pool or the partials: canary rows around the
    partials stay intact and the other sequences keep their results."""
    wl = W.make_custom("promise", dtype, 8, 2, 128, 16, [100, 300, 64], seed=63)
    d = util.DeviceWorkload(wl)
    binding.cache_append(d.k_new, d.v_new, d.k_cache, d.v_cache, d.slot_mapping)
    want = util.oracle_attention(wl)
    P, maxP = 64, 5
    lens = wl.context_lens.clone()
    lens[1] = 300 + 64 * 40                         # far past max_partitions * P and past the page table
    rows = wl.B * wl.Hq * maxP
    po = torch.full((rows + 2 * wl.Hq, wl.D), 7.0, device="cuda:0", dtype=torch.float32)   # canaries before and after
    pl = torch.full((rows + 2 * wl.Hq,), 7.0, device="cuda:0", dtype=torch.float32)
    po_in = po[wl.Hq: wl.Hq + rows].view(wl.B, wl.Hq, maxP, wl.D)
    pl_in = pl[wl.Hq: wl.Hq + rows].view(wl.B, wl.Hq, maxP)
    decode = binding.paged_attention_decode_simt if simt else binding.paged_attention_decode
    decode(None, d.q, d.k_cache, d.v_cache, d.block_tables, lens.cuda(), d.alibi_slopes, wl.scale, partition_size=P,
           partial_out=po_in, partial_lse=pl_in, max_partitions=maxP)
    binding.paged_attention_reduce(d.out, po_in, pl_in, lens.cuda(), P)
    decode(d.out, d.q, d.k_cache, d.v_cache, d.block_tables, lens.cuda(), d.alibi_slopes, wl.scale)   # single pass too
    binding.paged_attention_reduce(d.out, po_in, pl_in, lens.cuda(), P)
    torch.cuda.synchronize()
    assert binding.device_status() == 0
    assert bool((po[: wl.Hq] == 7.0).all()) and bool((po[wl.Hq + rows:] == 7.0).all())
    assert bool((pl[: wl.Hq] == 7.0).all()) and bool((pl[wl.Hq + rows:] == 7.0).all())
    got = d.out.double().cpu().numpy()
    for s in (0, 2):
        assert np.max(np.abs(got[s] - want[s])) <= util.TOL[dtype]


def test_a_bounded_wait_that_runs_out_is_reported_and_leaves_the_device_usable():
    """Failure detection without a fault: one warp waits, with a short limit, for bytes nobody sends; the kernel
    records the timeout in the status word and returns.  The status reads -6 once, then 0, and decode still works."""
    assert binding.device_status() == 0
    binding.debug_wait_timeout(1 << 16)
    torch.cuda.synchronize()
    assert binding.device_status() == -6
    assert binding.status_string(-6) == "a bounded device-side wait ran out"
    assert binding.device_status() == 0
    with pytest.raises(binding.OptGqaError):
        binding.debug_wait_timeout(1 << 30)          # limits are capped: no long waits on request
    wl = W.make_custom("after", "bf16", 8, 2, 128, 16, [700, 33], seed=64)
    _check(wl, partition_size=256, balanced=True)
    _check(wl)


def test_read_stream_probe_reads_every_chunk():
    """The read-only probe of the benchmark: its checksum is the XOR of one 16-byte word per 256 bytes."""
    n = 8192 * 301
    src = torch.randint(-2**31, 2**31 - 1, (n // 4,), dtype=torch.int32, device="cuda:0")
    chk = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    binding.debug_read_stream(src, chk)
    torch.cuda.synchronize()
    assert binding.device_status() == 0
    words = src.cpu().numpy().view(np.uint32).reshape(-1, 64)[:, :4]       # the first 16 bytes of every 256
    assert int(chk.cpu().numpy().view(np.uint32)[0]) == int(np.bitwise_xor.reduce(words.reshape(-1)))


def test_undersized_workspace_is_refused_before_anything_runs():
    wl = W.make_custom("ws", "bf16", 8, 2, 128, 16, [700, 33], seed=65)
    d = util.DeviceWorkload(wl)
    P, maxP = 64, 11
    need = binding.workspace_bytes(wl.B, wl.Hq, wl.D, maxP)
    small = torch.empty(need // 2, dtype=torch.uint8, device="cuda:0")
    d.out.fill_(3.0)
    for call in (
        lambda: binding.paged_attention_decode_balanced(d.q, d.k_cache, d.v_cache, d.block_tables, d.context_lens,
                                                        d.alibi_slopes, wl.scale, P, small, maxP),
        lambda: binding.paged_attention_reduce_balanced(d.out, small, d.context_lens, wl.Hkv, P, maxP),
        lambda: binding.paged_attention_decode_local(d.out, d.q, d.k_cache, d.v_cache, d.block_tables, d.context_lens,
                                                     d.alibi_slopes, wl.scale, P, small, maxP, 100),
        lambda: binding.decode_step(d.out, d.q, d.k_new, d.v_new, d.slot_mapping, d.k_cache, d.v_cache, d.block_tables,
                                    d.context_lens, d.alibi_slopes, wl.scale, partition_size=P, workspace=small,
                                    max_partitions=maxP),
    ):
        with pytest.raises(binding.OptGqaError) as e:
            call()
        assert e.value.code == -2
    torch.cuda.synchronize()
    assert bool((d.out == 3.0).all())
    assert torch.equal(d.k_cache.cpu(), wl.k_cache)        # the fused append did not run either


def test_first_calls_from_several_host_threads_at_once():
    """The per-device caches (symbol addresses, kernel attributes, SM count) are filled by whichever calls come
    first; here four host threads of a fresh process make their first calls together, each on its own stream and
    buffers, and every one must give the oracle's result."""
    import subprocess
    import sys
    import textwrap

    code = textwrap.dedent("""
        import sys, threading
        import numpy as np, torch
        sys.path.insert(0, %r)
        from paper_2505_02351_b200 import binding, workloads as W
        from tests import util
        binding.load()
        torch.cuda.init()
        wls = [W.make_custom("thr%%d" %% i, "bf16" if i %% 2 == 0 else "fp32", 8, 2, 128 if i < 2 else 64, 16,
                             [700 + 37 * i, 33, 0, 260], seed=120 + i) for i in range(4)]
        want = [util.oracle_attention(w) for w in wls]
        devs = [util.DeviceWorkload(w) for w in wls]
        streams = [torch.cuda.Stream() for _ in wls]
        torch.cuda.synchronize()
        barrier = threading.Barrier(len(wls))
        errs = [None] * len(wls)

        def work(i):
            wl, d = wls[i], devs[i]
            try:
                barrier.wait()
                with torch.cuda.stream(streams[i]):
                    binding.cache_append(d.k_new, d.v_new, d.k_cache, d.v_cache, d.slot_mapping)
                    if wl.dtype == "bf16":
                        ws = torch.empty(binding.workspace_bytes(wl.B, wl.Hq, wl.D, 4), dtype=torch.uint8, device="cuda:0")
                        binding.paged_attention_decode_balanced(d.q, d.k_cache, d.v_cache, d.block_tables, d.context_lens,
                                                                d.alibi_slopes, wl.scale, 256, ws, 4)
                        binding.paged_attention_reduce_balanced(d.out, ws, d.context_lens, wl.Hkv, 256, 4)
                    else:
                        binding.paged_attention_decode(d.out, d.q, d.k_cache, d.v_cache, d.block_tables, d.context_lens,
                                                       d.alibi_slopes, wl.scale)
                streams[i].synchronize()
                errs[i] = float(np.max(np.abs(d.out.double().cpu().numpy() - want[i])))
            except Exception as e:          # noqa: BLE001
                errs[i] = repr(e)

        threads = [threading.Thread(target=work, args=(i,)) for i in range(len(wls))]
        [t.start() for t in threads]
        [t.join() for t in threads]
        assert binding.device_status() == 0
        for i, e in enumerate(errs):
            assert isinstance(e, float) and e <= util.TOL[wls[i].dtype], (i, e)
        print("threads ok", errs)
    """ % util.ROOT)
    out = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stdout + out.stderr
    assert "threads ok" in out.stdout
