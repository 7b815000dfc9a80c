"""Parity of the tensor-core chunked-prefill variant (append -> prefill, through the C ABI) with the CPU oracle."""
import numpy as np
import pytest
import torch

from paper_2505_02351_b200 import binding
from paper_2505_02351_b200 import workloads as W
from tests import util

pytestmark = pytest.mark.gpu
TOL = util.TOL["bf16"]


def _check(wl, **kw):
    got, d = util.gpu_prefill(wl, **kw)
    want = util.oracle_attention(wl, **kw)
    assert np.isfinite(got).all()
    err = np.max(np.abs(got - want)) if got.size else 0.0
    assert err <= TOL, f"{wl.name}: max-abs error {err}"
    return got, want, d


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (4, 2), (8, 2), (8, 1)])
@pytest.mark.parametrize("bs", [16, 32])
def test_shape_matrix_ragged_chunks(D, Hq, Hkv, bs):
    # new-token counts that end inside a query block, span several, equal the context (no history), or are 1
    lens = [200, 77, 33, 130, 1, 64, 300]
    qls = [70, 77, 1, 129, 1, 16, 17]
    wl = W.make_custom("pf", "bf16", Hq, Hkv, D, bs, lens, q_lens=qls, seed=D + Hq + bs, poison=True)
    _check(wl)                   # the default entry point runs on tcgen05 for both head dimensions
    _check(wl, slopes=False)
    _check(wl, mma=True)         # the warp-level kernel


def test_tiles_and_blocks_boundaries_on_tcgen05():
    # contexts and chunks around the 128-key tile and the 128-row query block: exactly full, one over, one under
    for G, Hkv in ((4, 2), (8, 1), (1, 2), (2, 2)):
        TQ = 128 // G
        lens = [128, 129, 127, 256 + TQ, 3 * 128 + 1, 640, 5]
        qls = [min(a, b) for a, b in zip(lens, [128, 1, TQ, TQ + 1, 2 * TQ - 1, 640, 5])]
        wl = W.make_custom("edge", "bf16", G * Hkv, Hkv, 128, 16, lens, q_lens=qls, seed=50 + G, poison=True)
        _check(wl)


def test_large_maximum_drift_forces_rescales():
    # scores that keep growing along the context (steep negative ALiBi slope is the usual case; here the values of
    # q.k themselves grow), so the running maximum moves by more than the rescale threshold many times
    wl = W.make_custom("drift", "bf16", 4, 1, 128, 16, [1500], q_lens=[300], seed=51,
                       slopes=torch.tensor([4.0, 1.0, 0.25, 0.0]), scale=1.0)
    _check(wl)
    _check(wl, mma=True)


def test_config5_shrunk():
    # the named workload with every length divided by 8: 512 existing + 256 new tokens per sequence
    wl = W.make_config(5, shrink=8, poison=True)
    assert wl.T == 4 * 256
    _check(wl)
    _check(wl, mma=True)


def test_prefill_with_one_new_token_is_the_decode_result():
    wl = W.make_custom("pf1", "bf16", 8, 2, 128, 16, [300, 41, 1000], q_lens=[1, 1, 1], seed=31)
    got, _ = util.gpu_prefill(wl)
    wl_dec = W.Workload(**{**wl.__dict__, "q_start_loc": None})
    dec, _ = util.gpu_decode(wl_dec)
    want = util.oracle_attention(wl)
    assert np.max(np.abs(got - want)) <= TOL
    assert np.max(np.abs(got - dec)) <= TOL


@pytest.mark.parametrize("scale", [0.0, -0.05, 0.5])
def test_scales_that_are_not_the_usual_one(scale):
    """The tcgen05 kernel takes the row maximum on the raw scores, which needs a positive factor: a negative scale
    negates Q inside the tensor-core instruction, a zero scale leaves the dot products out.  Both kernels, both head
    dimensions: the result is the oracle's."""
    for D in (128, 64):
        wl = W.make_custom("pfs", "bf16", 8, 2, D, 16, [300, 70], q_lens=[130, 70], seed=37)
        wl.scale = scale
        _check(wl)
        _check(wl, slopes=False)
        _check(wl, mma=True)


def test_steep_and_flat_slopes_on_the_tensor_core_bias():
    """slope / scale is split over three bf16 values inside the kernel: check slopes far from the usual ones."""
    for mult in (0.0, 1e-3, 7.0):
        wl = W.make_custom("pfb", "bf16", 8, 2, 128, 16, [700, 129], q_lens=[200, 129], seed=38)
        wl.alibi_slopes = wl.alibi_slopes * mult
        _check(wl)


def test_empty_sequences_and_no_new_tokens():
    # a sequence that contributes no new tokens leaves no row; the others are unaffected
    wl = W.make_custom("pf0", "bf16", 4, 2, 128, 16, [50, 64, 20], q_lens=[0, 64, 20], seed=32, poison=True)
    _check(wl)


def test_config5_full_size_every_row():
    """The full workload in the configuration the benchmark times (a query block sees up to 96 key tiles), every one
    of its 8192 x 32 output rows against the oracle (about half a minute of fp64 on the host cores)."""
    wl = W.make_config(5)
    got, _ = util.gpu_prefill(wl)
    assert np.isfinite(got).all()
    want = util.oracle_attention(wl)
    assert got.shape == want.shape == (4 * 2048, 32, 128)
    err = np.max(np.abs(got - want))
    assert err <= TOL, err


def test_config5_full_size_on_the_warp_level_kernel_sampled_rows():
    """The same workload through opt_gqa_paged_attention_prefill_mma; the oracle checks sampled rows one by one."""
    wl = W.make_config(5)
    got, _ = util.gpu_prefill(wl, mma=True)
    assert np.isfinite(got).all()
    rng = np.random.default_rng(5)
    rows = np.unique(np.concatenate([rng.integers(0, wl.T, size=24), [0, 2047, 2048, wl.T - 1]]))
    want = util.oracle_prefill_rows(wl, rows)
    err = np.max(np.abs(got[rows] - want))
    assert err <= TOL, err
    # property that holds at any size: every output lies in the convex hull of V's value range
    assert np.abs(got).max() <= float(wl.v_cache.float().abs().max().item()) + float(wl.v_new.float().abs().max().item())


# ------------------------------------------------------------------ the prompt branch with empty caches (contiguous k, v)
def _prompt(wl, slopes=True):
    import oracle
    dev = "cuda:0"
    q, k, v, qsl = wl.q.to(dev), wl.k_new.to(dev), wl.v_new.to(dev), wl.q_start_loc.to(dev)
    sl = wl.alibi_slopes.to(dev) if slopes else None
    out = torch.full_like(q, float("nan"))
    lens = wl.q_start_loc.numpy()[1:] - wl.q_start_loc.numpy()[:-1]
    binding.prompt_attention(out, q, k, v, qsl, int(lens.max()), sl, wl.scale)
    torch.cuda.synchronize()
    assert binding.device_status() == 0
    want = oracle.prompt_attention(W.storage_numpy(wl.q), W.storage_numpy(wl.k_new), W.storage_numpy(wl.v_new),
                                   wl.q_start_loc.numpy(), wl.alibi_slopes.numpy().astype(np.float64) if slopes else None,
                                   wl.scale, "bf16")
    got = out.double().cpu().numpy()
    assert np.isfinite(got).all()
    assert np.max(np.abs(got - want)) <= TOL, wl.name
    return got


@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (4, 2), (8, 2), (8, 1), (32, 8)])
def test_prompt_attention_contiguous(Hq, Hkv):
    lens = [200, 77, 1, 129, 64, 300, 128]
    wl = W.make_custom("prompt", "bf16", Hq, Hkv, 128, 16, lens, q_lens=lens, seed=70 + Hq)
    _prompt(wl)
    _prompt(wl, slopes=False)


def test_prompt_attention_equals_prefill_over_the_appended_cache():
    lens = [513, 40, 1000]
    wl = W.make_custom("prompt2", "bf16", 8, 2, 128, 16, lens, q_lens=lens, seed=75)
    got = _prompt(wl)
    paged, _ = util.gpu_prefill(wl)           # append the same tokens into pages, then prefill over the pages
    assert np.array_equal(got, paged)         # same kernel, same tiles, same order: bitwise equal


@pytest.mark.parametrize("scale", [None, 0.0, -0.1])
def test_prompt_attention_head_dim_64_and_other_scales(scale):
    for D in (64, 128):
        lens = [200, 77, 1, 129, 64]
        wl = W.make_custom("prompt3", "bf16", 8, 2, D, 16, lens, q_lens=lens, seed=76, scale=scale)
        _prompt(wl)
        _prompt(wl, slopes=False)


def test_prompt_attention_rejects_what_it_does_not_support():
    wl = W.make_custom("prompt4", "bf16", 4, 2, 64, 16, [10], q_lens=[10], seed=77)
    q = wl.q.cuda()
    with pytest.raises(binding.OptGqaError) as e:
        binding.prompt_attention(torch.empty_like(q), q.float(), wl.k_new.cuda().float(), wl.v_new.cuda().float(),
                                 wl.q_start_loc.cuda(), 10, None, wl.scale)
    assert e.value.code == -3                 # fp32 tensors: the entry point is bf16 only
