"""Parity of the ratio-free selection variants (SparK-p, SparK-g) and of sampled recovery (Gaussian,
Exponential) against the CPU oracle, through the C ABI, on identical seeded inputs.

Bar: kept-channel masks bit-exact; mu and the all-channel statistics within 1e-6 relative; attention output
max|delta| <= 1e-5 (fp32 storage) / 2e-3 (bf16 storage).  The draws of sampled recovery come from the same
counter-based generator on both sides, so the recovered keys agree to rounding.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_15212_b200 import binding as B
from paper_2508_15212_b200 import build as spark_build
from paper_2508_15212_b200.cache import SparkCache
from workloads import inputs
from workloads.batches import permuted_block_table

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 2e-3}


@pytest.fixture(scope="module", autouse=True)
def built():
    spark_build.build()
    B.lib()


def make(dtype, Bn, Hq, Hkv, lens, W, seed):
    return inputs.make_workload(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, seq_lens=lens, window=W, dtype=dtype,
                                sigma_s=1.0 if dtype == "bf16" else 0.5, seed=seed, device="cuda")


def to_np(t):
    t = t.detach().cpu()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def check_selection(wl, cap, *, top_p=None, group_prune=None, block_table=None, n_pool_pages=None):
    """Compress with a variant rule, compare masks / mu / kept values with the oracle, then the decode output."""
    Bn, Hq, Hkv, W, D, S = wl.shape
    wl_cpu = wl.to("cpu")
    _, a = oracle.window_mean(wl_cpu.q_win, Hkv)
    ref = oracle.select_variant(wl_cpu.k, wl_cpu.seq_lens, a, top_p=top_p, cap=cap if top_p is not None else None,
                                group_prune=group_prune)
    cache = SparkCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, window=W, keep=cap, dtype=wl.dtype, max_tokens=S,
                       top_p=top_p, group_prune=group_prune, block_table=block_table, n_pool_pages=n_pool_pages,
                       guard=True)
    cache.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
    assert cache.status() == 0
    assert np.array_equal(cache.qnorm.cpu().numpy(), a)
    u = cache.unpack()
    mask = u["mask"].cpu().numpy().view(np.uint32)
    assert np.array_equal(mask, ref["mask"]), "kept-channel masks must be bit-exact"
    assert np.allclose(u["mu"].cpu().numpy(), ref["mu"], rtol=1e-6, atol=0)
    # kept values: the first count slots hold the kept channels in ascending order, the rest of the row is zero
    kk, vals = to_np(wl_cpu.k), to_np(u["vals"])
    bits = ((ref["mask"][..., None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(Bn, Hkv, S, D).astype(bool)
    lens = wl_cpu.seq_lens.tolist()
    rng = np.random.default_rng(0)
    for _ in range(200):
        b, h = int(rng.integers(Bn)), int(rng.integers(Hkv))
        if lens[b] == 0:
            continue
        t = int(rng.integers(lens[b]))
        n = int(ref["count"][b, h, t])
        assert np.array_equal(vals[b, h, t, :n], kk[b, h, t][bits[b, h, t]]) and not vals[b, h, t, n:].any()
    if top_p is not None and block_table is None:
        # SparK-p pools carry, behind the pages, how many slot rows of each page are in use: the largest kept
        # count among the page's live tokens (the decode step copies only that much of a page)
        n_pages, pb = cache.params.n_pool_pages, cache.page_bytes
        off = (n_pages * pb + 255) // 256 * 256
        assert cache.pages.numel() == B.spark_pool_bytes(cache.params) == off + 4 * n_pages
        rows = cache.pages[off:off + 4 * n_pages].view(torch.int32).cpu().numpy().reshape(Bn, Hkv, cache.table_blocks)
        cnt = np.zeros((Bn, Hkv, cache.table_blocks * 16), np.int32)
        cnt[:, :, :S] = ref["count"]
        assert np.array_equal(rows, cnt.reshape(Bn, Hkv, cache.table_blocks, 16).max(axis=-1))
    out_ref, lse_ref = oracle.decode_attn(wl_cpu.q, wl_cpu.k, wl_cpu.v, wl_cpu.seq_lens, ref["mask"], ref["mu"], a)
    lse = cache.alloc_lse()
    out = cache.decode(wl.q, lse=lse)
    assert cache.status() == 0 and cache.broken_guards() == []
    d = float(np.abs(out.cpu().numpy() - out_ref).max())
    assert d <= TOL[wl.dtype], f"max|delta| {d:.3e}"
    fin = np.isfinite(lse_ref)
    assert np.allclose(lse.cpu().numpy()[fin], lse_ref[fin], rtol=0, atol=1e-3 if wl.dtype == "bf16" else 2e-5)
    return ref


@pytest.mark.parametrize("dtype,p,cap", [("bf16", 0.99, 128), ("bf16", 0.9, 96), ("bf16", 0.5, 128), ("f32", 0.95, 128),
                                         ("bf16", 0.99, 40)])
def test_top_p_selection_and_decode(dtype, p, cap):
    wl = make(dtype, 3, 8, 2, [1, 37, 530], 8, seed=500 + cap)
    ref = check_selection(wl, cap, top_p=p)
    live = ref["count"][ref["count"] > 0]
    assert live.min() >= 1 and live.max() <= cap
    if cap >= 96:
        assert len(np.unique(live)) > 3                    # the count really varies per token
    else:
        assert (live == cap).any()                         # the page capacity binds


def test_top_p_paged_pool_gqa7():
    lens = [700, 33, 1200, 16]
    wl = make("bf16", 4, 28, 4, lens, 32, seed=510)
    table, n_pages = permuted_block_table(4, 4, lens, "cuda", seed=3, spare=5)
    check_selection(wl, 128, top_p=0.99, block_table=table, n_pool_pages=n_pages)


@pytest.mark.parametrize("dtype,ratios", [("bf16", [0.25, 0.5, 0.75, 1.0]), ("bf16", [0.1, 0.3, 0.5, 0.7, 0.9]),
                                          ("f32", [0.0, 0.5, 1.0]), ("bf16", [0.5])])
def test_rank_group_selection_and_decode(dtype, ratios):
    wl = make(dtype, 3, 8, 2, [1, 37, 530], 8, seed=520 + len(ratios))
    cap = B.spark_group_keep(128, ratios)
    ref = check_selection(wl, cap, group_prune=ratios)
    assert (ref["count"][ref["count"] > 0] == cap).all()
    if len(ratios) == 1:                                   # one group is the fixed-ratio rule
        fixed = SparkCache(batch=3, n_q_heads=8, n_kv_heads=2, window=8, keep=cap, dtype=dtype, max_tokens=530)
        fixed.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
        assert np.array_equal(fixed.unpack(want_vals=False, want_v=False)["mask"].cpu().numpy().view(np.uint32), ref["mask"])
    with pytest.raises(B.SparkError):                      # a page that cannot hold the kept channels is refused
        SparkCache(batch=1, n_q_heads=4, n_kv_heads=1, window=4, keep=cap - 1, dtype=dtype, max_tokens=16,
                   group_prune=ratios)


def test_append_under_top_p_equals_compressing_the_longer_sequence():
    lens0, extra = [37, 16], 19
    wl = make("bf16", 2, 8, 2, [n + extra for n in lens0], 8, seed=530)
    Bn, Hq, Hkv, W, D, S = wl.shape
    kw = dict(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, window=W, keep=128, dtype="bf16", max_tokens=S, top_p=0.97)
    full, grown = SparkCache(**kw), SparkCache(**kw)
    full.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
    grown.compress(wl.q_win, wl.k, wl.v, torch.tensor(lens0, dtype=torch.int32, device="cuda"))
    for step in range(extra):
        idx = torch.tensor([n + step for n in lens0], device="cuda")
        grown.append(wl.k[torch.arange(Bn, device="cuda"), :, idx].contiguous(),
                     wl.v[torch.arange(Bn, device="cuda"), :, idx].contiguous())
    assert grown.status() == 0
    ua, ub = full.unpack(), grown.unpack()
    for key in ("mask", "mu", "vals", "v"):
        assert torch.equal(ua[key], ub[key]), key
    assert torch.equal(full.decode(wl.q), grown.decode(wl.q))


# ---------------------------------------------------------------- sampled recovery
def check_sampled(wl, keep, mode, seed, *, top_p=None, block_table=None, n_pool_pages=None):
    Bn, Hq, Hkv, W, D, S = wl.shape
    wl_cpu = wl.to("cpu")
    _, a = oracle.window_mean(wl_cpu.q_win, Hkv)
    if top_p is None:
        c = oracle.compress(wl_cpu.k, wl_cpu.seq_lens, keep, a, want_stats=True)
    else:
        c = oracle.select_variant(wl_cpu.k, wl_cpu.seq_lens, a, top_p=top_p, cap=keep, want_stats=True)
    out_ref, lse_ref = oracle.decode_attn_sampled(wl_cpu.q, wl_cpu.k, wl_cpu.v, wl_cpu.seq_lens, c["mask"], c["mu_all"],
                                                  c["sigma_all"], a, mode=mode, seed=seed)
    cache = SparkCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, window=W, keep=keep, dtype=wl.dtype, max_tokens=S,
                       recovery=mode, seed=seed, top_p=top_p, block_table=block_table, n_pool_pages=n_pool_pages,
                       guard=True)
    cache.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
    u = cache.unpack(want_vals=False, want_stats=True)
    assert np.array_equal(u["mask"].cpu().numpy().view(np.uint32), c["mask"])
    assert np.allclose(u["mu_all"].cpu().numpy(), c["mu_all"], rtol=1e-6, atol=0)
    assert np.allclose(u["sigma_all"].cpu().numpy(), c["sigma_all"], rtol=1e-6, atol=0)
    assert np.array_equal(to_np(u["v"])[0, 0, :wl_cpu.seq_lens[0]], to_np(wl_cpu.v)[0, 0, :wl_cpu.seq_lens[0]])
    lse = cache.alloc_lse()
    out = cache.decode(wl.q, lse=lse)
    out2 = cache.decode(wl.q)
    assert cache.status() == 0 and cache.broken_guards() == []
    assert torch.equal(out, out2)                          # the draws are fixed: every step sees the same keys
    d = float(np.abs(out.cpu().numpy() - out_ref).max())
    assert d <= TOL[wl.dtype], f"max|delta| {d:.3e} (max|out| {np.abs(out_ref).max():.3e})"
    fin = np.isfinite(lse_ref)
    assert np.array_equal(np.isneginf(lse.cpu().numpy()), np.isneginf(lse_ref))
    assert np.allclose(lse.cpu().numpy()[fin], lse_ref[fin], rtol=2e-6, atol=1e-3 if wl.dtype == "bf16" else 3e-5)
    # a different seed gives different keys
    other = SparkCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, window=W, keep=keep, dtype=wl.dtype, max_tokens=S,
                       recovery=mode, seed=seed + 1, top_p=top_p, block_table=block_table, n_pool_pages=n_pool_pages)
    other.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
    if keep < 128 and max(wl_cpu.seq_lens.tolist()) > 1:
        assert not torch.equal(other.decode(wl.q), out)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("mode", [B.SPARK_RECOVER_GAUSSIAN, B.SPARK_RECOVER_EXPONENTIAL])
@pytest.mark.parametrize("keep", [64, 25])
def test_sampled_recovery_ragged_lengths(dtype, mode, keep):
    wl = make(dtype, 3, 8, 2, [0, 37, 530], 8, seed=540 + keep + mode)
    inputs.enforce_saliency_gap(wl, keep)
    check_sampled(wl, keep, mode, seed=11)


@pytest.mark.parametrize("G,mode", [(1, 1), (7, 2), (8, 1)])
def test_sampled_recovery_group_sizes_and_paged_pool(G, mode):
    lens = [300, 47]
    wl = make("bf16", 2, 2 * G, 2, lens, 16, seed=560 + G)
    inputs.enforce_saliency_gap(wl, 38)
    table, n_pages = permuted_block_table(2, 2, lens, "cuda", seed=9, spare=3)
    check_sampled(wl, 38, mode, seed=5, block_table=table, n_pool_pages=n_pages)


def test_sampled_recovery_with_nothing_pruned_is_dense_attention():
    wl = make("bf16", 1, 4, 1, [200], 8, seed=570)
    check_sampled(wl, 128, B.SPARK_RECOVER_EXPONENTIAL, seed=2)


def test_sampled_recovery_on_top_p_selection():
    wl = make("bf16", 2, 8, 2, [150, 260], 8, seed=580)
    check_sampled(wl, 128, B.SPARK_RECOVER_EXPONENTIAL, seed=3, top_p=0.95)


def test_sampled_recovery_many_ctas_share_a_unit():
    """A sequence long enough that every unit is split over several CTAs (partials, tickets, last-arriver merge)."""
    wl = make("bf16", 1, 8, 2, [20000], 16, seed=590)
    inputs.enforce_saliency_gap(wl, 64)
    check_sampled(wl, 64, B.SPARK_RECOVER_GAUSSIAN, seed=4)


def test_sampled_recovery_refuses_pruned_value_rows():
    with pytest.raises(B.SparkError) as e:
        SparkCache(batch=1, n_q_heads=4, n_kv_heads=1, window=4, keep=64, dtype="bf16", max_tokens=16,
                   recovery=B.SPARK_RECOVER_GAUSSIAN, keep_v=64)
    assert e.value.code == 3
