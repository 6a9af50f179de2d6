"""The benchmark configurations at full size, in the launch configuration bench.py times.

The oracle cannot redo these sizes whole in seconds, so: sampled (sequence, KV head) units are compared
with the oracle in full (masks bit-exact, mu, attention output of the unit's G query heads), and
properties that hold at any size are checked on everything (popcount(mask) == T on every token, kept
values' saliency >= pruned saliency on a sample, lengths, status word).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_15212_b200 import binding as B
from paper_2508_15212_b200 import build as spark_build
from paper_2508_15212_b200.cache import SparkCache
from workloads import inputs
from workloads.batches import build_evicted_batch, permuted_block_table

pytestmark = pytest.mark.gpu
TOL = 2e-3          # bf16 storage, fp32 accumulation


@pytest.fixture(scope="module", autouse=True)
def built():
    spark_build.build()
    B.lib()


def to_np(t):
    t = t.detach().cpu()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def popcounts(mask_i32: torch.Tensor) -> torch.Tensor:
    """popcount of each token's 128-bit mask, on the device, independent of the library."""
    m = mask_i32.to(torch.int64) & 0xFFFFFFFF
    cnt = torch.zeros(m.shape[:-1], dtype=torch.int64, device=m.device)
    for w in range(4):
        x = m[..., w]
        for _ in range(32):
            cnt += x & 1
            x = x >> 1
    return cnt


def check_unit(wl, cache, out, b, h, keep, lens, keep_v=0):
    """Full oracle parity of one (sequence, KV head) unit, including its G query heads' outputs."""
    Bn, Hq, Hkv, W, D, S = wl.shape
    G = Hq // Hkv
    n = lens[b]
    q_win = wl.q_win[b:b + 1, h * G:(h + 1) * G].cpu()
    k = wl.k[b:b + 1, h:h + 1, :n].cpu().contiguous()
    v = wl.v[b:b + 1, h:h + 1, :n].cpu().contiguous()
    q = wl.q[b:b + 1, h * G:(h + 1) * G].cpu()
    _, a = oracle.window_mean(q_win, 1)
    assert np.array_equal(cache.qnorm[b, h].cpu().numpy(), a[0, 0])
    c = oracle.compress(k, [n], keep, a)
    c["vmask"] = oracle.prune_values(v, [n], keep_v) if 0 < keep_v < 128 else None
    ref, _ = oracle.decode_attn(q, k, v, [n], c["mask"], c["mu"], a, vmask=c["vmask"])
    return c, ref[0]


def test_config3_4x128k_ratio08_sampled_units():
    cfg = inputs.CONFIGS[2]
    for keep in (B.spark_keep_count(128, cfg["ratio"]), 26):        # floor rule (25) and the rounded count (26)
        wl = inputs.config_workload(2, device="cuda")
        inputs.enforce_saliency_gap(wl, keep)
        Bn, Hq, Hkv, W, D, S = wl.shape
        lens = wl.seq_lens.tolist()
        cache = SparkCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, window=W, keep=keep, dtype=wl.dtype, max_tokens=S)
        cache.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
        out = cache.decode(wl.q)
        assert cache.status() == 0
        u = cache.unpack(want_vals=False, want_v=False)
        assert bool((popcounts(u["mask"]) == keep).all())
        G = Hq // Hkv
        for b, h in ((0, 0), (3, 7), (1, 4)):
            c, ref = check_unit(wl, cache, out, b, h, keep, lens)
            assert np.array_equal(u["mask"][b, h].cpu().numpy().view(np.uint32), c["mask"][0, 0])
            assert np.allclose(u["mu"][b, h].cpu().numpy(), c["mu"][0, 0], rtol=1e-6, atol=0)
            d = float(np.abs(out[b, h * G:(h + 1) * G].cpu().numpy() - ref).max())
            assert d <= TOL, f"T={keep} unit ({b},{h}) max|delta| {d:.3e}"
        del wl, cache, u
        torch.cuda.empty_cache()


def test_config4_evicted_batch_pruning_and_decode():
    """All 32 prompts, as benchmarked: 256 units of 2048 tokens on 148 CTAs, i.e. the whole-units plan with
    two units in each of the first 108 CTAs and one in each of the remaining 40."""
    cfg = dict(inputs.CONFIGS[3])
    keep = B.spark_keep_count(128, cfg["ratio"])
    n_prompts = cfg["batch"]
    assert n_prompts == 32
    cache, q, kept, dense = build_evicted_batch(cfg, keep, n_prompts=n_prompts, keep_prompts=(0, 27, 31), guard=True)
    Hq, Hkv, W, budget, S = cfg["n_q_heads"], cfg["n_kv_heads"], cfg["window"], cfg["token_budget"], cfg["seq_lens"]
    G = Hq // Hkv
    assert cache.packed_lens.cpu().tolist() == [budget] * n_prompts
    kept_np = kept.cpu().numpy()
    assert (np.diff(kept_np, axis=-1) > 0).all() and (kept_np[..., -W:] == np.arange(S - W, S)).all()
    out = cache.decode(q)
    assert cache.status() == 0 and cache.broken_guards() == []
    u = cache.unpack(want_vals=False, want_v=False)
    assert bool((popcounts(u["mask"]) == keep).all())
    # units (0,0) and (0,1) are the first and second unit of CTA 0; (0,5) sits in CTA 2; units of prompts 27..31
    # (unit index >= 216) are alone in their CTA
    checks = [(0, 0, True), (0, 1, False), (0, 5, True), (27, 3, True), (31, 7, False)]
    for b, h, with_eviction in checks:
        wl = dense[b]
        q_win = wl.q_win[:, h * G:(h + 1) * G].cpu()
        if with_eviction:                                  # the oracle needs ~4 GFLOP per unit
            k = wl.k[:, h:h + 1].cpu().contiguous()
            ref_kept, n, vote, pooled = oracle.evict(q_win, k, [S], budget, cfg["pool_kernel"], want_votes=True)
            srt = np.sort(pooled[0, 0, :S - W])[::-1]
            gap = (srt[budget - W - 1] - srt[budget - W]) / srt[budget - W - 1]
            same = np.array_equal(kept_np[b, h], ref_kept[0, 0])
            overlap = len(set(kept_np[b, h].tolist()) & set(ref_kept[0, 0].tolist()))
            assert same or (gap <= 1e-4 and overlap >= budget - 2), f"unit ({b},{h}): overlap {overlap}, gap {gap:.2e}"
        # pruning + decode of this unit on the evicted token set fed to both sides
        idx = torch.from_numpy(kept_np[b, h].astype(np.int64))
        kg = wl.k[0, h].cpu()[idx].view(1, 1, budget, 128).contiguous()
        vg = wl.v[0, h].cpu()[idx].view(1, 1, budget, 128).contiguous()
        _, a = oracle.window_mean(q_win, 1)
        assert np.array_equal(cache.qnorm[b, h].cpu().numpy(), a[0, 0])
        c = oracle.compress(kg, [budget], keep, a)
        ref, _ = oracle.decode_attn(q[b:b + 1, h * G:(h + 1) * G].cpu(), kg, vg, [budget], c["mask"], c["mu"], a)
        assert np.array_equal(u["mask"][b, h].cpu().numpy().view(np.uint32), c["mask"][0, 0])
        d = float(np.abs(out[b, h * G:(h + 1) * G].cpu().numpy() - ref[0]).max())
        assert d <= TOL, f"unit ({b},{h}) max|delta| {d:.3e}"


@pytest.mark.parametrize("ratio", [0.3, 0.5, 0.7, 0.8])
def test_config5_qwen_paged_variable_lengths(ratio):
    cfg = inputs.CONFIGS[4]
    keep = B.spark_keep_count(128, ratio)
    for layer in (0, 27):
        wl = inputs.config_workload(4, device="cuda", seed_offset=layer)
        Bn, Hq, Hkv, W, D, S = wl.shape
        lens = wl.seq_lens.tolist()
        assert Bn == 16 and min(lens) >= 8192 and max(lens) <= 131072
        order = np.argsort(lens)
        sample = [int(order[0]), int(order[-1]), int(order[len(order) // 2])]     # shortest, longest, a middle one
        for b in sample:                                   # the saliency gap is enforced on the checked slices
            sub = inputs.Workload(q_win=wl.q_win[b:b + 1], k=wl.k[b:b + 1, :, :lens[b]], v=wl.v[b:b + 1],
                                  q=wl.q[b:b + 1], seq_lens=wl.seq_lens[b:b + 1], dtype=wl.dtype, meta={})
            inputs.enforce_saliency_gap(sub, keep)
        table, n_pages = permuted_block_table(Bn, Hkv, lens, "cuda", seed=1000 * layer + int(ratio * 10))
        cache = SparkCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, window=W, keep=keep, dtype=wl.dtype,
                           max_tokens=S, block_table=table, n_pool_pages=n_pages)
        cache.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
        out = cache.decode(wl.q)
        assert cache.status() == 0
        assert cache.packed_lens.cpu().tolist() == lens
        G = Hq // Hkv
        u = cache.unpack(want_vals=False, want_v=False)
        valid = torch.arange(S, device="cuda")[None, None, :] < wl.seq_lens[:, None, None]
        pc = popcounts(u["mask"])
        assert bool((pc[valid.expand_as(pc)] == keep).all()) and bool((pc[~valid.expand_as(pc)] == 0).all())
        for b in sample:
            h = (b + layer) % Hkv
            c, ref = check_unit(wl, cache, out, b, h, keep, lens)
            n = lens[b]
            assert np.array_equal(u["mask"][b, h, :n].cpu().numpy().view(np.uint32), c["mask"][0, 0])
            d = float(np.abs(out[b, h * G:(h + 1) * G].cpu().numpy() - ref).max())
            assert d <= TOL, f"ratio {ratio} layer {layer} unit ({b},{h}) max|delta| {d:.3e}"
        del wl, cache, u
        torch.cuda.empty_cache()


def test_config5_qwen_paged_with_value_pruning():
    """Layer 0 of the Qwen-shaped configuration with (0.5 + 0.5) key + value channel pruning."""
    keep = keep_v = B.spark_keep_count(128, 0.5)
    wl = inputs.config_workload(4, device="cuda", seed_offset=0)
    Bn, Hq, Hkv, W, D, S = wl.shape
    lens = wl.seq_lens.tolist()
    order = np.argsort(lens)
    sample = [int(order[0]), int(order[-1])]
    for b in sample:
        sub = inputs.Workload(q_win=wl.q_win[b:b + 1], k=wl.k[b:b + 1, :, :lens[b]], v=wl.v[b:b + 1],
                              q=wl.q[b:b + 1], seq_lens=wl.seq_lens[b:b + 1], dtype=wl.dtype, meta={})
        inputs.enforce_saliency_gap(sub, keep)
    table, n_pages = permuted_block_table(Bn, Hkv, lens, "cuda", seed=4242)
    cache = SparkCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, window=W, keep=keep, dtype=wl.dtype,
                       max_tokens=S, block_table=table, n_pool_pages=n_pages, keep_v=keep_v)
    cache.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
    out = cache.decode(wl.q)
    assert cache.status() == 0
    G = Hq // Hkv
    u = cache.unpack(want_vals=False, want_v=False, want_vmask=True)
    valid = torch.arange(S, device="cuda")[None, None, :] < wl.seq_lens[:, None, None]
    for name, want in (("mask", keep), ("vmask", keep_v)):
        pc = popcounts(u[name])
        assert bool((pc[valid.expand_as(pc)] == want).all()) and bool((pc[~valid.expand_as(pc)] == 0).all())
    for b in sample:
        h = b % Hkv
        c, ref = check_unit(wl, cache, out, b, h, keep, lens, keep_v=keep_v)
        n = lens[b]
        assert np.array_equal(u["mask"][b, h, :n].cpu().numpy().view(np.uint32), c["mask"][0, 0])
        assert np.array_equal(u["vmask"][b, h, :n].cpu().numpy().view(np.uint32), c["vmask"][0, 0])
        d = float(np.abs(out[b, h * G:(h + 1) * G].cpu().numpy() - ref).max())
        assert d <= TOL, f"unit ({b},{h}) max|delta| {d:.3e}"
