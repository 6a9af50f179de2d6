"""Pins for the oracle's adaptive selection rules (SparK-p, SparK-g) and sampled recovery.

Sec. "Ablation Studies" (adaptive variants) and Sec. "Channel Recovery" (Gaussian / Exponential
distributions) with the statistics of App. "Caching Pruned Channel Statistics".  Expected values come from
the already pinned fixed-T oracle, from independent NumPy expressions, from the published test vectors of
the splitmix64 mixer, and from the closed-form moments and tail probabilities of the two distributions.
"""
import itertools
import math

import numpy as np
import pytest

import oracle


def rand_case(rng, B=1, Hq=1, Hkv=1, W=4, D=8, S=5):
    q_win = rng.standard_normal((B, Hq, W, D)).astype(np.float32)
    k = rng.standard_normal((B, Hkv, S, D)).astype(np.float32)
    v = rng.standard_normal((B, Hkv, S, D)).astype(np.float32)
    q = rng.standard_normal((B, Hq, D)).astype(np.float32)
    return q_win, k, v, q


def bits_of(mask_row, D):
    return [j for j in range(D) if (int(mask_row[j // 32]) >> (j % 32)) & 1]


def saliency(a, k):
    return (a[:, :, None, :] * np.abs(k)).astype(np.float32)        # one fp32 multiply, as the method fixes it


def dense_attention(q, K, V):
    q, K, V = np.asarray(q, np.float64), np.asarray(K, np.float64), np.asarray(V, np.float64)
    s = K @ q / math.sqrt(K.shape[1])
    e = np.exp(s - s.max())
    return (e / e.sum()) @ V, s.max() + math.log(e.sum())


# ---------------------------------------------------------------- SparK-p
@pytest.mark.parametrize("D,p", [(8, 0.5), (8, 0.9), (16, 0.99), (128, 0.99), (128, 0.7)])
def test_top_p_keeps_the_smallest_prefix_that_reaches_the_mass(D, p):
    rng = np.random.default_rng(100 + D)
    B, Hkv, S = 2, 2, 40
    q_win, k, v, q = rand_case(rng, B, Hkv, Hkv, 4, D, S)
    lens = [S, S - 7]
    _, a = oracle.window_mean(q_win, Hkv)
    sel = oracle.select_variant(k, lens, a, top_p=p)
    w = saliency(a, k).astype(np.float64)
    counts = set()
    for b, h, t in itertools.product(range(B), range(Hkv), range(S)):
        kept = bits_of(sel["mask"][b, h, t], D)
        if t >= lens[b]:
            assert kept == [] and sel["count"][b, h, t] == 0
            continue
        n = int(sel["count"][b, h, t])
        counts.add(n)
        assert n >= 1 and len(kept) == n
        srt = np.sort(w[b, h, t])[::-1]
        total = srt.sum()
        # minimality, with a margin so that summation order cannot matter
        assert srt[:n].sum() >= np.float32(p) * total * (1 - 1e-12)
        if n > 1:
            assert srt[:n - 1].sum() < np.float32(p) * total * (1 + 1e-12)
        assert w[b, h, t][kept].min() >= np.delete(w[b, h, t], kept).max() if n < D else True
        pruned = np.delete(w[b, h, t], kept)
        want_mu = pruned.mean() if n < D else 0.0
        assert abs(sel["mu"][b, h, t] - want_mu) <= 1e-6 * max(abs(want_mu), 1e-30)
    assert len(counts) > 1, "case too weak: every token kept the same number of channels"
    # the kept set of a token with count n is exactly the fixed-T oracle's set for T = n
    for n in counts:
        fixed = oracle.compress(k, lens, n, a)["mask"]
        same = sel["count"] == n
        assert np.array_equal(sel["mask"][same], fixed[same])


def test_top_p_limits_cap_and_monotonicity():
    rng = np.random.default_rng(7)
    D, S = 32, 50
    q_win, k, v, q = rand_case(rng, 1, 2, 2, 4, D, S)
    _, a = oracle.window_mean(q_win, 2)
    tiny = oracle.select_variant(k, [S], a, top_p=1e-6)
    assert (tiny["count"] == 1).all()                                   # the most salient channel alone
    assert np.array_equal(tiny["mask"], oracle.compress(k, [S], 1, a)["mask"])
    full = oracle.select_variant(k, [S], a, top_p=1.0)
    assert (full["count"] >= D - 2).all() and (full["count"] <= D).all()   # all the mass: (almost) every channel
    prev = np.zeros_like(full["count"])
    for p in (0.3, 0.6, 0.9, 0.99):
        cur = oracle.select_variant(k, [S], a, top_p=p)["count"]
        assert (cur >= prev).all()
        prev = cur
    capped = oracle.select_variant(k, [S], a, top_p=0.99, cap=5)
    free = oracle.select_variant(k, [S], a, top_p=0.99)
    assert np.array_equal(capped["count"], np.minimum(free["count"], 5))
    assert np.array_equal(capped["mask"][free["count"] <= 5], free["mask"][free["count"] <= 5])


def test_top_p_hand_row():
    # saliencies (a = 1): 8 4 2 1 1 0 0 0 -> total 16; 50 % -> {0}; 75 % -> {0,1}; 90 % -> 14.4 -> {0,1,2,3} (15)
    k = np.array([8, 4, 2, 1, 1, 0, 0, 0], np.float32).reshape(1, 1, 1, 8)
    a = np.ones((1, 1, 8), np.float32)
    for p, want in ((0.5, [0]), (0.75, [0, 1]), (0.9, [0, 1, 2, 3]), (0.94, [0, 1, 2, 3, 4]), (0.8, [0, 1, 2])):
        sel = oracle.select_variant(k, [1], a, top_p=p)
        assert bits_of(sel["mask"][0, 0, 0], 8) == want, p
    sel = oracle.select_variant(k, [1], a, top_p=0.9)
    assert sel["mu"][0, 0, 0] == np.float32(0.25)                       # pruned: 1 0 0 0


# ---------------------------------------------------------------- SparK-g
def test_groups_hand_row_and_counts():
    # ranks by saliency: channels 7 6 5 4 3 2 1 0; four groups of two ranks with ratios 0, .5, .5, 1
    k = np.arange(1, 9, dtype=np.float32).reshape(1, 1, 1, 8)
    a = np.ones((1, 1, 8), np.float32)
    sel = oracle.select_variant(k, [1], a, group_prune=[0.0, 0.5, 0.5, 1.0])
    assert bits_of(sel["mask"][0, 0, 0], 8) == [3, 5, 6, 7] and sel["count"][0, 0, 0] == 4
    assert sel["mu"][0, 0, 0] == np.float32((5 + 3 + 2 + 1) / 4)
    # D = 128: the paper's two ratio lists give 48 and 63 kept channels (overall ratios 0.625 and 0.508)
    rng = np.random.default_rng(3)
    q_win, k, v, q = rand_case(rng, 1, 1, 1, 4, 128, 6)
    _, a = oracle.window_mean(q_win, 1)
    g4 = oracle.select_variant(k, [6], a, group_prune=[0.25, 0.5, 0.75, 1.0])
    g5 = oracle.select_variant(k, [6], a, group_prune=[0.1, 0.3, 0.5, 0.7, 0.9])
    assert (g4["count"] == 24 + 16 + 8 + 0).all() and (g5["count"] == 23 + 18 + 13 + 7 + 2).all()


@pytest.mark.parametrize("D,ratios", [(128, [0.25, 0.5, 0.75, 1.0]), (128, [0.1, 0.3, 0.5, 0.7, 0.9]),
                                      (20, [0.0, 0.34, 1.0]), (16, [0.5])])
def test_groups_keep_the_head_of_every_rank_segment(D, ratios):
    rng = np.random.default_rng(11 + D + len(ratios))
    S = 30
    q_win, k, v, q = rand_case(rng, 1, 2, 2, 4, D, S)
    _, a = oracle.window_mean(q_win, 2)
    sel = oracle.select_variant(k, [S], a, group_prune=ratios)
    w = saliency(a, k)
    g = len(ratios)
    for h, t in itertools.product(range(2), range(S)):
        order = sorted(range(D), key=lambda j: (-float(w[0, h, t, j]), j))
        want, start = [], 0
        for i in range(g):
            size = D // g + (1 if i < D % g else 0)
            kp = int(math.floor((1.0 - float(np.float32(ratios[i]))) * size + 1e-9))
            want += order[start:start + kp]
            start += size
        assert bits_of(sel["mask"][0, h, t], D) == sorted(want)
    if g == 1:                                                     # one group = the fixed-ratio rule
        T = int(math.floor((1 - ratios[0]) * D + 1e-9))
        assert np.array_equal(sel["mask"], oracle.compress(k, [S], T, a)["mask"])
        assert np.array_equal(sel["mu"], oracle.compress(k, [S], T, a)["mu"])


# ---------------------------------------------------------------- the counter-based generator
def test_generator_matches_the_published_splitmix64_vectors():
    """seed * golden + counter 0 is the state after `seed` increments of a splitmix64 stream started at 0; its
    first outputs are 0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F."""
    for seed, z in ((1, 0xE220A8397B1DCDAF), (2, 0x6E789E6AA1B965F4), (3, 0x06C45D188009454F)):
        u1, u2 = oracle.draw_uniforms(seed, 0, 0, 0)
        assert u1 == ((z >> 40) + 0.5) / 2 ** 24 and u2 == (((z >> 16) & 0xFFFFFF) + 0.5) / 2 ** 24


def test_generator_is_keyed_uniform_and_inside_the_open_interval():
    n = 60000
    us = np.array([oracle.draw_uniforms(9, 3, t, j) for t in range(n // 100) for j in range(100)])
    assert us.min() > 0.0 and us.max() < 1.0
    assert abs(us.mean(axis=0) - 0.5).max() < 0.005 and abs(us.var(axis=0) - 1 / 12).max() < 0.002
    assert abs(np.corrcoef(us[:, 0], us[:, 1])[0, 1]) < 0.02
    hist = np.histogram(us[:, 0], bins=20, range=(0, 1))[0]
    assert abs(hist / n - 0.05).max() < 0.005
    assert oracle.draw_uniforms(9, 3, 5, 6) == oracle.draw_uniforms(9, 3, 5, 6)
    keys = {oracle.draw_uniforms(s, u, t, j) for s in (1, 2) for u in (0, 1) for t in (0, 1, 256) for j in (0, 1, 127)}
    assert len(keys) == 2 * 2 * 3 * 3                                 # every part of the key matters


# ---------------------------------------------------------------- sampled recovery
def recovery_case(seed=21, D=64, S=400, T=24, Hkv=2, G=2):
    rng = np.random.default_rng(seed)
    q_win, k, v, q = rand_case(rng, 1, Hkv * G, Hkv, 4, D, S)
    lens = [S]
    _, a = oracle.window_mean(q_win, Hkv)
    c = oracle.compress(k, lens, T, a, want_stats=True, want_saliency=True)
    return q_win, k, v, q, lens, a, c


def test_statistics_are_the_all_channel_mean_and_population_deviation():
    q_win, k, v, q, lens, a, c = recovery_case()
    w = c["saliency"].astype(np.float64)
    assert np.allclose(c["mu_all"], w.mean(axis=-1), rtol=1e-6)
    assert np.allclose(c["sigma_all"], w.std(axis=-1), rtol=1e-6)      # numpy's default is the population form


@pytest.mark.parametrize("mode", [1, 2])
def test_sampled_decode_is_textbook_attention_over_the_recovered_keys(mode):
    """Independent restatement: K~ = K where kept, recovered / a elsewhere; then dense attention."""
    q_win, k, v, q, lens, a, c = recovery_case()
    out, lse, rec = oracle.decode_attn_sampled(q, k, v, lens, c["mask"], c["mu_all"], c["sigma_all"], a,
                                               mode=mode, seed=5, want_recovered=True)
    D = k.shape[-1]
    bits = ((c["mask"][..., None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(k.shape).astype(bool)
    assert (rec[bits] == 0).all() and (rec[~bits] != 0).any()
    kt = np.where(bits, k.astype(np.float64), rec / a[:, :, None, :].astype(np.float64))
    G = q.shape[1] // k.shape[1]
    for i in range(q.shape[1]):
        ref, ref_lse = dense_attention(q[0, i], kt[0, i // G], v[0, i // G])
        assert np.allclose(out[0, i], ref, rtol=0, atol=3e-7) and abs(lse[0, i] - ref_lse) < 2e-6 + 1e-6 * abs(ref_lse)
    out2, _ = oracle.decode_attn_sampled(q, k, v, lens, c["mask"], c["mu_all"], c["sigma_all"], a, mode=mode, seed=5)
    out3, _ = oracle.decode_attn_sampled(q, k, v, lens, c["mask"], c["mu_all"], c["sigma_all"], a, mode=mode, seed=6)
    assert np.array_equal(out, out2) and not np.array_equal(out, out3)  # fixed per seed, different across seeds


def test_exponential_draws_have_the_distributions_moments_and_tail():
    q_win, k, v, q, lens, a, c = recovery_case(S=600)
    _, _, rec = oracle.decode_attn_sampled(q, k, v, lens, c["mask"], c["mu_all"], None, a, mode=2, seed=77,
                                           want_recovered=True)
    bits = ((c["mask"][..., None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(k.shape).astype(bool)
    x = (rec / c["mu_all"][..., None].astype(np.float64))[~bits]         # ~ Exp(1)
    assert x.size > 40000 and x.min() > 0
    se = 1 / math.sqrt(x.size)
    assert abs(x.mean() - 1.0) < 5 * se and abs(x.var() - 1.0) < 15 * se
    assert abs((x > 1).mean() - math.exp(-1)) < 5 * 0.5 * se and abs((x > 3).mean() - math.exp(-3)) < 5 * 0.25 * se


def test_gaussian_draws_have_the_distributions_moments_and_mass():
    q_win, k, v, q, lens, a, c = recovery_case(S=600)
    _, _, rec = oracle.decode_attn_sampled(q, k, v, lens, c["mask"], c["mu_all"], c["sigma_all"], a, mode=1, seed=78,
                                           want_recovered=True)
    bits = ((c["mask"][..., None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(k.shape).astype(bool)
    z = ((rec - c["mu_all"][..., None]) / c["sigma_all"][..., None].astype(np.float64))[~bits]   # ~ N(0, 1)
    se = 1 / math.sqrt(z.size)
    assert abs(z.mean()) < 5 * se and abs(z.var() - 1.0) < 10 * se
    assert abs((np.abs(z) < 1).mean() - 0.682689) < 5 * 0.5 * se and abs((z > 2).mean() - 0.0227501) < 5 * 0.15 * se
    assert (z < 0).any()                                                 # draws are not clamped


def test_gaussian_without_spread_is_the_degenerate_rule_on_the_all_channel_mean():
    q_win, k, v, q, lens, a, c = recovery_case(S=50)
    zero = np.zeros_like(c["sigma_all"])
    out, lse = oracle.decode_attn_sampled(q, k, v, lens, c["mask"], c["mu_all"], zero, a, mode=1, seed=1)
    ref, ref_lse = oracle.decode_attn(q, k, v, lens, c["mask"], c["mu_all"], a)       # mu := all-channel mean
    assert np.allclose(out, ref, rtol=0, atol=1e-7) and np.allclose(lse, ref_lse, rtol=0, atol=1e-6)


@pytest.mark.parametrize("mode", [1, 2])
def test_nothing_pruned_means_dense_attention_whatever_the_distribution(mode):
    q_win, k, v, q, lens, a, c = recovery_case(S=30, T=64, D=64)
    out, lse = oracle.decode_attn_sampled(q, k, v, lens, c["mask"], c["mu_all"], c["sigma_all"], a, mode=mode, seed=3)
    G = q.shape[1] // k.shape[1]
    for i in range(q.shape[1]):
        ref, _ = dense_attention(q[0, i], k[0, i // G], v[0, i // G])
        assert np.allclose(out[0, i], ref, rtol=0, atol=3e-7)
