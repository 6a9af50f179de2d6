"""Pins for the CPU oracle: checks against what the paper and the mathematics fix.

Nothing here re-types the oracle's own loops: every expected value is a closed
form, a brute-force enumeration, a textbook routine written independently in
NumPy, or the hand-worked fixture under tests/golden/.
"""
import itertools
import json
import math
import os

import numpy as np
import pytest

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def dense_attention(q, K, V, scale=None):
    """Textbook softmax(q K^T / sqrt(D)) V for one head, float64 (Sec. Preliminaries)."""
    q, K, V = np.asarray(q, np.float64), np.asarray(K, np.float64), np.asarray(V, np.float64)
    s = K @ q * (scale if scale else 1.0 / math.sqrt(K.shape[1]))
    e = np.exp(s - s.max())
    return (e / e.sum()) @ V, s.max() + math.log(e.sum())


def rand_case(rng, B=1, Hq=1, Hkv=1, W=4, D=8, S=5, scale=1.0):
    q_win = rng.standard_normal((B, Hq, W, D)).astype(np.float32) * scale
    k = rng.standard_normal((B, Hkv, S, D)).astype(np.float32) * scale
    v = rng.standard_normal((B, Hkv, S, D)).astype(np.float32)
    q = rng.standard_normal((B, Hq, D)).astype(np.float32)
    return q_win, k, v, q


def bits_of(mask_row, D):
    return [j for j in range(D) if (int(mask_row[j // 32]) >> (j % 32)) & 1]


# ---------------------------------------------------------------- hand-worked fixture
def test_hand_example_whole_chain():
    g = json.load(open(os.path.join(GOLD, "hand_example.json")))
    D, T = g["D"], g["T"]
    q_win = np.array(g["q_win"], np.float32).reshape(1, 1, g["W"], D)
    k = np.array(g["k"], np.float32).reshape(1, 1, 3, D)
    v = np.zeros((1, 1, 3, D), np.float32)
    v[0, 0, :, :2] = np.array(g["v"], np.float32)
    q = np.array(g["q"], np.float32).reshape(1, 1, D)
    qbar, a = oracle.window_mean(q_win, 1)
    assert np.array_equal(qbar[0, 0], np.array(g["qbar"], np.float32))
    assert np.array_equal(a[0, 0], np.abs(np.array(g["qbar"], np.float32)))
    c = oracle.compress(k, [3], T, a, want_idx=True, want_saliency=True)
    assert np.array_equal(c["saliency"][0, 0], np.array(g["saliency"], np.float32))
    assert [int(x) for x in c["mask"][0, 0, :, 0]] == g["mask"]
    assert np.array_equal(c["mu"][0, 0], np.array(g["mu"], np.float32))
    for path in (0, 1):
        out, lse, sc = oracle.decode_attn(q, k, v, [3], c["mask"], c["mu"], a, path=path, want_scores=True)
        assert np.allclose(sc[0, 0], g["scores"], rtol=0, atol=5e-8)
        assert np.allclose(out[0, 0, :2], g["out"], rtol=0, atol=1e-7)   # float32 output
    # the recovered key rows of the fixture reproduce its scores (checks the fixture itself)
    kr = np.array(g["k_recovered"])
    assert np.allclose(kr @ np.array(g["q"]) / math.sqrt(D), g["scores"], atol=5e-8)


# ---------------------------------------------------------------- window mean
def test_window_mean_pools_group_queries_exactly():
    rng = np.random.default_rng(1)
    B, Hq, Hkv, W, D = 2, 6, 2, 8, 16
    # small integers / 8: sums are exact in any order, so the mean has one right answer
    q_win = (rng.integers(-40, 41, (B, Hq, W, D)) / 8.0).astype(np.float32)
    qbar, a = oracle.window_mean(q_win, Hkv, eps=0.3)
    G = Hq // Hkv
    want = q_win.astype(np.float64).reshape(B, Hkv, G, W, D).sum(axis=(2, 3)) / (G * W)
    assert np.array_equal(qbar, want.astype(np.float32))
    assert np.array_equal(a, np.maximum(np.abs(want.astype(np.float32)), np.float32(0.3)))
    assert (a >= np.float32(0.3)).all() and (np.abs(qbar) < 0.3).any()   # the floor is exercised


def test_window_mean_bf16_input_is_widened_exactly():
    torch = pytest.importorskip("torch")
    x = torch.tensor([[[[1.0, -2.5, 0.15625, 3.0]] * 2]], dtype=torch.bfloat16)   # [1,1,2,4]
    qbar, a = oracle.window_mean(x, 1)
    assert np.array_equal(qbar[0, 0], np.array([1.0, -2.5, 0.15625, 3.0], np.float32))


# ---------------------------------------------------------------- selection (Eq. cal)
@pytest.mark.parametrize("D", [8, 10])
def test_top_t_equals_brute_force_argmax_of_linear_objective(D):
    rng = np.random.default_rng(D)
    q_win, k, v, q = rand_case(rng, D=D, S=6)
    _, a = oracle.window_mean(q_win, 1)
    w = (a[0, 0][None, :] * np.abs(k[0, 0])).astype(np.float64)       # saliency, Sec. Problem Formulation
    for T in range(1, D + 1):
        c = oracle.compress(k, [6], T, a, want_idx=True)
        for t in range(6):
            best = max(itertools.combinations(range(D), T), key=lambda s: sum(w[t, j] for j in s))
            assert bits_of(c["mask"][0, 0, t], D) == list(best)
            assert list(c["kept_idx"][0, 0, t]) == list(best)


def test_ties_keep_lower_channel():
    D, T = 8, 3
    a = np.ones((1, 1, D), np.float32)
    k = np.array([[[[2, 1, 1, 1, 1, 0.5, 2, 1]]]], np.float32)        # w: two 2s, five 1s
    c = oracle.compress(k, [1], T, a)
    assert bits_of(c["mask"][0, 0, 0], D) == [0, 1, 6]                 # 2s, then the FIRST of the 1s
    k2 = np.ones((1, 1, 1, D), np.float32)
    c2 = oracle.compress(k2, [1], 5, a)
    assert bits_of(c2["mask"][0, 0, 0], D) == [0, 1, 2, 3, 4]


def test_popcount_separation_and_mu_on_random_heads():
    rng = np.random.default_rng(3)
    B, Hq, Hkv, W, D, S = 2, 4, 2, 8, 128, 40
    q_win, k, v, q = rand_case(rng, B, Hq, Hkv, W, D, S, scale=2.0)
    _, a = oracle.window_mean(q_win, Hkv)
    for T in (1, 25, 64, 127, 128):
        c = oracle.compress(k, [S, S - 7], T, a, want_idx=True, want_saliency=True)
        for b, h, t in itertools.product(range(B), range(Hkv), range(S)):
            kept = bits_of(c["mask"][b, h, t], D)
            if t >= [S, S - 7][b]:
                assert kept == [] and c["mu"][b, h, t] == 0
                continue
            assert len(kept) == T                                       # sum_j z_j = T
            assert kept == sorted(kept) == list(c["kept_idx"][b, h, t])
            w = a[b, h] * np.abs(k[b, h, t])                            # fp32 product
            assert np.array_equal(w, c["saliency"][b, h, t])
            pruned = [j for j in range(D) if j not in kept]
            if pruned:
                assert w[kept].min() >= w[pruned].max()
                assert np.isclose(c["mu"][b, h, t], w[pruned].astype(np.float64).mean(), rtol=1e-6)
            else:
                assert c["mu"][b, h, t] == 0


def test_all_channel_statistics_are_population_moments():
    rng = np.random.default_rng(5)
    q_win, k, v, q = rand_case(rng, D=32, S=9)
    _, a = oracle.window_mean(q_win, 1)
    c = oracle.compress(k, [9], 16, a, want_saliency=True, want_stats=True)
    w = c["saliency"][0, 0].astype(np.float64)
    assert np.allclose(c["mu_all"][0, 0], w.mean(axis=1), rtol=1e-6)
    assert np.allclose(c["sigma_all"][0, 0], w.std(axis=1), rtol=1e-6)   # 1/|C| normalisation


def test_strided_token_major_layout_matches_head_major():
    rng = np.random.default_rng(6)
    q_win, k, v, q = rand_case(rng, B=2, Hq=4, Hkv=2, D=16, S=7)
    _, a = oracle.window_mean(q_win, 2)
    c1 = oracle.compress(k, [7, 5], 6, a)
    k_tm = np.ascontiguousarray(k.transpose(0, 2, 1, 3)).transpose(0, 2, 1, 3)   # [B,S,H,D] storage
    v_tm = np.ascontiguousarray(v.transpose(0, 2, 1, 3)).transpose(0, 2, 1, 3)
    assert k_tm.strides != k.strides
    c2 = oracle.compress(k_tm, [7, 5], 6, a)
    assert np.array_equal(c1["mask"], c2["mask"]) and np.array_equal(c1["mu"], c2["mu"])
    o1, l1 = oracle.decode_attn(q, k, v, [7, 5], c1["mask"], c1["mu"], a)
    o2, l2 = oracle.decode_attn(q, k_tm, v_tm, [7, 5], c1["mask"], c1["mu"], a)
    assert np.array_equal(o1, o2) and np.array_equal(l1, l2)


# ---------------------------------------------------------------- recovery + attention
def test_ratio_zero_is_dense_attention_with_gqa_mapping():
    rng = np.random.default_rng(7)
    B, Hq, Hkv, W, D, S = 2, 6, 2, 4, 32, 50
    q_win, k, v, q = rand_case(rng, B, Hq, Hkv, W, D, S)
    lens = [S, 31]
    _, a = oracle.window_mean(q_win, Hkv)
    c = oracle.compress(k, lens, D, a)
    assert (c["mu"] == 0).all()
    for b in range(B):
        assert (c["mask"][b, :, :lens[b]] == 0xFFFFFFFF).all()
    for path in (0, 1):
        out, lse = oracle.decode_attn(q, k, v, lens, c["mask"], c["mu"], a, path=path)
        for b, i in itertools.product(range(B), range(Hq)):
            h = i // (Hq // Hkv)
            want, want_lse = dense_attention(q[b, i], k[b, h, :lens[b]], v[b, h, :lens[b]])
            assert np.allclose(out[b, i], want, rtol=0, atol=1e-6)
            assert np.isclose(lse[b, i], want_lse, rtol=0, atol=1e-5)


def test_zero_fill_mode_equals_dense_attention_on_masked_keys():
    rng = np.random.default_rng(8)
    q_win, k, v, q = rand_case(rng, B=1, Hq=2, Hkv=1, W=4, D=64, S=33)
    _, a = oracle.window_mean(q_win, 1)
    c = oracle.compress(k, [33], 20, a)
    dense_mask = np.array([[(int(c["mask"][0, 0, t, j // 32]) >> (j % 32)) & 1 for j in range(64)]
                           for t in range(33)], np.float64)
    out, lse = oracle.decode_attn(q, k, v, [33], c["mask"], np.zeros_like(c["mu"]), a)
    for i in range(2):
        want, _ = dense_attention(q[0, i], k[0, 0] * dense_mask, v[0, 0])
        assert np.allclose(out[0, i], want, atol=1e-6)


def test_mass_preservation_of_recovered_entries():
    """sum over pruned j of |q-bar_j| * k~_j equals the pruned saliency mass (D-T) mu."""
    rng = np.random.default_rng(9)
    D, S, T = 32, 12, 10
    q_win, k, v, _ = rand_case(rng, W=6, D=D, S=S)
    qbar, a = oracle.window_mean(q_win, 1)
    c = oracle.compress(k, [S], T, a, want_saliency=True)
    # probe query = a itself, scale 1: scores are sum_kept a_j k_j + sum_pruned a_j (mu/a_j)
    _, _, sc = oracle.decode_attn(a.reshape(1, 1, D), k, v, [S], c["mask"], c["mu"], a,
                                  scale=1.0, want_scores=True)
    for t in range(S):
        kept = bits_of(c["mask"][0, 0, t], D)
        pruned = [j for j in range(D) if j not in kept]
        kept_part = float((a[0, 0, kept].astype(np.float64) * k[0, 0, t, kept]).sum())
        pruned_mass = float(c["saliency"][0, 0, t, pruned].astype(np.float64).sum())
        assert np.isclose(sc[0, 0, t] - kept_part, pruned_mass, rtol=1e-6)
        assert np.isclose(pruned_mass, (D - T) * float(c["mu"][0, 0, t]), rtol=1e-6)


@pytest.mark.parametrize("T", [1, 5, 16, 31])
def test_positive_case_collapses_to_dense_attention_for_every_ratio(T):
    """q-bar > 0, K >= 0, one head, decode query = q-bar: q.K~ = sum_j w_j = q-bar.K for every T."""
    rng = np.random.default_rng(10 + T)
    D, S, W = 32, 20, 4
    base = (rng.integers(1, 64, D) / 16.0).astype(np.float32)            # exactly representable
    q_win = np.broadcast_to(base, (1, 1, W, D)).copy()                    # mean == base exactly
    k = (rng.integers(0, 256, (1, 1, S, D)) / 32.0).astype(np.float32)
    v = rng.standard_normal((1, 1, S, D)).astype(np.float32)
    qbar, a = oracle.window_mean(q_win, 1)
    assert np.array_equal(qbar[0, 0], base)
    c = oracle.compress(k, [S], T, a)
    want, want_lse = dense_attention(base, k[0, 0], v[0, 0])
    for path in (0, 1):
        out, lse = oracle.decode_attn(base.reshape(1, 1, D), k, v, [S], c["mask"], c["mu"], a, path=path)
        assert np.allclose(out[0, 0], want, atol=2e-6)
        assert np.isclose(lse[0, 0], want_lse, atol=1e-5)


def test_two_score_paths_agree_and_splits_merge_by_lse():
    rng = np.random.default_rng(11)
    B, Hq, Hkv, W, D, S = 1, 4, 2, 8, 128, 200
    q_win, k, v, q = rand_case(rng, B, Hq, Hkv, W, D, S, scale=1.5)
    _, a = oracle.window_mean(q_win, Hkv)
    c = oracle.compress(k, [S], 40, a)
    o0, l0, s0 = oracle.decode_attn(q, k, v, [S], c["mask"], c["mu"], a, path=0, want_scores=True)
    o1, l1, s1 = oracle.decode_attn(q, k, v, [S], c["mask"], c["mu"], a, path=1, want_scores=True)
    assert np.allclose(s0, s1, rtol=1e-12, atol=1e-12)
    assert np.allclose(o0, o1, atol=1e-7)
    # split the tokens 77 | 123, attend separately, merge with log-sum-exp weights
    cut = 77
    parts = []
    for lo, hi in ((0, cut), (cut, S)):
        o, l = oracle.decode_attn(q, k[:, :, lo:hi], v[:, :, lo:hi], [hi - lo],
                                  np.ascontiguousarray(c["mask"][:, :, lo:hi]),
                                  np.ascontiguousarray(c["mu"][:, :, lo:hi]), a)
        parts.append((o.astype(np.float64), l.astype(np.float64)))
    m = np.maximum(parts[0][1], parts[1][1])
    w0, w1 = np.exp(parts[0][1] - m), np.exp(parts[1][1] - m)
    merged = (parts[0][0] * w0[..., None] + parts[1][0] * w1[..., None]) / (w0 + w1)[..., None]
    assert np.allclose(merged, o0, atol=2e-6)
    assert np.allclose(m + np.log(w0 + w1), l0, atol=1e-5)


def test_scale_argument_and_default():
    rng = np.random.default_rng(12)
    q_win, k, v, q = rand_case(rng, D=16, S=6)
    _, a = oracle.window_mean(q_win, 1)
    c = oracle.compress(k, [6], 16, a)
    o_def, _ = oracle.decode_attn(q, k, v, [6], c["mask"], c["mu"], a)
    o_exp, _ = oracle.decode_attn(q, k, v, [6], c["mask"], c["mu"], a, scale=0.25)   # 1/sqrt(16)
    assert np.array_equal(o_def, o_exp)
    o_one, _ = oracle.decode_attn(q, k, v, [6], c["mask"], c["mu"], a, scale=1.0)
    want, _ = dense_attention(q[0, 0], k[0, 0], v[0, 0], scale=1.0)
    assert np.allclose(o_one[0, 0], want, atol=1e-6)


def test_empty_sequence_gives_zero_output():
    rng = np.random.default_rng(13)
    q_win, k, v, q = rand_case(rng, B=2, D=16, S=4)
    _, a = oracle.window_mean(q_win, 1)
    c = oracle.compress(k, [0, 4], 8, a)
    out, lse = oracle.decode_attn(q, k, v, [0, 4], c["mask"], c["mu"], a)
    assert (out[0] == 0).all() and np.isneginf(lse[0]).all() and np.isfinite(out[1]).all()


def test_memory_accounting_of_kept_values():
    """Kept key values are T/D of the dense keys; at ratio 0.8 K+V values are 60 % (a 40 % cut)."""
    D = 128

    def keep_count(d, lam):                                            # T = floor((1 - lambda) D)
        return int(math.floor((1.0 - lam) * d + 1e-9))
    assert keep_count(D, 0.5) == 64 and keep_count(D, 0.8) == 25       # floor((1-lambda) D)
    assert keep_count(D, 0.3) == 89 and keep_count(D, 0.7) == 38 and keep_count(D, 0.0) == 128
    lam = 0.8
    assert math.isclose(((1 - lam) * D + D) / (2 * D), 0.6)


# ---------------------------------------------------------------- eviction (own invariants only)
def test_eviction_identity_budget_and_window_always_kept():
    rng = np.random.default_rng(14)
    B, Hq, Hkv, W, D, S = 1, 4, 2, 4, 16, 40
    q_win, k, v, q = rand_case(rng, B, Hq, Hkv, W, D, S)
    kept, n = oracle.evict(q_win, k, [S], budget=64, pool=7)
    assert n[0] == S and (kept[0, :, :S] == np.arange(S)).all() and (kept[0, :, S:] == -1).all()
    kept, n = oracle.evict(q_win, k, [S], budget=12, pool=7)
    assert n[0] == 12
    for h in range(Hkv):
        row = list(kept[0, h])
        assert row == sorted(row) and len(set(row)) == 12
        assert row[-W:] == list(range(S - W, S))


def test_eviction_pool_one_is_plain_top_k_of_causal_window_votes():
    rng = np.random.default_rng(15)
    B, Hq, Hkv, W, D, S, budget = 1, 2, 1, 3, 8, 17, 9
    q_win, k, v, q = rand_case(rng, B, Hq, Hkv, W, D, S)
    kept, n, vote, pooled = oracle.evict(q_win, k, [S], budget=budget, pool=1, want_votes=True)
    P = S - W
    want_vote = np.zeros(P)
    for g in range(Hq):
        for w in range(W):
            last = P + w
            s = k[0, 0, :last + 1].astype(np.float64) @ q_win[0, g, w].astype(np.float64) / math.sqrt(D)
            e = np.exp(s - s.max())
            want_vote += (e / e.sum())[:P]
    assert np.allclose(vote[0, 0, :P], want_vote, rtol=1e-12)
    assert np.array_equal(pooled[0, 0, :P], vote[0, 0, :P])
    top = sorted(sorted(range(P), key=lambda t: (-want_vote[t], t))[:budget - W])
    assert list(kept[0, 0]) == top + list(range(P, S))
    # pooling: each pooled value is the max of its clamped 5-neighbourhood
    _, _, vote5, pooled5 = oracle.evict(q_win, k, [S], budget=budget, pool=5, want_votes=True)
    for t in range(P):
        assert pooled5[0, 0, t] == vote5[0, 0, max(0, t - 2):min(P, t + 3)].max()


def independent_votes(q_win, k, S, W, D):
    """Causal observation-window votes of one KV head, written directly with NumPy (group summed)."""
    P = S - W
    vote = np.zeros(P)
    for g in range(q_win.shape[0]):
        for w in range(W):
            last = P + w
            s = k[:last + 1].astype(np.float64) @ q_win[g, w].astype(np.float64) / math.sqrt(D)
            e = np.exp(s - s.max())
            vote += (e / e.sum())[:P]
    return vote


@pytest.mark.parametrize("pool,S,W,budget,seed", [(7, 61, 4, 20, 16), (7, 200, 8, 40, 17), (3, 33, 2, 9, 18),
                                                  (7, 12, 3, 6, 19)])
def test_eviction_kept_set_is_top_k_of_the_POOLED_votes(pool, S, W, budget, seed):
    """End to end at pool > 1: independent votes -> independent clamped max-pool -> top-(budget - W) with ties
    to the lower position -> + window.  An oracle that ranked the raw votes would fail here."""
    rng = np.random.default_rng(seed)
    B, Hq, Hkv, D = 1, 4, 2, 16
    q_win, k, v, q = rand_case(rng, B, Hq, Hkv, W, D, S)
    kept, n = oracle.evict(q_win, k, [S], budget=budget, pool=pool)
    assert n[0] == budget
    P, half, G = S - W, (pool - 1) // 2, Hq // Hkv
    differs_from_raw_ranking = False
    for h in range(Hkv):
        vote = independent_votes(q_win[0, h * G:(h + 1) * G], k[0, h], S, W, D)
        pooled = np.array([vote[max(0, t - half):min(P, t + half + 1)].max() for t in range(P)])
        order = sorted(range(P), key=lambda t: (-pooled[t], t))
        want = sorted(order[:budget - W]) + list(range(P, S))
        assert list(kept[0, h]) == want
        # max-pooling makes equal pooled values routine: the boundary of this case must cut through a tie
        # group somewhere in the sweep, which exercises the lower-position rule
        raw = sorted(sorted(range(P), key=lambda t: (-vote[t], t))[:budget - W]) + list(range(P, S))
        differs_from_raw_ranking |= (raw != want)
    assert differs_from_raw_ranking, "case too weak: pooled and raw rankings keep the same tokens"


def test_eviction_boundary_inside_a_run_of_equal_pooled_values():
    """One dominant key makes `pool` neighbours share the same pooled value; a budget that ends inside that
    run must keep the LOWER positions of the run."""
    B, Hq, Hkv, W, D, S, pool = 1, 1, 1, 2, 8, 30, 7
    rng = np.random.default_rng(20)
    q_win = rng.standard_normal((B, Hq, W, D)).astype(np.float32)
    k = (0.01 * rng.standard_normal((B, Hkv, S, D))).astype(np.float32)
    k[0, 0, 15] = 4.0 * q_win[0, 0].mean(axis=0)                       # token 15 takes nearly all attention
    P = S - W
    vote = independent_votes(q_win[0], k[0, 0], S, W, D)
    pooled = np.array([vote[max(0, t - 3):min(P, t + 4)].max() for t in range(P)])
    run = [t for t in range(P) if pooled[t] == pooled[15]]
    assert run == list(range(12, 19))                                  # the 7-neighbourhood of the dominant token
    for extra in range(1, 7):                                          # budget ends inside the run
        kept, n = oracle.evict(q_win, k, [S], budget=W + extra, pool=pool)
        assert list(kept[0, 0]) == run[:extra] + list(range(P, S))


def test_eviction_votes_in_closed_form_uniform_and_one_hot_attention():
    """Two cases whose votes are known without computing a softmax.  (a) All keys equal: every causal softmax
    is uniform, so vote[t] = G * sum_w 1 / (S - W + w + 1) for every prefix token, all pooled values tie and the
    lower positions are kept.  (b) Keys that are huge multiples of orthogonal directions, each window query
    aligned with one prefix key: attention is one-hot, so vote[t] = number of (head, window row) pairs that
    point at t, pooled[t] = the largest count within three positions, and the kept set follows by hand."""
    B, Hq, Hkv, W, D, S = 1, 2, 1, 3, 8, 20
    P = S - W
    rng = np.random.default_rng(21)
    q_win = rng.standard_normal((B, Hq, W, D)).astype(np.float32)
    k = np.broadcast_to(rng.standard_normal((1, 1, 1, D)).astype(np.float32), (B, Hkv, S, D)).copy()
    kept, n, vote, pooled = oracle.evict(q_win, k, [S], budget=9, pool=7, want_votes=True)
    uniform = Hq * sum(1.0 / (P + w + 1) for w in range(W))
    assert np.allclose(vote[0, 0, :P], uniform, rtol=1e-12) and np.allclose(pooled[0, 0, :P], uniform, rtol=1e-12)
    assert list(kept[0, 0]) == list(range(9 - W)) + list(range(P, S))
    # (b) one-hot attention: window query (g, w) points at prefix token target[g][w]
    target = [[2, 2, 11], [2, 11, 15]]                                # counts: token 2 -> 3, token 11 -> 2, token 15 -> 1
    k = np.zeros((B, Hkv, S, D), dtype=np.float32)
    q_win = np.zeros((B, Hq, W, D), dtype=np.float32)
    for j, tkn in enumerate((2, 11, 15)):
        k[0, 0, tkn, j] = 1.0
    for g in range(Hq):
        for w in range(W):
            q_win[0, g, w, (2, 11, 15).index(target[g][w])] = 400.0   # logit 400 / sqrt(8) against 0: one-hot in double
    kept, n, vote, pooled = oracle.evict(q_win, k, [S], budget=W + 9, pool=7, want_votes=True)
    want_vote = np.zeros(P)
    want_vote[2], want_vote[11], want_vote[15] = 3.0, 2.0, 1.0
    assert np.allclose(vote[0, 0, :P], want_vote, atol=1e-12)
    want_pooled = np.zeros(P)
    want_pooled[0:6] = 3.0                                            # |t - 2| <= 3, clamped at 0
    want_pooled[8:15] = 2.0                                           # |t - 11| <= 3
    want_pooled[15:17] = 1.0                                          # |t - 15| <= 3 where 11 does not reach (t = 15, 16; P = 17)
    assert np.allclose(pooled[0, 0, :P], want_pooled, atol=1e-12)
    # nine prefix tokens: the six at 3.0, then the three lowest of the seven at 2.0
    assert list(kept[0, 0]) == [0, 1, 2, 3, 4, 5, 8, 9, 10] + list(range(P, S))


# ---------------------------------------------------------------- value-channel pruning (App. "Pruning Value Cache Channels")
def test_value_pruning_hand_rows_and_ties():
    # |v| = (3, 1, 0.5, 4, 1, 0, 2, 4): the three largest are channels 3 and 7 (4, tie -> lower first) and 0 (3)
    v = np.array([3, -1, 0.5, -4, 1, 0, -2, 4], np.float32).reshape(1, 1, 1, 8)
    assert bits_of(oracle.prune_values(v, [1], 3)[0, 0, 0], 8) == [0, 3, 7]
    assert bits_of(oracle.prune_values(v, [1], 2)[0, 0, 0], 8) == [3, 7]
    assert bits_of(oracle.prune_values(v, [1], 1)[0, 0, 0], 8) == [3]          # tie 3 vs 7: lower channel
    assert bits_of(oracle.prune_values(v, [1], 5)[0, 0, 0], 8) == [0, 1, 3, 6, 7]  # tie 1 vs 4 at |v| = 1
    assert bits_of(oracle.prune_values(v, [1], 8)[0, 0, 0], 8) == list(range(8))


@pytest.mark.parametrize("D,T_v", [(6, 2), (8, 5), (40, 13)])
def test_value_pruning_maximises_kept_magnitude(D, T_v):
    """The kept set is the T_v-subset with the largest sum of |v| (brute force for small D, separation beyond)."""
    rng = np.random.default_rng(11 + D)
    v = rng.standard_normal((2, 2, 4, D)).astype(np.float32)
    vm = oracle.prune_values(v, [4, 3], T_v)
    for b, h, t in itertools.product(range(2), range(2), range(4)):
        kept = bits_of(vm[b, h, t], D)
        if t >= [4, 3][b]:
            assert kept == []
            continue
        assert len(kept) == T_v
        mag = np.abs(v[b, h, t].astype(np.float64))
        if D <= 8:
            best = max(itertools.combinations(range(D), T_v), key=lambda c: mag[list(c)].sum())
            assert kept == list(best)
        else:
            assert mag[kept].min() >= np.delete(mag, kept).max()


def test_value_pruning_bf16_input_and_full_keep_is_identity():
    rng = np.random.default_rng(5)
    q_win, k, v, q = rand_case(rng, B=1, Hq=2, Hkv=1, W=3, D=32, S=9)
    v16 = (v.view(np.uint32) >> 16).astype(np.uint16)                  # truncated bf16 patterns
    vf = (v16.astype(np.uint32) << 16).view(np.float32)
    assert np.array_equal(oracle.prune_values(v16, [9], 7), oracle.prune_values(vf, [9], 7))
    _, a = oracle.window_mean(q_win, 1)
    c = oracle.compress(k, [9], 16, a)
    full = oracle.prune_values(v, [9], 32)
    assert (full == 0xFFFFFFFF).all()
    o0, l0 = oracle.decode_attn(q, k, v, [9], c["mask"], c["mu"], a)
    o1, l1 = oracle.decode_attn(q, k, v, [9], c["mask"], c["mu"], a, vmask=full)
    assert np.array_equal(o0, o1) and np.array_equal(l0, l1)


def test_value_pruned_decode_equals_dense_routine_on_zeroed_values():
    """Pruned value entries contribute nothing: same result as textbook attention over values zeroed by hand,
    with the scores untouched (the key side is unaffected by the value mask)."""
    rng = np.random.default_rng(8)
    q_win, k, v, q = rand_case(rng, B=2, Hq=4, Hkv=2, W=4, D=16, S=11)
    lens = [11, 6]
    _, a = oracle.window_mean(q_win, 2)
    c = oracle.compress(k, lens, 16, a)                                # keys dense -> scores are textbook scores
    vm = oracle.prune_values(v, lens, 5)
    out, lse = oracle.decode_attn(q, k, v, lens, c["mask"], c["mu"], a, vmask=vm)
    for b, i in itertools.product(range(2), range(4)):
        h, n = i // 2, lens[b]
        vz = np.zeros((n, 16))
        for t in range(n):
            order = sorted(range(16), key=lambda j: (-abs(float(v[b, h, t, j])), j))[:5]
            vz[t, order] = v[b, h, t, order]
        ref, ref_lse = dense_attention(q[b, i], k[b, h, :n], vz)
        assert np.allclose(out[b, i], ref, rtol=0, atol=2e-7)
        assert abs(lse[b, i] - ref_lse) < 1e-6
