"""Seeded random shapes through the whole path (compress -> unpack -> decode) against the oracle.

Each case draws batch, head counts, group size, window, kept-channel count, storage type, value pruning,
ragged lengths (with empty sequences and lengths that end on / one past a page boundary mixed in), and
whether the pages sit in a shared pool behind a permuted block table with spare pages or in a contiguous
cache.  The checks are check_case's: masks / kept values / value rows / qnorm bit-exact, mu, output and lse
within the tolerances of the parity bar, guard bands intact, two decode calls identical.
"""
import random

import pytest
import torch

from test_gpu_parity import built, check_case, check_eviction_case, make  # noqa: F401  (fixture + helpers)
from workloads.batches import permuted_block_table

pytestmark = pytest.mark.gpu


def draw_case(seed):
    rnd = random.Random(seed)
    dtype = rnd.choice(["bf16", "bf16", "f32"])
    G = rnd.choice([1, 2, 3, 4, 4, 5, 6, 7, 8])
    Hkv = rnd.choice([1, 2, 3, 4])
    Bn = rnd.choice([1, 2, 3, 5, 9, 20, 40])                # up to 160 units: more units than CTAs
    W = rnd.choice([1, 4, 8, 32])
    keep = rnd.choice([1, 2, 16, 25, 38, 64, 64, 89, 127, 128])
    keep_v = rnd.choice([0, 0, 0, 64, 25]) if keep < 128 or rnd.random() < 0.5 else 0
    cap = rnd.choice([40, 150, 600, 1500, 4000])
    while Bn * Hkv * G * cap > 1_500_000:               # keeps the oracle's share of a case under a second or two
        cap //= 2
    equal = rnd.random() < 0.25                         # equal lengths: the aligned / whole-units divisions
    lens = []
    for _ in range(Bn):
        kind = rnd.random()
        if kind < 0.12:
            n = 0
        elif kind < 0.3:
            n = 16 * rnd.randint(1, max(1, cap // 16)) + rnd.choice([0, 1, -1])     # around a page boundary
        else:
            n = rnd.randint(1, cap)
        lens.append(max(0, min(n, cap)))
    if equal:
        lens = [max(lens[0], 1)] * Bn
    paged = rnd.random() < 0.5
    return dict(dtype=dtype, G=G, Hkv=Hkv, Bn=Bn, W=W, keep=keep, keep_v=keep_v, lens=lens, paged=paged)


@pytest.mark.parametrize("seed", list(range(300, 396)))
def test_random_shape(seed):
    c = draw_case(seed)
    sigma = 1.0 if c["dtype"] == "bf16" else 0.5
    wl = make(c["dtype"], c["Bn"], c["G"] * c["Hkv"], c["Hkv"], c["lens"], c["W"], c["keep"], seed=seed, sigma=sigma)
    table, n_pool = None, None
    if c["paged"]:
        table, n_pages = permuted_block_table(c["Bn"], c["Hkv"], c["lens"], "cuda", seed=seed)
        n_pool = n_pages + 3                            # spare pages that nothing may touch
    check_case(wl, c["keep"], block_table=table, n_pool_pages=n_pool, keep_v=c["keep_v"])


def draw_eviction_case(seed):
    rnd = random.Random(seed)
    dtype = rnd.choice(["bf16", "bf16", "f32"])
    W = rnd.choice([4, 8, 16, 32, 64])
    G = rnd.choice([1, 2, 4, 4, 7, 8])                  # G * W above 256 leaves the tensor-core votes for the fallback
    Hkv = rnd.choice([1, 2, 3])
    budget = W + rnd.choice([1, 5, 30, 64, 200, 448])
    pool = rnd.choice([1, 3, 7, 7, 7])
    keep = rnd.choice([25, 64, 64, 100])
    Bn = rnd.choice([1, 2, 4])
    lens = []
    for _ in range(Bn):
        kind = rnd.random()
        if kind < 0.2:
            n = rnd.randint(max(1, W // 2), budget)                        # nothing to evict (at or under the budget)
        elif kind < 0.35:
            n = budget + rnd.randint(1, 3)                                 # evicts one to three tokens
        else:
            n = rnd.randint(budget + 1, budget + rnd.choice([50, 700, 3000]))
        lens.append(n)
    return dict(dtype=dtype, lens=lens, W=W, budget=budget, G=G, keep=keep, Hkv=Hkv, pool=pool)


@pytest.mark.parametrize("seed", list(range(500, 540)))
def test_random_eviction_shape(seed):
    c = draw_eviction_case(seed)
    check_eviction_case(c["dtype"], c["lens"], c["W"], c["budget"], c["G"], keep=c["keep"], Hkv=c["Hkv"],
                        pool=c["pool"], seed=seed)


@pytest.mark.parametrize("seed", list(range(700, 724)))
def test_random_append_mix(seed):
    """Prefill a random ragged batch, then grow it by a random mix of one-token appends and block appends (in a
    paged pool or a contiguous cache, with or without value pruning): the cache must equal the oracle's pruning of
    the full sequences with the prefill window statistics, and the decode output must match."""
    import numpy as np
    from test_gpu_parity import TOL, oracle_side
    from paper_2508_15212_b200.cache import SparkCache
    rnd = random.Random(seed)
    dtype = rnd.choice(["bf16", "bf16", "f32"])
    G, Hkv, Bn = rnd.choice([1, 2, 4, 7]), rnd.choice([1, 2, 3]), rnd.choice([1, 2, 4])
    keep = rnd.choice([25, 38, 64, 127, 128])
    keep_v = rnd.choice([0, 0, 64])
    lens0 = [rnd.choice([0, 1, 15, 16, 17, rnd.randint(1, 300)]) for _ in range(Bn)]
    n_app = rnd.randint(1, 70)
    lens1 = [l + n_app for l in lens0]
    S = max(lens1)
    full = make(dtype, Bn, G * Hkv, Hkv, lens1, 8, keep, seed=seed, sigma=1.0 if dtype == "bf16" else 0.5)
    table, n_pool = None, None
    if rnd.random() < 0.5:
        table, n_pages = permuted_block_table(Bn, Hkv, lens1, "cuda", seed=seed)
        n_pool = n_pages + 2
    cache = SparkCache(batch=Bn, n_q_heads=G * Hkv, n_kv_heads=Hkv, window=8, keep=keep, dtype=dtype, max_tokens=S,
                       block_table=table, n_pool_pages=n_pool, keep_v=keep_v, guard=True)
    lens0_t = torch.tensor(lens0, dtype=torch.int32, device="cuda")
    cache.compress(full.q_win, full.k, full.v, lens0_t)
    done = 0
    while done < n_app:
        n = min(n_app - done, rnd.choice([1, 1, 2, 5, 16, 33]))
        idx = (lens0_t.long().view(Bn, 1, 1, 1) + done + torch.arange(n, device="cuda").view(1, 1, n, 1))
        idx = idx.expand(Bn, Hkv, n, 128)
        k_blk, v_blk = full.k.gather(2, idx).contiguous(), full.v.gather(2, idx).contiguous()
        if n == 1 and rnd.random() < 0.7:
            cache.append(k_blk[:, :, 0].contiguous(), v_blk[:, :, 0].contiguous())
        else:
            cache.append_block(k_blk, v_blk)
        done += n
    assert cache.status() == 0 and cache.broken_guards() == []
    assert cache.packed_lens.cpu().tolist() == lens1
    a, c, o_ref, _ = oracle_side(full.to("cpu"), keep, keep_v)
    u = cache.unpack(want_vmask=True)
    assert np.array_equal(u["mask"].cpu().numpy().view(np.uint32), c["mask"])
    assert np.allclose(u["mu"].cpu().numpy(), c["mu"], rtol=1e-6, atol=0)
    if c["vmask"] is not None:
        assert np.array_equal(u["vmask"].cpu().numpy().view(np.uint32), c["vmask"])
    out = cache.decode(full.q)
    assert cache.status() == 0 and cache.broken_guards() == []
    assert float(np.abs(out.cpu().numpy() - o_ref).max()) <= TOL[dtype]


@pytest.mark.parametrize("seed", list(range(800, 830)) + [2031, 2095, 2139, 2195])     # the last four: fp32 storage, large outputs
def test_random_variant_shape(seed):
    """The ratio-free selection rules (Sec. "Ablation Studies", adaptive variants) and the sampled recovery
    distributions (Sec. "Channel Recovery") on random ragged batches, paged or contiguous."""
    import test_gpu_variants as V
    from paper_2508_15212_b200 import binding as B
    rnd = random.Random(seed)
    dtype = rnd.choice(["bf16", "bf16", "f32"])
    G, Hkv, Bn = rnd.choice([1, 2, 4, 5, 7, 8]), rnd.choice([1, 2, 3]), rnd.choice([1, 2, 3, 6])
    cap_len = rnd.choice([40, 200, 900])
    lens = [rnd.choice([0, 16, 17, rnd.randint(1, cap_len)]) for _ in range(Bn)]
    if max(lens) == 0:
        lens[0] = cap_len
    wl = V.make(dtype, Bn, G * Hkv, Hkv, lens, rnd.choice([4, 8, 32]), seed)
    table, n_pool = None, None
    if rnd.random() < 0.4:
        table, n_pages = permuted_block_table(Bn, Hkv, lens, "cuda", seed=seed)
        n_pool = n_pages + 2
    kind = rnd.choice(["top_p", "groups", "gaussian", "exponential", "sampled_top_p"])
    if kind == "top_p":
        V.check_selection(wl, rnd.choice([128, 96, 40]), top_p=rnd.choice([0.5, 0.9, 0.99, 0.999]),
                          block_table=table, n_pool_pages=n_pool)
    elif kind == "groups":
        ratios = rnd.choice([[0.25, 0.5, 0.75, 1.0], [0.1, 0.3, 0.5, 0.7, 0.9], [0.0, 1.0], [0.5], [0.2, 0.4, 0.6]])
        V.check_selection(wl, B.spark_group_keep(128, ratios), group_prune=ratios, block_table=table, n_pool_pages=n_pool)
    elif kind == "sampled_top_p":
        V.check_sampled(wl, 128, rnd.choice([1, 2]), seed, top_p=0.95, block_table=table, n_pool_pages=n_pool)
    else:
        V.check_sampled(wl, rnd.choice([25, 64, 100]), 1 if kind == "gaussian" else 2, seed,
                        block_table=table, n_pool_pages=n_pool)
