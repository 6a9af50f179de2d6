"""Parity of the CUDA path (through the C ABI) against the CPU oracle on identical seeded inputs.

Bar: kept-channel masks, kept values, value rows and qnorm bit-exact; mu within 1e-6 relative; attention
output max|delta| <= 1e-5 (fp32 storage) / 2e-3 (bf16 storage), fp32 accumulation on the GPU.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_15212_b200 import binding as B
from paper_2508_15212_b200 import build as spark_build
from workloads import inputs
from workloads.batches import permuted_block_table
from paper_2508_15212_b200.cache import SparkCache

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 2e-3}


@pytest.fixture(scope="module", autouse=True)
def built():
    spark_build.build()
    B.lib()


def to_np(t):
    t = t.detach().cpu()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def oracle_side(wl_cpu, keep, keep_v=0):
    Hkv = wl_cpu.k.shape[1]
    _, a = oracle.window_mean(wl_cpu.q_win, Hkv)
    c = oracle.compress(wl_cpu.k, wl_cpu.seq_lens, keep, a, want_idx=True)
    c["vmask"] = oracle.prune_values(wl_cpu.v, wl_cpu.seq_lens, keep_v) if 0 < keep_v < 128 else None
    out, lse = oracle.decode_attn(wl_cpu.q, wl_cpu.k, wl_cpu.v, wl_cpu.seq_lens, c["mask"], c["mu"], a,
                                  vmask=c["vmask"])
    return a, c, out, lse


def check_case(wl, keep, block_table=None, n_pool_pages=None, check_vals=True, keep_v=0):
    """wl lives on the GPU; returns max|delta| of the attention output."""
    Bn, Hq, Hkv, W, D, S = wl.shape
    wl_cpu = wl.to("cpu")
    a, c, o_ref, lse_ref = oracle_side(wl_cpu, keep, keep_v)
    cache = SparkCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, window=W, keep=keep, dtype=wl.dtype,
                       max_tokens=S, block_table=block_table, n_pool_pages=n_pool_pages, keep_v=keep_v, guard=True)
    cache.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
    lens = wl_cpu.seq_lens.tolist()
    assert cache.packed_lens.cpu().tolist() == lens
    assert np.array_equal(cache.qnorm.cpu().numpy(), a), "qnorm must be bit-exact"
    u = cache.unpack(want_vmask=True)
    mask = u["mask"].cpu().numpy().view(np.uint32)
    assert np.array_equal(mask, c["mask"]), "kept-channel masks must be bit-exact"
    vmask = u["vmask"].cpu().numpy().view(np.uint32)
    if c["vmask"] is not None:
        assert np.array_equal(vmask, c["vmask"]), "value-channel masks must be bit-exact"
    else:
        live = np.arange(S)[None, None, :, None] < np.asarray(lens)[:, None, None, None]
        assert np.array_equal(vmask, np.where(live, np.uint32(0xFFFFFFFF), np.uint32(0)) + np.zeros_like(vmask))
    mu = u["mu"].cpu().numpy()
    assert np.allclose(mu, c["mu"], rtol=1e-6, atol=0)
    if check_vals:
        kk = to_np(wl_cpu.k)
        want_vals = np.take_along_axis(kk, c["kept_idx"].astype(np.int64), axis=-1)
        vv = to_np(wl_cpu.v).copy()
        for b, n in enumerate(lens):
            want_vals[b, :, n:] = 0
            vv[b, :, n:] = 0
        assert np.array_equal(to_np(u["vals"]), want_vals), "kept values must be bit-identical copies"
        if c["vmask"] is not None:                                   # dropped value entries read back as zero
            bits = (c["vmask"][..., None] >> np.arange(32, dtype=np.uint32)) & 1
            vv = np.where(bits.reshape(vv.shape).astype(bool), vv, np.zeros_like(vv))
        assert np.array_equal(to_np(u["v"]), vv)
    lse = cache.alloc_lse()
    out = cache.decode(wl.q, lse=lse)
    out2 = cache.decode(wl.q)                                    # tickets self-reset; result reproducible
    assert cache.status() == 0
    assert torch.equal(out, out2)
    assert cache.broken_guards() == [], "a kernel wrote outside one of its buffers"
    d = float(np.abs(out.cpu().numpy() - o_ref).max())
    assert d <= TOL[wl.dtype], f"max|delta| {d:.3e} (max|out| {np.abs(o_ref).max():.3e})"
    l = lse.cpu().numpy()
    fin = np.isfinite(lse_ref)
    assert np.array_equal(np.isneginf(l), np.isneginf(lse_ref))
    assert np.allclose(l[fin], lse_ref[fin], rtol=0, atol=1e-3 if wl.dtype == "bf16" else 2e-5)
    return d


def make(dtype, Bn, Hq, Hkv, lens, W, keep, seed, sigma=1.0, gap=True):
    wl = inputs.make_workload(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, seq_lens=lens, window=W, dtype=dtype,
                              sigma_s=sigma, seed=seed, device="cuda")
    if gap:
        inputs.enforce_saliency_gap(wl, keep)
    return wl


def test_config1_tiny_fp32_full():
    c = inputs.CONFIGS[0]
    wl = inputs.config_workload(0, device="cuda")
    keep = B.spark_keep_count(128, c["ratio"])
    assert keep == 64
    inputs.enforce_saliency_gap(wl, keep)
    check_case(wl, keep)


@pytest.mark.parametrize("keep", [1, 25, 26, 38, 64, 89, 127, 128])
def test_bf16_gqa4_ragged_lengths_every_keep(keep):
    wl = make("bf16", 3, 8, 2, [1, 37, 530], 8, keep, seed=10 + keep)
    check_case(wl, keep)


@pytest.mark.parametrize("G,keep", [(1, 64), (2, 38), (3, 64), (5, 25), (6, 89), (7, 64), (8, 64)])
def test_group_sizes_bf16(G, keep):
    wl = make("bf16", 2, 2 * G, 2, [300, 47], 16, keep, seed=40 + G)
    check_case(wl, keep)


@pytest.mark.parametrize("G,keep", [(1, 64), (2, 38), (4, 25), (7, 64), (8, 100)])
def test_group_sizes_fp32(G, keep):
    wl = make("f32", 2, 2 * G, 2, [200, 33], 8, keep, seed=60 + G, sigma=0.5)
    check_case(wl, keep)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_selection_is_exact_on_subnormal_saliencies(dtype):
    """Saliencies around 1e-39 (fp32 subnormals, whose upper 16 bits are bf16 subnormals): the selection must still
    order them exactly -- nothing may be flushed to zero on the way to the kept set."""
    wl = make(dtype, 2, 4, 2, [70, 33], 8, 64, seed=75, sigma=1.0 if dtype == "bf16" else 0.5, gap=False)
    tdt = wl.k.dtype
    wl.k = (wl.k.float() * 2e-38).to(tdt)                       # the divisor's floor keeps a[j] ordinary: shrink K alone
    wl_cpu = wl.to("cpu")
    _, a = oracle.window_mean(wl_cpu.q_win, 2)
    sal = oracle.compress(wl_cpu.k, wl_cpu.seq_lens, 64, a, want_saliency=True)["saliency"]
    live = sal[0, 0, :70]
    assert 0 < live[live > 0].min() < 1.1754944e-38 and live.max() < 1e-36      # really in the subnormal range
    for keep in (64, 25):
        cache = SparkCache(batch=2, n_q_heads=4, n_kv_heads=2, window=8, keep=keep, dtype=dtype, max_tokens=70)
        cache.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
        c = oracle.compress(wl_cpu.k, wl_cpu.seq_lens, keep, a)
        u = cache.unpack(want_vals=False, want_v=False)
        assert np.array_equal(cache.qnorm.cpu().numpy(), a)
        assert np.array_equal(u["mask"].cpu().numpy().view(np.uint32), c["mask"])
        assert np.allclose(u["mu"].cpu().numpy(), c["mu"], rtol=1e-6, atol=0)


def test_single_token_and_empty_sequence():
    wl = make("bf16", 3, 8, 2, [0, 1, 16], 4, 64, seed=70)
    check_case(wl, 64)


def test_all_sequences_empty():
    wl = make("bf16", 2, 8, 2, [0, 0], 4, 64, seed=71, gap=False)
    Bn, Hq, Hkv, W, D, S = wl.shape
    cache = SparkCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, window=W, keep=64, dtype="bf16", max_tokens=16)
    cache.compress(wl.q_win, wl.k[:, :, :0].contiguous() if S == 0 else wl.k, wl.v, wl.seq_lens)
    lse = torch.full((Bn, Hq), 1.0, dtype=torch.float32, device="cuda")
    out = cache.decode(wl.q, out=torch.full((Bn, Hq, 128), 7.0, dtype=torch.float32, device="cuda"), lse=lse)
    assert cache.status() == 0
    assert bool((out == 0).all()) and bool(torch.isneginf(lse).all())


@pytest.mark.parametrize("W", [1, 64])
def test_window_sizes(W):
    wl = make("bf16", 2, 8, 2, [70, 200], W, 38, seed=72 + W)
    check_case(wl, 38)


def test_paged_pool_with_permuted_block_table_qwen_shape():
    lens = [700, 33, 1200, 16]
    wl = make("bf16", 4, 28, 4, lens, 32, 38, seed=80)
    max_blocks = (max(lens) + 15) // 16 + 3                      # table wider than needed
    n_pages = 4 * 4 * max_blocks + 11
    g = torch.Generator().manual_seed(5)
    perm = torch.randperm(n_pages, generator=g)[: 4 * 4 * max_blocks].to(torch.int32)
    bt = perm.view(4, 4, max_blocks).cuda()
    check_case(wl, 38, block_table=bt, n_pool_pages=n_pages)


def test_token_major_kv_layout():
    wl = make("bf16", 2, 8, 2, [100, 260], 8, 64, seed=90)
    k_tm = wl.k.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)      # [B,S,H,D] storage
    v_tm = wl.v.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    assert k_tm.stride() != wl.k.stride()
    wl.k, wl.v = k_tm, v_tm
    check_case(wl, 64)


def test_many_units_cross_cta_boundaries():
    """More (sequence, head) units than CTAs, lengths that make CTA ranges straddle units."""
    lens = [64 + 37 * i for i in range(40)]
    wl = make("bf16", 40, 16, 8, lens, 8, 64, seed=100, gap=False)
    check_case(wl, 64, check_vals=False)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_largest_batch_with_empty_and_one_page_sequences(dtype):
    """1024 sequences (the most one call takes), lengths 0..33: empty ones, single tokens, page tails."""
    rng = np.random.default_rng(1024)
    lens = rng.integers(0, 34, size=1024).tolist()
    lens[0], lens[1], lens[-1] = 0, 33, 0
    wl = make(dtype, 1024, 2, 1, lens, 4, 38, seed=110, sigma=1.0 if dtype == "bf16" else 0.5, gap=False)
    check_case(wl, 38, check_vals=False)


@pytest.mark.parametrize("Bn,Hkv,n", [(37, 8, 150), (145, 2, 70)])
def test_more_equal_units_than_ctas_whole_units_per_cta(Bn, Hkv, n):
    """296 and 290 equal-length units on 148 CTAs: every CTA takes two whole units (or two and one)."""
    wl = make("bf16", Bn, 2 * Hkv, Hkv, [n] * Bn, 8, 64, seed=120 + Bn, gap=False)
    check_case(wl, 64, check_vals=False)


def test_config2_llama_32k_full():
    c = inputs.CONFIGS[1]
    wl = inputs.config_workload(1, device="cuda")
    keep = B.spark_keep_count(128, c["ratio"])
    inputs.enforce_saliency_gap(wl, keep)
    d = check_case(wl, keep)
    print(f"config 2 max|delta| = {d:.3e}")


def test_bad_page_id_is_recorded_not_dereferenced():
    wl = make("bf16", 1, 4, 1, [64], 4, 64, seed=110, gap=False)
    cache = SparkCache(batch=1, n_q_heads=4, n_kv_heads=1, window=4, keep=64, dtype="bf16", max_tokens=64,
                       block_table=B.identity_block_table(1, 1, 4, "cuda"))
    cache.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
    assert cache.status() == 0
    cache.block_table[0, 0, 1] = 1 << 20                       # outside the pool
    cache.decode(wl.q)
    assert B.spark_read_status(cache.ws_decode) == 6            # SPARK_ERR_DEVICE_BOUNDS


def oracle_evicted_sets(wl_cpu, budget, pool):
    """Oracle eviction: kept tokens, lengths and the relative gap of the pooled votes at the budget boundary."""
    Bn, Hq, Hkv, W, D, S = wl_cpu.shape
    lens = wl_cpu.seq_lens.tolist()
    kept, n, vote, pooled = oracle.evict(wl_cpu.q_win, wl_cpu.k, lens, budget, pool, want_votes=True)
    gaps = np.full((Bn, Hkv), np.inf)
    for b in range(Bn):
        if lens[b] <= budget:
            continue
        P, k = lens[b] - W, budget - W
        for h in range(Hkv):
            srt = np.sort(pooled[b, h, :P])[::-1]
            gaps[b, h] = (srt[k - 1] - srt[k]) / max(srt[k - 1], 1e-300)
    return kept, n, gaps


def oracle_on_kept_tokens(wl_cpu, kept, n, keep):
    """Oracle pruning + decode over the tokens listed in `kept` ([B][Hkv][budget], first n[b] valid)."""
    Bn, Hq, Hkv, W, D, S = wl_cpu.shape
    budget = kept.shape[-1]
    kk, vv = to_np(wl_cpu.k), to_np(wl_cpu.v)
    kg, vg = np.zeros((Bn, Hkv, budget, D), kk.dtype), np.zeros((Bn, Hkv, budget, D), vv.dtype)
    for b in range(Bn):
        for h in range(Hkv):
            idx = kept[b, h, :n[b]]
            kg[b, h, :n[b]] = kk[b, h, idx]
            vg[b, h, :n[b]] = vv[b, h, idx]
    _, a = oracle.window_mean(wl_cpu.q_win, Hkv)
    c = oracle.compress(kg, n, keep, a)
    out, _ = oracle.decode_attn(to_np(wl_cpu.q), kg, vg, n, c["mask"], c["mu"], a)
    return c, out, kg, vg


@pytest.mark.parametrize("dtype,lens,W,budget,G", [("bf16", [600, 90, 300], 8, 128, 4),
                                                   ("bf16", [2000], 32, 256, 7),
                                                   ("f32", [500, 64], 16, 96, 2)])
def test_eviction_then_pruning_against_oracle(dtype, lens, W, budget, G):
    check_eviction_case(dtype, lens, W, budget, G)


def check_eviction_case(dtype, lens, W, budget, G, keep=64, Hkv=2, pool=7, seed=None):
    """Three checks, none of them conditional on the other: (1) the evicted token sets against the oracle's
    (exact where the pooled votes at the budget boundary are not a near-tie); (2) pruning and decode of the
    evicting call against the oracle run on the SAME token set (the one the GPU kept); (3) pruning and decode
    of the oracle's token set, gathered and fed to both sides through the non-evicting call.  A near-tie in
    (1) can therefore never hide a pruning or decode error."""
    Bn = len(lens)
    wl = make(dtype, Bn, Hkv * G, Hkv, lens, W, keep, seed=130 + G if seed is None else seed,
              sigma=1.0 if dtype == "bf16" else 0.5, gap=False)
    wl_cpu = wl.to("cpu")
    kept_ref, n_ref, gaps = oracle_evicted_sets(wl_cpu, budget, pool)
    cache = SparkCache(batch=Bn, n_q_heads=Hkv * G, n_kv_heads=Hkv, window=W, keep=keep, dtype=dtype,
                       max_tokens=max(lens), token_budget=budget, pool_kernel=pool, guard=True)
    cache.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
    assert cache.status() == 0
    assert cache.packed_lens.cpu().tolist() == n_ref.tolist()
    kept = cache.kept_tokens.cpu().numpy()
    # (1) token sets
    for b in range(Bn):
        for h in range(Hkv):
            a_, r_ = kept[b, h, :n_ref[b]], kept_ref[b, h, :n_ref[b]]
            assert (np.diff(a_) > 0).all()
            if lens[b] >= W:
                assert a_[-W:].tolist() == list(range(lens[b] - W, lens[b]))
            if gaps[b, h] > 1e-4:
                assert np.array_equal(a_, r_), f"evicted set differs at unit ({b},{h}), gap {gaps[b, h]:.2e}"
            else:
                assert len(set(a_.tolist()) & set(r_.tolist())) >= n_ref[b] - 2
    # (2) the evicting call's pages and output against the oracle on the GPU's own token set
    c_gpu, out_gpu_ref, _, _ = oracle_on_kept_tokens(wl_cpu, kept, n_ref, keep)
    u = cache.unpack(want_vals=False, want_v=False)
    m = min(max(lens), budget)                              # tokens a unit can hold: the unpacked and the oracle arrays
    assert int(n_ref.max()) <= m                            # are sized max(lens) and budget
    assert np.array_equal(u["mask"].cpu().numpy().view(np.uint32)[:, :, :m], c_gpu["mask"][:, :, :m])
    assert np.allclose(u["mu"].cpu().numpy()[:, :, :m], c_gpu["mu"][:, :, :m], rtol=1e-6, atol=0)
    out = cache.decode(wl.q)
    assert cache.status() == 0
    d = float(np.abs(out.cpu().numpy() - out_gpu_ref).max())
    assert d <= TOL[dtype], f"evicting call: max|delta| {d:.3e}"
    assert cache.broken_guards() == []
    # (3) the oracle's token set, gathered, through the non-evicting call
    c_ref, out_ref, kg, vg = oracle_on_kept_tokens(wl_cpu, kept_ref, n_ref, keep)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    as_t = (lambda x: torch.from_numpy(x.view(np.int16)).view(torch.bfloat16)) if dtype == "bf16" else torch.from_numpy
    kg_t, vg_t = as_t(kg).cuda(), as_t(vg).cuda()
    assert kg_t.dtype == tdt
    plain = SparkCache(batch=Bn, n_q_heads=Hkv * G, n_kv_heads=Hkv, window=W, keep=keep, dtype=dtype,
                       max_tokens=budget, guard=True)
    plain.compress(wl.q_win, kg_t, vg_t, torch.from_numpy(n_ref).cuda())
    u = plain.unpack(want_vals=False, want_v=False)
    assert np.array_equal(u["mask"].cpu().numpy().view(np.uint32), c_ref["mask"])
    out = plain.decode(wl.q)
    assert plain.status() == 0
    d = float(np.abs(out.cpu().numpy() - out_ref).max())
    assert d <= TOL[dtype], f"oracle's token set: max|delta| {d:.3e}"
    assert plain.broken_guards() == []


def test_overlap_flag_gives_identical_results_back_to_back():
    """Programmatic dependent launch: same workspace, consecutive steps, bitwise the same output."""
    wl = make("bf16", 2, 16, 4, [4000, 1500], 16, 64, seed=140, gap=False)
    outs = []
    for flags in (0, B.SPARK_FLAG_OVERLAP_PREVIOUS):
        cache = SparkCache(batch=2, n_q_heads=16, n_kv_heads=4, window=16, keep=64, dtype="bf16", max_tokens=4000,
                           flags=flags)
        cache.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
        o = [cache.decode(wl.q) for _ in range(6)]             # launched back to back on one stream
        assert cache.status() == 0
        assert all(torch.equal(o[0], x) for x in o[1:])
        outs.append(o[0])
    assert torch.equal(outs[0], outs[1])
    with pytest.raises(B.SparkError):
        SparkCache(batch=1, n_q_heads=4, n_kv_heads=1, window=4, keep=64, dtype="bf16", max_tokens=64, flags=6)


@pytest.mark.parametrize("dtype,keep", [("bf16", 64), ("bf16", 25), ("f32", 38)])
def test_append_tokens_equals_compressing_the_longer_sequence(dtype, keep):
    """Prefill S0 tokens, append n more one at a time: the cache must equal what pruning all S0 + n
    tokens with the same window queries gives (oracle), and the decode output must match."""
    lens0, n_app = [37, 530, 16], 21
    full = make(dtype, 3, 8, 2, [l + n_app for l in lens0], 8, keep, seed=150, sigma=1.0 if dtype == "bf16" else 0.5)
    S = max(lens0) + n_app
    cache = SparkCache(batch=3, n_q_heads=8, n_kv_heads=2, window=8, keep=keep, dtype=dtype, max_tokens=S)
    lens0_t = torch.tensor(lens0, dtype=torch.int32, device="cuda")
    cache.compress(full.q_win, full.k, full.v, lens0_t)                  # prefill sees the first S0 tokens only
    for i in range(n_app):
        idx = (lens0_t.long() + i).view(3, 1, 1, 1).expand(3, 2, 1, 128)
        cache.append(full.k.gather(2, idx).squeeze(2).contiguous(), full.v.gather(2, idx).squeeze(2).contiguous())
        assert B.lib().spark_last_launch_count() == 1             # a CTA per sequence, a warp per KV head
    assert cache.status() == 0
    assert cache.packed_lens.cpu().tolist() == [l + n_app for l in lens0]
    wl_cpu = full.to("cpu")
    a, c, o_ref, _ = oracle_side(wl_cpu, keep)
    u = cache.unpack()
    assert np.array_equal(u["mask"].cpu().numpy().view(np.uint32), c["mask"])
    assert np.allclose(u["mu"].cpu().numpy(), c["mu"], rtol=1e-6, atol=0)
    out = cache.decode(full.q)
    assert float(np.abs(out.cpu().numpy() - o_ref).max()) <= TOL[dtype]
    # a full sequence is left unchanged and the condition is recorded
    small = SparkCache(batch=1, n_q_heads=4, n_kv_heads=1, window=8, keep=keep, dtype=dtype, max_tokens=16)
    one = make(dtype, 1, 4, 1, [16], 8, keep, seed=151, gap=False)
    small.compress(one.q_win, one.k, one.v, one.seq_lens)
    small.append(one.k[:, :, 0].contiguous(), one.v[:, :, 0].contiguous())
    assert small.packed_lens.cpu().tolist() == [16] and B.spark_read_status(small.ws_compress) == 6


def test_append_with_more_than_32_kv_heads():
    """Up to 32 KV heads a CTA per sequence appends all heads in one launch; beyond that the per-head launch plus
    the length update is used.  Same result either way (oracle pruning of the longer sequence)."""
    lens0, n_app, Hkv, keep = [20, 5], 14, 40, 64
    full = make("bf16", 2, Hkv, Hkv, [l + n_app for l in lens0], 4, keep, seed=154)
    S = max(lens0) + n_app
    cache = SparkCache(batch=2, n_q_heads=Hkv, n_kv_heads=Hkv, window=4, keep=keep, dtype="bf16", max_tokens=S, guard=True)
    lens0_t = torch.tensor(lens0, dtype=torch.int32, device="cuda")
    cache.compress(full.q_win, full.k, full.v, lens0_t)
    for i in range(n_app):
        idx = (lens0_t.long() + i).view(2, 1, 1, 1).expand(2, Hkv, 1, 128)
        cache.append(full.k.gather(2, idx).squeeze(2).contiguous(), full.v.gather(2, idx).squeeze(2).contiguous())
        assert B.lib().spark_last_launch_count() == 2
    assert cache.status() == 0 and cache.broken_guards() == []
    assert cache.packed_lens.cpu().tolist() == [l + n_app for l in lens0]
    a, c, o_ref, _ = oracle_side(full.to("cpu"), keep)
    u = cache.unpack(want_vals=False, want_v=False)
    assert np.array_equal(u["mask"].cpu().numpy().view(np.uint32), c["mask"])
    assert float(np.abs(cache.decode(full.q).cpu().numpy() - o_ref).max()) <= TOL["bf16"]


def test_block_append_equals_appending_one_token_at_a_time():
    lens0, n = [37, 530, 16], 45
    full = make("bf16", 3, 8, 2, [l + n for l in lens0], 8, 38, seed=152)
    S = max(lens0) + n
    lens0_t = torch.tensor(lens0, dtype=torch.int32, device="cuda")
    idx = (lens0_t.long().view(3, 1, 1, 1) + torch.arange(n, device="cuda").view(1, 1, n, 1)).expand(3, 2, n, 128)
    k_blk, v_blk = full.k.gather(2, idx).contiguous(), full.v.gather(2, idx).contiguous()
    one, blk = (SparkCache(batch=3, n_q_heads=8, n_kv_heads=2, window=8, keep=38, dtype="bf16", max_tokens=S,
                           guard=True) for _ in range(2))
    for c in (one, blk):
        c.compress(full.q_win, full.k, full.v, lens0_t)
    for i in range(n):
        one.append(k_blk[:, :, i].contiguous(), v_blk[:, :, i].contiguous())
    blk.append_block(k_blk, v_blk)
    assert one.status() == 0 and blk.status() == 0 and blk.broken_guards() == []
    assert blk.packed_lens.cpu().tolist() == [l + n for l in lens0]
    ua, ub = one.unpack(), blk.unpack()
    for key in ("mask", "mu", "vals", "v"):
        assert torch.equal(ua[key], ub[key]), key
    # more tokens than there is room for: the sequence is filled up and the condition recorded
    small = SparkCache(batch=1, n_q_heads=4, n_kv_heads=1, window=8, keep=38, dtype="bf16", max_tokens=32)
    w1 = make("bf16", 1, 4, 1, [40], 8, 38, seed=153, gap=False)
    small.compress(w1.q_win, w1.k[:, :, :20].contiguous(), w1.v[:, :, :20].contiguous(), torch.tensor([20], dtype=torch.int32, device="cuda"))
    small.append_block(w1.k[:, :, 20:40].contiguous(), w1.v[:, :, 20:40].contiguous())
    assert small.packed_lens.cpu().tolist() == [32] and B.spark_read_status(small.ws_compress) == 6


@pytest.mark.parametrize("dtype,block,n_app", [("bf16", 16, 41), ("bf16", None, 30), ("f32", 8, 19)])
def test_dense_tail_equals_the_oracle_with_appended_keys_left_dense(dtype, block, n_app):
    """Pruned prefix + dense tail (the paper's literal K <- Cat[K, k]): the oracle attends over all tokens with
    the prefill-pruned mask on the prefix (handed-over blocks included) and every channel kept on the tail."""
    from paper_2508_15212_b200.cache import DenseTailCache
    keep, lens0 = 38, [50, 200]
    full = make(dtype, 2, 8, 2, [l + n_app for l in lens0], 8, keep, seed=160, sigma=1.0 if dtype == "bf16" else 0.5)
    S = max(lens0) + n_app
    cache = DenseTailCache(batch=2, n_q_heads=8, n_kv_heads=2, window=8, keep=keep, dtype=dtype, max_tokens=S,
                           tail_block=block, max_tail=64)
    lens0_t = torch.tensor(lens0, dtype=torch.int32, device="cuda")
    cache.compress(full.q_win, full.k, full.v, lens0_t)
    wl_cpu = full.to("cpu")
    _, a = oracle.window_mean(wl_cpu.q_win, 2)
    c = oracle.compress(wl_cpu.k, wl_cpu.seq_lens, keep, a)
    for i in range(n_app):
        idx = (lens0_t.long() + i).view(2, 1, 1, 1).expand(2, 2, 1, 128)
        cache.append(full.k.gather(2, idx).squeeze(2).contiguous(), full.v.gather(2, idx).squeeze(2).contiguous())
        if i in (0, n_app // 2, n_app - 1):
            n_dense = (i + 1) if block is None else (i + 1) % block
            mask, mu, lens_now = c["mask"].copy(), c["mu"].copy(), [l + i + 1 for l in lens0]
            for b, l in enumerate(lens_now):                 # the last n_dense tokens are still dense
                mask[b, :, l - n_dense:l] = 0xFFFFFFFF
                mu[b, :, l - n_dense:l] = 0.0
            ref, ref_lse = oracle.decode_attn(wl_cpu.q, wl_cpu.k, wl_cpu.v, lens_now, mask, mu, a)
            lse = torch.empty(2, 8, dtype=torch.float32, device="cuda")
            out = cache.decode(full.q, lse=lse)
            assert cache.status() == 0
            d = float(np.abs(out.cpu().numpy() - ref).max())
            assert d <= TOL[dtype], f"after {i + 1} appended tokens: max|delta| {d:.3e}"
            assert np.allclose(lse.cpu().numpy(), ref_lse, rtol=0, atol=1e-3 if dtype == "bf16" else 2e-5)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_host_entry_point_staged_and_mapped_equal_the_device_call(dtype):
    """spark_decode_attn_host: query and result in page-locked host memory, with staging copies or (flag) with the
    kernel addressing the host buffers itself.  Both must give the device call's output bit for bit (which the
    other tests tie to the oracle)."""
    wl = make(dtype, 2, 8, 2, [700, 64], 8, 38, seed=170, sigma=1.0 if dtype == "bf16" else 0.5)
    cache = SparkCache(batch=2, n_q_heads=8, n_kv_heads=2, window=8, keep=38, dtype=dtype, max_tokens=700)
    cache.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
    ref = cache.decode(wl.q)
    wl_cpu = wl.to("cpu")
    a, c, o_ref, _ = oracle_side(wl_cpu, 38)
    assert float(np.abs(ref.cpu().numpy() - o_ref).max()) <= TOL[dtype]
    q_host = wl.q.cpu().pin_memory()
    for flags in (0, B.SPARK_FLAG_HOST_MAPPED):
        out_host = torch.full((2, 8, 128), float("nan"), dtype=torch.float32).pin_memory()
        cache.params.flags = flags
        call = cache.bind_decode_host(q_host, out_host)
        call()
        torch.cuda.synchronize()
        assert torch.equal(out_host, ref.cpu()), f"flags={flags}"
    cache.params.flags = 0
    assert cache.status() == 0


@pytest.mark.parametrize("batch", [1, 3, 4])
def test_host_mapped_query_travels_with_the_launch_when_it_fits(batch):
    """SPARK_FLAG_HOST_MAPPED, bf16 storage: a query of up to 24 KB is read during the call and rides in the
    launch (8 KB and 24 KB parameter blocks: batch 1 and 3 at 32 heads), so q_host may be overwritten as soon as
    the call returns; a larger one (batch 4) is read by the kernel in stream order.  Same bits as the device
    call, which is checked against the oracle here."""
    lens = [200, 64, 17, 333][:batch]
    wl = make("bf16", batch, 32, 8, lens, 8, 64, seed=171 + batch, sigma=1.0)
    cache = SparkCache(batch=batch, n_q_heads=32, n_kv_heads=8, window=8, keep=64, dtype="bf16", max_tokens=max(lens))
    cache.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
    ref = cache.decode(wl.q)
    _, _, o_ref, _ = oracle_side(wl.to("cpu"), 64)
    assert float(np.abs(ref.cpu().numpy() - o_ref).max()) <= TOL["bf16"]
    q_host = wl.q.cpu().pin_memory()
    out_host = torch.full((batch, 32, 128), float("nan"), dtype=torch.float32).pin_memory()
    cache.params.flags = B.SPARK_FLAG_HOST_MAPPED
    call = cache.bind_decode_host(q_host, out_host)
    by_value = batch * 32 * 256 <= 24 * 1024
    for _ in range(2):
        call()
        if by_value:
            q_host.zero_()                                      # the bytes were taken during the call
        torch.cuda.synchronize()
        assert torch.equal(out_host, ref.cpu())
        q_host.copy_(wl.q.cpu())
        out_host.fill_(float("nan"))
    cache.params.flags = 0
    assert cache.status() == 0


def test_merge_attn_handles_empty_sides():
    o = torch.randn(2, 4, 128, device="cuda")
    zero = torch.zeros_like(o)
    l = torch.tensor([[0.5, -1.0, 2.0, 0.0]] * 2, device="cuda")
    ninf = torch.full_like(l, float("-inf"))
    out, lse = torch.empty_like(o), torch.empty_like(l)
    B.spark_merge_attn(o, l, zero, ninf, out, lse)
    assert torch.equal(out, o) and torch.equal(lse, l)
    B.spark_merge_attn(zero, ninf, zero, ninf, out, lse)
    assert bool((out == 0).all()) and bool(torch.isneginf(lse).all())
    B.spark_merge_attn(o, l, o, l, out, lse)                    # equal halves: same output, lse + ln 2
    assert torch.allclose(out, o, atol=1e-6) and torch.allclose(lse, l + 0.6931472, atol=1e-6)


# ---- value-channel pruning (App. "Pruning Value Cache Channels") ------------------------------------
@pytest.mark.parametrize("keep,keep_v", [(64, 64), (64, 89), (25, 25), (38, 1), (128, 64), (64, 127)])
def test_value_pruning_bf16_ragged(keep, keep_v):
    wl = make("bf16", 3, 8, 2, [1, 37, 530], 8, keep, seed=300 + keep + keep_v)
    check_case(wl, keep, keep_v=keep_v)


@pytest.mark.parametrize("G,keep,keep_v", [(1, 64, 64), (7, 38, 64), (8, 64, 25)])
def test_value_pruning_group_sizes_and_paged_pool(G, keep, keep_v):
    lens = [300, 47]
    wl = make("bf16", 2, 2 * G, 2, lens, 16, keep, seed=340 + G)
    table, n_pages = permuted_block_table(2, 2, lens, "cuda", seed=7, spare=3)
    check_case(wl, keep, block_table=table, n_pool_pages=n_pages, keep_v=keep_v)


def test_value_pruning_fp32_storage():
    wl = make("f32", 2, 4, 2, [130, 33], 8, 64, seed=360, sigma=0.5)
    check_case(wl, 64, keep_v=48)


def test_value_pruning_llama_32k_half_half():
    """The (0.5 + 0.5) setting at the 32K shape: several CTAs per unit, last-arriver merge."""
    wl = inputs.config_workload(1, device="cuda")
    inputs.enforce_saliency_gap(wl, 64)
    d = check_case(wl, 64, check_vals=False, keep_v=64)
    assert d <= 2e-3


def test_value_pruning_append_matches_compressing_the_longer_sequence():
    lens0, extra = [37, 16], 20
    wl = make("bf16", 2, 8, 2, [n + extra for n in lens0], 8, 64, seed=370)
    Bn, Hq, Hkv, W, D, S = wl.shape
    full = SparkCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, window=W, keep=64, dtype="bf16", max_tokens=S, keep_v=40)
    full.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
    grown = SparkCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, window=W, keep=64, dtype="bf16", max_tokens=S, keep_v=40)
    grown.compress(wl.q_win, wl.k, wl.v, torch.tensor(lens0, dtype=torch.int32, device="cuda"))
    for step in range(extra):
        idx = torch.tensor([n + step for n in lens0], device="cuda")
        k_new = wl.k[torch.arange(Bn, device="cuda"), :, idx].contiguous()
        v_new = wl.v[torch.arange(Bn, device="cuda"), :, idx].contiguous()
        grown.append(k_new, v_new)
    assert grown.status() == 0 and grown.packed_lens.cpu().tolist() == wl.seq_lens.cpu().tolist()
    ua, ub = full.unpack(want_vmask=True), grown.unpack(want_vmask=True)
    for key in ("mask", "mu", "vals", "v", "vmask"):
        assert torch.equal(ua[key], ub[key]), key
    assert torch.equal(full.decode(wl.q), grown.decode(wl.q))
