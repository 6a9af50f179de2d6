"""Packed caches of the benchmark configurations: block tables of a paged pool and the evicted batch.

Harness code for the tests and the benchmark (buffer plumbing around the library calls; all arithmetic
is in the library).
"""
from __future__ import annotations

import torch

from paper_2508_15212_b200.cache import SparkCache

from . import inputs


def permuted_block_table(batch: int, n_kv_heads: int, lens, device, seed: int, spare: int = 0):
    """Block table of a paged pool: every (sequence, head) unit gets exactly the pages it needs, drawn
    from a seeded random permutation of the pool.  Returns (table [B,Hkv,max_blocks] int32, n_pool_pages)."""
    blocks = [(int(n) + 15) // 16 for n in lens]
    max_blocks = max(max(blocks), 1)
    n_pages = n_kv_heads * sum(blocks) + spare
    g = torch.Generator().manual_seed(int(seed))
    perm = torch.randperm(n_pages, generator=g).to(torch.int32)
    table = torch.zeros(batch, n_kv_heads, max_blocks, dtype=torch.int32)
    pos = 0
    for b in range(batch):
        for h in range(n_kv_heads):
            table[b, h, :blocks[b]] = perm[pos:pos + blocks[b]]
            pos += blocks[b]
    return table.to(device), max(n_pages, 1)


def build_evicted_batch(config: dict, keep: int, device="cuda", n_prompts: int = None, seed_offset: int = 0,
                        keep_prompts=(), flags: int = 0, keep_v: int = 0,
                        guard: bool = False, keep_gathered: bool = False):
    """Configuration 4: prompts are generated, evicted to the token budget and pruned ONE AT A TIME (each
    prompt's dense K/V is freed before the next), into one shared page pool; the result is a batch cache
    whose decode step serves all prompts.  Returns (cache, q [B,Hq,D], kept_tokens [B,Hkv,budget], dense)
    where `dense` maps each prompt index listed in `keep_prompts` to its dense workload, for checks.  With
    `keep_gathered` the cache also carries `gathered = (q_win, k, v)`: every prompt's window queries and the keys
    and values of its kept tokens ([B,Hkv,budget,D]), the input an oracle needs to redo pruning and decode."""
    Bn = int(n_prompts or config["batch"])
    Hq, Hkv, W, S = config["n_q_heads"], config["n_kv_heads"], config["window"], int(config["seq_lens"])
    budget, pool = int(config["token_budget"]), int(config["pool_kernel"])
    batch = SparkCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, window=W, keep=keep, dtype=config["dtype"],
                       max_tokens=min(S, budget), device=device, flags=flags, keep_v=keep_v, guard=guard)
    blocks = batch.max_blocks
    from paper_2508_15212_b200 import binding as B
    rows = B.identity_block_table(Bn, Hkv, blocks, device)     # where each prompt's pages sit in the batch pool
    qs, kept, dense = [], [], {}
    gath = ([], [], []) if keep_gathered else None
    batch.prep_us = []                     # evict + prune time of each prompt (CUDA events)
    for b in range(Bn):
        wl = inputs.make_workload(batch=1, n_q_heads=Hq, n_kv_heads=Hkv, seq_lens=S, window=W,
                                  dtype=config["dtype"], sigma_s=config["sigma_s"],
                                  seed=int(config["seed"]) + 7 * b + 1000003 * seed_offset, device=device)
        one = SparkCache(batch=1, n_q_heads=Hq, n_kv_heads=Hkv, window=W, keep=keep, dtype=config["dtype"],
                         max_tokens=S, device=device, token_budget=budget, pool_kernel=pool,
                         block_table=rows[b:b + 1].contiguous(),
                         n_pool_pages=batch.params.n_pool_pages, pages=batch.pages, keep_v=keep_v)
        assert one.block_table.shape[-1] == blocks
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        one.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
        e1.record()
        e1.synchronize()
        batch.prep_us.append(e0.elapsed_time(e1) * 1e3)
        batch.qnorm[b].copy_(one.qnorm[0])
        batch.packed_lens[b:b + 1].copy_(one.packed_lens)
        qs.append(wl.q[0])
        kept.append(one.kept_tokens[0].clone())
        assert one.status() == 0
        if b in keep_prompts:
            dense[b] = wl
        if keep_gathered:
            idx = one.kept_tokens[0].long().unsqueeze(-1).expand(Hkv, budget, 128)
            gath[0].append(wl.q_win[0])
            gath[1].append(wl.k[0].gather(1, idx))
            gath[2].append(wl.v[0].gather(1, idx))
        del wl, one
    batch.gathered = tuple(torch.stack(x) for x in gath) if keep_gathered else None
    return batch, torch.stack(qs), torch.stack(kept), dense
