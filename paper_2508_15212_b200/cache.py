"""Device buffers of one packed SparK cache and the calls on it (plumbing around the C ABI)."""
from __future__ import annotations

from typing import Dict, Optional

import torch

from . import binding as B

_TDT = {"f32": torch.float32, "bf16": torch.bfloat16}


class SparkCache:
    """Owns the page pool, block table, qnorm, lens and workspaces for B sequences.

    ``block_table`` defaults to the identity (contiguous cache); pass a permuted
    table for a paged pool.  All arithmetic happens inside the library.
    """

    def __init__(self, *, batch: int, n_q_heads: int, n_kv_heads: int, window: int, keep: int, dtype: str,
                 max_tokens: int, device="cuda", block_table: Optional[torch.Tensor] = None,
                 n_pool_pages: Optional[int] = None, token_budget: int = 0, pool_kernel: int = 7,
                 softmax_scale: float = 0.0, pages: Optional[torch.Tensor] = None, flags: int = 0,
                 keep_v: int = 0):
        self.device = torch.device(device)
        self.dtype = dtype
        self.max_src_tokens = int(max_tokens)
        packed_max = min(max_tokens, token_budget) if token_budget > 0 else max_tokens
        self.max_tokens = int(packed_max)
        self.max_blocks = max(1, (self.max_tokens + 15) // 16)
        if block_table is None:
            block_table = B.identity_block_table(batch, n_kv_heads, self.max_blocks, self.device)
        self.block_table = block_table.to(self.device, torch.int32).contiguous()
        assert self.block_table.shape == (batch, n_kv_heads, self.block_table.shape[-1])
        assert self.block_table.shape[-1] >= self.max_blocks
        if n_pool_pages is None:
            n_pool_pages = batch * n_kv_heads * self.block_table.shape[-1]
        self.params = B.make_params(batch=batch, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, window=window,
                                    keep=keep, dtype=_TDT[dtype], n_pool_pages=n_pool_pages,
                                    token_budget=token_budget, pool_kernel=pool_kernel,
                                    softmax_scale=softmax_scale, flags=flags, keep_v=keep_v)
        self.page_bytes = B.spark_page_bytes(self.params)
        assert self.page_bytes > 0
        self.pages = pages if pages is not None else torch.zeros(n_pool_pages * self.page_bytes,
                                                                   dtype=torch.uint8, device=self.device)
        self.qnorm = torch.empty(batch, n_kv_heads, 128, dtype=torch.float32, device=self.device)
        self.packed_lens = torch.zeros(batch, dtype=torch.int32, device=self.device)
        self.kept_tokens = (torch.empty(batch, n_kv_heads, token_budget, dtype=torch.int32, device=self.device)
                            if token_budget > 0 else None)
        cb, db = B.spark_workspace_bytes(self.params, self.max_src_tokens)
        self.ws_compress = torch.empty(cb, dtype=torch.uint8, device=self.device)
        self.ws_decode = torch.empty(db, dtype=torch.uint8, device=self.device)
        B.spark_workspace_init(self.ws_compress)
        B.spark_workspace_init(self.ws_decode)

    # -- the two calls of the method ------------------------------------------------------------
    def compress(self, q_win, k, v, seq_lens) -> None:
        B.spark_compress(self.params, q_win, k, v, seq_lens, self.max_src_tokens, self.pages, self.block_table,
                         self.qnorm, self.packed_lens, self.kept_tokens, self.ws_compress)

    def append(self, k_new, v_new) -> None:
        """One new token per sequence ([B, Hkv, D]), pruned with the prefill statistics."""
        B.spark_append(self.params, k_new, v_new, self.pages, self.block_table, self.qnorm, self.packed_lens,
                       self.ws_compress)

    def decode(self, q, out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None):
        p = self.params
        if out is None:
            out = torch.empty(p.batch, p.n_q_heads, 128, dtype=torch.float32, device=self.device)
        B.spark_decode_attn(p, q, self.pages, self.block_table, self.packed_lens, self.qnorm, out, lse,
                            self.ws_decode)
        return out

    # -- inspection ------------------------------------------------------------------------------
    def unpack(self, want_vals=True, want_v=True, want_vmask=False) -> Dict[str, torch.Tensor]:
        p, n = self.params, self.max_tokens
        tdt = _TDT[self.dtype]
        out = dict(mask=torch.empty(p.batch, p.n_kv_heads, n, 4, dtype=torch.int32, device=self.device),
                   mu=torch.empty(p.batch, p.n_kv_heads, n, dtype=torch.float32, device=self.device))
        if want_vals:
            out["vals"] = torch.empty(p.batch, p.n_kv_heads, n, p.keep, dtype=tdt, device=self.device)
        if want_v:
            out["v"] = torch.empty(p.batch, p.n_kv_heads, n, 128, dtype=tdt, device=self.device)
        B.spark_unpack_pages(p, self.pages, self.block_table, self.packed_lens, n, out["mask"], out["mu"],
                             out.get("vals"), out.get("v"))
        if want_vmask:
            out["vmask"] = torch.empty(p.batch, p.n_kv_heads, n, 4, dtype=torch.int32, device=self.device)
            B.spark_unpack_value_masks(p, self.pages, self.block_table, self.packed_lens, n, out["vmask"])
        return out

    def status(self) -> int:
        s = B.spark_read_status(self.ws_compress)
        return s if s else B.spark_read_status(self.ws_decode)

    @property
    def algorithmic_bytes_per_token(self) -> int:
        return B.spark_algorithmic_bytes_per_token(self.params)


# ---------------------------------------------------------------------------------------------------
# Packed caches of the benchmark configurations (buffer plumbing; all arithmetic is in the library)
# ---------------------------------------------------------------------------------------------------
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
                        keep_prompts: int = 0, flags: int = 0, keep_v: int = 0):
    """Configuration 4: prompts are generated, evicted to the token budget and pruned ONE AT A TIME (each
    prompt's dense K/V is freed before the next), into one shared page pool; the result is a batch cache
    whose decode step serves all prompts.  Returns (cache, q [B,Hq,D], kept_tokens [B,Hkv,budget], dense)
    where `dense` holds the first `keep_prompts` prompts' workloads for checks."""
    from . import inputs
    Bn = int(n_prompts or config["batch"])
    Hq, Hkv, W, S = config["n_q_heads"], config["n_kv_heads"], config["window"], int(config["seq_lens"])
    budget, pool = int(config["token_budget"]), int(config["pool_kernel"])
    batch = SparkCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, window=W, keep=keep, dtype=config["dtype"],
                       max_tokens=min(S, budget), device=device, flags=flags, keep_v=keep_v)
    blocks = batch.max_blocks
    qs, kept, dense = [], [], []
    batch.prep_us = []                     # evict + prune time of each prompt (CUDA events)
    for b in range(Bn):
        wl = inputs.make_workload(batch=1, n_q_heads=Hq, n_kv_heads=Hkv, seq_lens=S, window=W,
                                  dtype=config["dtype"], sigma_s=config["sigma_s"],
                                  seed=int(config["seed"]) + 7 * b + 1000003 * seed_offset, device=device)
        one = SparkCache(batch=1, n_q_heads=Hq, n_kv_heads=Hkv, window=W, keep=keep, dtype=config["dtype"],
                         max_tokens=S, device=device, token_budget=budget, pool_kernel=pool,
                         block_table=batch.block_table[b:b + 1].contiguous(),
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
        if b < keep_prompts:
            dense.append(wl)
        del wl, one
    return batch, torch.stack(qs), torch.stack(kept), dense
