"""Device buffers of one packed SparK cache and the calls on it (plumbing around the C ABI)."""
from __future__ import annotations

from typing import Dict, Optional

import torch

from . import binding as B

_TDT = {"f32": torch.float32, "bf16": torch.bfloat16}
GUARD_BYTES = 4096          # canary band on each side of a guarded buffer
GUARD_VALUE = 0xA5


class SparkCache:
    """Owns the page pool, block table, qnorm, lens and workspaces for B sequences.

    Without a ``block_table`` the cache is contiguous (the library is given no table: unit (b, h) owns
    ``max_blocks`` consecutive pages); pass a table for a paged pool.  All arithmetic happens inside the
    library.
    """

    def __init__(self, *, batch: int, n_q_heads: int, n_kv_heads: int, window: int, keep: int, dtype: str,
                 max_tokens: int, device="cuda", block_table: Optional[torch.Tensor] = None,
                 n_pool_pages: Optional[int] = None, token_budget: int = 0, pool_kernel: int = 7,
                 softmax_scale: float = 0.0, pages: Optional[torch.Tensor] = None, flags: int = 0,
                 keep_v: int = 0, guard: bool = False, top_p: Optional[float] = None, group_prune=None,
                 recovery: int = 0, seed: int = 0):
        self.device = torch.device(device)
        self.guard = bool(guard)          # debugging aid: canary bands around every buffer the library writes
        self._bands = []                  # (name, raw uint8 tensor, payload bytes)
        self.dtype = dtype
        self.max_src_tokens = int(max_tokens)
        packed_max = min(max_tokens, token_budget) if token_budget > 0 else max_tokens
        self.max_tokens = int(packed_max)
        self.max_blocks = max(1, (self.max_tokens + 15) // 16)
        if block_table is None:
            self.block_table = None                       # contiguous cache: the calls get a NULL table
            self.table_blocks = self.max_blocks
        else:
            self.block_table = block_table.to(self.device, torch.int32).contiguous()
            assert self.block_table.shape == (batch, n_kv_heads, self.block_table.shape[-1])
            assert self.block_table.shape[-1] >= self.max_blocks
            self.table_blocks = int(self.block_table.shape[-1])
        if n_pool_pages is None:
            n_pool_pages = batch * n_kv_heads * self.table_blocks
        self.params = B.make_params(batch=batch, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, window=window,
                                    keep=keep, dtype=_TDT[dtype], n_pool_pages=n_pool_pages,
                                    token_budget=token_budget, pool_kernel=pool_kernel,
                                    softmax_scale=softmax_scale, flags=flags, keep_v=keep_v, top_p=top_p,
                                    group_prune=group_prune, recovery=recovery, seed=seed)
        self.page_bytes = B.spark_page_bytes(self.params)
        assert self.page_bytes > 0
        self.pages = pages if pages is not None else self._alloc("pages", B.spark_pool_bytes(self.params), zero=True)
        self.qnorm = self._alloc("qnorm", batch * n_kv_heads * 128 * 4).view(torch.float32).view(batch, n_kv_heads, 128)
        self.packed_lens = self._alloc("packed_lens", batch * 4, zero=True).view(torch.int32)
        self.kept_tokens = (self._alloc("kept_tokens", batch * n_kv_heads * token_budget * 4).view(torch.int32)
                            .view(batch, n_kv_heads, token_budget) if token_budget > 0 else None)
        cb, db = B.spark_workspace_bytes(self.params, self.max_src_tokens)
        self.ws_compress = self._alloc("ws_compress", cb)
        self.ws_decode = self._alloc("ws_decode", db)
        B.spark_workspace_init(self.ws_compress)
        B.spark_workspace_init(self.ws_decode)

    # -- buffers ----------------------------------------------------------------------------------
    def _alloc(self, name: str, nbytes: int, zero: bool = False) -> torch.Tensor:
        """A uint8 device buffer of `nbytes`; with guard=True it sits between two canary bands."""
        if not self.guard:
            return (torch.zeros if zero else torch.empty)(nbytes, dtype=torch.uint8, device=self.device)
        raw = torch.full((nbytes + 2 * GUARD_BYTES,), GUARD_VALUE, dtype=torch.uint8, device=self.device)
        payload = raw[GUARD_BYTES:GUARD_BYTES + nbytes]
        if zero:
            payload.zero_()
        self._bands.append((name, raw, nbytes))
        return payload

    def alloc_out(self) -> torch.Tensor:
        p = self.params
        return self._alloc("out", p.batch * p.n_q_heads * 128 * 4).view(torch.float32).view(p.batch, p.n_q_heads, 128)

    def alloc_lse(self) -> torch.Tensor:
        p = self.params
        return self._alloc("lse", p.batch * p.n_q_heads * 4).view(torch.float32).view(p.batch, p.n_q_heads)

    def broken_guards(self):
        """Names of guarded buffers whose canary bands were written to (empty list: all intact)."""
        bad = []
        for name, raw, nbytes in self._bands:
            head, tail = raw[:GUARD_BYTES], raw[GUARD_BYTES + nbytes:]
            if not (bool((head == GUARD_VALUE).all()) and bool((tail == GUARD_VALUE).all())):
                bad.append(name)
        return bad

    # -- the two calls of the method ------------------------------------------------------------
    def compress(self, q_win, k, v, seq_lens) -> None:
        B.spark_compress(self.params, q_win, k, v, seq_lens, self.max_src_tokens, self.pages, self.block_table,
                         self.qnorm, self.packed_lens, self.kept_tokens, self.ws_compress, max_blocks=self.table_blocks)

    def append(self, k_new, v_new) -> None:
        """One new token per sequence ([B, Hkv, D]), pruned with the prefill statistics."""
        B.spark_append(self.params, k_new, v_new, self.pages, self.block_table, self.qnorm, self.packed_lens,
                       self.ws_compress, max_blocks=self.table_blocks)

    def append_block(self, k_new, v_new) -> None:
        """n new tokens per sequence ([B, Hkv, n, D]), each pruned with the prefill statistics."""
        B.spark_append_block(self.params, k_new, v_new, self.pages, self.block_table, self.qnorm, self.packed_lens,
                             self.ws_compress, max_blocks=self.table_blocks)

    def decode(self, q, out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None):
        p = self.params
        if out is None:
            out = self.alloc_out()
        B.spark_decode_attn(p, q, self.pages, self.block_table, self.packed_lens, self.qnorm, out, lse,
                            self.ws_decode, max_blocks=self.table_blocks)
        return out

    def bind_decode(self, q, out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                    stream: Optional[int] = None) -> "B.BoundDecode":
        """The decode step on fixed buffers, marshalled once (for decode loops); call the result to enqueue it."""
        if out is None:
            out = self.alloc_out()
        return B.BoundDecode(self.params, q, self.pages, self.block_table, self.packed_lens, self.qnorm, out, lse,
                             self.ws_decode, max_blocks=self.table_blocks, stream=stream)

    def bind_decode_host(self, q_host, out_host, stream: Optional[int] = None) -> "B.BoundDecodeHost":
        """The decode step for a query and a result in page-locked host tensors (copy-in, step, copy-out in one
        call, nothing synchronised); the device staging buffers are allocated here, once."""
        q_dev = torch.empty(q_host.shape, dtype=q_host.dtype, device=self.device)
        return B.BoundDecodeHost(self.params, q_host, q_dev, self.pages, self.block_table, self.packed_lens,
                                 self.qnorm, self.alloc_out(), out_host, self.ws_decode,
                                 max_blocks=self.table_blocks, stream=stream)

    # -- inspection ------------------------------------------------------------------------------
    def unpack(self, want_vals=True, want_v=True, want_vmask=False, want_stats=False) -> Dict[str, torch.Tensor]:
        p, n = self.params, self.max_tokens
        tdt = _TDT[self.dtype]
        out = dict(mask=torch.empty(p.batch, p.n_kv_heads, n, 4, dtype=torch.int32, device=self.device),
                   mu=torch.empty(p.batch, p.n_kv_heads, n, dtype=torch.float32, device=self.device))
        if want_vals:
            out["vals"] = torch.empty(p.batch, p.n_kv_heads, n, p.keep, dtype=tdt, device=self.device)
        if want_v:
            out["v"] = torch.empty(p.batch, p.n_kv_heads, n, 128, dtype=tdt, device=self.device)
        B.spark_unpack_pages(p, self.pages, self.block_table, self.packed_lens, n, out["mask"], out["mu"],
                             out.get("vals"), out.get("v"), max_blocks=self.table_blocks)
        if want_vmask:
            out["vmask"] = torch.empty(p.batch, p.n_kv_heads, n, 4, dtype=torch.int32, device=self.device)
            B.spark_unpack_value_masks(p, self.pages, self.block_table, self.packed_lens, n, out["vmask"],
                                       max_blocks=self.table_blocks)
        if want_stats:
            out["mu_all"] = torch.empty(p.batch, p.n_kv_heads, n, dtype=torch.float32, device=self.device)
            out["sigma_all"] = torch.empty(p.batch, p.n_kv_heads, n, dtype=torch.float32, device=self.device)
            B.spark_unpack_stats(p, self.pages, self.block_table, self.packed_lens, n, out["mu_all"], out["sigma_all"],
                                 max_blocks=self.table_blocks)
        return out

    def status(self) -> int:
        s = B.spark_read_status(self.ws_compress)
        return s if s else B.spark_read_status(self.ws_decode)

    @property
    def algorithmic_bytes_per_token(self) -> int:
        return B.spark_algorithmic_bytes_per_token(self.params)


class DenseTailCache:
    """A sequence held as a pruned prefix plus a DENSE tail of recently appended tokens.

    The paper appends the keys of generated tokens as they are (K <- Cat[K, k], Sec. "Preliminaries") and prunes
    "during prefill"; this object is that reading.  Appended tokens go, unpruned, into a small second cache whose
    pages keep all 128 channels; every `tail_block` appended tokens the dense copies that this object also keeps
    are handed to the prefix in one spark_append_block call (pruned with the prefill statistics) and the tail
    starts over.  `tail_block=None` never hands them over: the literal "dense appended keys".  A decode step is
    the prefix step, the tail step and their log-sum-exp merge (spark_merge_attn); all arithmetic is in the
    library.
    """

    def __init__(self, *, batch: int, n_q_heads: int, n_kv_heads: int, window: int, keep: int, dtype: str,
                 max_tokens: int, tail_block: Optional[int] = 64, max_tail: int = 1024, device="cuda", **prefix_kw):
        self.block = int(tail_block) if tail_block else None
        cap = self.block if self.block else int(max_tail)
        self.prefix = SparkCache(batch=batch, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, window=window, keep=keep,
                                 dtype=dtype, max_tokens=max_tokens, device=device, **prefix_kw)
        self.tail = SparkCache(batch=batch, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, window=window, keep=128,
                               dtype=dtype, max_tokens=cap, device=device)
        tdt = _TDT[dtype]
        self.k_tail = torch.zeros(batch, n_kv_heads, cap, 128, dtype=tdt, device=device)
        self.v_tail = torch.zeros(batch, n_kv_heads, cap, 128, dtype=tdt, device=device)
        self.n_tail = 0
        p = self.prefix.params
        self._o = [torch.empty(p.batch, p.n_q_heads, 128, dtype=torch.float32, device=device) for _ in range(2)]
        self._l = [torch.empty(p.batch, p.n_q_heads, dtype=torch.float32, device=device) for _ in range(2)]

    def compress(self, q_win, k, v, seq_lens) -> None:
        self.prefix.compress(q_win, k, v, seq_lens)
        self.tail.qnorm.copy_(self.prefix.qnorm)           # the tail is dense: qnorm only has to be a valid divisor
        self.tail.packed_lens.zero_()
        self.n_tail = 0

    def append(self, k_new, v_new) -> None:
        """One new token per sequence ([B, Hkv, D]); it stays dense until its block is handed to the prefix."""
        self.tail.append(k_new, v_new)
        self.k_tail[:, :, self.n_tail].copy_(k_new)
        self.v_tail[:, :, self.n_tail].copy_(v_new)
        self.n_tail += 1
        if self.block and self.n_tail == self.block:
            self.prefix.append_block(self.k_tail, self.v_tail)
            self.tail.packed_lens.zero_()
            self.n_tail = 0

    def decode(self, q, out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None):
        if out is None:
            out = torch.empty_like(self._o[0])
        self.prefix.decode(q, out=self._o[0], lse=self._l[0])
        self.tail.decode(q, out=self._o[1], lse=self._l[1])
        B.spark_merge_attn(self._o[0], self._l[0], self._o[1], self._l[1], out, lse)
        return out

    def status(self) -> int:
        s = self.prefix.status()
        return s if s else self.tail.status()
