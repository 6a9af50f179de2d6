"""The allocation-free decode entry point against the regular one.

spark_decode_attn_noalloc serves callers that are handed device tensors but may not allocate (no
workspace to pass): it runs the same kernels on a scratch array built into the library.  The check: on
the same packed cache its output equals the regular entry point's AND the CPU oracle's (same tolerance as
the parity tests), on two calls in a row (the second call finds the scratch as the first left it), and
problems beyond the built-in scratch are refused before anything is launched.  Collected last on purpose.
"""
import numpy as np
import pytest
import torch

import oracle

from paper_2508_15212_b200 import binding as B
from paper_2508_15212_b200 import build as spark_build
from paper_2508_15212_b200.cache import SparkCache
from workloads import inputs

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 2e-3}


@pytest.fixture(scope="module", autouse=True)
def built():
    spark_build.build()
    B.lib()


@pytest.mark.parametrize("dtype,Bn,Hq,Hkv,lens,keep,keep_v", [
    ("bf16", 2, 16, 4, [2100, 333], 64, 0),     # several CTAs share a unit: partials and tickets in use
    ("bf16", 1, 28, 4, [5000], 38, 0),
    ("f32", 2, 4, 2, [700, 64], 25, 0),
    ("bf16", 2, 16, 4, [2100, 333], 64, 64),    # pruned value rows
])
def test_noalloc_matches_regular_entry_point_twice(dtype, Bn, Hq, Hkv, lens, keep, keep_v):
    wl = inputs.make_workload(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, seq_lens=lens, window=16, dtype=dtype,
                              sigma_s=1.0 if dtype == "bf16" else 0.5, seed=321, device="cuda")
    # one case with an explicit block table, the others contiguous (no table)
    table = B.identity_block_table(Bn, Hkv, (max(lens) + 15) // 16, "cuda") if keep == 38 else None
    cache = SparkCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, window=16, keep=keep, dtype=dtype,
                       max_tokens=max(lens), keep_v=keep_v, block_table=table)
    cache.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
    lse_ref = torch.empty(Bn, Hq, dtype=torch.float32, device="cuda")
    ref = cache.decode(wl.q, lse=lse_ref)
    assert cache.status() == 0
    # the oracle on the same inputs: an error common to both entry points cannot pass
    wl_cpu = wl.to("cpu")
    _, a = oracle.window_mean(wl_cpu.q_win, Hkv)
    c = oracle.compress(wl_cpu.k, wl_cpu.seq_lens, keep, a)
    vm = oracle.prune_values(wl_cpu.v, wl_cpu.seq_lens, keep_v) if 0 < keep_v < 128 else None
    o_ref, l_ref = oracle.decode_attn(wl_cpu.q, wl_cpu.k, wl_cpu.v, wl_cpu.seq_lens, c["mask"], c["mu"], a, vmask=vm)
    for call in range(2):
        out = torch.full((Bn, Hq, 128), float("nan"), dtype=torch.float32, device="cuda")
        lse = torch.full((Bn, Hq), float("nan"), dtype=torch.float32, device="cuda")
        B.spark_decode_attn_noalloc(cache.params, wl.q, cache.pages, cache.block_table, cache.packed_lens,
                                    cache.qnorm, out, lse, max_blocks=cache.table_blocks)
        torch.cuda.synchronize()
        d = float((out - ref).abs().max())
        assert d <= TOL[dtype], f"call {call}: max|delta| {d:.3e}"
        assert float((lse - lse_ref).abs().max()) <= 1e-3
        d = float(np.abs(out.cpu().numpy() - o_ref).max())
        assert d <= TOL[dtype], f"call {call}: max|delta| vs oracle {d:.3e}"
        assert float(np.abs(lse.cpu().numpy() - l_ref).max()) <= (1e-3 if dtype == "bf16" else 2e-5)


def test_noalloc_refuses_problems_beyond_its_scratch():
    p = B.make_params(batch=65, n_q_heads=4, n_kv_heads=1, window=4, keep=64, dtype=torch.bfloat16,
                      n_pool_pages=65)
    dummy = torch.zeros(1 << 12, dtype=torch.uint8, device="cuda")
    bt = torch.zeros(65, 1, 1, dtype=torch.int32, device="cuda")
    with pytest.raises(B.SparkError) as e:
        B.spark_decode_attn_noalloc(p, dummy, dummy, bt, dummy, dummy, dummy, None)
    assert e.value.code == 4            # SPARK_ERR_WORKSPACE, nothing launched
