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

from test_gpu_parity import built, check_case, make                      # noqa: F401  (fixture + helpers)
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
