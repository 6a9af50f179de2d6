"""The seeded generators: determinism, value structure, and the conditioning the benchmark asks for."""
import math
import numpy as np
import torch

import oracle
from workloads import inputs


def small(seed=0, dtype="bf16", **kw):
    args = dict(batch=2, n_q_heads=8, n_kv_heads=2, head_dim=128, seq_lens=[96, 50], window=8,
                dtype=dtype, sigma_s=1.0, seed=seed)
    args.update(kw)
    return inputs.make_workload(**args)


def test_same_seed_same_bytes_other_seed_other_bytes():
    a, b, c = small(3), small(3), small(4)
    assert torch.equal(a.k.view(torch.int16), b.k.view(torch.int16))
    assert torch.equal(a.q_win.view(torch.int16), b.q_win.view(torch.int16))
    assert not torch.equal(a.k.view(torch.int16), c.k.view(torch.int16))
    assert a.k.dtype == torch.bfloat16 and a.seq_lens.tolist() == [96, 50]


def test_outlier_key_channels_and_window_mean_floor():
    wl = small(5, seq_lens=[4096, 4096])
    rms = wl.k.float().pow(2).mean(dim=2).sqrt()                  # [B,Hkv,D]
    ratio = rms.max(dim=-1).values / rms.median(dim=-1).values
    assert (ratio > 4).all()                                      # a few channels dominate
    qbar, a = oracle.window_mean(wl.q_win, 2)
    assert (np.abs(qbar) > 1e-3).all()


def test_saliency_gap_is_enforced_as_seen_by_the_oracle():
    for dtype, keep in (("bf16", 64), ("f32", 25)):
        wl = small(6, dtype=dtype)
        inputs.enforce_saliency_gap(wl, keep)
        _, a = oracle.window_mean(wl.q_win, 2)
        c = oracle.compress(wl.k, wl.seq_lens, keep, a, want_saliency=True)
        for b, n in enumerate(wl.seq_lens.tolist()):
            w = np.sort(c["saliency"][b, :, :n], axis=-1)[..., ::-1]
            wT, wN = w[..., keep - 1], w[..., keep]
            assert ((wT - wN) >= 2.0 ** -7 * wT).all()


def test_config_table_shapes():
    assert len(inputs.CONFIGS) == 5
    wl = inputs.config_workload(0)
    assert wl.shape == (1, 1, 1, 32, 128, 1024) and wl.dtype == "f32"
    wl = inputs.config_workload(4, batch=3, seed_offset=1, seq_lens=[40, 17, 33])
    assert wl.shape[:5] == (3, 28, 4, 32, 128)
    c5 = inputs.config_workload.__globals__["CONFIGS"][4]
    assert [int(math.floor((1.0 - r) * 128 + 1e-9)) for r in c5["ratio"]] == [89, 64, 38, 25]
