"""Seeded synthetic workloads for the SparK hot path.

This module serves both the CPU oracle and the CUDA path with identical bytes.
It draws tensors with the structure the paper reports for key/query
activations (strong per-channel magnitude differences, a few outlier key
channels, token-dependent saliency; Sec. "Motivations and Observations" and the
heat maps of App. "Observations") at the attention shapes of the benchmark
configurations.  Nothing here packs, scores or attends.

Two conditioning steps look at the data they produce, because the benchmark
definition asks for them:

* ``_floor_window_mean``  redraws window-query columns whose mean is close to
  zero, so the recovery divisor |q-bar_j| (Sec. "Channel Recovery") stays away
  from 0;
* ``enforce_saliency_gap`` nudges a key entry wherever the T-th and (T+1)-th
  largest saliencies of a token (Sec. "Problem Formulation", w = |q-bar_j| |k_j|)
  are closer than a relative gap, so that top-T selection has no near-ties.

Both are written directly with torch ops and share no code with ``oracle/`` or
with the CUDA sources.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional, Sequence, Union

import torch

_DTYPES = {"f32": torch.float32, "bf16": torch.bfloat16}


@dataclasses.dataclass
class Workload:
    """One batch of attention-layer tensors in the storage dtype."""

    q_win: torch.Tensor      # [B, Hq, W, D]   observation-window queries
    k: torch.Tensor          # [B, Hkv, S_max, D]
    v: torch.Tensor          # [B, Hkv, S_max, D]
    q: torch.Tensor          # [B, Hq, D]      one decode query per sequence
    seq_lens: torch.Tensor   # [B] int32
    dtype: str               # "f32" | "bf16"
    meta: Dict[str, object]

    @property
    def shape(self):
        B, Hq, W, D = self.q_win.shape
        return B, Hq, self.k.shape[1], W, D, self.k.shape[2]

    def to(self, device) -> "Workload":
        return dataclasses.replace(
            self,
            q_win=self.q_win.to(device), k=self.k.to(device), v=self.v.to(device),
            q=self.q.to(device), seq_lens=self.seq_lens.to(device))


def _lognormal(gen, shape, sigma, device):
    z = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    return torch.exp(sigma * z)


def _floor_window_mean(q_win, scale_q, G, gen, floor_rel=0.05, max_tries=64):
    """Redraw window columns whose pooled mean over the G*W group queries is small."""
    B, Hq, W, D = q_win.shape
    Hkv = Hq // G
    for _ in range(max_tries):
        grp = q_win.view(B, Hkv, G, W, D).double()
        qbar = grp.mean(dim=(2, 3))                                    # [B,Hkv,D]
        ref = scale_q.view(1, Hkv, G, D).double().mean(dim=2)          # [1,Hkv,D]
        bad = qbar.abs() < floor_rel * ref                             # [B,Hkv,D]
        if not bool(bad.any()):
            return q_win
        z = torch.randn(q_win.shape, generator=gen, device=q_win.device, dtype=torch.float32)
        fresh = z * scale_q.view(1, Hq, 1, D)
        sel = bad.view(B, Hkv, 1, 1, D).expand(B, Hkv, G, W, D).reshape(B, Hq, W, D)
        q_win = torch.where(sel, fresh, q_win)
    raise RuntimeError("window-mean floor not reached")


def make_workload(*, batch: int, n_q_heads: int, n_kv_heads: int, head_dim: int = 128,
                  seq_lens: Union[int, Sequence[int]], window: int, dtype: str = "bf16",
                  sigma_s: float = 1.0, n_outliers: int = 4, outlier_gain: float = 8.0,
                  seed: int = 0, device: str = "cpu") -> Workload:
    """Draw Q_win, K, V, q.

    X[..., j] = z * scale_X[head][j], z ~ N(0,1), scale ~ LogNormal(0, sigma_s)
    drawn per tensor and per head; ``n_outliers`` random key channels per KV head
    are multiplied by ``outlier_gain``.  The decode query shares its head's
    window-query scales.  Everything is rounded to the storage dtype before use.
    """
    assert n_q_heads % n_kv_heads == 0
    B, Hq, Hkv, D, W = batch, n_q_heads, n_kv_heads, head_dim, window
    G = Hq // Hkv
    lens = [int(seq_lens)] * B if isinstance(seq_lens, int) else [int(x) for x in seq_lens]
    assert len(lens) == B
    S_max = max(max(lens), 1)
    tdt = _DTYPES[dtype]
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))

    scale_q = _lognormal(gen, (Hq, D), sigma_s, device)
    scale_k = _lognormal(gen, (B, Hkv, D), sigma_s, device)
    scale_v = _lognormal(gen, (B, Hkv, D), sigma_s, device)
    # outlier key channels: the first n_outliers entries of a random permutation
    if n_outliers > 0:
        perm = torch.rand((B, Hkv, D), generator=gen, device=device).argsort(dim=-1)
        out_idx = perm[..., :n_outliers]
        gain = torch.ones((B, Hkv, D), device=device)
        gain.scatter_(-1, out_idx, outlier_gain)
        scale_k = scale_k * gain

    q_win = torch.randn((B, Hq, W, D), generator=gen, device=device) * scale_q.view(1, Hq, 1, D)
    q_win = _floor_window_mean(q_win, scale_q, G, gen)
    k = torch.empty((B, Hkv, S_max, D), device=device, dtype=tdt)
    v = torch.empty((B, Hkv, S_max, D), device=device, dtype=tdt)
    for b in range(B):          # per sequence, to bound the fp32 temporaries
        zk = torch.randn((Hkv, S_max, D), generator=gen, device=device)
        k[b] = (zk * scale_k[b].view(Hkv, 1, D)).to(tdt)
        del zk
        zv = torch.randn((Hkv, S_max, D), generator=gen, device=device)
        v[b] = (zv * scale_v[b].view(Hkv, 1, D)).to(tdt)
        del zv
    q = torch.randn((B, Hq, D), generator=gen, device=device) * scale_q.view(1, Hq, D)

    return Workload(q_win=q_win.to(tdt), k=k, v=v, q=q.to(tdt),
                    seq_lens=torch.tensor(lens, dtype=torch.int32, device=device),
                    dtype=dtype,
                    meta=dict(batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, window=W,
                              sigma_s=sigma_s, seed=seed, seq_lens=lens))


def enforce_saliency_gap(wl: Workload, keep: int, rel_gap: float = 2.0 ** -6,
                         bump: float = 1.0 + 2.0 ** -4, max_rounds: int = 16,
                         qnorm_eps: float = 1e-12) -> int:
    """Make every token's T-th and (T+1)-th largest saliency differ by > rel_gap.

    Saliency here is |mean window query|_j * |K[t][j]| with the mean pooled over
    the G*W queries that share the KV head.  Where the gap is too small the key
    entry holding the T-th largest saliency is multiplied by ``bump`` in the
    storage dtype, and the check repeats.  Modifies ``wl.k`` in place and returns
    the number of entries changed.  No-op when keep == head_dim.
    """
    B, Hq, Hkv, W, D, S_max = wl.shape
    if keep >= D:
        return 0
    G = Hq // Hkv
    grp = wl.q_win.view(B, Hkv, G, W, D).double()
    a = grp.mean(dim=(2, 3)).float().abs().clamp_min(qnorm_eps)       # [B,Hkv,D]
    changed = 0
    for b in range(B):
        for h in range(Hkv):
            kk = wl.k[b, h]                                            # [S_max, D] view
            for _ in range(max_rounds):
                w = a[b, h].view(1, D) * kk.float().abs()
                top, idx = torch.topk(w, keep + 1, dim=-1, sorted=True)
                wT, wN = top[:, keep - 1], top[:, keep]
                close = (wT - wN) < rel_gap * wT
                n = int(close.sum())
                if n == 0:
                    break
                rows = close.nonzero(as_tuple=True)[0]
                cols = idx[rows, keep - 1]
                kk[rows, cols] = (kk[rows, cols].float() * bump).to(kk.dtype)
                changed += n
            else:
                raise RuntimeError("saliency gap not reached")
    return changed


# --------------------------------------------------------------------------------------
# The benchmark configurations (shapes, lengths and value structure of BASELINE configs).
# --------------------------------------------------------------------------------------

CONFIGS: List[Dict[str, object]] = [
    dict(name="tiny_fp32", batch=1, n_q_heads=1, n_kv_heads=1, head_dim=128, seq_lens=1024,
         window=32, dtype="f32", sigma_s=0.5, ratio=0.5, seed=0),
    dict(name="llama8b_32k", batch=1, n_q_heads=32, n_kv_heads=8, head_dim=128, seq_lens=32768,
         window=32, dtype="bf16", sigma_s=1.0, ratio=0.5, seed=2),
    dict(name="llama8b_4x128k", batch=4, n_q_heads=32, n_kv_heads=8, head_dim=128, seq_lens=131072,
         window=64, dtype="bf16", sigma_s=1.0, ratio=0.8, seed=3),
    dict(name="llama8b_evict2048_b32", batch=32, n_q_heads=32, n_kv_heads=8, head_dim=128,
         seq_lens=131072, window=32, dtype="bf16", sigma_s=1.0, ratio=0.5, seed=4,
         token_budget=2048, pool_kernel=7),
    dict(name="qwen7b_paged_b16", batch=16, n_q_heads=28, n_kv_heads=4, head_dim=128,
         seq_lens=("uniform", 8192, 131072), window=32, dtype="bf16", sigma_s=1.0,
         ratio=(0.3, 0.5, 0.7, 0.8), seed=5, n_layers=28),
]


def config_workload(index: int, device: str = "cpu", *, seq_lens=None, batch=None,
                    seed_offset: int = 0) -> Workload:
    """Build the workload of benchmark configuration ``index`` (0-based).

    ``seq_lens`` / ``batch`` shrink the configuration for parity slices; the
    value structure (scales, outliers, dtype, heads) stays that of the config.
    """
    c = dict(CONFIGS[index])
    B = int(batch if batch is not None else c["batch"])
    sl = seq_lens if seq_lens is not None else c["seq_lens"]
    if isinstance(sl, tuple) and sl[0] == "uniform":
        g = torch.Generator().manual_seed(int(c["seed"]) + 7919 * seed_offset)
        sl = torch.randint(int(sl[1]), int(sl[2]) + 1, (B,), generator=g).tolist()
    return make_workload(batch=B, n_q_heads=c["n_q_heads"], n_kv_heads=c["n_kv_heads"],
                         head_dim=c["head_dim"], seq_lens=sl, window=c["window"],
                         dtype=c["dtype"], sigma_s=c["sigma_s"],
                         seed=int(c["seed"]) + 1000003 * seed_offset, device=device)
