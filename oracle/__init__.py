"""Python face of the SparK CPU oracle -- TEST INFRASTRUCTURE, NOT A PRODUCT PATH.

Compiles ``spark_oracle.c`` with gcc (no CUDA, no code shared with the CUDA
library) and exposes its functions on host arrays.  Only the tests, the smoke
check and the benchmark's cpu_baseline / reference arm may import this package.

Tensors may be numpy arrays or CPU torch tensors; bf16 is carried as the raw
16-bit pattern.  Layouts are logical (unpaged): K/V ``[B, Hkv, S, D]`` (or any
layout with a contiguous last axis, described by strides), masks
``[B, Hkv, S, ceil(D/32)]`` uint32, statistics ``[B, Hkv, S]`` float32.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spark_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None

F32, BF16 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc; returns the library path."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-fopenmp",
           "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_threads.restype = ctypes.c_int
    return _lib


def threads() -> int:
    return int(lib().oracle_threads())


# ------------------------------------------------------------------ array plumbing
def _as_np(x) -> Tuple[np.ndarray, int]:
    """Return (array, dtype code); bf16 torch tensors become uint16 arrays."""
    try:
        import torch
        if isinstance(x, torch.Tensor):
            x = x.detach().cpu()
            if x.dtype == torch.bfloat16:
                return x.view(torch.int16).numpy().view(np.uint16), BF16
            return x.numpy(), F32 if x.dtype == torch.float32 else -1
    except ImportError:
        pass
    x = np.asarray(x)
    if x.dtype == np.uint16:
        return x, BF16
    if x.dtype == np.float32:
        return x, F32
    return x, -1


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _kv_strides(k: np.ndarray) -> Tuple[int, int, int]:
    assert k.ndim == 4 and k.strides[-1] == k.itemsize, "last axis must be contiguous"
    return tuple(int(s // k.itemsize) for s in k.strides[:3])


def _i32(x) -> np.ndarray:
    try:
        import torch
        if isinstance(x, torch.Tensor):
            x = x.detach().cpu().numpy()
    except ImportError:
        pass
    return np.ascontiguousarray(np.asarray(x, dtype=np.int32))


# ------------------------------------------------------------------ oracle calls
def window_mean(q_win, n_kv_heads: int, eps: float = 1e-12):
    """Sec. "SparK": pooled mean window query and a = max(|q-bar|, eps).  -> (qbar, a)"""
    q, dt = _as_np(q_win)
    q = np.ascontiguousarray(q)
    B, Hq, W, D = q.shape
    qbar = np.empty((B, n_kv_heads, D), np.float32)
    a = np.empty((B, n_kv_heads, D), np.float32)
    rc = lib().oracle_window_mean(_ptr(q), dt, B, Hq, n_kv_heads, W, D, ctypes.c_float(eps),
                                  _ptr(qbar), _ptr(a))
    assert rc == 0, rc
    return qbar, a


def compress(k, seq_lens, keep: int, a, *, want_idx=False, want_saliency=False, want_stats=False):
    """Eq. (cal) top-T selection per token.  -> dict(mask, mu[, kept_idx, saliency, mu_all, sigma_all])"""
    kk, dt = _as_np(k)
    B, Hkv, S, D = kk.shape
    sb, sh, st = _kv_strides(kk)
    lens = _i32(seq_lens)
    a = np.ascontiguousarray(a, dtype=np.float32)
    MW = (D + 31) // 32
    mask = np.empty((B, Hkv, S, MW), np.uint32)
    mu = np.empty((B, Hkv, S), np.float32)
    idx = np.empty((B, Hkv, S, keep), np.int32) if want_idx else None
    sal = np.empty((B, Hkv, S, D), np.float32) if want_saliency else None
    mu_all = np.empty((B, Hkv, S), np.float32) if want_stats else None
    sg_all = np.empty((B, Hkv, S), np.float32) if want_stats else None
    rc = lib().oracle_compress(_ptr(kk), dt, B, Hkv, D, ctypes.c_int64(sb), ctypes.c_int64(sh),
                               ctypes.c_int64(st), _ptr(lens), S, int(keep), _ptr(a), _ptr(mask),
                               _ptr(mu), _ptr(idx), _ptr(sal), _ptr(mu_all), _ptr(sg_all))
    assert rc == 0, rc
    out = dict(mask=mask, mu=mu)
    if want_idx:
        out["kept_idx"] = idx
    if want_saliency:
        out["saliency"] = sal
    if want_stats:
        out["mu_all"], out["sigma_all"] = mu_all, sg_all
    return out


def prune_values(v, seq_lens, keep_v: int):
    """App. "Pruning Value Cache Channels": per-token top-T_v value channels by magnitude.  -> vmask"""
    vv, dt = _as_np(v)
    B, Hkv, S, D = vv.shape
    sb, sh, st = _kv_strides(vv)
    lens = _i32(seq_lens)
    vmask = np.empty((B, Hkv, S, (D + 31) // 32), np.uint32)
    rc = lib().oracle_prune_values(_ptr(vv), dt, B, Hkv, D, ctypes.c_int64(sb), ctypes.c_int64(sh),
                                   ctypes.c_int64(st), _ptr(lens), S, int(keep_v), _ptr(vmask))
    assert rc == 0, rc
    return vmask


def decode_attn(q, k, v, lens, mask, mu, a, *, scale: float = 0.0, path: int = 0,
                want_scores: bool = False, vmask=None):
    """Sec. "Channel Recovery" + softmax attention.  -> (out [B,Hq,D] f32, lse [B,Hq] f32[, scores])"""
    qq, dtq = _as_np(q)
    kk, dt = _as_np(k)
    vv, dtv = _as_np(v)
    assert dtq == dt == dtv
    qq = np.ascontiguousarray(qq)
    B, Hkv, S, D = kk.shape
    Hq = qq.shape[1]
    sb, sh, st = _kv_strides(kk)
    assert _kv_strides(vv) == (sb, sh, st)
    lens = _i32(lens)
    mask = np.ascontiguousarray(mask, dtype=np.uint32)
    mu = np.ascontiguousarray(mu, dtype=np.float32)
    a = np.ascontiguousarray(a, dtype=np.float32)
    assert mask.shape[:3] == (B, Hkv, S) and mu.shape == (B, Hkv, S)
    out = np.empty((B, Hq, D), np.float32)
    lse = np.empty((B, Hq), np.float32)
    scores = np.zeros((B, Hq, S), np.float64) if want_scores else None
    if vmask is not None:
        vmask = np.ascontiguousarray(vmask, dtype=np.uint32)
        assert vmask.shape == mask.shape
    rc = lib().oracle_decode_attn(_ptr(qq), _ptr(kk), _ptr(vv), dt, B, Hq, Hkv, D,
                                  ctypes.c_int64(sb), ctypes.c_int64(sh), ctypes.c_int64(st),
                                  _ptr(lens), S, _ptr(mask), _ptr(mu), _ptr(a),
                                  ctypes.c_double(scale), int(path), _ptr(out), _ptr(lse),
                                  _ptr(scores), _ptr(vmask))
    assert rc == 0, rc
    return (out, lse, scores) if want_scores else (out, lse)


def evict(q_win, k, seq_lens, budget: int, pool: int = 7, *, want_votes: bool = False):
    """Benchmark eviction rule (parity unpinned against the paper).  -> (kept_tok, out_len[, vote, pooled])"""
    q, dtq = _as_np(q_win)
    kk, dt = _as_np(k)
    assert dtq == dt
    q = np.ascontiguousarray(q)
    B, Hq, W, D = q.shape
    Hkv, S = kk.shape[1], kk.shape[2]
    sb, sh, st = _kv_strides(kk)
    lens = _i32(seq_lens)
    kept = np.empty((B, Hkv, budget), np.int32)
    out_len = np.empty((B,), np.int32)
    vote = np.zeros((B, Hkv, S), np.float64) if want_votes else None
    pooled = np.zeros((B, Hkv, S), np.float64) if want_votes else None
    rc = lib().oracle_evict(_ptr(q), _ptr(kk), dt, B, Hq, Hkv, W, D, ctypes.c_int64(sb),
                            ctypes.c_int64(sh), ctypes.c_int64(st), _ptr(lens), S, int(budget),
                            int(pool), _ptr(kept), _ptr(out_len), _ptr(vote), _ptr(pooled))
    assert rc == 0, rc
    return (kept, out_len, vote, pooled) if want_votes else (kept, out_len)


def select_variant(k, seq_lens, a, *, top_p: float = None, cap: int = None, group_prune=None, want_stats=False):
    """Adaptive selection (Sec. "Ablation Studies"): SparK-p when `top_p` is given (at most `cap` channels),
    SparK-g when `group_prune` (ratios from the most salient rank group to the least) is given.
    -> dict(mask, mu, count[, mu_all, sigma_all])"""
    kk, dt = _as_np(k)
    B, Hkv, S, D = kk.shape
    sb, sh, st = _kv_strides(kk)
    lens = _i32(seq_lens)
    a = np.ascontiguousarray(a, dtype=np.float32)
    MW = (D + 31) // 32
    mask = np.empty((B, Hkv, S, MW), np.uint32)
    mu = np.empty((B, Hkv, S), np.float32)
    count = np.empty((B, Hkv, S), np.int32)
    mu_all = np.empty((B, Hkv, S), np.float32) if want_stats else None
    sg_all = np.empty((B, Hkv, S), np.float32) if want_stats else None
    assert (top_p is None) != (group_prune is None)
    if top_p is not None:
        variant, n_groups, prune = 1, 0, None
        cap = D if cap is None else int(cap)
    else:
        variant, top_p, cap = 2, 0.0, D
        prune = np.ascontiguousarray(group_prune, dtype=np.float32)
        n_groups = int(prune.size)
    rc = lib().oracle_select_variant(_ptr(kk), dt, B, Hkv, D, ctypes.c_int64(sb), ctypes.c_int64(sh),
                                     ctypes.c_int64(st), _ptr(lens), S, _ptr(a), variant,
                                     ctypes.c_float(top_p), int(cap), n_groups, _ptr(prune), _ptr(mask),
                                     _ptr(mu), _ptr(count), _ptr(mu_all), _ptr(sg_all))
    assert rc == 0, rc
    out = dict(mask=mask, mu=mu, count=count)
    if want_stats:
        out["mu_all"], out["sigma_all"] = mu_all, sg_all
    return out


def draw_uniforms(seed: int, unit: int, t: int, j: int):
    """The two 24-bit uniforms of the sampled-recovery draw of entry (unit, t, j)."""
    u1, u2 = ctypes.c_double(0), ctypes.c_double(0)
    lib().oracle_draw_uniforms(ctypes.c_uint32(seed), ctypes.c_int64(unit), ctypes.c_int64(t), int(j),
                               ctypes.byref(u1), ctypes.byref(u2))
    return u1.value, u2.value


def decode_attn_sampled(q, k, v, lens, mask, mu_all, sigma_all, a, *, mode: int, seed: int, scale: float = 0.0,
                        want_recovered: bool = False):
    """Sec. "Channel Recovery" with a Gaussian (mode 1) or Exponential (mode 2) recovery distribution.
    -> (out, lse[, recovered saliencies [B,Hkv,S,D] float64])"""
    qq, dtq = _as_np(q)
    kk, dt = _as_np(k)
    vv, dtv = _as_np(v)
    assert dtq == dt == dtv
    qq = np.ascontiguousarray(qq)
    B, Hkv, S, D = kk.shape
    Hq = qq.shape[1]
    sb, sh, st = _kv_strides(kk)
    assert _kv_strides(vv) == (sb, sh, st)
    lens = _i32(lens)
    mask = np.ascontiguousarray(mask, dtype=np.uint32)
    mu_all = np.ascontiguousarray(mu_all, dtype=np.float32)
    sigma_all = None if sigma_all is None else np.ascontiguousarray(sigma_all, dtype=np.float32)
    a = np.ascontiguousarray(a, dtype=np.float32)
    out = np.empty((B, Hq, D), np.float32)
    lse = np.empty((B, Hq), np.float32)
    rec = np.zeros((B, Hkv, S, D), np.float64) if want_recovered else None
    rc = lib().oracle_decode_attn_sampled(_ptr(qq), _ptr(kk), _ptr(vv), dt, B, Hq, Hkv, D,
                                          ctypes.c_int64(sb), ctypes.c_int64(sh), ctypes.c_int64(st),
                                          _ptr(lens), S, _ptr(mask), _ptr(mu_all), _ptr(sigma_all), _ptr(a),
                                          ctypes.c_double(scale), int(mode), ctypes.c_uint32(seed),
                                          _ptr(out), _ptr(lse), _ptr(rec))
    assert rc == 0, rc
    return (out, lse, rec) if want_recovered else (out, lse)
