"""ctypes binding of ``libspark.so`` -- same names as ``include/spark.h``, argument marshalling only.

Every step of the hot path runs in the library's CUDA kernels; PyTorch supplies device memory and the
stream.  There is no fallback: if the library is missing the import of a function fails loudly.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspark.so")

SPARK_OK = 0
STATUS_NAMES = {0: "SPARK_OK", 1: "SPARK_ERR_NULL", 2: "SPARK_ERR_BAD_SHAPE", 3: "SPARK_ERR_UNSUPPORTED",
                4: "SPARK_ERR_WORKSPACE", 5: "SPARK_ERR_CUDA", 6: "SPARK_ERR_DEVICE_BOUNDS",
                7: "SPARK_ERR_DEVICE_TIMEOUT"}
SPARK_F32, SPARK_BF16 = 0, 1
_DTYPE_CODE = {torch.float32: SPARK_F32, torch.bfloat16: SPARK_BF16}
EXPORTS = ["spark_version", "spark_last_launch_count", "spark_keep_count", "spark_page_bytes", "spark_pool_bytes",
           "spark_algorithmic_bytes_per_token", "spark_workspace_bytes", "spark_workspace_init",
           "spark_compress", "spark_append", "spark_append_block", "spark_merge_attn", "spark_decode_attn", "spark_decode_attn_host", "spark_decode_attn_noalloc", "spark_unpack_pages",
           "spark_unpack_value_masks", "spark_unpack_stats", "spark_group_keep", "spark_read_status"]


class SparkError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where}: {STATUS_NAMES.get(code, code)}")
        self.code = code


class spark_params(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("window", ctypes.c_int32), ("keep", ctypes.c_int32),
                ("page_tokens", ctypes.c_int32), ("dtype", ctypes.c_int32), ("token_budget", ctypes.c_int32),
                ("pool_kernel", ctypes.c_int32), ("qnorm_eps", ctypes.c_float),
                ("softmax_scale", ctypes.c_float), ("n_pool_pages", ctypes.c_int64),
                ("flags", ctypes.c_int32), ("keep_v", ctypes.c_int32),
                ("select", ctypes.c_int32), ("top_p", ctypes.c_float), ("n_groups", ctypes.c_int32),
                ("group_prune", ctypes.c_float * 8), ("recovery", ctypes.c_int32), ("seed", ctypes.c_uint32)]


SPARK_FLAG_OVERLAP_PREVIOUS = 1
SPARK_FLAG_HOST_MAPPED = 2
SPARK_SELECT_FIXED, SPARK_SELECT_TOP_P, SPARK_SELECT_GROUPS = 0, 1, 2
SPARK_RECOVER_DEGENERATE, SPARK_RECOVER_GAUSSIAN, SPARK_RECOVER_EXPONENTIAL = 0, 1, 2


_lib = None


def lib() -> ctypes.CDLL:
    """Load the library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2508_15212_b200.build`; "
                               "there is no fallback path")
        L = ctypes.CDLL(LIB_PATH)
        P, vp, i32, i64, sz = ctypes.POINTER(spark_params), ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
        L.spark_version.restype = i32
        L.spark_last_launch_count.restype = i32
        L.spark_keep_count.restype = i32
        L.spark_keep_count.argtypes = [i32, ctypes.c_double]
        L.spark_page_bytes.restype = sz
        L.spark_page_bytes.argtypes = [P]
        L.spark_pool_bytes.restype = sz
        L.spark_pool_bytes.argtypes = [P]
        L.spark_algorithmic_bytes_per_token.restype = sz
        L.spark_algorithmic_bytes_per_token.argtypes = [P]
        L.spark_workspace_bytes.restype = i32
        L.spark_workspace_bytes.argtypes = [P, i64, ctypes.POINTER(sz), ctypes.POINTER(sz)]
        L.spark_workspace_init.restype = i32
        L.spark_workspace_init.argtypes = [vp, sz, vp]
        L.spark_compress.restype = i32
        L.spark_compress.argtypes = [P, vp, vp, vp, i64, i64, i64, vp, i32, vp, vp, i32, vp, vp, vp, vp, sz, vp]
        L.spark_append.restype = i32
        L.spark_append.argtypes = [P, vp, vp, vp, vp, i32, vp, vp, vp, sz, vp]
        L.spark_append_block.restype = i32
        L.spark_append_block.argtypes = [P, vp, vp, i32, vp, vp, i32, vp, vp, vp, sz, vp]
        L.spark_merge_attn.restype = i32
        L.spark_merge_attn.argtypes = [i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
        L.spark_decode_attn.restype = i32
        L.spark_decode_attn.argtypes = [P, vp, vp, vp, i32, vp, vp, vp, vp, vp, sz, vp]
        L.spark_decode_attn_host.restype = i32
        L.spark_decode_attn_host.argtypes = [P, vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.spark_decode_attn_noalloc.restype = i32
        L.spark_decode_attn_noalloc.argtypes = [P, vp, vp, vp, i32, vp, vp, vp, vp, vp]
        L.spark_unpack_pages.restype = i32
        L.spark_unpack_pages.argtypes = [P, vp, vp, i32, vp, i32, vp, vp, vp, vp, vp]
        L.spark_unpack_value_masks.restype = i32
        L.spark_unpack_value_masks.argtypes = [P, vp, vp, i32, vp, i32, vp, vp]
        L.spark_unpack_stats.restype = i32
        L.spark_unpack_stats.argtypes = [P, vp, vp, i32, vp, i32, vp, vp, vp]
        L.spark_group_keep.restype = i32
        L.spark_group_keep.argtypes = [i32, i32, ctypes.POINTER(ctypes.c_float)]
        L.spark_read_status.restype = i32
        L.spark_read_status.argtypes = [vp, vp]
        _lib = L
    return _lib


def _check(code: int, where: str) -> None:
    if code != SPARK_OK:
        raise SparkError(code, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _blocks(block_table, max_blocks) -> int:
    """Table width: the table's last dimension, or `max_blocks` for a contiguous cache (no table)."""
    if block_table is not None:
        return int(block_table.shape[-1])
    assert max_blocks is not None, "a contiguous cache (block_table=None) needs max_blocks"
    return int(max_blocks)


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_params(*, batch, n_q_heads, n_kv_heads, window, keep, dtype, n_pool_pages, head_dim=128,
                page_tokens=16, token_budget=0, pool_kernel=7, qnorm_eps=0.0, softmax_scale=0.0,
                flags=0, keep_v=0, top_p=None, group_prune=None, recovery=0, seed=0) -> spark_params:
    """A parameter block.  `top_p` selects SparK-p, `group_prune` (ratios, most salient rank group first)
    selects SparK-g; `keep` is then the capacity of a token's slot list."""
    code = dtype if isinstance(dtype, int) else _DTYPE_CODE[dtype]
    assert top_p is None or group_prune is None
    select = SPARK_SELECT_TOP_P if top_p is not None else (SPARK_SELECT_GROUPS if group_prune is not None else SPARK_SELECT_FIXED)
    ratios = list(group_prune) if group_prune is not None else []
    assert len(ratios) <= 8
    arr = (ctypes.c_float * 8)(*(ratios + [0.0] * (8 - len(ratios))))
    return spark_params(batch, n_q_heads, n_kv_heads, head_dim, window, keep, page_tokens, code,
                        token_budget, pool_kernel, qnorm_eps, softmax_scale, n_pool_pages, flags, keep_v,
                        select, float(top_p) if top_p is not None else 0.0, len(ratios), arr, int(recovery), int(seed))


# ---- host-only helpers -----------------------------------------------------------------------------
def spark_version() -> int:
    return int(lib().spark_version())


def spark_last_launch_count() -> int:
    return int(lib().spark_last_launch_count())


def spark_keep_count(head_dim: int, ratio: float) -> int:
    return int(lib().spark_keep_count(head_dim, ratio))


def spark_group_keep(head_dim: int, group_prune) -> int:
    ratios = list(group_prune)
    arr = (ctypes.c_float * len(ratios))(*ratios)
    return int(lib().spark_group_keep(head_dim, len(ratios), arr))


def spark_page_bytes(p: spark_params) -> int:
    return int(lib().spark_page_bytes(ctypes.byref(p)))


def spark_pool_bytes(p: spark_params) -> int:
    return int(lib().spark_pool_bytes(ctypes.byref(p)))


def spark_algorithmic_bytes_per_token(p: spark_params) -> int:
    return int(lib().spark_algorithmic_bytes_per_token(ctypes.byref(p)))


def spark_workspace_bytes(p: spark_params, max_seq_tokens: int):
    c, d = ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(lib().spark_workspace_bytes(ctypes.byref(p), max_seq_tokens, ctypes.byref(c), ctypes.byref(d)),
           "spark_workspace_bytes")
    return int(c.value), int(d.value)


# ---- device calls ----------------------------------------------------------------------------------
def spark_workspace_init(workspace: torch.Tensor) -> None:
    _check(lib().spark_workspace_init(_ptr(workspace), workspace.numel() * workspace.element_size(), _stream()),
           "spark_workspace_init")


def spark_compress(p: spark_params, q_win, k, v, seq_lens, max_seq_tokens, pages, block_table, qnorm,
                   packed_lens, kept_tokens, workspace, max_blocks=None) -> None:
    assert k.stride(-1) == 1 and v.stride() == k.stride() and q_win.is_contiguous()
    sb, sh, st = k.stride(0), k.stride(1), k.stride(2)
    _check(lib().spark_compress(ctypes.byref(p), _ptr(q_win), _ptr(k), _ptr(v), sb, sh, st, _ptr(seq_lens),
                                int(max_seq_tokens), _ptr(pages), _ptr(block_table), _blocks(block_table, max_blocks),
                                _ptr(qnorm), _ptr(packed_lens), _ptr(kept_tokens), _ptr(workspace),
                                workspace.numel() * workspace.element_size(), _stream()),
           "spark_compress")


def spark_append(p: spark_params, k_new, v_new, pages, block_table, qnorm, packed_lens, workspace,
                 max_blocks=None) -> None:
    assert k_new.is_contiguous() and v_new.is_contiguous()
    _check(lib().spark_append(ctypes.byref(p), _ptr(k_new), _ptr(v_new), _ptr(pages), _ptr(block_table),
                              _blocks(block_table, max_blocks), _ptr(qnorm), _ptr(packed_lens), _ptr(workspace),
                              workspace.numel() * workspace.element_size(), _stream()),
           "spark_append")


def spark_append_block(p: spark_params, k_new, v_new, pages, block_table, qnorm, packed_lens, workspace,
                       max_blocks=None) -> None:
    """k_new, v_new: [B, Hkv, n_new, D] contiguous; every sequence grows by n_new tokens."""
    assert k_new.is_contiguous() and v_new.is_contiguous() and k_new.shape == v_new.shape and k_new.dim() == 4
    _check(lib().spark_append_block(ctypes.byref(p), _ptr(k_new), _ptr(v_new), int(k_new.shape[2]), _ptr(pages),
                                    _ptr(block_table), _blocks(block_table, max_blocks), _ptr(qnorm),
                                    _ptr(packed_lens), _ptr(workspace),
                                    workspace.numel() * workspace.element_size(), _stream()),
           "spark_append_block")


def spark_merge_attn(out_a, lse_a, out_b, lse_b, out, lse=None) -> None:
    """Merge two partial attention results ([B, Hq, 128] fp32 with their [B, Hq] log-sum-exp)."""
    Bn, Hq, D = out_a.shape
    _check(lib().spark_merge_attn(Bn, Hq, D, _ptr(out_a), _ptr(lse_a), _ptr(out_b), _ptr(lse_b), _ptr(out), _ptr(lse),
                                  _stream()),
           "spark_merge_attn")


def spark_decode_attn(p: spark_params, q, pages, block_table, packed_lens, qnorm, out, lse, workspace,
                      max_blocks=None) -> None:
    _check(lib().spark_decode_attn(ctypes.byref(p), _ptr(q), _ptr(pages), _ptr(block_table),
                                   _blocks(block_table, max_blocks), _ptr(packed_lens), _ptr(qnorm), _ptr(out), _ptr(lse),
                                   _ptr(workspace), workspace.numel() * workspace.element_size(), _stream()),
           "spark_decode_attn")


class BoundDecodeHost:
    """spark_decode_attn_host with every argument marshalled once: query and result in page-locked host
    tensors, device staging owned by this object's caller.  Calling it enqueues copy-in, the step and
    copy-out on the stream; it does not synchronise."""

    def __init__(self, p: spark_params, q_host, q_dev, pages, block_table, packed_lens, qnorm, out_dev, out_host,
                 workspace, max_blocks=None, stream: Optional[int] = None):
        assert q_host.is_pinned() and out_host.is_pinned() and q_host.is_contiguous() and out_host.is_contiguous()
        self._alive = (p, q_host, q_dev, pages, block_table, packed_lens, qnorm, out_dev, out_host, workspace)
        self._fn = lib().spark_decode_attn_host
        self._args = (ctypes.byref(p), _ptr(q_host), _ptr(q_dev), _ptr(pages), _ptr(block_table),
                      _blocks(block_table, max_blocks), _ptr(packed_lens), _ptr(qnorm), _ptr(out_dev), _ptr(out_host),
                      None, None, _ptr(workspace), workspace.numel() * workspace.element_size())
        self._stream = None if stream is None else ctypes.c_void_p(stream)
        self.out_host = out_host

    def __call__(self) -> None:
        code = self._fn(*self._args, self._stream if self._stream is not None else _stream())
        if code != SPARK_OK:
            raise SparkError(code, "spark_decode_attn_host")


class BoundDecode:
    """spark_decode_attn with every argument marshalled once.

    A decode loop calls the same entry point with the same buffers step after step; this object converts
    the pointers and sizes to C values a single time, so a call costs one foreign-function call (the
    stream is the only thing looked up per call, unless a fixed stream handle is given).
    """

    def __init__(self, p: spark_params, q, pages, block_table, packed_lens, qnorm, out, lse, workspace,
                 max_blocks=None, stream: Optional[int] = None):
        self._alive = (p, q, pages, block_table, packed_lens, qnorm, out, lse, workspace)     # keep the buffers
        self._fn = lib().spark_decode_attn
        self._args = (ctypes.byref(p), _ptr(q), _ptr(pages), _ptr(block_table), _blocks(block_table, max_blocks),
                      _ptr(packed_lens), _ptr(qnorm), _ptr(out), _ptr(lse), _ptr(workspace),
                      workspace.numel() * workspace.element_size())
        self._stream = None if stream is None else ctypes.c_void_p(stream)
        self.out = out

    def __call__(self) -> None:
        code = self._fn(*self._args, self._stream if self._stream is not None else _stream())
        if code != SPARK_OK:
            raise SparkError(code, "spark_decode_attn")


def spark_decode_attn_noalloc(p: spark_params, q, pages, block_table, packed_lens, qnorm, out, lse,
                              max_blocks=None) -> None:
    """Decode step that brings its own fixed scratch (batch * n_kv_heads <= 64); allocates nothing."""
    _check(lib().spark_decode_attn_noalloc(ctypes.byref(p), _ptr(q), _ptr(pages), _ptr(block_table),
                                           _blocks(block_table, max_blocks), _ptr(packed_lens), _ptr(qnorm), _ptr(out),
                                           _ptr(lse), _stream()),
           "spark_decode_attn_noalloc")


def spark_unpack_pages(p: spark_params, pages, block_table, packed_lens, max_tokens, mask=None, mu=None,
                       vals=None, v=None, max_blocks=None) -> None:
    _check(lib().spark_unpack_pages(ctypes.byref(p), _ptr(pages), _ptr(block_table), _blocks(block_table, max_blocks),
                                    _ptr(packed_lens), int(max_tokens), _ptr(mask), _ptr(mu), _ptr(vals),
                                    _ptr(v), _stream()),
           "spark_unpack_pages")


def spark_unpack_value_masks(p: spark_params, pages, block_table, packed_lens, max_tokens, vmask,
                             max_blocks=None) -> None:
    _check(lib().spark_unpack_value_masks(ctypes.byref(p), _ptr(pages), _ptr(block_table), _blocks(block_table, max_blocks),
                                          _ptr(packed_lens), int(max_tokens), _ptr(vmask), _stream()),
           "spark_unpack_value_masks")


def spark_unpack_stats(p: spark_params, pages, block_table, packed_lens, max_tokens, mu_all, sigma_all,
                       max_blocks=None) -> None:
    _check(lib().spark_unpack_stats(ctypes.byref(p), _ptr(pages), _ptr(block_table), _blocks(block_table, max_blocks),
                                    _ptr(packed_lens), int(max_tokens), _ptr(mu_all), _ptr(sigma_all), _stream()),
           "spark_unpack_stats")


def spark_read_status(workspace: torch.Tensor) -> int:
    return int(lib().spark_read_status(_ptr(workspace), _stream()))


# ---- allocation helpers (plumbing, no arithmetic) ---------------------------------------------------
def identity_block_table(batch: int, n_kv_heads: int, max_blocks: int, device) -> torch.Tensor:
    """Page ids for a contiguous cache: unit (b, h) owns pages [u*max_blocks, (u+1)*max_blocks)."""
    return torch.arange(batch * n_kv_heads * max_blocks, dtype=torch.int32, device=device).view(
        batch, n_kv_heads, max_blocks)


def alloc_workspace(p: spark_params, max_seq_tokens: int, device, which: str = "decode") -> torch.Tensor:
    c, d = spark_workspace_bytes(p, max_seq_tokens)
    ws = torch.empty(c if which == "compress" else d, dtype=torch.uint8, device=device)
    spark_workspace_init(ws)
    return ws
