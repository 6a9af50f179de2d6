"""Host-side checks of the C ABI: the library loads, exports what include/spark.h declares, and the
host-only entry points and argument checks behave (no kernel is launched here)."""
import ctypes
import os
import re

import pytest

from paper_2508_15212_b200 import binding as B
from paper_2508_15212_b200 import build as spark_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    spark_build.build()
    return B.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "spark.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(spark_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert set(names) == set(B.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_keep_count_is_floor(lib):
    assert B.spark_keep_count(128, 0.5) == 64
    assert B.spark_keep_count(128, 0.8) == 25          # floor(25.6), not round
    assert B.spark_keep_count(128, 0.3) == 89
    assert B.spark_keep_count(128, 0.7) == 38
    assert B.spark_keep_count(128, 0.0) == 128
    assert B.spark_keep_count(128, 1.0) == -1 and B.spark_keep_count(128, -0.1) == -1


def params(**kw):
    import torch
    base = dict(batch=1, n_q_heads=32, n_kv_heads=8, window=32, keep=64, dtype=torch.bfloat16, n_pool_pages=8)
    base.update(kw)
    return B.make_params(**base)


def test_page_and_algorithmic_bytes(lib):
    import torch
    # bf16: 16 tokens * (2T + 16 + 4 + 256) bytes exactly
    assert B.spark_page_bytes(params(keep=64)) == 16 * 404
    assert B.spark_page_bytes(params(keep=25)) == 16 * 326
    assert B.spark_page_bytes(params(keep=128)) == 16 * (256 + 20 + 256)
    assert B.spark_page_bytes(params(keep=64, dtype=torch.float32)) == 16 * 788
    assert B.spark_page_bytes(params(keep=0)) == 0 and B.spark_page_bytes(params(keep=129)) == 0
    assert B.spark_algorithmic_bytes_per_token(params(keep=64)) == 404
    assert B.spark_algorithmic_bytes_per_token(params(keep=25)) == 326
    assert B.spark_algorithmic_bytes_per_token(params(keep=64, dtype=torch.float32)) == 788
    # kept key values are T/D of the dense keys (the paper's memory claim at ratio 0.8: 60 % of K+V values)
    assert (2 * 25 + 256) / 512 < 0.6 + 1e-9


def test_workspace_sizes_and_param_checks(lib):
    c, d = B.spark_workspace_bytes(params(), 32768)
    assert c >= 256 and d >= 256 and c % 256 == 0 and d % 256 == 0
    for bad in (dict(head_dim=64), dict(page_tokens=32), dict(n_q_heads=72, n_kv_heads=8),
                dict(batch=2000)):
        with pytest.raises(B.SparkError) as e:
            B.spark_workspace_bytes(params(**bad), 128)
        assert e.value.code == 3
    for bad in (dict(keep=0), dict(keep=129), dict(n_q_heads=30), dict(batch=0), dict(n_pool_pages=0)):
        with pytest.raises(B.SparkError) as e:
            B.spark_workspace_bytes(params(**bad), 128)
        assert e.value.code == 2


def test_null_and_shape_errors_come_before_any_launch(lib):
    p = params()
    null = ctypes.c_void_p(None)
    one = ctypes.c_void_p(4096)          # never dereferenced on the host
    rc = lib.spark_decode_attn(ctypes.byref(p), null, one, one, 4, one, one, one, null, one, 1 << 20, null)
    assert rc == 1
    rc = lib.spark_decode_attn(ctypes.byref(p), one, one, one, 4, one, one, one, null, null, 0, null)
    assert rc == 1
    rc = lib.spark_decode_attn(ctypes.byref(p), one, one, one, 4, one, one, one, null, one, 16, null)
    assert rc == 4                       # workspace too small
    rc = lib.spark_decode_attn(ctypes.byref(p), one, one, one, 4, one, one, one, null,
                               ctypes.c_void_p(4096 + 8), 1 << 30, null)
    assert rc == 4                       # workspace misaligned
    rc = lib.spark_compress(ctypes.byref(p), one, one, one, 0, 0, 128, one, 64, one, one, 2, one, one, null,
                            one, 1 << 20, null)
    assert rc == 2                       # 64 tokens need 4 blocks, table has 2
    rc = lib.spark_compress(ctypes.byref(p), one, one, one, 0, 0, 64, one, 64, one, one, 4, one, one, null,
                            one, 1 << 20, null)
    assert rc == 2                       # token stride shorter than a row
    rc = lib.spark_compress(ctypes.byref(p), null, one, one, 0, 0, 128, one, 64, one, one, 4, one, one, null,
                            one, 1 << 20, null)
    assert rc == 1
    rc = lib.spark_unpack_pages(ctypes.byref(p), null, one, 4, one, 64, null, null, null, null, null)
    assert rc == 1
    assert lib.spark_read_status(null, null) == 1
    assert lib.spark_workspace_init(null, 1024, null) == 1
    assert B.spark_version() >= 100


def test_misaligned_pointers_and_oversized_tables_are_refused_on_the_host(lib):
    """q, qnorm and out are accessed with 16-byte vector loads / stores: a pointer that is not 16-byte aligned
    would fault on the device, so it is turned away here.  16 * max_blocks must fit a 32-bit int."""
    p = params()
    null, one, ws = ctypes.c_void_p(None), ctypes.c_void_p(4096), ctypes.c_void_p(8192)
    off8, off4 = ctypes.c_void_p(4096 + 8), ctypes.c_void_p(4096 + 4)

    def decode(q=one, qnorm=one, out=one, lse=null, max_blocks=4):
        return lib.spark_decode_attn(ctypes.byref(p), q, one, one, max_blocks, one, qnorm, out, lse, ws, 1 << 30, null)

    assert decode(q=off8) == 2 and decode(qnorm=off8) == 2 and decode(out=off4) == 2
    assert decode(lse=ctypes.c_void_p(4096 + 2)) == 2
    assert decode(max_blocks=(2 ** 31 - 1) // 16 + 1) == 2

    def noalloc(q=one, qnorm=one, out=one, max_blocks=4):
        return lib.spark_decode_attn_noalloc(ctypes.byref(p), q, one, one, max_blocks, one, qnorm, out, null, null)

    assert noalloc(q=off8) == 2 and noalloc(qnorm=off8) == 2 and noalloc(out=off4) == 2
    assert noalloc(max_blocks=(2 ** 31 - 1) // 16 + 1) == 2
    # spark_compress writes qnorm and the page kernel reads it back four floats at a time
    rc = lib.spark_compress(ctypes.byref(p), one, one, one, 0, 0, 128, one, 64, one, one, 4, off8, one, null,
                            ws, 1 << 30, null)
    assert rc == 2
    rc = lib.spark_compress(ctypes.byref(p), one, one, one, 0, 0, 128, one, 64, one, one, (2 ** 31 - 1) // 16 + 1,
                            one, one, null, ws, 1 << 30, null)
    assert rc == 2
    rc = lib.spark_append(ctypes.byref(p), one, one, one, one, 4, off8, one, ws, 1 << 20, null)
    assert rc == 2
