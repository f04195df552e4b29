"""Host-side checks that need no GPU: the shared library loads, exports every
symbol the header declares, sizes workspaces, and rejects bad arguments before
touching the device."""
import ctypes as C
import os
import re

import pytest

import paper_2410_08584_b200 as z
from paper_2410_08584_b200 import build as zbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    zbuild.build()
    return z.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "zipvl.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(zipvl_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert len(names) >= 10
    for n in names:
        assert hasattr(lib, n), f"libzipvl.so does not export {n}"
    assert set(z.EXPORTS) == set(names)
    assert lib.zipvl_version() >= 100


def test_struct_layout_matches_header():
    assert C.sizeof(z.zipvl_layer) == 48
    assert C.sizeof(z.zipvl_decode_desc) == 24


def test_workspace_sizes(lib):
    lay = z.zipvl_layer(2944, 32, 32, 128, z.ZIPVL_BF16, 0, 0, 0, 0.0, 0)
    assert z.zipvl_workspace_bytes(z.OP_SCORE, lay, 128) > 0
    assert z.zipvl_workspace_bytes(z.OP_SCORE, lay, 0) == 0
    assert z.zipvl_workspace_bytes(z.OP_DECODE, lay, 0, 16) >= 16 * 32 * 130 * 4
    assert z.zipvl_workspace_bytes(z.OP_DECODE, lay, 0, 0) == 0
    bad = z.zipvl_layer(0, 32, 32, 128, 0, 0, 0, 0, 0.0, 0)
    assert z.zipvl_workspace_bytes(z.OP_SCORE, bad, 128) == 0
    assert z.zipvl_workspace_bytes(99, lay, 128) == 0


def test_argument_validation_without_a_device(lib):
    ok = z.zipvl_layer(128, 4, 2, 64, z.ZIPVL_BF16, 0, 0, 0, 0.0, 0)
    p = C.c_void_p(0x1000)          # never dereferenced: validation fails first
    null = C.c_void_p(0)
    I, U = z.ZipvlError, None

    def status(call):
        rc = call()
        text = lib.zipvl_last_error().decode()
        return rc, text

    rc, text = status(lambda: lib.zipvl_score(C.byref(ok), null, p, p, 8, p, p, None, p, 1 << 20, None, None))
    assert rc == 1 and "NULL" in text
    rc, _ = status(lambda: lib.zipvl_score(C.byref(ok), p, p, p, 0, p, p, None, p, 1 << 20, None, None))
    assert rc == 1
    rc, text = status(lambda: lib.zipvl_score(C.byref(ok), p, p, p, 8, p, p, None, p, 16, None, None))
    assert rc == 3 and "workspace" in text
    rc, _ = status(lambda: lib.zipvl_score(C.byref(ok), C.c_void_p(0x1004), p, p, 8, p, p, None, p, 1 << 20, None, None))
    assert rc == 1
    for bad in (z.zipvl_layer(128, 4, 3, 64, 0, 0, 0, 0, 0.0, 0),      # heads do not divide
                z.zipvl_layer(0, 4, 2, 64, 0, 0, 0, 0, 0.0, 0),        # L < 1
                z.zipvl_layer(128, 4, 2, 64, 0, 0, 100, 0, 0.0, 0)):   # stride too small
        rc, _ = status(lambda: lib.zipvl_score(C.byref(bad), p, p, p, 8, p, p, None, p, 1 << 20, None, None))
        assert rc == 1
    for bad in (z.zipvl_layer(128, 4, 2, 80, 0, 0, 0, 0, 0.0, 0),      # head_dim
                z.zipvl_layer(128, 4, 2, 64, 7, 0, 0, 0, 0.0, 0)):     # dtype
        rc, _ = status(lambda: lib.zipvl_score(C.byref(bad), p, p, p, 8, p, p, None, p, 1 << 20, None, None))
        assert rc == 2
    # select: tau outside (0, 1], NaN, bad mode, bad L
    for tau in (0.0, -0.5, 1.5, float("nan")):
        rc, _ = status(lambda: lib.zipvl_select(128, p, p, tau, 0, 0, p, p, None, None, 0, None, None))
        assert rc == 1
    assert lib.zipvl_select(128, p, p, 0.9, 8, 0, p, p, None, None, 0, None, None) == 1
    assert lib.zipvl_select(128, p, p, 0.9, 0x84, 0, p, p, None, None, 0, None, None) == 1   # a stray low bit
    assert lib.zipvl_select(0, p, p, 0.9, 0, 0, p, p, None, None, 0, None, None) == 1
    assert lib.zipvl_select(128, p, null, 0.9, 0, 0, p, p, None, None, 0, None, None) == 1
    assert lib.zipvl_select(128, p, p, 0.9, 0, -1, p, p, None, None, 0, None, None) == 1
    # sparse prefill / compaction: k_max range, out_mode, capacity
    assert lib.zipvl_sparse_prefill(C.byref(ok), p, p, p, p, p, 0, p, 0, p, 1 << 20, None, None) == 1
    assert lib.zipvl_sparse_prefill(C.byref(ok), p, p, p, p, p, 129, p, 0, p, 1 << 20, None, None) == 1
    assert lib.zipvl_sparse_prefill(C.byref(ok), p, p, p, p, p, 128, p, 5, p, 1 << 20, None, None) == 1
    assert lib.zipvl_compact_kv(C.byref(ok), p, p, p, p, 128, p, p, 0, p, None, None) == 1
    assert lib.zipvl_compact_kv(C.byref(ok), p, p, p, p, 128, p, null, 128, p, None, None) == 1
    # the fused call validates like the two it replaces
    f = lib.zipvl_sparse_prefill_compact
    assert f(C.byref(ok), p, p, p, p, p, 0, p, 0, p, p, 128, p, p, 1 << 20, None, None) == 1      # k_max
    assert f(C.byref(ok), p, p, p, p, p, 128, p, 5, p, p, 128, p, p, 1 << 20, None, None) == 1    # out_mode
    assert f(C.byref(ok), p, p, p, p, p, 128, p, 0, p, p, 0, p, p, 1 << 20, None, None) == 1      # capacity
    assert f(C.byref(ok), p, p, p, p, p, 128, p, 0, null, p, 128, p, p, 1 << 20, None, None) == 1  # NULL cache
    assert f(C.byref(ok), p, p, p, p, p, 128, p, 0, p, p, 128, null, p, 1 << 20, None, None) == 1  # NULL len_out
    assert lib.zipvl_release_host_scratch() in (0, 4)     # nothing to release; no device here
    # decode
    d = z.zipvl_decode_desc(2, 4, 2, 64, 0, 0.0)
    assert lib.zipvl_decode(None, p, p, p, p, p, p, p, p, 10, p, p, 1 << 20, None, None) == 1
    assert lib.zipvl_decode(C.byref(d), p, p, null, p, p, p, p, p, 10, p, p, 1 << 20, None, None) == 1
    assert lib.zipvl_decode(C.byref(d), p, p, p, p, p, p, p, p, 0, p, p, 1 << 20, None, None) == 1
    assert lib.zipvl_decode(C.byref(d), p, p, p, p, p, p, p, p, 10, p, p, 8, None, None) == 3
    # query heads per kv head: beyond 8 in fp32, beyond 32 in 16-bit storage
    d9 = z.zipvl_decode_desc(2, 18, 2, 64, z.ZIPVL_F32, 0.0)
    assert lib.zipvl_decode(C.byref(d9), p, p, p, p, p, p, p, p, 10, p, p, 1 << 20, None, None) == 2
    d33 = z.zipvl_decode_desc(2, 66, 2, 64, z.ZIPVL_BF16, 0.0)
    assert lib.zipvl_decode(C.byref(d33), p, p, p, p, p, p, p, p, 10, p, p, 1 << 20, None, None) == 2
    # decode without a workspace: the same validation, and the size check of its built-in
    # scratch, before anything is launched
    na = lib.zipvl_decode_noalloc
    assert na(C.byref(d), null, None, None, p, p, p, p, p, 128, p, None, None) == 1
    assert na(C.byref(d), p, p, null, p, p, p, p, p, 128, p, None, None) == 1
    big = z.zipvl_decode_desc(16, 32, 32, 128, 0, 0.0)
    rc, text = status(lambda: na(C.byref(big), p, None, None, p, p, p, p, p, 32768, p, None, None))
    assert rc == 3 and "scratch" in text
    # the mixed-precision cache: storage type, head grouping, batch, NULL blocks
    lay16 = z.zipvl_layer(128, 4, 2, 64, z.ZIPVL_BF16, 0, 0, 0, 0.0, 0)
    lay32 = z.zipvl_layer(128, 4, 2, 64, z.ZIPVL_F32, 0, 0, 0, 0.0, 0)
    qk = lib.zipvl_quantize_kv
    assert qk(C.byref(lay32), p, p, p, p, 128, p, p, p, 8, p, p, p, 8, p, None, None) == 2
    assert qk(C.byref(lay16), p, p, p, p, 0, p, p, p, 8, p, p, p, 8, p, None, None) == 1
    assert qk(C.byref(lay16), p, p, p, p, 128, null, p, p, 8, p, p, p, 8, p, None, None) == 1
    assert qk(C.byref(lay16), p, p, p, p, 128, p, p, p, 0, p, p, p, 8, p, None, None) == 1
    dq = lib.zipvl_decode_quant
    d1 = z.zipvl_decode_desc(1, 4, 2, 64, 0, 0.0)
    assert dq(C.byref(d), p, None, None, p, p, p, 8, p, p, p, 8, p, 16, p, p, 1 << 20, None, None) == 2   # batch 2
    assert dq(C.byref(d1), p, p, None, p, p, p, 8, p, p, p, 8, p, 16, p, p, 1 << 20, None, None) == 1
    assert dq(C.byref(d1), p, None, None, p, p, p, 8, p, p, p, 8, p, 16, p, p, 8, None, None) == 3
    d3 = z.zipvl_decode_desc(1, 6, 2, 64, 0, 0.0)
    assert dq(C.byref(d3), p, None, None, p, p, p, 8, p, p, p, 8, p, 16, p, p, 1 << 20, None, None) == 2  # 3 heads per KV head
    # ... and its batched form: the table, the workspace for the whole batch, the same shapes
    dqb = lib.zipvl_decode_quant_batch
    assert dqb(C.byref(d), p, None, None, null, 16, p, p, 1 << 20, None, None) == 1             # no table
    assert dqb(C.byref(d), p, None, None, C.c_void_p(0x1004), 16, p, p, 1 << 20, None, None) == 1
    assert dqb(C.byref(d), p, p, None, p, 16, p, p, 1 << 20, None, None) == 1                   # k_new without v_new
    assert dqb(C.byref(d), p, None, None, p, 16, p, p, 8, None, None) == 3
    assert dqb(C.byref(d3), p, None, None, p, 16, p, p, 1 << 20, None, None) == 2               # 3 heads per KV head
    # the wait self-test: limits outside [1, 2^20] and a missing status word are refused
    assert lib.zipvl_selftest_wait_timeout(0, None, p, None) == 1
    assert lib.zipvl_selftest_wait_timeout(1 << 21, None, p, None) == 1
    assert lib.zipvl_selftest_wait_timeout(1000, None, None, None) == 1
    assert lib.zipvl_status_string(3).decode() == "workspace too small"
    assert lib.zipvl_status_string(0).decode() == "ok"


def test_binding_refuses_host_tensors():
    import torch
    lay = z.zipvl_layer(8, 1, 1, 64, 0, 0, 0, 0, 0.0, 0)
    q = torch.zeros(8, 1, 64, dtype=torch.bfloat16)
    with pytest.raises(ValueError):
        z.zipvl_score(lay, q, q, torch.arange(8, dtype=torch.int32))
