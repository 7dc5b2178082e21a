"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, and rejects bad arguments before any launch."""
import ctypes
import os
import re

import pytest

from paper_2609_33503_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def declared_functions():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        src = open(os.path.join(ROOT, "include", fn)).read()
        src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
        names |= set(re.findall(r"\b(relaxkv_[a-z0-9_]+)\s*\(", src))
    return names


def test_library_exports_every_declared_symbol():
    lib = B.lib()
    declared = declared_functions()
    assert len(declared) >= 10
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(B.ENTRY_POINTS)


def test_anchor_count_matches_the_paper_equation():
    for line in open(os.path.join(GOLDEN, "anchor_counts.txt")):
        if line.strip() and line[0] != "#":
            T, r, k = line.split()
            assert B.relaxkv_anchor_count(int(T), float(r)) == int(k)


def test_status_strings_and_workspace():
    assert B.status_string(B.OK) == "ok"
    assert "workspace" in B.status_string(B.ERR_WORKSPACE_TOO_SMALL)
    s = B.Shape(40, 8, 128, [32768], [128])
    ws = B.relaxkv_workspace_bytes(s, 40)
    assert ws >= 2 * 32768 * 8 * 128 * 2          # room for the materialised K~ and V~
    assert B.relaxkv_workspace_bytes(B.Shape(40, 8, 96, [128], [8]), 1) == 0     # unsupported head_dim
    assert B.relaxkv_workspace_bytes(B.Shape(40, 7, 128, [128], [8]), 1) == 0    # H % H_kv != 0


FAKE = ctypes.c_void_p(0x10000)      # aligned, never dereferenced: calls must fail before any launch
NULL = ctypes.c_void_p(None)
I64 = ctypes.c_int64


def _cache_struct(k=0x10000, v=0x20000, tok=1024, head=128):
    off = (ctypes.c_int64 * 1)(0)
    c = B._CacheView()
    c.k, c.v, c.token_stride, c.head_stride = k, v, tok, head
    c.h_req_token_offset = ctypes.cast(off, ctypes.POINTER(ctypes.c_int64))
    c._keep = off
    return c


def test_bad_arguments_are_rejected_on_the_host():
    lib = B.lib()
    ok_shape = B.Shape(8, 2, 128, [256], [4])
    i32 = B._i32
    cache = _cache_struct()
    # scatter: NULL fresh states, bad shapes, misaligned cache, odd strides
    args = lambda shape, c, kn: lib.relaxkv_scatter_kv(shape.ref(), ctypes.byref(c), kn, FAKE, FAKE, FAKE, FAKE, FAKE,
                                                       i32([4]), NULL)
    assert args(ok_shape, cache, NULL) == B.ERR_INVALID_ARG
    assert args(B.Shape(8, 2, 96, [256], [4]), cache, FAKE) == B.ERR_UNSUPPORTED_SHAPE
    assert args(B.Shape(8, 3, 128, [256], [4]), cache, FAKE) == B.ERR_INVALID_ARG
    assert args(B.Shape(8, 2, 128, [0], [4]), cache, FAKE) == B.ERR_INVALID_ARG
    assert args(ok_shape, _cache_struct(k=0x10002), FAKE) == B.ERR_INVALID_ARG
    assert args(ok_shape, _cache_struct(tok=1023), FAKE) == B.ERR_INVALID_ARG
    assert args(B.Shape(64, 2, 128, [256], [4]), cache, FAKE) == B.ERR_UNSUPPORTED_SHAPE      # group of 32
    # attention: workspace too small / unaligned, negative bounds, k_new without v_new
    att = lambda ws, nbytes, mt, kn=FAKE, vn=FAKE: lib.relaxkv_sparse_ctx_attention(
        ok_shape.ref(), 0, ctypes.byref(cache), FAKE, kn, vn, FAKE, FAKE, FAKE, FAKE, I64(16), i32([mt]), i32([16]),
        FAKE, NULL, ws, ctypes.c_size_t(nbytes), NULL)
    need = B.relaxkv_workspace_bytes(ok_shape, 1)
    assert att(FAKE, need - 1, 16) == B.ERR_WORKSPACE_TOO_SMALL
    assert att(ctypes.c_void_p(0x10010), need, 16) == B.ERR_INVALID_ARG
    assert att(FAKE, need, -1) == B.ERR_INVALID_ARG
    assert att(FAKE, need, 16, kn=FAKE, vn=NULL) == B.ERR_INVALID_ARG
    assert lib.relaxkv_sparse_ctx_attention(ok_shape.ref(), 7, ctypes.byref(cache), FAKE, FAKE, FAKE, FAKE, FAKE, FAKE,
                                            FAKE, I64(16), i32([16]), i32([16]), FAKE, NULL, FAKE,
                                            ctypes.c_size_t(need), NULL) == B.ERR_INVALID_ARG
    # score_select: k out of range, missing q_len, zero layers
    qs = (ctypes.c_void_p * 1)(0x10000)
    caches = (B._CacheView * 1)(cache)
    sc = lambda shape, n_layers, k: lib.relaxkv_score_select(shape.ref(), n_layers, qs, caches, NULL, i32([k]), FAKE,
                                                             NULL, FAKE, FAKE, ctypes.c_size_t(need), NULL)
    assert sc(ok_shape, 1, 0) == B.ERR_INVALID_ARG
    assert sc(ok_shape, 1, 257) == B.ERR_INVALID_ARG
    assert sc(ok_shape, 0, 8) == B.ERR_INVALID_ARG
    assert sc(B.Shape(8, 2, 128, [256], None), 1, 8) == B.ERR_INVALID_ARG
    # a workspace that is not 256-byte aligned is refused by every call that takes one
    odd = ctypes.c_void_p(0x10010)
    assert lib.relaxkv_score_select(ok_shape.ref(), 1, qs, caches, NULL, i32([8]), FAKE, NULL, FAKE, odd,
                                    ctypes.c_size_t(need), NULL) == B.ERR_INVALID_ARG
    assert lib.relaxkv_build_active_sets(ok_shape.ref(), 1, i32([8]), FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, NULL,
                                         odd, ctypes.c_size_t(need), NULL) == B.ERR_INVALID_ARG
    assert lib.relaxkv_scale_scores(ok_shape.ref(), 1, FAKE, ctypes.c_float(0.0), NULL) == B.ERR_INVALID_ARG
    # build_active_sets: NULL outputs
    assert lib.relaxkv_build_active_sets(ok_shape.ref(), 1, i32([8]), FAKE, NULL, FAKE, FAKE, FAKE, FAKE, FAKE, NULL,
                                         FAKE, ctypes.c_size_t(need), NULL) == B.ERR_INVALID_ARG
    # select / gather
    assert lib.relaxkv_select_topk(ok_shape.ref(), 1, i32([300]), FAKE, NULL, FAKE, NULL) == B.ERR_INVALID_ARG
    assert lib.relaxkv_gather_kv(ok_shape.ref(), 0, ctypes.byref(cache), FAKE, FAKE, FAKE, FAKE, FAKE, FAKE,
                                 i32([200]), FAKE, FAKE, I64(100), NULL) == B.ERR_INVALID_ARG     # too few rows


def test_block_work_calls_reject_bad_arguments_on_the_host():
    """The projections and the fused norm + rotary call check pointers, alignment and shapes before any launch."""
    lib = B.lib()
    F32 = ctypes.c_float
    lin = lambda x, w, y, rows, n_out, n_in, res=NULL: lib.relaxkv_linear(x, w, res, y, I64(rows), n_out, n_in, NULL)
    assert lin(NULL, FAKE, FAKE, 4, 64, 64) == B.ERR_INVALID_ARG
    assert lin(FAKE, FAKE, ctypes.c_void_p(0x10002), 4, 64, 64) == B.ERR_INVALID_ARG          # output not 16-byte aligned
    assert lin(FAKE, FAKE, FAKE, 4, 60, 64) == B.ERR_UNSUPPORTED_SHAPE                        # widths are multiples of 8
    assert lin(FAKE, FAKE, FAKE, -1, 64, 64) == B.ERR_UNSUPPORTED_SHAPE
    assert lin(FAKE, FAKE, FAKE, 0, 64, 64) == B.OK                                           # nothing to do
    qkv = lambda x, w, q, k, v, rows, n_q, n_kv, n_in: lib.relaxkv_linear_qkv(x, w, q, k, v, I64(rows), n_q, n_kv, n_in, NULL)
    assert qkv(FAKE, FAKE, FAKE, NULL, FAKE, 4, 64, 16, 64) == B.ERR_INVALID_ARG
    assert qkv(FAKE, ctypes.c_void_p(0x10008), FAKE, FAKE, FAKE, 4, 64, 16, 64) == B.ERR_INVALID_ARG
    assert qkv(FAKE, FAKE, FAKE, FAKE, FAKE, 4, 64, 12, 64) == B.ERR_UNSUPPORTED_SHAPE
    assert qkv(FAKE, FAKE, FAKE, FAKE, FAKE, 0, 64, 16, 64) == B.OK
    assert lib.relaxkv_linear_swiglu(FAKE, FAKE, FAKE, I64(4), 100, 64, NULL) == B.ERR_UNSUPPORTED_SHAPE   # 128-feature blocks
    nr = lambda q, k, rows, hq, hkv, d, wq, wk, eps, pos, theta: lib.relaxkv_qk_norm_rope(
        q, k, I64(rows), hq, hkv, d, wq, wk, F32(eps), pos, F32(theta), NULL)
    assert nr(FAKE, NULL, 4, 8, 2, 128, NULL, NULL, 1e-6, FAKE, 1e6) == B.ERR_INVALID_ARG
    assert nr(FAKE, FAKE, 4, 8, 2, 128, FAKE, NULL, 1e-6, FAKE, 1e6) == B.ERR_INVALID_ARG     # one norm weight without the other
    assert nr(FAKE, FAKE, 4, 8, 2, 128, NULL, NULL, 1e-6, NULL, 1e6) == B.ERR_INVALID_ARG     # no positions
    assert nr(FAKE, FAKE, 4, 8, 2, 128, NULL, NULL, 1e-6, FAKE, 1.0) == B.ERR_INVALID_ARG     # theta must exceed 1
    assert nr(FAKE, FAKE, 4, 8, 2, 96, NULL, NULL, 1e-6, FAKE, 1e6) == B.ERR_UNSUPPORTED_SHAPE
    assert nr(FAKE, FAKE, 0, 8, 2, 128, NULL, NULL, 1e-6, FAKE, 1e6) == B.OK


def test_chained_launch_switch_is_host_state_only():
    """relaxkv_set_chained_launch returns the previous setting and launches nothing (chained is the default)."""
    assert B.relaxkv_set_chained_launch(False) is True
    assert B.relaxkv_set_chained_launch(False) is False
    assert B.relaxkv_set_chained_launch(True) is False
    assert B.relaxkv_set_chained_launch(True) is True


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", "/nonexistent/librelaxkv.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        B.lib()
