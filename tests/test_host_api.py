"""CPU-only checks of the boundary: the library loads, exports every declared symbol, and
host-side validation returns error codes without touching a GPU."""
import ctypes
import os
import re

import pytest

from paper_2506_19225_b200 import binding as vb
from paper_2506_19225_b200 import build as vbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    vbuild.build_library()
    return vb.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "vxl.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vxl_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = declared_symbols()
    assert set(vb.EXPORTS) == set(names)
    for n in names:
        assert getattr(lib, n) is not None


def test_status_strings(lib):
    assert vb.status_str(vb.VXL_OK) == "ok"
    seen = {vb.status_str(c) for c in range(7)}
    assert len(seen) == 7


def _shape(**kw):
    base = dict(B=1, T=256, Hq=2, Hkv=1, D=64, q_strides=(256 * 128, 128, 64),
                kv_strides=(256 * 64, 64, 64))
    base.update(kw)
    return vb.make_shape(**base)


FAKE = ctypes.c_void_p(0x10000)      # aligned, never dereferenced: every call below fails on the host


def test_prefill_rejects_bad_arguments(lib):
    s = _shape()
    f = lib.vxl_chunk_prefill_attn
    ws = ctypes.c_void_p(0x20000)
    assert f(None, FAKE, FAKE, 64, FAKE, 8, FAKE, None, ctypes.byref(s), ws, 1 << 20, None) == vb.VXL_ERR_INVALID_ARG
    assert f(FAKE, FAKE, FAKE, 60, FAKE, 8, FAKE, None, ctypes.byref(s), ws, 1 << 20, None) == vb.VXL_ERR_INVALID_ARG
    assert f(FAKE, FAKE, FAKE, 64, None, 8, FAKE, None, ctypes.byref(s), ws, 1 << 20, None) == vb.VXL_ERR_INVALID_ARG
    assert f(FAKE, FAKE, FAKE, 64, FAKE, 65, FAKE, None, ctypes.byref(s), ws, 1 << 20, None) == vb.VXL_ERR_INVALID_ARG
    assert f(FAKE, FAKE, FAKE, 64, FAKE, 8, FAKE, None, ctypes.byref(s), None, 0, None) == vb.VXL_ERR_WORKSPACE
    assert f(FAKE, FAKE, FAKE, 64, FAKE, 8, FAKE, None, ctypes.byref(s), ctypes.c_void_p(0x20010), 1 << 20, None) == vb.VXL_ERR_WORKSPACE
    assert f(ctypes.c_void_p(0x10008), FAKE, FAKE, 64, FAKE, 8, FAKE, None, ctypes.byref(s), ws, 1 << 20, None) == vb.VXL_ERR_INVALID_ARG
    s2 = _shape(D=96, q_strides=(256 * 192, 192, 96), kv_strides=(256 * 96, 96, 96))
    assert f(FAKE, FAKE, FAKE, 64, FAKE, 8, FAKE, None, ctypes.byref(s2), ws, 1 << 20, None) == vb.VXL_ERR_UNSUPPORTED
    s3 = _shape(Hq=3, Hkv=2)
    assert f(FAKE, FAKE, FAKE, 64, FAKE, 8, FAKE, None, ctypes.byref(s3), ws, 1 << 20, None) == vb.VXL_ERR_INVALID_ARG
    s4 = _shape(kv_strides=(256 * 64, 60, 64))
    assert f(FAKE, FAKE, FAKE, 64, FAKE, 8, FAKE, None, ctypes.byref(s4), ws, 1 << 20, None) == vb.VXL_ERR_INVALID_ARG
    s5 = _shape()
    s5.struct_size = 8
    assert f(FAKE, FAKE, FAKE, 64, FAKE, 8, FAKE, None, ctypes.byref(s5), ws, 1 << 20, None) == vb.VXL_ERR_INVALID_ARG


def test_decode_and_scores_reject_bad_arguments(lib):
    s = _shape(B=2, T=512, Hq=28, Hkv=4, D=128, q_strides=(28 * 128, 0, 128),
               kv_strides=(512 * 512, 512, 128))
    ws = ctypes.c_void_p(0x20000)
    g = lib.vxl_chunk_scores
    assert g(FAKE, FAKE, None, 4, FAKE, 8, 0, None, FAKE, 2, FAKE, ctypes.byref(s), ws, 1 << 30, None) == vb.VXL_ERR_INVALID_ARG
    assert g(FAKE, FAKE, FAKE, 4, FAKE, 8, 0, None, FAKE, 5, FAKE, ctypes.byref(s), ws, 1 << 30, None) == vb.VXL_ERR_INVALID_ARG
    assert g(FAKE, FAKE, FAKE, 4, FAKE, 8, 16, None, FAKE, 2, FAKE, ctypes.byref(s), ws, 1 << 30, None) == vb.VXL_ERR_INVALID_ARG
    assert g(FAKE, FAKE, FAKE, 4, FAKE, 8, 0, None, FAKE, 2, FAKE, ctypes.byref(s), ws, 16, None) == vb.VXL_ERR_WORKSPACE
    f = lib.vxl_bilevel_decode_attn
    assert f(FAKE, FAKE, None, FAKE, 4, 128, FAKE, 8, 0, None, 2, None, FAKE, None, None, None,
             ctypes.byref(s), ws, 1 << 30, None) == vb.VXL_ERR_INVALID_ARG
    assert f(FAKE, FAKE, FAKE, FAKE, 4, 128, FAKE, 8, 0, None, 5, None, FAKE, None, None, None,
             ctypes.byref(s), ws, 1 << 30, None) == vb.VXL_ERR_INVALID_ARG
    assert f(FAKE, FAKE, FAKE, FAKE, 4, 0, FAKE, 8, 0, None, 2, None, FAKE, None, None, None,
             ctypes.byref(s), ws, 1 << 30, None) == vb.VXL_ERR_INVALID_ARG
    assert f(FAKE, FAKE, FAKE, FAKE, 4, 128, FAKE, 8, 0, None, 2, None, FAKE, None, None, None,
             ctypes.byref(s), ws, 64, None) == vb.VXL_ERR_WORKSPACE
    assert lib.vxl_device_status(None, None) == vb.VXL_ERR_WORKSPACE
    # an unknown relevance rule is refused before anything is launched
    s.score_mode = 7
    assert g(FAKE, FAKE, FAKE, 4, FAKE, 8, 0, None, FAKE, 2, FAKE, ctypes.byref(s), ws, 1 << 30, None) == vb.VXL_ERR_INVALID_ARG
    assert f(FAKE, FAKE, FAKE, FAKE, 4, 128, FAKE, 8, 0, None, 2, None, FAKE, None, None, None,
             ctypes.byref(s), ws, 1 << 30, None) == vb.VXL_ERR_INVALID_ARG


def test_prefill_block_range_is_checked(lib):
    s = _shape(B=1, T=1024, Hq=4, Hkv=2, D=128, q_strides=(1024 * 512, 512, 128), kv_strides=(1024 * 256, 256, 128))
    ws = ctypes.c_void_p(0x20000)
    f = lib.vxl_chunk_prefill_attn
    for begin, count in ((-1, 0), (0, -1), (5, 0), (2, 3), (4, 1)):          # four chunks of 256 rows
        s.block_begin, s.block_count = begin, count
        assert f(FAKE, FAKE, FAKE, 256, FAKE, 8, FAKE, None, ctypes.byref(s), ws, 1 << 30, None) == vb.VXL_ERR_INVALID_ARG


def test_workspace_sizes(lib):
    s = _shape(B=8, T=262144, Hq=28, Hkv=4, D=128, q_strides=(28 * 128, 0, 128),
               kv_strides=(262144 * 512, 512, 128))
    dec = vb.workspace_bytes(vb.VXL_OP_DECODE, s, 128, 128, 8, 2048)
    # partial slots: one per chunk plus at least one (at most 64) per selected chunk
    assert dec >= 8 * 28 * (128 + 8) * (128 + 2) * 4
    assert dec < 2 * 8 * 28 * (128 + 8 * 64) * (128 + 2) * 4
    assert vb.workspace_bytes(vb.VXL_OP_SCORES, s, 128, 128) < dec
    assert vb.workspace_bytes(vb.VXL_OP_PREFILL, s, 128, 128) >= 256
    assert vb.workspace_bytes(99, s, 128, 128) == 0


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    monkeypatch.setattr(vb, "_lib", None)
    monkeypatch.setattr(vb, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        vb.load()


def test_window_prefix_pool_multi_select_offline_reject_bad_arguments(lib):
    """Host-side checks of the entry points added after the first three (nothing is launched)."""
    ws = ctypes.c_void_p(0x20000)
    f = lib.vxl_chunk_prefill_attn
    s = _shape(step=48)                                           # 64 % 48 != 0
    assert f(FAKE, FAKE, FAKE, 64, FAKE, 8, FAKE, None, ctypes.byref(s), ws, 1 << 20, None) == vb.VXL_ERR_INVALID_ARG
    s = _shape(step=32, prefix_len=10)                            # (256 - 10) % 32 != 0
    assert f(FAKE, FAKE, FAKE, 64, FAKE, 8, FAKE, None, ctypes.byref(s), ws, 1 << 20, None) == vb.VXL_ERR_INVALID_ARG
    s = _shape(step=32)                                           # R > step
    assert f(FAKE, FAKE, FAKE, 64, FAKE, 33, FAKE, None, ctypes.byref(s), ws, 1 << 20, None) == vb.VXL_ERR_INVALID_ARG
    assert lib.vxl_prefill_kernel_kind(ctypes.byref(_shape(step=48)), 64, 8) == -1
    d = _shape(B=2, T=512, Hq=28, Hkv=4, D=128, q_strides=(28 * 128, 3584, 128), kv_strides=(512 * 512, 512, 128))
    p = lib.vxl_pool_sparse
    assert p(FAKE, FAKE, None, 4, 8, FAKE, FAKE, ctypes.byref(d), None) == vb.VXL_ERR_INVALID_ARG
    assert p(FAKE, FAKE, FAKE, 0, 8, FAKE, FAKE, ctypes.byref(d), None) == vb.VXL_ERR_INVALID_ARG
    assert p(FAKE, FAKE, FAKE, 4, 8, FAKE, ctypes.c_void_p(0x10008), ctypes.byref(d), None) == vb.VXL_ERR_INVALID_ARG
    assert p(FAKE, FAKE, FAKE, 4, 0, FAKE, FAKE, ctypes.byref(d), None) == vb.VXL_OK          # nothing to pool
    m = lib.vxl_chunk_scores_multi
    assert m(FAKE, 0, FAKE, FAKE, 4, FAKE, 8, 0, None, FAKE, 2, FAKE, ctypes.byref(d), ws, 1 << 30, None) == vb.VXL_ERR_INVALID_ARG
    d0 = _shape(B=2, T=512, Hq=28, Hkv=4, D=128, q_strides=(28 * 128, 0, 128), kv_strides=(512 * 512, 512, 128))
    assert m(FAKE, 3, FAKE, FAKE, 4, FAKE, 8, 0, None, FAKE, 2, FAKE, ctypes.byref(d0), ws, 1 << 30, None) == vb.VXL_ERR_INVALID_ARG
    assert m(FAKE, 3, FAKE, FAKE, 4, FAKE, 8, 0, None, FAKE, 2, FAKE, ctypes.byref(d), ws, 16, None) == vb.VXL_ERR_WORKSPACE
    t = lib.vxl_topk_select
    assert t(None, 2, 8, 2, FAKE, None) == vb.VXL_ERR_INVALID_ARG
    assert t(FAKE, 2, 8, 9, FAKE, None) == vb.VXL_ERR_INVALID_ARG
    assert t(FAKE, 2, 5000, 2, FAKE, None) == vb.VXL_ERR_UNSUPPORTED
    assert t(FAKE, 2, 8, 0, FAKE, None) == vb.VXL_OK
    o = lib.vxl_bilevel_decode_offline
    lvl = vb.VxlSparseLevel(0x10000, 0x10000)
    args = lambda shape, **kw: [kw.get("q", FAKE), FAKE, FAKE, FAKE, FAKE, 4, 128, kw.get("lvl", ctypes.byref(lvl)), 8,
                                kw.get("topk", 2), FAKE, FAKE, FAKE, FAKE, None, kw.get("scores", FAKE), FAKE,
                                ctypes.byref(shape), kw.get("ws", ws), kw.get("ws_bytes", 1 << 30), None, None]
    assert o(*args(d, lvl=None)) == vb.VXL_ERR_INVALID_ARG
    assert o(*args(d, scores=None)) == vb.VXL_ERR_INVALID_ARG
    assert o(*args(d, topk=5)) == vb.VXL_ERR_INVALID_ARG
    assert o(*args(d, ws_bytes=64)) == vb.VXL_ERR_WORKSPACE
    padded = _shape(B=2, T=512, Hq=28, Hkv=4, D=128, q_strides=(28 * 128, 0, 128), kv_strides=(512 * 640, 640, 128))
    assert o(*args(padded)) == vb.VXL_ERR_UNSUPPORTED               # token rows of the host cache are not contiguous


def test_host_prefill_rejects_bad_arguments(lib):
    """vxl_chunk_prefill_host: refused on the host before any copy or kernel is enqueued."""
    f = lib.vxl_chunk_prefill_host
    ws = ctypes.c_void_p(0x20000)
    s1, s2, s3 = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x2000), ctypes.c_void_p(0x3000)
    good = _shape(B=1, T=1024, Hq=4, Hkv=2, D=128, q_strides=(1024 * 512, 512, 128), kv_strides=(1024 * 256, 256, 128))

    def call(shape, *, q_host=FAKE, L=256, R=8, lse_host=None, lse_dev=None, ridx_dev=FAKE, per=1, wsb=1 << 30,
             streams=(s1, s2, s3)):
        return f(q_host, FAKE, FAKE, L, FAKE, R, FAKE, lse_host, FAKE, FAKE, FAKE, ridx_dev, FAKE, lse_dev, per,
                 ctypes.byref(shape), ws, wsb, *streams)

    assert call(good, q_host=None) == vb.VXL_ERR_INVALID_ARG
    assert call(good, L=300) == vb.VXL_ERR_INVALID_ARG                      # T % chunk_len != 0
    assert call(good, lse_host=FAKE) == vb.VXL_ERR_INVALID_ARG              # lse on one side only
    assert call(good, ridx_dev=None) == vb.VXL_ERR_INVALID_ARG
    assert call(good, per=-1) == vb.VXL_ERR_INVALID_ARG
    assert call(good, wsb=64) == vb.VXL_ERR_WORKSPACE
    assert call(good, streams=(s1, s1, s3)) == vb.VXL_ERR_INVALID_ARG       # the pipeline needs three streams
    assert call(good, streams=(s1, s2, s2)) == vb.VXL_ERR_INVALID_ARG
    padded = _shape(B=1, T=1024, Hq=4, Hkv=2, D=128, q_strides=(1024 * 640, 640, 128), kv_strides=(1024 * 256, 256, 128))
    assert call(padded) == vb.VXL_ERR_UNSUPPORTED                           # host and device rows are copied whole
    window = _shape(B=1, T=1024, Hq=4, Hkv=2, D=128, q_strides=(1024 * 512, 512, 128), kv_strides=(1024 * 256, 256, 128), step=128)
    assert call(window) == vb.VXL_ERR_UNSUPPORTED
    ranged = _shape(B=1, T=1024, Hq=4, Hkv=2, D=128, q_strides=(1024 * 512, 512, 128), kv_strides=(1024 * 256, 256, 128),
                    block_begin=1, block_count=1)
    assert call(ranged) == vb.VXL_ERR_UNSUPPORTED


def test_selftest_bounded_wait_rejects_bad_arguments(lib):
    f = lib.vxl_selftest_bounded_wait
    assert f(None, 1000, None) == vb.VXL_ERR_WORKSPACE
    assert f(ctypes.c_void_p(0x20010), 1000, None) == vb.VXL_ERR_WORKSPACE
    assert f(ctypes.c_void_p(0x20000), 0, None) == vb.VXL_ERR_INVALID_ARG
    assert f(ctypes.c_void_p(0x20000), 10**12, None) == vb.VXL_ERR_INVALID_ARG        # no long waits on request
