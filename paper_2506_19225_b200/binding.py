"""Thin ctypes binding over the C ABI in ``include/vxl.h``.

Argument marshalling only: tensors are PyTorch CUDA tensors (device memory and streams are
the only things PyTorch provides here), every step of the path runs in the library's CUDA
kernels.  There is no CPU fallback: loading fails loudly when ``libvxl.so`` is missing.
"""
from __future__ import annotations

import ctypes
import math
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libvxl.so")

VXL_OK = 0
VXL_ERR_INVALID_ARG, VXL_ERR_UNSUPPORTED, VXL_ERR_INVALID_INDEX = 1, 2, 3
VXL_ERR_WORKSPACE, VXL_ERR_CUDA, VXL_ERR_TIMEOUT = 4, 5, 6
VXL_BF16, VXL_F32 = 0, 1
VXL_OP_PREFILL, VXL_OP_SCORES, VXL_OP_DECODE = 0, 1, 2
VXL_SCORE_LSE, VXL_SCORE_MASS = 0, 1

EXPORTS = ("vxl_workspace_bytes", "vxl_chunk_prefill_attn", "vxl_chunk_prefill_host", "vxl_chunk_scores",
           "vxl_chunk_scores_static", "vxl_chunk_scores_multi", "vxl_topk_select", "vxl_bilevel_decode_attn", "vxl_bilevel_decode_offline", "vxl_pack_retained", "vxl_pool_sparse", "vxl_device_status", "vxl_selftest_bounded_wait",
           "vxl_status_str", "vxl_prefill_kernel_kind")


class VxlShape(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("B", ctypes.c_int32), ("T", ctypes.c_int32),
                ("Hq", ctypes.c_int32), ("Hkv", ctypes.c_int32), ("D", ctypes.c_int32),
                ("q_stride_b", ctypes.c_int64), ("q_stride_t", ctypes.c_int64), ("q_stride_h", ctypes.c_int64),
                ("kv_stride_b", ctypes.c_int64), ("kv_stride_t", ctypes.c_int64), ("kv_stride_h", ctypes.c_int64),
                ("out_stride_b", ctypes.c_int64), ("out_stride_t", ctypes.c_int64), ("out_stride_h", ctypes.c_int64),
                ("scale", ctypes.c_float), ("out_dtype", ctypes.c_int32), ("validate", ctypes.c_int32),
                ("force_general", ctypes.c_int32), ("prefill_gather4", ctypes.c_int32),
                ("prefill_step", ctypes.c_int32), ("prefix_len", ctypes.c_int32),
                ("block_begin", ctypes.c_int32), ("block_count", ctypes.c_int32), ("score_mode", ctypes.c_int32)]


class VxlSparseLevel(ctypes.Structure):
    _fields_ = [("k_sparse", ctypes.c_void_p), ("v_sparse", ctypes.c_void_p)]


class VxlError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_str(code)} (vxl_status {code})")


_lib = None


def load():
    """Load libvxl.so (built in-tree by ``paper_2506_19225_b200.build``).  Raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} not found: build it with `python -m paper_2506_19225_b200.build` "
                "(there is no CPU fallback)")
        lib = ctypes.CDLL(LIB_PATH)
        lib.vxl_workspace_bytes.restype = ctypes.c_size_t
        lib.vxl_workspace_bytes.argtypes = [ctypes.c_int32, ctypes.POINTER(VxlShape), ctypes.c_int32,
                                            ctypes.c_int32, ctypes.c_int32, ctypes.c_int32]
        lib.vxl_status_str.restype = ctypes.c_char_p
        lib.vxl_status_str.argtypes = [ctypes.c_int]
        lib.vxl_prefill_kernel_kind.restype = ctypes.c_int32
        lib.vxl_prefill_kernel_kind.argtypes = [ctypes.POINTER(VxlShape), ctypes.c_int32, ctypes.c_int32]
        vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
        lib.vxl_chunk_prefill_attn.restype = ctypes.c_int
        lib.vxl_chunk_prefill_attn.argtypes = [vp, vp, vp, i32, vp, i32, vp, vp, ctypes.POINTER(VxlShape),
                                               vp, sz, vp]
        lib.vxl_chunk_prefill_host.restype = ctypes.c_int
        lib.vxl_chunk_prefill_host.argtypes = [vp, vp, vp, i32, vp, i32, vp, vp, vp, vp, vp, vp, vp, vp, i32,
                                               ctypes.POINTER(VxlShape), vp, sz, vp, vp, vp]
        lib.vxl_chunk_scores.restype = ctypes.c_int
        lib.vxl_chunk_scores.argtypes = [vp, vp, vp, i32, vp, i32, i64, ctypes.POINTER(VxlSparseLevel),
                                         vp, i32, vp, ctypes.POINTER(VxlShape), vp, sz, vp]
        lib.vxl_chunk_scores_multi.restype = ctypes.c_int
        lib.vxl_chunk_scores_multi.argtypes = [vp, i32, vp, vp, i32, vp, i32, i64, ctypes.POINTER(VxlSparseLevel),
                                               vp, i32, vp, ctypes.POINTER(VxlShape), vp, sz, vp]
        lib.vxl_topk_select.restype = ctypes.c_int
        lib.vxl_topk_select.argtypes = [vp, i32, i32, i32, vp, vp]
        lib.vxl_chunk_scores_static.restype = ctypes.c_int
        lib.vxl_chunk_scores_static.argtypes = [vp, vp, vp, i32, vp, i32, i64, ctypes.POINTER(VxlSparseLevel),
                                                vp, i32, vp, vp, ctypes.POINTER(VxlShape), vp]
        lib.vxl_bilevel_decode_attn.restype = ctypes.c_int
        lib.vxl_bilevel_decode_attn.argtypes = [vp, vp, vp, vp, i32, i32, vp, i32, i64,
                                                ctypes.POINTER(VxlSparseLevel), i32, vp, vp, vp, vp, vp,
                                                ctypes.POINTER(VxlShape), vp, sz, vp]
        lib.vxl_bilevel_decode_offline.restype = ctypes.c_int
        lib.vxl_bilevel_decode_offline.argtypes = [vp, vp, vp, vp, vp, i32, i32, ctypes.POINTER(VxlSparseLevel), i32, i32,
                                                   vp, vp, vp, vp, vp, vp, vp, ctypes.POINTER(VxlShape), vp, sz, vp, vp]
        lib.vxl_pack_retained.restype = ctypes.c_int
        lib.vxl_pack_retained.argtypes = [vp, vp, vp, i32, i32, i64, vp, vp, ctypes.POINTER(VxlShape), vp]
        lib.vxl_pool_sparse.restype = ctypes.c_int
        lib.vxl_pool_sparse.argtypes = [vp, vp, vp, i32, i32, vp, vp, ctypes.POINTER(VxlShape), vp]
        lib.vxl_device_status.restype = ctypes.c_int
        lib.vxl_device_status.argtypes = [vp, vp]
        lib.vxl_selftest_bounded_wait.restype = ctypes.c_int
        lib.vxl_selftest_bounded_wait.argtypes = [vp, i64, vp]
        _lib = lib
    return _lib


def status_str(code: int) -> str:
    return load().vxl_status_str(int(code)).decode()


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _out_code(dtype) -> int:
    if dtype == torch.float32:
        return VXL_F32
    if dtype == torch.bfloat16:
        return VXL_BF16
    raise ValueError("out dtype must be float32 or bfloat16")


def _check_bf16(*ts):
    for t in ts:
        if t is not None and (t.dtype != torch.bfloat16 or not t.is_cuda or t.stride(-1) != 1):
            raise ValueError("q/k/v must be CUDA bf16 tensors with a contiguous last dim")


def make_shape(*, B, T, Hq, Hkv, D, q_strides, kv_strides, out_strides=(0, 0, 0), scale=0.0,
               out_dtype=VXL_F32, validate=False, force_general=False, gather4=False, step=0,
               prefix_len=0, score_mode=VXL_SCORE_LSE, block_begin=0, block_count=0) -> VxlShape:
    s = VxlShape()
    s.struct_size = ctypes.sizeof(VxlShape)
    s.B, s.T, s.Hq, s.Hkv, s.D = B, T, Hq, Hkv, D
    s.q_stride_b, s.q_stride_t, s.q_stride_h = q_strides
    s.kv_stride_b, s.kv_stride_t, s.kv_stride_h = kv_strides
    s.out_stride_b, s.out_stride_t, s.out_stride_h = out_strides
    s.scale = float(scale)
    s.out_dtype = out_dtype
    s.validate = int(bool(validate))
    s.force_general = int(bool(force_general))
    s.prefill_gather4 = int(bool(gather4))
    s.prefill_step = int(step)
    s.prefix_len = int(prefix_len)
    s.score_mode = int(score_mode)
    s.block_begin = int(block_begin)
    s.block_count = int(block_count)
    return s


def workspace_bytes(op: int, shape: VxlShape, C: int, R: int, topk: int = 0, max_chunk_len: int = 0) -> int:
    return int(load().vxl_workspace_bytes(op, ctypes.byref(shape), C, R, topk, max_chunk_len))


def new_workspace(nbytes: int, device) -> torch.Tensor:
    """Zero-filled, 256-byte aligned scratch (torch's caching allocator aligns to 512 bytes)."""
    return torch.zeros(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def device_status(workspace: torch.Tensor, stream=None) -> int:
    return int(load().vxl_device_status(_ptr(workspace), _stream(stream)))


def selftest_bounded_wait(workspace: torch.Tensor, limit_cycles: int = 2_000_000, stream=None) -> int:
    """Launches the probe whose wait must run out; returns the launch status (read the workspace afterwards)."""
    return int(load().vxl_selftest_bounded_wait(_ptr(workspace), int(limit_cycles), _stream(stream)))


def _prefill_shape(q, k, out, scale, validate, force_general, gather4=False, step=0, prefix_len=0,
                   block_begin=0, block_count=0):
    B, T, Hq, D = q.shape
    Hkv = k.shape[2]
    return make_shape(B=B, T=T, Hq=Hq, Hkv=Hkv, D=D,
                      q_strides=(q.stride(0), q.stride(1), q.stride(2)),
                      kv_strides=(k.stride(0), k.stride(1), k.stride(2)),
                      out_strides=(out.stride(0), out.stride(1), out.stride(2)),
                      scale=scale or 0.0, out_dtype=_out_code(out.dtype), validate=validate,
                      force_general=force_general, gather4=gather4, step=step, prefix_len=prefix_len,
                      block_begin=block_begin, block_count=block_count)


def prefill_workspace(*, B, T, Hq, Hkv, D, chunk_len, R, device) -> torch.Tensor:
    """A zeroed workspace large enough for vxl_chunk_prefill_attn on a contiguous problem."""
    shape = make_shape(B=B, T=T, Hq=Hq, Hkv=Hkv, D=D, q_strides=(T * Hq * D, Hq * D, D),
                       kv_strides=(T * Hkv * D, Hkv * D, D))
    return new_workspace(workspace_bytes(VXL_OP_PREFILL, shape, T // chunk_len, R, 0, chunk_len), device)


def chunk_prefill_attn(q, k, v, chunk_len: int, retained_idx, *, scale=None, out=None,
                       out_dtype=torch.float32, return_lse=False, lse=None, workspace=None,
                       validate=False, force_general=False, gather4=False, step=0, prefix_len=0,
                       block_begin=0, block_count=0, stream=None):
    """Chunk-based pre-filling attention.  q [B,T,Hq,D] (or [T,Hq,D]), k/v [B,T,Hkv,D] bf16 CUDA;
    retained_idx [C,R] int32 CUDA (or None).  Returns out (and lse [B,T,Hq] if asked).
    ``step`` (a divisor of chunk_len) turns the chunks into a sliding window and ``prefix_len``
    makes the first tokens visible to all later ones; retained_idx then has one row per block
    of ``step`` tokens after the prefix.  ``block_begin`` / ``block_count`` restrict the call to
    the rows of those chunks (blocks): nothing after the range is read, other rows of out stay."""
    squeeze = q.dim() == 3
    if squeeze:
        q, k, v = q[None], k[None], v[None]
        if out is not None:
            out = out[None]
    _check_bf16(q, k, v)
    if k.stride() != v.stride():
        raise ValueError("k and v must share strides")
    B, T, Hq, D = q.shape
    if out is None:
        out = torch.empty((B, T, Hq, D), dtype=out_dtype, device=q.device)
    if return_lse and lse is None:
        lse = torch.empty((B, T, Hq), dtype=torch.float32, device=q.device)
    R = 0 if retained_idx is None else int(retained_idx.shape[1])
    if retained_idx is not None and (retained_idx.dtype != torch.int32 or not retained_idx.is_contiguous()):
        raise ValueError("retained_idx must be contiguous int32")
    shape = _prefill_shape(q, k, out, scale, validate, force_general, gather4, step, prefix_len,
                           block_begin, block_count)
    blk = step if step > 0 else chunk_len
    C = (T - prefix_len) // blk if blk > 0 else 0
    if workspace is None:
        workspace = new_workspace(workspace_bytes(VXL_OP_PREFILL, shape, C, R, 0, chunk_len), q.device)
    rc = load().vxl_chunk_prefill_attn(_ptr(q), _ptr(k), _ptr(v), chunk_len, _ptr(retained_idx), R,
                                       _ptr(out), _ptr(lse), ctypes.byref(shape), _ptr(workspace),
                                       workspace.numel(), _stream(stream))
    if rc != VXL_OK:
        raise VxlError(rc, "vxl_chunk_prefill_attn")
    if squeeze:
        out = out[0]
        lse = None if lse is None else lse[0]
    return (out, lse) if return_lse else out


def prefill_kernel_kind(*, B, T, Hq, Hkv, D, chunk_len, R, force_general=False, step=0, prefix_len=0,
                        block_begin=0, block_count=0) -> int:
    """Which kernel a contiguous [B,T,H,D] problem would use: 1 = tcgen05, 0 = general, -1 = invalid."""
    shape = make_shape(B=B, T=T, Hq=Hq, Hkv=Hkv, D=D, q_strides=(T * Hq * D, Hq * D, D),
                       kv_strides=(T * Hkv * D, Hkv * D, D), force_general=force_general, step=step,
                       prefix_len=prefix_len, block_begin=block_begin, block_count=block_count)
    return int(load().vxl_prefill_kernel_kind(ctypes.byref(shape), chunk_len, R))


def _decode_shape(q, k_cache, out, scale, validate, score_mode=VXL_SCORE_LSE):
    B, Hq, D = q.shape
    _, T, Hkv, _ = k_cache.shape
    ostr = (0, 0, 0) if out is None else (out.stride(0), 0, out.stride(1))
    return make_shape(B=B, T=T, Hq=Hq, Hkv=Hkv, D=D,
                      q_strides=(q.stride(0), 0, q.stride(1)),
                      kv_strides=(k_cache.stride(0), k_cache.stride(1), k_cache.stride(2)),
                      out_strides=ostr, scale=scale or 0.0,
                      out_dtype=VXL_F32 if out is None else _out_code(out.dtype), validate=validate,
                      score_mode=score_mode)


def _ridx_args(retained_idx, C, sparse=None):
    if retained_idx is None:
        if sparse is not None and C > 0:
            return None, int(sparse[0].shape[1]) // C, 0      # a stored sparse level: R rows per chunk, no indices
        return None, 0, 0
    if retained_idx.dtype != torch.int32 or not retained_idx.is_contiguous():
        raise ValueError("retained_idx must be contiguous int32")
    R = int(retained_idx.shape[-1])
    stride_b = C * R if retained_idx.dim() == 3 else 0
    return retained_idx, R, stride_b


def _sparse_arg(sparse):
    if sparse is None:
        return None, None
    ks, vs = sparse
    lvl = VxlSparseLevel(ks.data_ptr(), 0 if vs is None else vs.data_ptr())
    return ctypes.byref(lvl), lvl


def chunk_scores(q, k_cache, chunk_offsets, retained_idx, *, topk=0, scale=None, sparse=None,
                 workspace=None, validate=False, score_mode=VXL_SCORE_LSE, stream=None):
    """Per-chunk relevance (+ top-k).  q [B,Hq,D], k_cache [B,T,Hkv,D].  Returns (scores [B,C] fp32,
    topk_idx [B,topk] int32 ascending or None)."""
    _check_bf16(q, k_cache)
    B = q.shape[0]
    C = int(chunk_offsets.numel()) - 1
    ridx, R, rsb = _ridx_args(retained_idx, C, sparse)
    shape = _decode_shape(q, k_cache, None, scale, validate, score_mode)
    scores = torch.empty((B, C), dtype=torch.float32, device=q.device)
    topk_idx = torch.empty((B, topk), dtype=torch.int32, device=q.device) if topk > 0 else None
    if workspace is None:
        workspace = new_workspace(workspace_bytes(VXL_OP_SCORES, shape, C, R), q.device)
    sp_ref, _keep = _sparse_arg(sparse)
    rc = load().vxl_chunk_scores(_ptr(q), _ptr(k_cache), _ptr(chunk_offsets), C, _ptr(ridx), R, rsb, sp_ref,
                                 _ptr(scores), topk, _ptr(topk_idx), ctypes.byref(shape), _ptr(workspace),
                                 workspace.numel(), _stream(stream))
    if rc != VXL_OK:
        raise VxlError(rc, "vxl_chunk_scores")
    return scores, topk_idx


def chunk_scores_multi(q, k_cache, chunk_offsets, retained_idx, *, topk=0, scale=None, sparse=None,
                       workspace=None, validate=False, stream=None):
    """Relevance for a query of several tokens.  q [B,Tq,Hq,D]; returns (scores [B,C], topk_idx or None)."""
    _check_bf16(q, k_cache)
    B, Tq, Hq, D = q.shape
    C = int(chunk_offsets.numel()) - 1
    ridx, R, rsb = _ridx_args(retained_idx, C, sparse)
    shape = make_shape(B=B, T=k_cache.shape[1], Hq=Hq, Hkv=k_cache.shape[2], D=D,
                       q_strides=(q.stride(0), q.stride(1), q.stride(2)),
                       kv_strides=(k_cache.stride(0), k_cache.stride(1), k_cache.stride(2)),
                       scale=scale or 0.0, validate=validate)
    scores = torch.empty((B, C), dtype=torch.float32, device=q.device)
    topk_idx = torch.empty((B, topk), dtype=torch.int32, device=q.device) if topk > 0 else None
    if workspace is None:
        workspace = new_workspace(workspace_bytes(VXL_OP_SCORES, shape, C, R), q.device)
    sp_ref, _keep = _sparse_arg(sparse)
    rc = load().vxl_chunk_scores_multi(_ptr(q), Tq, _ptr(k_cache), _ptr(chunk_offsets), C, _ptr(ridx), R, rsb, sp_ref,
                                       _ptr(scores), topk, _ptr(topk_idx), ctypes.byref(shape), _ptr(workspace),
                                       workspace.numel(), _stream(stream))
    if rc != VXL_OK:
        raise VxlError(rc, "vxl_chunk_scores_multi")
    return scores, topk_idx


def topk_select(scores, topk: int, *, stream=None):
    """Top-k chunks per sequence from given relevance scores [B,C] fp32 -> ascending ids [B,topk] int32."""
    if scores.dtype != torch.float32 or not scores.is_cuda or not scores.is_contiguous() or scores.dim() != 2:
        raise ValueError("scores must be a contiguous CUDA fp32 [B,C] tensor")
    B, C = scores.shape
    out = torch.empty((B, topk), dtype=torch.int32, device=scores.device)
    rc = load().vxl_topk_select(_ptr(scores), B, C, topk, _ptr(out), _stream(stream))
    if rc != VXL_OK:
        raise VxlError(rc, "vxl_topk_select")
    return out


STATIC_SCRATCH_BYTES = 1 << 20


def chunk_scores_static(q, k_cache, chunk_offsets, retained_idx, scores, *, topk=0, topk_idx=None,
                        device_status=None, scale=None, sparse=None, validate=False, stream=None):
    """vxl_chunk_scores for callers that may not allocate device memory (a plug-in living inside
    someone else's memory pool, a loop with a frozen memory budget): the scratch is a fixed
    1 MiB array inside the library instead of a workspace.  Unlike ``chunk_scores`` this wrapper
    allocates nothing either: the caller passes every output.

    scores [B,C] fp32, topk_idx [B,topk] int32 (required when topk > 0) and device_status (one
    int32, optional) are CUDA tensors the caller already owns.  Raises VxlError with
    VXL_ERR_WORKSPACE when the problem needs more scratch than the library holds.  Calls on one
    device share the scratch: do not let two of them overlap on the GPU."""
    _check_bf16(q, k_cache)
    C = int(chunk_offsets.numel()) - 1
    ridx, R, rsb = _ridx_args(retained_idx, C)
    if scores.dtype != torch.float32 or tuple(scores.shape) != (q.shape[0], C) or not scores.is_contiguous():
        raise ValueError("scores must be a contiguous fp32 [B,C] tensor")
    if topk > 0 and (topk_idx is None or topk_idx.dtype != torch.int32 or not topk_idx.is_contiguous()
                     or tuple(topk_idx.shape) != (q.shape[0], topk)):
        raise ValueError("topk_idx must be a contiguous int32 [B,topk] tensor")
    if device_status is not None and (device_status.dtype != torch.int32 or device_status.numel() < 1):
        raise ValueError("device_status must hold one int32")
    shape = _decode_shape(q, k_cache, None, scale, validate)
    sp_ref, _keep = _sparse_arg(sparse)
    rc = load().vxl_chunk_scores_static(_ptr(q), _ptr(k_cache), _ptr(chunk_offsets), C, _ptr(ridx), R, rsb,
                                        sp_ref, _ptr(scores), topk, _ptr(topk_idx) if topk > 0 else None,
                                        _ptr(device_status), ctypes.byref(shape), _stream(stream))
    if rc != VXL_OK:
        raise VxlError(rc, "vxl_chunk_scores_static")


def bilevel_decode_attn(q, k_cache, v_cache, chunk_offsets, retained_idx, topk: int, *, max_chunk_len: int,
                        selected=None, scale=None, sparse=None, out=None, out_dtype=torch.float32,
                        return_lse=False, return_scores=False, workspace=None, validate=False,
                        score_mode=VXL_SCORE_LSE, stream=None):
    """Bi-level KV decoding attention.  Returns a dict with ``out`` [B,Hq,D] and, on request,
    ``lse`` [B,Hq], ``scores`` [B,C], ``topk`` [B,topk] (only when the call selects itself)."""
    _check_bf16(q, k_cache, v_cache)
    if k_cache.stride() != v_cache.stride():
        raise ValueError("k_cache and v_cache must share strides")
    B, Hq, D = q.shape
    C = int(chunk_offsets.numel()) - 1
    ridx, R, rsb = _ridx_args(retained_idx, C, sparse)
    if out is None:
        out = torch.empty((B, Hq, D), dtype=out_dtype, device=q.device)
    shape = _decode_shape(q, k_cache, out, scale, validate, score_mode)
    lse = torch.empty((B, Hq), dtype=torch.float32, device=q.device) if return_lse else None
    scores = topk_out = None
    if selected is None and return_scores:
        scores = torch.empty((B, C), dtype=torch.float32, device=q.device)
        topk_out = torch.empty((B, max(topk, 1)), dtype=torch.int32, device=q.device)
    if selected is not None and (selected.dtype != torch.int32 or not selected.is_contiguous()):
        raise ValueError("selected must be contiguous int32")
    if workspace is None:
        workspace = new_workspace(workspace_bytes(VXL_OP_DECODE, shape, C, R, topk, max_chunk_len), q.device)
    sp_ref, _keep = _sparse_arg(sparse)
    rc = load().vxl_bilevel_decode_attn(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(chunk_offsets), C,
                                        max_chunk_len, _ptr(ridx), R, rsb, sp_ref, topk, _ptr(selected),
                                        _ptr(out), _ptr(lse), _ptr(scores), _ptr(topk_out), ctypes.byref(shape),
                                        _ptr(workspace), workspace.numel(), _stream(stream))
    if rc != VXL_OK:
        raise VxlError(rc, "vxl_bilevel_decode_attn")
    res = {"out": out}
    if lse is not None:
        res["lse"] = lse
    if scores is not None:
        res["scores"] = scores
        res["topk"] = topk_out[:, :topk]
    return res


class HostPrefill:
    """Chunk-based pre-filling of sequences whose tokens live in pinned host memory
    (vxl_chunk_prefill_host: copy chunk c in, attend chunk c, copy its output rows back, on three
    streams).  This class only holds what the call needs (device arrays, workspace, two copy streams),
    so that ``run`` allocates nothing; the pipeline itself is inside the library."""

    def __init__(self, T: int, Hq: int, Hkv: int, D: int, chunk_len: int, R: int, *, B: int = 1, device="cuda",
                 out_dtype=torch.float32, chunks_per_call: int = 1, scale=None, force_general=False, with_lse=False):
        if T % chunk_len:
            raise ValueError("T must be a multiple of chunk_len")
        self.B, self.T, self.Hq, self.Hkv, self.D, self.L, self.R = B, T, Hq, Hkv, D, chunk_len, R
        self.C = T // chunk_len
        self.per_call = max(1, int(chunks_per_call))
        self.q = torch.empty((B, T, Hq, D), dtype=torch.bfloat16, device=device)
        self.k = torch.empty((B, T, Hkv, D), dtype=torch.bfloat16, device=device)
        self.v = torch.empty_like(self.k)
        self.out = torch.empty((B, T, Hq, D), dtype=out_dtype, device=device)
        self.lse = torch.empty((B, T, Hq), dtype=torch.float32, device=device) if with_lse else None
        self.ridx = torch.empty((self.C, max(R, 1)), dtype=torch.int32, device=device)
        self.ws = prefill_workspace(B=B, T=T, Hq=Hq, Hkv=Hkv, D=D, chunk_len=chunk_len, R=R, device=device)
        self.s_in, self.s_out = torch.cuda.Stream(device=device), torch.cuda.Stream(device=device)
        self.shape = make_shape(B=B, T=T, Hq=Hq, Hkv=Hkv, D=D, q_strides=(T * Hq * D, Hq * D, D),
                                kv_strides=(T * Hkv * D, Hkv * D, D), scale=scale or 0.0,
                                out_dtype=_out_code(out_dtype), force_general=force_general)

    def run(self, q_host, k_host, v_host, retained_idx_host, out_host, lse_host=None, stream=None):
        """q_host [B,T,Hq,D] (or [T,Hq,D] when B = 1), k_host/v_host likewise with Hkv: pinned bf16 (or their
        bits as int16); retained_idx_host [C,R] int32; out_host pinned, of the output dtype.  Returns
        out_host; the copies into it are ordered before later work on the stream (synchronise it before
        reading)."""
        B, T = self.B, self.T
        for name, h, heads in (("q_host", q_host, self.Hq), ("k_host", k_host, self.Hkv), ("v_host", v_host, self.Hkv),
                               ("out_host", out_host, self.Hq)):
            if h.numel() != B * T * heads * self.D or not h.is_pinned() or not h.is_contiguous():
                raise ValueError(f"{name} must be a contiguous pinned host tensor of {B} x {T} x {heads} x {self.D} elements")
        if q_host.element_size() != 2 or k_host.element_size() != 2 or v_host.element_size() != 2:
            raise ValueError("q_host / k_host / v_host hold bf16 values (torch.bfloat16, or their bits as int16)")
        if out_host.dtype != self.out.dtype:
            raise ValueError("out_host must have the output dtype")
        if (lse_host is None) != (self.lse is None):
            raise ValueError("lse_host goes with with_lse=True")
        hp = lambda t: None if t is None else ctypes.c_void_p(t.data_ptr())
        rc = load().vxl_chunk_prefill_host(
            hp(q_host), hp(k_host), hp(v_host), self.L, hp(retained_idx_host) if self.R > 0 else None, self.R,
            hp(out_host), hp(lse_host), _ptr(self.q), _ptr(self.k), _ptr(self.v), _ptr(self.ridx), _ptr(self.out),
            _ptr(self.lse), self.per_call, ctypes.byref(self.shape), _ptr(self.ws), self.ws.numel(), _stream(stream),
            ctypes.c_void_p(self.s_in.cuda_stream), ctypes.c_void_p(self.s_out.cuda_stream))
        if rc != VXL_OK:
            raise VxlError(rc, "vxl_chunk_prefill_host")
        return out_host


class OfflineDecoder:
    """Bi-level decoding with the dense cache in pinned host memory (vxl_bilevel_decode_offline).

    Holds the buffers a call needs (staging slots for the selected chunks, the host copy of the
    selection, outputs, workspace, a copy stream), so that ``step`` itself allocates nothing."""

    def __init__(self, k_host, v_host, chunk_offsets_host, sparse, topk: int, max_chunk_len: int, Hq: int,
                 device="cuda", scale=None):
        if not (k_host.is_pinned() and v_host.is_pinned()):
            raise ValueError("k_host / v_host must be pinned host tensors")
        self.k_host, self.v_host, self.sparse = k_host, v_host, sparse
        B, T, Hkv, D = k_host.shape
        self.B, self.T, self.Hkv, self.D, self.Hq, self.topk, self.Lmax = B, T, Hkv, D, Hq, topk, max_chunk_len
        self.off_host = chunk_offsets_host.to(torch.int32).contiguous()
        self.off = self.off_host.to(device)
        self.C = int(self.off_host.numel()) - 1
        self.R = int(sparse[0].shape[1]) // self.C
        self.k_stage = torch.empty((B, topk, max_chunk_len, Hkv, D), dtype=torch.bfloat16, device=device)
        self.v_stage = torch.empty_like(self.k_stage)
        self.topk_host = torch.empty((B, topk), dtype=torch.int32).pin_memory()
        self.out = torch.empty((B, Hq, D), dtype=torch.float32, device=device)
        self.lse = torch.empty((B, Hq), dtype=torch.float32, device=device)
        self.scores = torch.empty((B, self.C), dtype=torch.float32, device=device)
        self.topk_out = torch.empty((B, topk), dtype=torch.int32, device=device)
        self.copy_stream = torch.cuda.Stream(device=device)
        self.shape = make_shape(B=B, T=T, Hq=Hq, Hkv=Hkv, D=D, q_strides=(Hq * D, 0, D),
                                kv_strides=(k_host.stride(0), k_host.stride(1), k_host.stride(2)),
                                scale=scale or 0.0)
        self.ws = new_workspace(workspace_bytes(VXL_OP_DECODE, self.shape, self.C, self.R, topk, max_chunk_len), device)
        self._lvl = VxlSparseLevel(sparse[0].data_ptr(), sparse[1].data_ptr())

    def step(self, q, stream=None):
        """q [B,Hq,D] bf16 CUDA, contiguous.  Returns (out, lse, scores, topk) views of the held buffers."""
        _check_bf16(q)
        rc = load().vxl_bilevel_decode_offline(
            _ptr(q), ctypes.c_void_p(self.k_host.data_ptr()), ctypes.c_void_p(self.v_host.data_ptr()),
            _ptr(self.off), ctypes.c_void_p(self.off_host.data_ptr()), self.C, self.Lmax, ctypes.byref(self._lvl),
            self.R, self.topk, _ptr(self.k_stage), _ptr(self.v_stage), ctypes.c_void_p(self.topk_host.data_ptr()),
            _ptr(self.out), _ptr(self.lse), _ptr(self.scores), _ptr(self.topk_out), ctypes.byref(self.shape),
            _ptr(self.ws), self.ws.numel(), _stream(stream), ctypes.c_void_p(self.copy_stream.cuda_stream))
        if rc != VXL_OK:
            raise VxlError(rc, "vxl_bilevel_decode_offline")
        return self.out, self.lse, self.scores, self.topk_out


def pack_retained(k_cache, v_cache, retained_idx, *, stream=None):
    """Build the contiguous sparse level [B, C*R, Hkv, D] for K and V."""
    _check_bf16(k_cache, v_cache)
    B, T, Hkv, D = k_cache.shape
    C = int(retained_idx.shape[-2])
    ridx, R, rsb = _ridx_args(retained_idx, C)
    ks = torch.empty((B, C * R, Hkv, D), dtype=torch.bfloat16, device=k_cache.device)
    vs = torch.empty_like(ks)
    shape = make_shape(B=B, T=T, Hq=Hkv, Hkv=Hkv, D=D, q_strides=(0, 0, D),
                       kv_strides=(k_cache.stride(0), k_cache.stride(1), k_cache.stride(2)))
    rc = load().vxl_pack_retained(_ptr(k_cache), _ptr(v_cache), _ptr(ridx), C, R, rsb, _ptr(ks), _ptr(vs),
                                  ctypes.byref(shape), _stream(stream))
    if rc != VXL_OK:
        raise VxlError(rc, "vxl_pack_retained")
    return ks, vs


def pool_sparse(k_cache, v_cache, chunk_offsets, R: int, *, stream=None):
    """Average-pooled sparse level [B, C*R, Hkv, D] for K and V (R pooled rows per chunk)."""
    _check_bf16(k_cache, v_cache)
    B, T, Hkv, D = k_cache.shape
    C = int(chunk_offsets.numel()) - 1
    ks = torch.empty((B, C * R, Hkv, D), dtype=torch.bfloat16, device=k_cache.device)
    vs = torch.empty_like(ks)
    shape = make_shape(B=B, T=T, Hq=Hkv, Hkv=Hkv, D=D, q_strides=(0, 0, D),
                       kv_strides=(k_cache.stride(0), k_cache.stride(1), k_cache.stride(2)))
    rc = load().vxl_pool_sparse(_ptr(k_cache), _ptr(v_cache), _ptr(chunk_offsets), C, R, _ptr(ks), _ptr(vs),
                                ctypes.byref(shape), _stream(stream))
    if rc != VXL_OK:
        raise VxlError(rc, "vxl_pool_sparse")
    return ks, vs


def bf16_from_bits(bits, device):
    """uint16 bit patterns (NumPy) -> bf16 CUDA tensor holding exactly those bytes."""
    import numpy as np
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.to(device).view(torch.bfloat16)
