"""vxl_chunk_scores_static: the scores/top-k call for callers that cannot allocate.

Some users of this library run where cudaMalloc is not an option: inside a host application
that has claimed the whole device heap, or in a serving loop whose memory is fixed at start-up.
For them the library offers one call whose scratch is a fixed array inside the library image.
This file checks, through the C ABI, that the call gives the same answer as the ordinary
vxl_chunk_scores (which takes a caller-allocated workspace), twice in a row on different
problems, so that whatever the first call leaves behind in the shared array cannot leak into
the second.  It is named to be collected last: it must pass after every other test has used
the GPU, and equally when run alone in a fresh process.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2506_19225_b200 import binding as vb
from paper_2506_19225_b200 import inputs
from oracle import ref
from tests.parity import LSE_ABS_ERR, TOPK_NEAR_TIE, to_gpu

pytestmark = pytest.mark.gpu


def _problem(B, T, L, R, topk, seed, packed):
    d = inputs.make_decode(B=B, T=T, L=L, R=R, Hq=28, Hkv=4, D=128, seed=seed, n_planted=2)
    q, k, v = to_gpu(d.q), to_gpu(d.k), to_gpu(d.v)
    off = torch.from_numpy(d.chunk_offsets).cuda()
    ridx = torch.from_numpy(np.ascontiguousarray(d.retained_idx)).cuda()
    sparse = vb.pack_retained(k, v, ridx) if packed else None
    return d, q, k, off, ridx, sparse, topk


def _compare(prob):
    d, q, k, off, ridx, sparse, topk = prob
    # reference: the existing entry point with its caller-allocated workspace
    want_scores, want_topk = vb.chunk_scores(q, k, off, ridx, topk=topk, scale=d.scale, sparse=sparse)
    # everything the static call writes is allocated before it runs
    scores = torch.full((d.B, d.C), float("nan"), dtype=torch.float32, device="cuda")
    topk_idx = torch.full((d.B, topk), -1, dtype=torch.int32, device="cuda")
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    vb.chunk_scores_static(q, k, off, ridx, scores, topk=topk, topk_idx=topk_idx, device_status=status,
                           scale=d.scale, sparse=sparse)
    torch.cuda.synchronize()
    assert int(status.item()) == vb.VXL_OK
    # the two entry points run the same kernels on the same inputs: equal bit for bit, not merely close
    assert torch.equal(scores, want_scores)
    assert torch.equal(topk_idx, want_topk)
    # and the answer is the right one: the fp64 oracle on the same bytes
    for b in range(d.B):
        _, sc = ref.scores(d.q[b], d.k[b], d.retained_idx, d.scale)
        idx, gap = ref.topk(sc, topk)
        err = np.abs(scores[b].double().cpu().numpy() - sc).max()
        assert err <= LSE_ABS_ERR, f"scores differ from the oracle by {err:.3e}"
        assert topk_idx[b].cpu().tolist() == idx.tolist() or gap < TOPK_NEAR_TIE


def test_static_scratch_matches_workspace_call_twice_in_a_row():
    first = _problem(B=3, T=8192, L=256, R=32, topk=5, seed=41, packed=True)     # 32 chunks, TMA stream path
    second = _problem(B=2, T=2048, L=128, R=16, topk=3, seed=42, packed=False)   # 16 chunks, rows by index
    _compare(first)
    _compare(second)      # smaller problem over the first call's leftovers
    _compare(first)       # and back again


def test_static_scratch_refuses_problems_beyond_its_size():
    lib = vb.load()
    C = 4096
    q = torch.zeros((16, 64, 128), dtype=torch.bfloat16, device="cuda")
    k = torch.zeros((16, C, 4, 128), dtype=torch.bfloat16, device="cuda")
    shape = vb._decode_shape(q, k, None, None, False)
    assert vb.workspace_bytes(vb.VXL_OP_SCORES, shape, C, 1) > vb.STATIC_SCRATCH_BYTES
    off = torch.arange(C + 1, dtype=torch.int32, device="cuda")
    ridx = torch.arange(C, dtype=torch.int32, device="cuda").reshape(C, 1)
    scores = torch.zeros((16, C), dtype=torch.float32, device="cuda")
    rc = lib.vxl_chunk_scores_static(vb._ptr(q), vb._ptr(k), vb._ptr(off), C, vb._ptr(ridx), 1, 0, None,
                                     vb._ptr(scores), 0, None, None, ctypes.byref(shape), vb._stream())
    assert rc == vb.VXL_ERR_WORKSPACE
    torch.cuda.synchronize()


def test_static_scratch_reports_a_bad_index_and_a_refused_call_touches_nothing():
    d, q, k, off, ridx, sparse, topk = _problem(B=2, T=2048, L=128, R=16, topk=3, seed=43, packed=False)
    scores = torch.zeros((d.B, d.C), dtype=torch.float32, device="cuda")
    topk_idx = torch.zeros((d.B, topk), dtype=torch.int32, device="cuda")
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    bad = ridx.clone()
    bad[1, 2] = d.T + 5                      # outside its chunk and the cache: clamped when read, reported under validate
    vb.chunk_scores_static(q, k, off, bad, scores, topk=topk, topk_idx=topk_idx, device_status=status,
                           scale=d.scale, validate=True)
    torch.cuda.synchronize()
    assert int(status.item()) == vb.VXL_ERR_INVALID_INDEX
    # a call refused on the host (topk > C) enqueues nothing: the status word of the call before it is still there
    lib = vb.load()
    shape = vb._decode_shape(q, k, None, None, False)
    rc = lib.vxl_chunk_scores_static(vb._ptr(q), vb._ptr(k), vb._ptr(off), d.C, vb._ptr(ridx), d.R, 0, None,
                                     vb._ptr(scores), d.C + 1, vb._ptr(topk_idx), vb._ptr(status),
                                     ctypes.byref(shape), vb._stream())
    assert rc == vb.VXL_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert int(status.item()) == vb.VXL_ERR_INVALID_INDEX
    # the next good call starts from a clean status word
    vb.chunk_scores_static(q, k, off, ridx, scores, topk=topk, topk_idx=topk_idx, device_status=status, scale=d.scale,
                           validate=True)
    torch.cuda.synchronize()
    assert int(status.item()) == vb.VXL_OK
