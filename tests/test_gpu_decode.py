"""GPU parity: vxl_chunk_scores / vxl_bilevel_decode_attn / vxl_pack_retained vs the fp64 oracle."""
import functools

import numpy as np
import pytest
import torch

from oracle import ref
from paper_2506_19225_b200 import binding as vb
from paper_2506_19225_b200 import inputs
from tests.parity import LSE_ABS_ERR, TOPK_NEAR_TIE, check_close, to_gpu

pytestmark = pytest.mark.gpu


def gpu_tensors(d):
    return (to_gpu(d.q), to_gpu(d.k), to_gpu(d.v), torch.from_numpy(d.chunk_offsets).cuda(),
            torch.from_numpy(np.ascontiguousarray(d.retained_idx)).cuda() if d.R > 0 else None)


def oracle_selection(d, b, topk, ridx=None):
    ridx = d.retained_idx if ridx is None else ridx
    _, sc = ref.scores(d.q[b], d.k[b], ridx, d.scale)
    idx, gap = ref.topk(sc, topk)
    return sc, idx, gap


def check_decode(d, topk, *, sparse=False, per_seq_ridx=False):
    q, k, v, off, ridx = gpu_tensors(d)
    ridx_np = d.retained_idx
    if per_seq_ridx:
        rng = np.random.default_rng(5)
        ridx_np = np.stack([inputs.make_retained_idx(rng, d.C, d.L, d.R) for _ in range(d.B)])
        ridx = torch.from_numpy(ridx_np).cuda()
    sp = vb.pack_retained(k, v, ridx) if (sparse and d.R > 0) else None
    ws = vb.new_workspace(vb.workspace_bytes(vb.VXL_OP_DECODE, vb._decode_shape(q, k, None, None, False),
                                             d.C, d.R, topk, d.L), "cuda")
    res = vb.bilevel_decode_attn(q, k, v, off, ridx, topk, max_chunk_len=d.L, scale=d.scale, sparse=sp,
                                 return_lse=True, return_scores=True, workspace=ws, validate=True)
    torch.cuda.synchronize()
    assert vb.device_status(ws) == vb.VXL_OK
    near_ties = []
    for b in range(d.B):
        rb = ridx_np[b] if per_seq_ridx else ridx_np
        sc, idx, gap = oracle_selection(d, b, topk, rb)
        if d.R > 0:
            check_close(res["scores"][b], sc, f"{d.name} scores b{b}", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)
        got = res["topk"][b].cpu().numpy()
        assert np.all(np.diff(got) > 0), "top-k ids must be ascending and distinct"
        if got.tolist() != idx.tolist():
            # only acceptable when the oracle's k-th and (k+1)-th scores are a near tie
            assert gap < TOPK_NEAR_TIE, f"{d.name} b{b}: top-k {got.tolist()} != {idx.tolist()} (gap {gap:.3e})"
            near_ties.append((b, gap))
            assert len(set(got.tolist()) ^ set(idx.tolist())) == 2
        want, want_lse = ref.decode(d.q[b], d.k[b], d.v[b], d.chunk_offsets, rb, got, d.scale)
        check_close(res["out"][b], want, f"{d.name} out b{b} k{topk}")
        check_close(res["lse"][b], want_lse, f"{d.name} lse b{b}", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)
    if near_ties:
        print(f"near ties reported: {near_ties}")
    return res


SMALL = [
    # B, T, L, R, Hq, Hkv, D, topk
    (2, 1024, 128, 16, 28, 4, 128, 3),
    (1, 1024, 128, 16, 28, 4, 128, 0),       # k = 0: sparse level only
    (1, 1024, 128, 16, 28, 4, 128, 8),       # k = C: dense attention
    (3, 768, 96, 5, 6, 2, 64, 2),            # D = 64, two heads per CTA, ragged tiles
    (2, 640, 160, 33, 9, 3, 128, 1),         # Hkv = 3 (one kv head per CTA), G = 3
    (1, 512, 128, 128, 16, 1, 128, 1),       # everything retained, G = 16
    (1, 2048, 512, 0, 8, 4, 128, 2),         # R = 0
    (2, 4096, 2048, 64, 28, 4, 128, 1),      # long chunks: several slices
]


@pytest.mark.parametrize("sparse", [False, True])
@pytest.mark.parametrize("B,T,L,R,Hq,Hkv,D,topk", SMALL)
def test_small_decode(B, T, L, R, Hq, Hkv, D, topk, sparse):
    d = inputs.make_decode(B=B, T=T, L=L, R=R, Hq=Hq, Hkv=Hkv, D=D, seed=100 + T + R + topk,
                           n_planted=min(2, T // L), name=f"small B{B} T{T} L{L} R{R} D{D}")
    check_decode(d, topk, sparse=sparse)


@pytest.mark.parametrize("B,T,L,R,Hq,Hkv,topk", [
    (40, 512, 128, 8, 8, 4, 1),        # one dense item per sequence, fewer items than SMs
    (200, 256, 64, 4, 8, 4, 2),        # 400 items in blocks of three: a CTA's block straddles sequences
    (24, 1024, 128, 16, 28, 4, 3),
    (300, 256, 64, 4, 4, 4, 4),        # B * topk beyond the in-kernel selection scratch: separate top-k launch
])
def test_many_sequences_over_a_packed_level(B, T, L, R, Hq, Hkv, topk):
    # the dense pass ranks the chunks itself when the sparse level is packed: its CTAs then own
    # contiguous blocks of items, whatever their alignment to the sequences
    d = inputs.make_decode(B=B, T=T, L=L, R=R, Hq=Hq, Hkv=Hkv, D=128, seed=300 + B, n_planted=min(2, T // L),
                           name=f"many B{B} T{T} L{L}")
    check_decode(d, topk, sparse=True)


def test_per_sequence_retained_idx():
    d = inputs.make_decode(B=3, T=1024, L=128, R=12, Hq=8, Hkv=2, D=128, seed=9, n_planted=2)
    check_decode(d, 2, per_seq_ridx=True)
    check_decode(d, 2, per_seq_ridx=True, sparse=True)


def test_user_selected_chunks_and_order():
    d = inputs.make_decode(B=2, T=1024, L=128, R=16, Hq=28, Hkv=4, D=128, seed=10, n_planted=2)
    q, k, v, off, ridx = gpu_tensors(d)
    sel = np.array([[5, 1, 6], [0, 7, 3]], dtype=np.int32)
    res = vb.bilevel_decode_attn(q, k, v, off, ridx, 3, max_chunk_len=d.L, scale=d.scale,
                                 selected=torch.from_numpy(sel).cuda(), return_lse=True)
    for b in range(d.B):
        want, want_lse = ref.decode(d.q[b], d.k[b], d.v[b], d.chunk_offsets, d.retained_idx, sel[b], d.scale)
        check_close(res["out"][b], want, f"selected b{b}")
        check_close(res["lse"][b], want_lse, f"selected lse b{b}", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)


def test_unequal_chunks():
    d = inputs.make_decode(B=1, T=1024, L=128, R=8, Hq=8, Hkv=2, D=128, seed=12, n_planted=1)
    off = np.array([0, 100, 300, 333, 700, 1000], dtype=np.int32)       # off[C] < T is allowed
    rng = np.random.default_rng(2)
    ridx = np.stack([np.sort(rng.choice(np.arange(off[c], off[c + 1]), size=8, replace=False))
                     for c in range(5)]).astype(np.int32)
    q, k, v = to_gpu(d.q), to_gpu(d.k), to_gpu(d.v)
    res = vb.bilevel_decode_attn(q, k, v, torch.from_numpy(off).cuda(), torch.from_numpy(ridx).cuda(), 2,
                                 max_chunk_len=367, scale=d.scale, return_lse=True, return_scores=True,
                                 validate=True)
    _, sc = ref.scores(d.q[0], d.k[0], ridx, d.scale)
    idx, gap = ref.topk(sc, 2)
    assert res["topk"][0].cpu().tolist() == idx.tolist() or gap < TOPK_NEAR_TIE
    want, _ = ref.decode(d.q[0], d.k[0], d.v[0], off, ridx, res["topk"][0].cpu().numpy(), d.scale)
    check_close(res["out"][0], want, "unequal chunks")


def test_chunk_scores_standalone_and_pack():
    d = inputs.make_decode(B=2, T=2048, L=128, R=16, Hq=28, Hkv=4, D=128, seed=14, n_planted=2)
    q, k, v, off, ridx = gpu_tensors(d)
    ks, vs = vb.pack_retained(k, v, ridx)
    flat = torch.from_numpy(d.retained_idx.reshape(-1).astype(np.int64)).cuda()
    assert torch.equal(ks, k[:, flat]) and torch.equal(vs, v[:, flat])     # byte-exact gather
    for sp in (None, (ks, None)):
        scores, topk = vb.chunk_scores(q, k, off, ridx, topk=4, scale=d.scale, sparse=sp)
        for b in range(d.B):
            sc, idx, gap = oracle_selection(d, b, 4)
            check_close(scores[b], sc, "scores", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)
            assert topk[b].cpu().tolist() == idx.tolist() or gap < TOPK_NEAR_TIE


def test_topk_tie_rule_on_equal_scores():
    """Identical chunks give bit-identical scores on the GPU: the lower chunk ids must win."""
    d = inputs.make_decode(B=1, T=512, L=64, R=8, Hq=4, Hkv=2, D=128, seed=15, n_planted=0)
    for c in range(1, d.C):
        d.k[0, c * 64:(c + 1) * 64] = d.k[0, :64]
    d.retained_idx = (d.retained_idx[0][None, :] + 64 * np.arange(d.C)[:, None]).astype(np.int32)
    q, k, v, off, ridx = gpu_tensors(d)
    _, topk = vb.chunk_scores(q, k, off, ridx, topk=3, scale=d.scale)
    assert topk[0].cpu().tolist() == [0, 1, 2]


@functools.lru_cache(maxsize=1)
def _cfg5(B):
    return inputs.make_decode_cfg5(B)          # the 8-sequence cache takes a while to draw: made once


@pytest.mark.parametrize("sparse", [True, False], ids=["packed_level", "rows_by_index"])
@pytest.mark.parametrize("B,topk", [(1, 8), (1, 16), (8, 8), (8, 16)])
def test_cfg5_full_size(B, topk, sparse):
    """The 262,144-token decode configuration, every output compared.  `packed_level` is the call the
    benchmark times (stored sparse level streamed by TMA, the dense pass ranking the chunks itself);
    `rows_by_index` gathers the sparse rows from the dense cache and ranks in a launch of its own."""
    d = _cfg5(B)
    res = check_decode(d, topk, sparse=sparse)
    for b in range(B):
        assert set(d.planted[b].tolist()) <= set(res["topk"][b].cpu().tolist())


def test_rows_past_the_end_of_an_item_never_reach_the_output():
    """Ragged chunks whose last 32-row tile runs into memory the call does not own: unwritten cache
    capacity after the last chunk (NaN here) and, for the dense level kept on the host, staging slots that
    still hold whatever was there before (NaN here).  Their probabilities are zero; their V rows must not
    turn the output into NaN."""
    d = inputs.make_decode(B=2, T=1024, L=128, R=8, Hq=8, Hkv=4, D=128, seed=13, n_planted=1)
    off = np.array([0, 100, 300, 333, 700, 933], dtype=np.int32)            # lengths 100 / 200 / 33 / 367 / 233
    C = len(off) - 1
    rng = np.random.default_rng(3)
    ridx = np.stack([np.sort(rng.choice(np.arange(off[c], off[c + 1]), size=8, replace=False))
                     for c in range(C)]).astype(np.int32)
    q, k, v = to_gpu(d.q), to_gpu(d.k), to_gpu(d.v)
    k[:, off[C]:] = float("nan"); v[:, off[C]:] = float("nan")             # capacity nobody has written
    off_t, ridx_t = torch.from_numpy(off).cuda(), torch.from_numpy(ridx).cuda()
    level = vb.pack_retained(k, v, ridx_t)
    for topk, sparse in ((2, None), (2, level), (C, level), (1, level)):
        res = vb.bilevel_decode_attn(q, k, v, off_t, ridx_t, topk, max_chunk_len=367, scale=d.scale, sparse=sparse,
                                     return_lse=True, return_scores=True, validate=True)
        torch.cuda.synchronize()
        assert torch.isfinite(res["out"]).all() and torch.isfinite(res["lse"]).all()
        for b in range(d.B):
            got = res["topk"][b].cpu().numpy()
            want, want_lse = ref.decode(d.q[b], d.k[b], d.v[b], off, ridx, got, d.scale)
            check_close(res["out"][b], want, f"ragged tail b{b} k{topk}")
            check_close(res["lse"][b], want_lse, "ragged tail lse", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)
    # dense level on the host, staging slots poisoned before every step
    k_host, v_host = to_gpu(d.k).cpu().pin_memory(), to_gpu(d.v).cpu().pin_memory()
    dec = vb.OfflineDecoder(k_host, v_host, torch.from_numpy(off), level, 3, 367, d.Hq, scale=d.scale)
    for _ in range(2):
        dec.k_stage.fill_(float("nan")); dec.v_stage.fill_(float("nan"))
        out, lse, _, sel = dec.step(q)
        torch.cuda.synchronize()
        assert vb.device_status(dec.ws) == vb.VXL_OK
        assert torch.isfinite(out).all() and torch.isfinite(lse).all()
        for b in range(d.B):
            want, _ = ref.decode(d.q[b], d.k[b], d.v[b], off, ridx, sel[b].cpu().numpy(), d.scale)
            check_close(out[b], want, f"offline ragged b{b}")


def test_a_selected_chunk_longer_than_max_chunk_len_is_reported():
    d = inputs.make_decode(B=1, T=2048, L=512, R=16, Hq=8, Hkv=4, D=128, seed=17, n_planted=1)
    q, k, v, off, ridx = gpu_tensors(d)
    level = vb.pack_retained(k, v, ridx)
    shape = vb._decode_shape(q, k, None, None, False)
    ws = vb.new_workspace(vb.workspace_bytes(vb.VXL_OP_DECODE, shape, d.C, d.R, 2, 512), "cuda")
    vb.bilevel_decode_attn(q, k, v, off, ridx, 2, max_chunk_len=256, scale=d.scale, sparse=level, workspace=ws)
    assert vb.device_status(ws) == vb.VXL_ERR_INVALID_ARG              # the bound was not a bound
    vb.bilevel_decode_attn(q, k, v, off, ridx, 2, max_chunk_len=512, scale=d.scale, sparse=level, workspace=ws)
    assert vb.device_status(ws) == vb.VXL_OK


# ------------------------------------------------------------------ pooled sparse level
@pytest.mark.parametrize("B,T,L,R,Hkv,D", [(2, 1024, 128, 16, 4, 128), (1, 768, 96, 5, 2, 64), (1, 512, 128, 128, 1, 128)])
def test_pool_sparse_matches_oracle(B, T, L, R, Hkv, D):
    d = inputs.make_decode(B=B, T=T, L=L, R=min(R, 8), Hq=Hkv, Hkv=Hkv, D=D, seed=50 + T + R, n_planted=1)
    k, v, off = to_gpu(d.k), to_gpu(d.v), torch.from_numpy(d.chunk_offsets).cuda()
    ks, vs = vb.pool_sparse(k, v, off, R)
    torch.cuda.synchronize()
    for b in range(B):
        for got, src in ((ks, d.k), (vs, d.v)):
            g = got[b].view(torch.int16).cpu().numpy().view(np.uint16)
            want = ref.pool(src[b], d.chunk_offsets, R)
            # the kernel sums and divides in fp64 in row order and rounds once: the same bytes as the oracle
            np.testing.assert_array_equal(g, want)
    if R == L:
        assert torch.equal(ks, k) and torch.equal(vs, v)           # windows of one row: a copy


def test_decode_over_pooled_sparse_level():
    """Scores, top-k and mixed attention when the sparse level is pooled (no retained indices)."""
    d = inputs.make_decode(B=2, T=2048, L=256, R=8, Hq=28, Hkv=4, D=128, seed=61, n_planted=2)
    R = 32
    q, k, v, off, _ = gpu_tensors(d)
    ks, vs = vb.pool_sparse(k, v, off, R)
    res = vb.bilevel_decode_attn(q, k, v, off, None, 3, max_chunk_len=d.L, scale=d.scale, sparse=(ks, vs),
                                 return_lse=True, return_scores=True)
    torch.cuda.synchronize()
    ks_np = ks.view(torch.int16).cpu().numpy().view(np.uint16)
    vs_np = vs.view(torch.int16).cpu().numpy().view(np.uint16)
    level_idx = np.arange(d.C * R, dtype=np.int32).reshape(d.C, R)
    for b in range(d.B):
        # both sides read the same stored level (its bytes were checked against the oracle's pooling above)
        _, sc = ref.scores(d.q[b], ks_np[b], level_idx, d.scale)
        idx, gap = ref.topk(sc, 3)
        check_close(res["scores"][b], sc, "pooled scores", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)
        got = res["topk"][b].cpu().numpy()
        assert got.tolist() == idx.tolist() or gap < TOPK_NEAR_TIE
        want, want_lse = ref.decode_levels(d.q[b], d.k[b], d.v[b], ks_np[b], vs_np[b], d.chunk_offsets, got, d.scale)
        check_close(res["out"][b], want, f"pooled decode b{b}")
        check_close(res["lse"][b], want_lse, f"pooled lse b{b}", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)


# ------------------------------------------------------------------ richer relevance
@pytest.mark.parametrize("packed", [False, True])
def test_scores_for_a_query_of_several_tokens(packed):
    d = inputs.make_decode(B=2, T=2048, L=128, R=16, Hq=28, Hkv=4, D=128, seed=71, n_planted=2)
    _, k, v, off, ridx = gpu_tensors(d)
    rng = np.random.default_rng(8)
    Tq = 5
    q_bits = inputs.f32_to_bf16_bits(rng.standard_normal((d.B, Tq, d.Hq, d.D), dtype=np.float32))
    q = to_gpu(q_bits)
    sp = (vb.pack_retained(k, v, ridx)[0], None) if packed else None
    scores, topk = vb.chunk_scores_multi(q, k, off, ridx, topk=4, scale=d.scale, sparse=sp, validate=True)
    for b in range(d.B):
        sc = ref.scores_multi(q_bits[b], d.k[b], d.retained_idx, d.scale)
        check_close(scores[b], sc, "multi-token scores", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)
        idx, gap = ref.topk(sc, 4)
        assert topk[b].cpu().tolist() == idx.tolist() or gap < TOPK_NEAR_TIE
    one, _ = vb.chunk_scores(q[:, 0].contiguous(), k, off, ridx, scale=d.scale, sparse=sp)
    first, _ = vb.chunk_scores_multi(q[:, :1], k, off, ridx, scale=d.scale, sparse=sp)
    assert (one - first).abs().max().item() < 1e-5       # one token: the same sparse pass, another summation order over the heads


@pytest.mark.parametrize("packed", [False, True])
@pytest.mark.parametrize("B,T,L,R,Hq,Hkv", [(2, 4096, 128, 16, 28, 4), (1, 3072, 256, 32, 16, 2)])
def test_attention_mass_relevance_scores_selection_and_decode(packed, B, T, L, R, Hq, Hkv):
    d = inputs.make_decode(B=B, T=T, L=L, R=R, Hq=Hq, Hkv=Hkv, D=128, seed=75 + B, n_planted=3)
    q, k, v, off, ridx = gpu_tensors(d)
    sp = vb.pack_retained(k, v, ridx) if packed else None
    scores, topk = vb.chunk_scores(q, k, off, ridx, topk=3, scale=d.scale, sparse=sp, validate=True,
                                   score_mode=vb.VXL_SCORE_MASS)
    res = vb.bilevel_decode_attn(q, k, v, off, ridx, 3, max_chunk_len=d.L, scale=d.scale, sparse=sp,
                                 return_scores=True, score_mode=vb.VXL_SCORE_MASS)
    for b in range(d.B):
        want = ref.scores_mass(d.q[b], d.k[b], d.retained_idx, d.scale)
        check_close(scores[b], want, "mass scores", max_err=2e-3, mean_err=2e-4)
        assert abs(scores[b].sum().item() - 1.0) < 1e-4
        idx, gap = ref.topk(want, 3)
        assert topk[b].cpu().tolist() == idx.tolist() or gap < TOPK_NEAR_TIE
        assert res["topk"][b].cpu().tolist() == topk[b].cpu().tolist()
        out, _ = ref.decode(d.q[b], d.k[b], d.v[b], d.chunk_offsets, d.retained_idx,
                            np.array(sorted(topk[b].cpu().tolist()), dtype=np.int32), d.scale)
        check_close(res["out"][b], out, "decode under mass relevance")
    # the two rules rank differently in general, and both leave the LSE path untouched
    lse_scores, _ = vb.chunk_scores(q, k, off, ridx, scale=d.scale, sparse=sp)
    _, want_lse = ref.scores(d.q[0], d.k[0], d.retained_idx, d.scale)
    check_close(lse_scores[0], want_lse, "lse scores after a mass call", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)


def test_topk_select_from_given_scores_and_decode_with_it():
    rng = np.random.default_rng(9)
    sc = rng.standard_normal((3, 200)).astype(np.float32)
    sc[1, 17] = sc[1, 3] = sc[1, 150] = 9.0                # ties: the lower ids win
    got = vb.topk_select(torch.from_numpy(sc).cuda(), 2).cpu().numpy()
    for b in range(3):
        idx, _ = ref.topk(sc[b].astype(np.float64), 2)
        assert got[b].tolist() == idx.tolist()
    assert got[1].tolist() == [3, 17]
    # the selection drives the decode call
    d = inputs.make_decode(B=1, T=1024, L=128, R=16, Hq=28, Hkv=4, D=128, seed=72, n_planted=1)
    q, k, v, off, ridx = gpu_tensors(d)
    ext = torch.tensor([[0.1, 5.0, 0.2, 0.0, 4.0, -1.0, 0.3, 0.25]], dtype=torch.float32, device="cuda")
    sel = vb.topk_select(ext, 2)
    assert sel.cpu().tolist() == [[1, 4]]
    res = vb.bilevel_decode_attn(q, k, v, off, ridx, 2, max_chunk_len=d.L, scale=d.scale, selected=sel)
    want, _ = ref.decode(d.q[0], d.k[0], d.v[0], d.chunk_offsets, d.retained_idx, np.array([1, 4], dtype=np.int32), d.scale)
    check_close(res["out"][0], want, "decode with external scores")


# ------------------------------------------------------------------ dense level kept in host memory
@pytest.mark.parametrize("B,T,L,R,topk,pooled", [(2, 4096, 512, 32, 3, False), (1, 2048, 256, 16, 2, True),
                                                  (3, 1536, 192, 8, 8, False)])
def test_offline_store_decode_matches_oracle_and_the_in_memory_call(B, T, L, R, topk, pooled):
    d = inputs.make_decode(B=B, T=T, L=L, R=R, Hq=28, Hkv=4, D=128, seed=80 + T + topk, n_planted=2)
    q, k, v, off, ridx = gpu_tensors(d)
    level = vb.pool_sparse(k, v, off, R) if pooled else vb.pack_retained(k, v, ridx)
    k_host, v_host = k.cpu().pin_memory(), v.cpu().pin_memory()
    dec = vb.OfflineDecoder(k_host, v_host, torch.from_numpy(d.chunk_offsets), level, topk, d.L, d.Hq, scale=d.scale)
    for _ in range(2):                                   # the second step reuses the staging slots
        out, lse, scores, sel = dec.step(q)
        torch.cuda.synchronize()
        assert vb.device_status(dec.ws) == vb.VXL_OK
        res = vb.bilevel_decode_attn(q, k, v, off, None if pooled else ridx, topk, max_chunk_len=d.L, scale=d.scale,
                                     sparse=level, return_lse=True, return_scores=True)
        assert torch.equal(sel, res["topk"])
        assert (out - res["out"]).abs().max().item() < 1e-5 and (lse - res["lse"]).abs().max().item() < 1e-5
        assert torch.equal(dec.topk_host, sel.cpu())
        ks_np = level[0].view(torch.int16).cpu().numpy().view(np.uint16)
        vs_np = level[1].view(torch.int16).cpu().numpy().view(np.uint16)
        for b in range(B):
            want, want_lse = ref.decode_levels(d.q[b], d.k[b], d.v[b], ks_np[b], vs_np[b], d.chunk_offsets,
                                               sel[b].cpu().numpy(), d.scale)
            check_close(out[b], want, f"offline decode b{b}")
            check_close(lse[b], want_lse, f"offline lse b{b}", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)


@pytest.mark.parametrize("mode", ["index", "packed"])
def test_many_short_chunks(mode):
    """2048 chunks of 16 tokens: the ranking runs over more chunks than threads in a warp or a CTA row."""
    d = inputs.make_decode(B=2, T=32768, L=16, R=4, Hq=8, Hkv=2, D=64, seed=95, n_planted=3)
    check_decode(d, 37, sparse=(mode == "packed"))


def test_a_wait_that_runs_out_is_reported_and_the_workspace_stays_usable():
    """Failure path shared by every kernel: a bounded wait on a barrier nothing completes gives up after its
    limit (two million clocks here, about a millisecond), the status word says so, and the next call works."""
    d = inputs.make_decode(B=1, T=1024, L=128, R=16, Hq=8, Hkv=4, D=128, seed=19, n_planted=1)
    q, k, v, off, ridx = gpu_tensors(d)
    shape = vb._decode_shape(q, k, None, None, False)
    ws = vb.new_workspace(vb.workspace_bytes(vb.VXL_OP_DECODE, shape, d.C, d.R, 2, d.L), "cuda")
    assert vb.selftest_bounded_wait(ws, 2_000_000) == vb.VXL_OK           # the launch itself succeeds
    assert vb.device_status(ws) == vb.VXL_ERR_TIMEOUT
    assert vb.device_status(ws) == vb.VXL_OK                               # cleared by the read
    res = vb.bilevel_decode_attn(q, k, v, off, ridx, 2, max_chunk_len=d.L, scale=d.scale, workspace=ws, return_scores=True)
    torch.cuda.synchronize()
    assert vb.device_status(ws) == vb.VXL_OK
    want, _ = ref.decode(d.q[0], d.k[0], d.v[0], d.chunk_offsets, d.retained_idx, res["topk"][0].cpu().numpy(), d.scale)
    check_close(res["out"][0], want, "decode after a reported timeout")
