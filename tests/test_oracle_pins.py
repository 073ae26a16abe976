"""Pins for the fp64 oracle: what the paper and the mathematics fix, independent of the oracle.

Each test names the statement it checks.  The comparisons are against library routines
(torch scaled_dot_product_attention in fp64, numpy sort/logsumexp), closed forms, a
hand-computed rational fixture and an independent brute-force twin.
"""
import json
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import brute, ref
from paper_2506_19225_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden", "hand_case.json")


def _bits(a):
    return inputs.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def _sdpa(q, k, v, scale, causal):
    """Library dense attention in fp64.  q [T,Hq,D], k/v [T,Hkv,D] -> [T,Hq,D]."""
    G = q.shape[1] // k.shape[1]
    qt = torch.from_numpy(q).permute(1, 0, 2)[None]
    kt = torch.from_numpy(np.repeat(k, G, axis=1)).permute(1, 0, 2)[None]
    vt = torch.from_numpy(np.repeat(v, G, axis=1)).permute(1, 0, 2)[None]
    o = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=causal, scale=scale)
    return o[0].permute(1, 0, 2).numpy()


def small_case(T=96, L=32, R=5, Hq=4, Hkv=2, D=16, seed=7, **kw):
    return inputs.make_prefill(T=T, L=L, R=R, Hq=Hq, Hkv=Hkv, D=D, seed=seed, **kw)


# ---------------------------------------------------------------- hand-computed fixture
def test_hand_fixture_prefill():
    g = json.load(open(GOLD))
    p = g["prefill"]
    q = _bits(p["q"]).reshape(g["T"], p["Hq"], g["D"])
    k = _bits(g["k"]).reshape(g["T"], 1, g["D"])
    v = _bits(g["v"]).reshape(g["T"], 1, g["D"])
    out, lse = ref.prefill(q, k, v, g["L"], np.array(g["retained_idx"]), math.log(2.0))
    want = np.array([[float(Fraction(*x)) for x in row] for row in p["out"]])
    np.testing.assert_allclose(out[:, 0, :], want, rtol=0, atol=1e-14)
    want_lse = np.log([float(Fraction(*x)) for x in p["exp_lse"]])
    np.testing.assert_allclose(lse[:, 0], want_lse, rtol=0, atol=1e-14)


def test_hand_fixture_decode():
    g = json.load(open(GOLD))
    d = g["decode"]
    ln2 = math.log(2.0)
    q = _bits(d["q"]).reshape(d["Hq"], g["D"])
    k = _bits(g["k"]).reshape(g["T"], 1, g["D"])
    v = _bits(g["v"]).reshape(g["T"], 1, g["D"])
    ridx = np.array(g["retained_idx"])
    lse_hc, sc = ref.scores(q, k, ridx, ln2)
    np.testing.assert_allclose(np.exp(lse_hc), [[float(Fraction(*x)) for x in r] for r in d["exp_lse_hc"]],
                               rtol=1e-14)
    np.testing.assert_allclose(sc, [float(Fraction(*x)) * ln2 for x in d["scores_in_ln2"]], rtol=1e-14)
    idx, gap = ref.topk(sc, 1)
    assert idx.tolist() == d["top1"]
    assert abs(gap - 2.5 * ln2) < 1e-14
    for sel, ko, kl in (([1], "sel1_out", "sel1_exp_lse"), ([], "sel_none_out", "sel_none_exp_lse")):
        out, lse = ref.decode(q, k, v, d["chunk_offsets"], ridx, sel, ln2)
        want = np.array([[float(Fraction(*x)) for x in row] for row in d[ko]])
        np.testing.assert_allclose(out, want, rtol=0, atol=1e-14)
        np.testing.assert_allclose(np.exp(lse), [float(Fraction(*x)) for x in d[kl]], rtol=1e-13)


# ---------------------------------------------------------------- reductions to textbook attention
def test_all_retained_equals_dense_causal():
    """R = L with every position retained: the sparsification vanishes (dense causal)."""
    c = small_case(T=96, L=32, R=32)
    out, _ = ref.prefill(c.q, c.k, c.v, c.L, c.retained_idx, c.scale)
    want = _sdpa(inputs.bf16_bits_to_f64(c.q), inputs.bf16_bits_to_f64(c.k),
                 inputs.bf16_bits_to_f64(c.v), c.scale, causal=True)
    np.testing.assert_allclose(out, want, rtol=0, atol=1e-12)


def test_single_chunk_equals_causal():
    c = small_case(T=64, L=64, R=3)
    out, _ = ref.prefill(c.q, c.k, c.v, c.L, c.retained_idx, c.scale)
    want = _sdpa(inputs.bf16_bits_to_f64(c.q), inputs.bf16_bits_to_f64(c.k),
                 inputs.bf16_bits_to_f64(c.v), c.scale, causal=True)
    np.testing.assert_allclose(out, want, rtol=0, atol=1e-12)


def test_no_retained_is_block_diagonal_causal():
    """R = 0: the 'naive' variant in which each chunk attends only to itself."""
    c = small_case(T=96, L=32, R=0)
    out, _ = ref.prefill(c.q, c.k, c.v, c.L, c.retained_idx, c.scale)
    qf, kf, vf = (inputs.bf16_bits_to_f64(x) for x in (c.q, c.k, c.v))
    for ch in range(c.C):
        s = slice(ch * c.L, (ch + 1) * c.L)
        want = _sdpa(qf[s], kf[s], vf[s], c.scale, causal=True)
        np.testing.assert_allclose(out[s], want, rtol=0, atol=1e-12)


def test_later_chunk_sees_only_retained_history():
    """Changing a non-retained K/V row of an earlier chunk must not change later chunks;
    changing a retained one must."""
    c = small_case(T=96, L=32, R=4, seed=11)
    base, _ = ref.prefill(c.q, c.k, c.v, c.L, c.retained_idx, c.scale)
    keep = set(c.retained_idx[0].tolist())
    free = next(p for p in range(32) if p not in keep)
    k2, v2 = c.k.copy(), c.v.copy()
    k2[free] = _bits(np.full(k2[free].shape, 3.0))
    v2[free] = _bits(np.full(v2[free].shape, -5.0))
    out2, _ = ref.prefill(c.q, k2, v2, c.L, c.retained_idx, c.scale)
    np.testing.assert_array_equal(out2[32:], base[32:])
    assert np.abs(out2[free:32] - base[free:32]).max() > 1e-3
    k3 = c.k.copy()
    p = int(c.retained_idx[0, 0])
    k3[p] = _bits(np.full(k3[p].shape, 3.0))
    out3, _ = ref.prefill(c.q, k3, c.v, c.L, c.retained_idx, c.scale)
    assert np.abs(out3[32:] - base[32:]).max() > 1e-6
    # retained rows of the token's own chunk and of later chunks are not extra keys
    ridx2 = c.retained_idx.copy()
    ridx2[2] = ridx2[2][::-1]
    out4, _ = ref.prefill(c.q, c.k, c.v, c.L, ridx2, c.scale)
    np.testing.assert_array_equal(out4, base)


# ---------------------------------------------------------------- invariants and closed forms
def test_softmax_rows_sum_to_one_and_lse_consistent():
    c = small_case()
    out, lse = ref.prefill(c.q, c.k, c.v, c.L, c.retained_idx, c.scale)
    M = brute.chunk_mask(c.T, c.L, c.retained_idx)
    qf, kf = inputs.bf16_bits_to_f64(c.q), inputs.bf16_bits_to_f64(c.k)
    G = c.Hq // c.Hkv
    for h in range(c.Hq):
        x = c.scale * qf[:, h] @ kf[:, h // G].T
        p = np.where(M, np.exp(x - lse[:, h:h + 1]), 0.0)
        np.testing.assert_allclose(p.sum(axis=1), 1.0, rtol=0, atol=1e-12)
    # V constant -> output equals that constant (weights sum to one)
    vc = _bits(np.full(c.v.shape, 0.75))
    outc, _ = ref.prefill(c.q, c.k, vc, c.L, c.retained_idx, c.scale)
    np.testing.assert_allclose(outc, 0.75, rtol=0, atol=1e-12)


def test_zero_query_gives_mean_of_allowed_values():
    c = small_case(seed=3)
    q0 = np.zeros_like(c.q)
    out, lse = ref.prefill(q0, c.k, c.v, c.L, c.retained_idx, c.scale)
    M = brute.chunk_mask(c.T, c.L, c.retained_idx)
    vf = inputs.bf16_bits_to_f64(c.v)
    G = c.Hq // c.Hkv
    for i in range(c.T):
        want = vf[M[i]].mean(axis=0)                      # [Hkv, D]
        np.testing.assert_allclose(out[i], np.repeat(want, G, axis=0), rtol=0, atol=1e-13)
        np.testing.assert_allclose(lse[i], math.log(M[i].sum()), rtol=0, atol=1e-13)
    # number of allowed keys: (i mod L) + 1 in-chunk plus c*R retained
    i = 2 * c.L + 7
    assert M[i].sum() == 8 + 2 * c.R


def test_permutation_of_retained_set_changes_nothing():
    c = small_case(seed=5)
    rng = np.random.default_rng(0)
    ridx = c.retained_idx.copy()
    for row in ridx:
        rng.shuffle(row)
    a, la = ref.prefill(c.q, c.k, c.v, c.L, c.retained_idx, c.scale)
    b, lb = ref.prefill(c.q, c.k, c.v, c.L, ridx, c.scale)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-12)
    np.testing.assert_allclose(la, lb, rtol=0, atol=1e-12)


def test_rows_argument_matches_full():
    c = small_case(seed=9)
    full, lfull = ref.prefill(c.q, c.k, c.v, c.L, c.retained_idx, c.scale)
    rows = np.array([0, 31, 32, 33, 95, 64], dtype=np.int32)
    sub, lsub = ref.prefill(c.q, c.k, c.v, c.L, c.retained_idx, c.scale, rows=rows)
    np.testing.assert_array_equal(sub, full[rows])
    np.testing.assert_array_equal(lsub, lfull[rows])


# ---------------------------------------------------------------- brute-force twin
@pytest.mark.parametrize("T,L,R,Hq,Hkv,D,seed", [
    (64, 16, 3, 2, 1, 8, 1), (96, 32, 5, 4, 2, 16, 2), (120, 24, 24, 6, 2, 4, 3),
    (256, 64, 8, 2, 1, 64, 4), (48, 48, 0, 3, 3, 8, 5)])
def test_brute_force_twin_prefill(T, L, R, Hq, Hkv, D, seed):
    c = inputs.make_prefill(T=T, L=L, R=R, Hq=Hq, Hkv=Hkv, D=D, seed=seed, chunk_mean_std=0.5)
    a, la = ref.prefill(c.q, c.k, c.v, c.L, c.retained_idx, c.scale)
    b, lb = brute.prefill(c.q, c.k, c.v, c.L, c.retained_idx, c.scale)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-10)
    np.testing.assert_allclose(la, lb, rtol=0, atol=1e-10)


def small_decode(B=2, T=192, L=32, R=4, Hq=6, Hkv=2, D=16, seed=21):
    return inputs.make_decode(B=B, T=T, L=L, R=R, Hq=Hq, Hkv=Hkv, D=D, seed=seed, n_planted=2)


def test_brute_force_twin_decode_scores_topk():
    d = small_decode()
    for b in range(d.B):
        lse_hc, sc = ref.scores(d.q[b], d.k[b], d.retained_idx, d.scale)
        lse2, sc2 = brute.scores(d.q[b], d.k[b], d.retained_idx, d.scale)
        np.testing.assert_allclose(lse_hc, lse2, rtol=0, atol=1e-10)
        np.testing.assert_allclose(sc, sc2, rtol=0, atol=1e-10)
        for k in (0, 1, 2, 3, d.C):
            idx, gap = ref.topk(sc, k)
            assert idx.tolist() == brute.topk(sc, k).tolist()
            out, lse = ref.decode(d.q[b], d.k[b], d.v[b], d.chunk_offsets, d.retained_idx, idx, d.scale)
            o2, l2 = brute.decode(d.q[b], d.k[b], d.v[b], d.chunk_offsets, d.retained_idx, idx, d.scale)
            np.testing.assert_allclose(out, o2, rtol=0, atol=1e-10)
            np.testing.assert_allclose(lse, l2, rtol=0, atol=1e-10)


# ---------------------------------------------------------------- decode special cases
def _dense_decode(d, b):
    qf = inputs.bf16_bits_to_f64(d.q[b])[None]
    kf, vf = inputs.bf16_bits_to_f64(d.k[b]), inputs.bf16_bits_to_f64(d.v[b])
    G = d.Hq // d.Hkv
    qt = torch.from_numpy(qf).permute(1, 0, 2)[None]
    kt = torch.from_numpy(np.repeat(kf, G, axis=1)).permute(1, 0, 2)[None]
    vt = torch.from_numpy(np.repeat(vf, G, axis=1)).permute(1, 0, 2)[None]
    o = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, scale=d.scale)
    return o[0, :, 0, :].numpy()


def test_decode_all_selected_is_dense_attention():
    d = small_decode()
    out, _ = ref.decode(d.q[0], d.k[0], d.v[0], d.chunk_offsets, d.retained_idx,
                        np.arange(d.C), d.scale)
    np.testing.assert_allclose(out, _dense_decode(d, 0), rtol=0, atol=1e-12)


def test_decode_everything_retained_is_dense_for_any_k():
    d = small_decode(R=32)
    want = _dense_decode(d, 1)
    for sel in ([], [2], [0, 5]):
        out, _ = ref.decode(d.q[1], d.k[1], d.v[1], d.chunk_offsets, d.retained_idx, sel, d.scale)
        np.testing.assert_allclose(out, want, rtol=0, atol=1e-12)


def test_decode_none_selected_is_attention_over_sparse_level():
    d = small_decode()
    out, lse, rows = ref.decode(d.q[0], d.k[0], d.v[0], d.chunk_offsets, d.retained_idx, [],
                                d.scale, return_rows=True)
    assert sorted(rows.tolist()) == sorted(d.retained_idx.reshape(-1).tolist())
    sub_k = d.k[0][d.retained_idx.reshape(-1)]
    sub_v = d.v[0][d.retained_idx.reshape(-1)]
    dd = inputs.DecodeCase(name="x", B=1, T=sub_k.shape[0], L=1, R=0, Hq=d.Hq, Hkv=d.Hkv, D=d.D,
                           seed=0, n_planted=0)
    dd.q, dd.k, dd.v = d.q[:1], sub_k[None], sub_v[None]
    np.testing.assert_allclose(out, _dense_decode(dd, 0), rtol=0, atol=1e-12)
    # per-head LSE over the whole sparse level = logsumexp over chunks of the chunk LSEs
    lse_hc, _ = ref.scores(d.q[0], d.k[0], d.retained_idx, d.scale)
    np.testing.assert_allclose(np.log(np.exp(lse_hc).sum(axis=1)), lse, rtol=0, atol=1e-12)


def test_decode_mixed_row_list_and_order_independence():
    d = small_decode()
    sel = [4, 1]
    out, lse, rows = ref.decode(d.q[0], d.k[0], d.v[0], d.chunk_offsets, d.retained_idx, sel,
                                d.scale, return_rows=True)
    want = []
    for c in range(d.C):
        want += list(range(c * d.L, (c + 1) * d.L)) if c in sel else d.retained_idx[c].tolist()
    assert rows.tolist() == want                      # either dense or sparse, never both
    out2, lse2 = ref.decode(d.q[0], d.k[0], d.v[0], d.chunk_offsets, d.retained_idx, sel[::-1], d.scale)
    np.testing.assert_array_equal(out, out2)
    np.testing.assert_array_equal(lse, lse2)


def test_topk_matches_full_sort_and_tie_rule():
    rng = np.random.default_rng(4)
    sc = rng.standard_normal(37)
    for k in (0, 1, 5, 36, 37):
        idx, gap = ref.topk(sc, k)
        order = np.argsort(-sc, kind="stable")
        assert idx.tolist() == sorted(order[:k].tolist())
        if 0 < k < 37:
            assert gap == sc[order[k - 1]] - sc[order[k]]
    tie = np.array([1.0, 3.0, 3.0, 0.0, 3.0])
    assert ref.topk(tie, 2)[0].tolist() == [1, 2]      # equal scores: lower chunk index wins
    assert ref.topk(tie, 2)[1] == 0.0


def test_planted_chunks_are_selected():
    d = inputs.make_decode(B=2, T=64 * 256, L=256, R=32, Hq=28, Hkv=4, D=128, seed=33, n_planted=4)
    for b in range(d.B):
        _, sc = ref.scores(d.q[b], d.k[b], d.retained_idx, d.scale)
        idx, _ = ref.topk(sc, 8)
        assert set(d.planted[b].tolist()) <= set(idx.tolist())


def test_prefill_row_equals_decode_over_same_key_set():
    """Ties the two halves together: a prefill row is a decode over (earlier chunks sparse,
    own chunk dense and truncated at the row)."""
    c = small_case(T=128, L=32, R=6, Hq=4, Hkv=2, D=16, seed=13)
    out, lse = ref.prefill(c.q, c.k, c.v, c.L, c.retained_idx, c.scale)
    for i in (0, 31, 40, 100, 127):
        ch = i // c.L
        off = np.array([cc * c.L for cc in range(ch + 1)] + [i + 1], dtype=np.int32)
        o2, l2 = ref.decode(c.q[i], c.k[:i + 1], c.v[:i + 1], off, c.retained_idx[:ch + 1], [ch], c.scale)
        np.testing.assert_allclose(out[i], o2, rtol=0, atol=1e-12)
        np.testing.assert_allclose(lse[i], l2, rtol=0, atol=1e-12)


def test_inputs_are_bf16_exact_and_seeded():
    a = small_case(seed=99)
    b = small_case(seed=99)
    assert np.array_equal(a.q, b.q) and np.array_equal(a.retained_idx, b.retained_idx)
    x = np.array([1.0, 1.00390625, 1.005859375, -2.5, 3.1415927], dtype=np.float32)
    bits = inputs.f32_to_bf16_bits(x)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, want)
    for row, ch in zip(a.retained_idx, range(a.C)):
        assert np.all(np.diff(row) > 0) and row.min() >= ch * a.L and row.max() < (ch + 1) * a.L


# ---------------------------------------------------------------- sliding chunk window + prefix
def window_case(T_vis=96, L=32, step=16, prefix_len=7, R=3, Hq=4, Hkv=2, D=16, seed=31):
    return inputs.make_prefill_window(T_vis=T_vis, L=L, step=step, prefix_len=prefix_len, R=R, Hq=Hq,
                                      Hkv=Hkv, D=D, seed=seed)


def test_window_hand_fixture_visibility_sets():
    """Each token's key set, read off through one-hot values with a zero query, equals the sets
    written out by hand in the fixture."""
    with open(os.path.join(os.path.dirname(GOLD), "window_mask_case.json")) as f:
        g = json.load(f)
    T, D = g["T"], 16
    q = _bits(np.zeros((T, 1, D)))
    k = _bits(np.random.default_rng(0).standard_normal((T, 1, D)))
    v = np.zeros((T, 1, D), dtype=np.float32)
    v[np.arange(T), 0, np.arange(T)] = 1.0           # T <= D: value row j is the j-th unit vector
    out, lse = ref.prefill_window(q, k, _bits(v), g["L"], g["step"], g["prefix_len"],
                                  np.array(g["retained_idx"], dtype=np.int32), 1.0)
    for i in range(T):
        vis = g["visible"][str(i)]
        want = np.zeros(D)
        want[vis] = 1.0 / len(vis)
        np.testing.assert_allclose(out[i, 0], want, atol=1e-12)
        np.testing.assert_allclose(lse[i, 0], np.log(len(vis)), atol=1e-12)


def test_window_with_step_equal_to_chunk_and_no_prefix_is_the_plain_chunked_form():
    c = small_case()
    a, al = ref.prefill(c.q, c.k, c.v, c.L, c.retained_idx, c.scale)
    b, bl = ref.prefill_window(c.q, c.k, c.v, c.L, c.L, 0, c.retained_idx, c.scale)
    np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(al, bl)


@pytest.mark.parametrize("T_vis,L,step,prefix_len,R", [(96, 32, 16, 7, 3), (64, 32, 8, 0, 2), (60, 20, 10, 13, 0),
                                                        (48, 48, 12, 5, 4), (40, 8, 8, 3, 2)])
def test_window_brute_force_twin(T_vis, L, step, prefix_len, R):
    c = window_case(T_vis=T_vis, L=L, step=step, prefix_len=prefix_len, R=R)
    a, al = ref.prefill_window(c.q, c.k, c.v, c.L, c.step, c.prefix_len, c.retained_idx, c.scale)
    b, bl = brute.prefill_window(c.q, c.k, c.v, c.L, c.step, c.prefix_len, c.retained_idx, c.scale)
    np.testing.assert_allclose(a, b, atol=1e-10)
    np.testing.assert_allclose(al, bl, atol=1e-10)


def test_window_covering_everything_or_everything_retained_is_dense_causal():
    c = window_case(T_vis=64, L=64, step=16, prefix_len=9, R=2)          # one window holds all visual tokens
    q, k, v = (inputs.bf16_bits_to_f64(x) for x in (c.q, c.k, c.v))
    want = _sdpa(q, k, v, c.scale, True)
    got, _ = ref.prefill_window(c.q, c.k, c.v, c.L, c.step, c.prefix_len, c.retained_idx, c.scale)
    np.testing.assert_allclose(got, want, atol=1e-10)
    c = window_case(T_vis=64, L=32, step=16, prefix_len=5, R=16)         # every token of every block retained
    q, k, v = (inputs.bf16_bits_to_f64(x) for x in (c.q, c.k, c.v))
    want = _sdpa(q, k, v, c.scale, True)
    got, _ = ref.prefill_window(c.q, c.k, c.v, c.L, c.step, c.prefix_len, c.retained_idx, c.scale)
    np.testing.assert_allclose(got, want, atol=1e-10)


def test_window_prefix_rows_are_causal_over_the_prefix_and_visual_rows_see_all_of_it():
    c = window_case(prefix_len=11)
    P0 = c.prefix_len
    q, k, v = (inputs.bf16_bits_to_f64(x) for x in (c.q, c.k, c.v))
    got, _ = ref.prefill_window(c.q, c.k, c.v, c.L, c.step, P0, c.retained_idx, c.scale)
    np.testing.assert_allclose(got[:P0], _sdpa(q[:P0], k[:P0], v[:P0], c.scale, True), atol=1e-10)
    # changing a prefix value row changes every visual row; changing a visual row outside a token's
    # window and retained set does not change that token
    v2 = c.v.copy()
    v2[3] = _bits(inputs.bf16_bits_to_f32(c.v[3]) + 1.0)
    moved, _ = ref.prefill_window(c.q, c.k, v2, c.L, c.step, P0, c.retained_idx, c.scale)
    assert np.all(np.abs(moved[P0:] - got[P0:]).max(axis=(1, 2)) > 0)
    far = P0 + 1                                       # first-block token, not retained?
    if far not in set(c.retained_idx.reshape(-1).tolist()):
        v3 = c.v.copy()
        v3[far] = _bits(inputs.bf16_bits_to_f32(c.v[far]) + 1.0)
        moved, _ = ref.prefill_window(c.q, c.k, v3, c.L, c.step, P0, c.retained_idx, c.scale)
        last = c.T - 1                                 # its window starts well after token `far`
        np.testing.assert_array_equal(moved[last], got[last])


def test_window_key_count_closed_form():
    """q = 0: lse = ln(number of visible keys) = ln(prefix + window part + retained blocks)."""
    c = window_case(T_vis=128, L=48, step=16, prefix_len=6, R=3)
    q0 = _bits(np.zeros((c.T, c.Hq, c.D)))
    _, lse = ref.prefill_window(q0, c.k, c.v, c.L, c.step, c.prefix_len, c.retained_idx, c.scale)
    for i in range(c.T):
        if i < c.prefix_len:
            n = i + 1
        else:
            iv = i - c.prefix_len
            ws = max(0, (iv // c.step + 1) * c.step - c.L)
            n = c.prefix_len + (iv - ws + 1) + c.R * (ws // c.step)
        np.testing.assert_allclose(lse[i], np.log(n), atol=1e-12)


# ---------------------------------------------------------------- pooled sparse level
def test_pool_window_one_is_identity_and_constant_windows_stay_constant():
    d = small_decode()
    off = d.chunk_offsets
    same = ref.pool(d.k[0], off, d.L)                       # R = chunk length: windows of one row
    np.testing.assert_array_equal(same, d.k[0])
    x = d.k[0].copy()
    x[:] = np.repeat(x[::4], 4, axis=0)                     # rows constant within groups of 4
    np.testing.assert_array_equal(ref.pool(x, off, d.L // 4), x[::4])


def test_pool_hand_values_and_rounding_to_nearest_even():
    # one kv head, D = 2, one chunk of 4 rows pooled to 2: means of (1,2) and (3,4); (1, 1+2^-7) -> tie
    x = np.array([[[1.0, 1.0]], [[2.0, 1.0 + 2.0 ** -7]], [[3.0, -5.0]], [[4.0, -5.5]]], dtype=np.float32)
    got = inputs.bf16_bits_to_f64(ref.pool(_bits(x), np.array([0, 4], dtype=np.int32), 2))
    np.testing.assert_array_equal(got[:, 0, 0], [1.5, 3.5])
    assert got[0, 0, 1] == 1.0                              # 1 + 2^-8 lies halfway between 1 and 1 + 2^-7: even wins
    assert got[1, 0, 1] == -5.25
    # unequal windows: chunk of 5 rows pooled to 2 -> rows [0,2) and [2,5)
    y = np.arange(1, 6, dtype=np.float32).reshape(5, 1, 1)
    got = inputs.bf16_bits_to_f64(ref.pool(_bits(y), np.array([0, 5], dtype=np.int32), 2))
    np.testing.assert_array_equal(got[:, 0, 0], [1.5, 4.0])


def test_pool_rounding_in_the_subnormal_range_of_bf16():
    # bf16 below 2^-126 counts in units of 2^-133 (bit patterns 0x0001 .. 0x007f).  Means of two rows, by hand:
    #   (3u, 2u) -> 2.5u: tie, even wins -> 2u        (3u, 4u) -> 3.5u: tie -> 4u
    #   (127u, 128u) -> 127.5u: tie -> 128u = the smallest normal 0x0080 (the encoding runs on)
    #   (-1u, -2u) -> -1.5u: tie -> -2u               (1u, 0) -> 0.5u: tie -> 0
    #   (5u, 2u) -> 3.5u -> 4u ; (6u, 1u) -> 3.5u -> 4u ; (1u, 2u) -> 1.5u -> 2u
    rows = np.array([[0x0003, 0x0003, 0x007F, 0x8001, 0x0001, 0x0005, 0x0006, 0x0001],
                     [0x0002, 0x0004, 0x0080, 0x8002, 0x0000, 0x0002, 0x0001, 0x0002]], dtype=np.uint16)
    got = ref.pool(rows.reshape(2, 1, 8), np.array([0, 2], dtype=np.int32), 1).reshape(-1)
    assert got.tolist() == [0x0002, 0x0004, 0x0080, 0x8002, 0x0000, 0x0004, 0x0004, 0x0002]


def test_pool_matches_numpy_mean_within_half_an_ulp():
    d = small_decode(T=256, L=64, R=4)
    got = inputs.bf16_bits_to_f64(ref.pool(d.v[1], d.chunk_offsets, 8))
    want = brute.pool(d.v[1], 64, 8)
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(want), 1e-30))) - 7)
    assert np.all(np.abs(got - want) <= 0.5 * ulp + 1e-300)


def test_decode_levels_with_retained_rows_as_the_sparse_level_equals_decode():
    d = small_decode()
    for b in range(d.B):
        ks, vs = d.k[b][d.retained_idx.reshape(-1)], d.v[b][d.retained_idx.reshape(-1)]
        sel = np.array([1, 4], dtype=np.int32)
        a, al = ref.decode(d.q[b], d.k[b], d.v[b], d.chunk_offsets, d.retained_idx, sel, d.scale)
        c, cl = ref.decode_levels(d.q[b], d.k[b], d.v[b], ks, vs, d.chunk_offsets, sel, d.scale)
        np.testing.assert_allclose(a, c, atol=1e-12)
        np.testing.assert_allclose(al, cl, atol=1e-12)


def test_decode_levels_with_identity_pooling_is_dense_attention():
    d = small_decode()
    ks, vs = ref.pool(d.k[0], d.chunk_offsets, d.L), ref.pool(d.v[0], d.chunk_offsets, d.L)
    got, _ = ref.decode_levels(d.q[0], d.k[0], d.v[0], ks, vs, d.chunk_offsets, np.array([2], dtype=np.int32), d.scale)
    np.testing.assert_allclose(got, _dense_decode(d, 0), atol=1e-10)


# ---------------------------------------------------------------- query of several tokens
def test_scores_multi_is_the_mean_over_tokens_and_does_not_depend_on_their_order():
    d = small_decode()
    rng = np.random.default_rng(3)
    qs = _bits(rng.standard_normal((5, d.Hq, d.D)))
    one = [ref.scores(qs[t], d.k[0], d.retained_idx, d.scale)[1] for t in range(5)]
    got = ref.scores_multi(qs, d.k[0], d.retained_idx, d.scale)
    np.testing.assert_allclose(got, np.mean(one, axis=0), atol=1e-12)
    np.testing.assert_allclose(ref.scores_multi(qs[::-1].copy(), d.k[0], d.retained_idx, d.scale), got, atol=1e-12)
    np.testing.assert_array_equal(ref.scores_multi(qs[:1], d.k[0], d.retained_idx, d.scale), one[0])
    twice = np.concatenate([qs[2:3], qs[2:3]])
    np.testing.assert_allclose(ref.scores_multi(twice, d.k[0], d.retained_idx, d.scale), one[2], atol=1e-12)
    # brute-force twin, token by token
    bt = np.mean([brute.scores(qs[t], d.k[0], d.retained_idx, d.scale)[1] for t in range(5)], axis=0)
    np.testing.assert_allclose(got, bt, atol=1e-10)


# ---------------------------------------------------------------- other relevance forms
def test_mass_scores_sum_to_one_and_match_softmax_over_the_whole_sparse_level():
    d = small_decode()
    got = ref.scores_mass(d.q[0], d.k[0], d.retained_idx, d.scale)
    np.testing.assert_allclose(got.sum(), 1.0, atol=1e-12)
    # by definition: softmax of one head over ALL sparse rows, summed per chunk, then the mean over heads
    q, k = inputs.bf16_bits_to_f64(d.q[0]), inputs.bf16_bits_to_f64(d.k[0])
    G = d.Hq // d.Hkv
    want = np.zeros(d.C)
    flat = d.retained_idx.reshape(-1)
    for h in range(d.Hq):
        x = d.scale * (k[flat, h // G, :] @ q[h])
        pm = np.exp(x - x.max()); pm /= pm.sum()
        want += pm.reshape(d.C, d.R).sum(axis=1)
    np.testing.assert_allclose(got, want / d.Hq, atol=1e-12)


def test_mean_logit_relevance_is_the_lse_score_over_a_one_row_pooled_level():
    """The mean over a chunk's rows of scale*q.k is the logit against the chunk's mean key, and the
    log-sum-exp of a single logit is that logit: pooling with R = 1 turns the LSE score into it."""
    d = small_decode()
    pooled = inputs.bf16_bits_to_f64(ref.pool(d.k[0], d.chunk_offsets, 1))         # [C,Hkv,D], rounded to bf16
    _, got = ref.scores(d.q[0], ref.pool(d.k[0], d.chunk_offsets, 1), np.arange(d.C, dtype=np.int32).reshape(d.C, 1), d.scale)
    q = inputs.bf16_bits_to_f64(d.q[0])
    G = d.Hq // d.Hkv
    want = np.mean([d.scale * (pooled[:, h // G, :] @ q[h]) for h in range(d.Hq)], axis=0)
    np.testing.assert_allclose(got, want, atol=1e-12)
    # and against the unrounded mean key it differs only by the bf16 rounding of the pooled row
    k = inputs.bf16_bits_to_f64(d.k[0]).reshape(d.C, d.L, d.Hkv, d.D).mean(axis=1)
    exact = np.mean([d.scale * (k[:, h // G, :] @ q[h]) for h in range(d.Hq)], axis=0)
    assert np.abs(got - exact).max() < 2e-2
