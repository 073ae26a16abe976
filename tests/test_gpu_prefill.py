"""GPU parity: vxl_chunk_prefill_attn (through the C ABI) against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2506_19225_b200 import binding as vb
from paper_2506_19225_b200 import inputs
from tests.parity import LSE_ABS_ERR, check_close, sample_rows, to_gpu

pytestmark = pytest.mark.gpu


def run_gpu(case, *, force_general=False, out_dtype=torch.float32, ridx=None, validate=False, gather4=False):
    q, k, v = (to_gpu(x) for x in (case.q, case.k, case.v))
    ridx = case.retained_idx if ridx is None else ridx
    ridx_t = torch.from_numpy(np.ascontiguousarray(ridx)).cuda() if case.R > 0 else None
    ws = vb.prefill_workspace(B=1, T=case.T, Hq=case.Hq, Hkv=case.Hkv, D=case.D, chunk_len=case.L, R=case.R,
                              device="cuda")
    out, lse = vb.chunk_prefill_attn(q, k, v, case.L, ridx_t, scale=case.scale, return_lse=True,
                                     out_dtype=out_dtype, force_general=force_general, workspace=ws,
                                     validate=validate, gather4=gather4)
    torch.cuda.synchronize()
    assert vb.device_status(ws) == vb.VXL_OK
    return out, lse


def compare_full(case, **kw):
    out, lse = run_gpu(case, **kw)
    want, want_lse = ref.prefill(case.q, case.k, case.v, case.L, case.retained_idx, case.scale)
    tol = dict(max_err=2e-2, mean_err=2e-3) if kw.get("out_dtype") == torch.bfloat16 else {}
    check_close(out, want, f"{case.name} out", **tol)
    check_close(lse, want_lse, f"{case.name} lse", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)


def compare_sampled(case, rows, **kw):
    out, lse = run_gpu(case, **kw)
    want, want_lse = ref.prefill(case.q, case.k, case.v, case.L, case.retained_idx, case.scale, rows=rows)
    idx = torch.from_numpy(rows.astype(np.int64)).cuda()
    check_close(out[idx], want, f"{case.name} out[rows]")
    check_close(lse[idx], want_lse, f"{case.name} lse[rows]", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)
    assert torch.isfinite(out).all()


@pytest.mark.parametrize("force_general", [False, True])
def test_cfg1_tiny(force_general):
    compare_full(inputs.make_prefill("cfg1_tiny"), force_general=force_general)


EDGE = [
    # T, L, R, Hq, Hkv, D
    (512, 256, 0, 4, 2, 128),        # R = 0: block-diagonal causal
    (512, 256, 256, 2, 1, 128),      # R = L: dense causal
    (256, 256, 16, 2, 2, 128),       # one chunk
    (768, 256, 24, 7, 1, 128),       # G = 7, R*c not a multiple of the key tile
    (1024, 512, 100, 4, 4, 128),     # R not a multiple of 4
    (320, 64, 8, 2, 1, 64),          # chunk shorter than a tile, D = 64
    (288, 96, 5, 3, 1, 64),          # chunk length not a multiple of the tile
    (2048, 1024, 64, 2, 1, 128),     # several tile pairs per chunk
    (1200, 300, 20, 4, 2, 128),      # chunk length off the tile grid: second pair holds 44 rows, its second tile none
    (1540, 385, 33, 7, 1, 128),      # one row into the second tile of the second pair
    (1280, 640, 64, 2, 1, 128),      # two and a half pairs
    (1808, 452, 452, 2, 2, 128),     # everything retained, ragged chunks: dense causal
    (1024, 512, 48, 4, 2, 64),       # head dimension 64: one 64-column panel per tile
    (1536, 384, 384, 6, 2, 64),      # head dimension 64, everything retained
    (640, 128, 16, 4, 2, 128),       # one query tile per chunk: the pair's second tile is surplus
    (800, 40, 7, 2, 1, 128),         # twenty chunks shorter than a third of a tile
    (1210, 110, 30, 3, 1, 64),       # short ragged chunks, head dimension 64
]


@pytest.mark.parametrize("force_general", [False, True])
@pytest.mark.parametrize("T,L,R,Hq,Hkv,D", EDGE)
def test_edge_shapes(T, L, R, Hq, Hkv, D, force_general):
    case = inputs.make_prefill(T=T, L=L, R=R, Hq=Hq, Hkv=Hkv, D=D, seed=T + 7 * R + D, chunk_mean_std=0.5)
    case.name = f"edge T{T} L{L} R{R} Hq{Hq} Hkv{Hkv} D{D} gen{int(force_general)}"
    compare_full(case, force_general=force_general)


@pytest.mark.parametrize("force_general", [False, True])
def test_unsorted_retained_and_stamps_pattern(force_general):
    case = inputs.make_prefill(T=1024, L=256, R=36, Hq=4, Hkv=2, D=128, seed=77, pattern="stamps")
    rng = np.random.default_rng(1)
    shuffled = case.retained_idx.copy()
    for row in shuffled:
        rng.shuffle(row)
    out, lse = run_gpu(case, force_general=force_general, ridx=shuffled, validate=True)
    want, want_lse = ref.prefill(case.q, case.k, case.v, case.L, case.retained_idx, case.scale)
    check_close(out, want, "unsorted out")
    check_close(lse, want_lse, "unsorted lse", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)


@pytest.mark.parametrize("T,L,R,Hq,Hkv,D", [EDGE[3], EDGE[4], EDGE[7]])
def test_gather4_variant(T, L, R, Hq, Hkv, D):
    """Retained rows fetched with TMA gather4 straight from K/V instead of the packed level."""
    case = inputs.make_prefill(T=T, L=L, R=R, Hq=Hq, Hkv=Hkv, D=D, seed=T + R, chunk_mean_std=0.5)
    compare_full(case, gather4=True)


def test_bf16_output_and_batch_strides():
    case = inputs.make_prefill(T=512, L=256, R=32, Hq=4, Hkv=2, D=128, seed=5)
    compare_full(case, out_dtype=torch.bfloat16)
    # batch of two with different data, non-contiguous q (padded head stride)
    c2 = inputs.make_prefill(T=512, L=256, R=32, Hq=4, Hkv=2, D=128, seed=6)
    q = torch.stack([to_gpu(case.q), to_gpu(c2.q)])
    k = torch.stack([to_gpu(case.k), to_gpu(c2.k)])
    v = torch.stack([to_gpu(case.v), to_gpu(c2.v)])
    qpad = torch.zeros((2, 512, 4, 136), dtype=torch.bfloat16, device="cuda")
    qpad[..., :128] = q
    ridx = torch.from_numpy(case.retained_idx).cuda()
    for fg in (False, True):
        out = vb.chunk_prefill_attn(qpad[..., :128], k, v, 256, ridx, scale=case.scale, force_general=fg)
        for b, cc in enumerate((case, c2)):
            want, _ = ref.prefill(cc.q, cc.k, cc.v, cc.L, case.retained_idx, cc.scale)
            check_close(out[b], want, f"batch {b} gen{int(fg)}")


def test_validate_flags_bad_index():
    case = inputs.make_prefill(T=512, L=256, R=8, Hq=2, Hkv=1, D=128, seed=8)
    bad = case.retained_idx.copy()
    bad[0, 3] = 300                                  # outside chunk 0
    q, k, v = (to_gpu(x) for x in (case.q, case.k, case.v))
    ws = vb.prefill_workspace(B=1, T=case.T, Hq=case.Hq, Hkv=case.Hkv, D=case.D, chunk_len=case.L, R=case.R,
                              device="cuda")
    vb.chunk_prefill_attn(q, k, v, case.L, torch.from_numpy(bad).cuda(), workspace=ws, validate=True)
    assert vb.device_status(ws) == vb.VXL_ERR_INVALID_INDEX
    assert vb.device_status(ws) == vb.VXL_OK          # cleared by the read
    dup = case.retained_idx.copy()
    dup[0, 1] = dup[0, 0]
    vb.chunk_prefill_attn(q, k, v, case.L, torch.from_numpy(dup).cuda(), workspace=ws, validate=True)
    assert vb.device_status(ws) == vb.VXL_ERR_INVALID_INDEX


def test_kernel_kind_selection():
    for name in ("cfg2_16k", "cfg3_64k", "cfg4_256k", "sweep_L512", "sweep_L1024", "sweep_L2048", "sweep_L4096"):
        c = inputs.prefill_shape(name)
        kw = dict(B=1, T=c.T, Hq=c.Hq, Hkv=c.Hkv, D=c.D, chunk_len=c.L, R=c.R)
        assert vb.prefill_kernel_kind(**kw) == 1                     # tcgen05 kernel
        assert vb.prefill_kernel_kind(force_general=True, **kw) == 0
    # plain chunks of any length and both head dimensions run on the tcgen05 kernel; a call over a range of
    # chunks needs the chunk to end on a key-tile boundary; window steps must be multiples of 128
    assert vb.prefill_kernel_kind(B=1, T=1200, Hq=4, Hkv=2, D=128, chunk_len=300, R=20) == 1
    assert vb.prefill_kernel_kind(B=1, T=1000, Hq=4, Hkv=2, D=128, chunk_len=200, R=20) == 1
    assert vb.prefill_kernel_kind(B=1, T=1000, Hq=4, Hkv=2, D=64, chunk_len=40, R=3) == 1
    assert vb.prefill_kernel_kind(B=1, T=1000, Hq=4, Hkv=2, D=128, chunk_len=200, R=20, block_begin=1, block_count=2) == 0
    assert vb.prefill_kernel_kind(B=1, T=1200, Hq=4, Hkv=2, D=128, chunk_len=600, R=20, step=300) == 0
    assert vb.prefill_kernel_kind(B=1, T=1920, Hq=4, Hkv=2, D=128, chunk_len=960, R=20, step=320) == 0
    assert vb.prefill_kernel_kind(B=1, T=1536, Hq=4, Hkv=2, D=128, chunk_len=384, R=20, step=128) == 1
    c = inputs.prefill_shape("cfg1_tiny")
    assert vb.prefill_kernel_kind(B=1, T=c.T, Hq=c.Hq, Hkv=c.Hkv, D=c.D, chunk_len=c.L, R=c.R) == 1
    assert vb.prefill_kernel_kind(B=1, T=100, Hq=2, Hkv=1, D=64, chunk_len=64, R=0) == -1


@pytest.mark.parametrize("name", ["cfg2_16k", "cfg3_64k", "sweep_L512", "sweep_L1024", "sweep_L2048", "sweep_L4096"])
def test_full_size_sampled(name):
    case = inputs.make_prefill(name)
    rows = sample_rows(case.T, case.L, 24, seed=case.seed)
    compare_sampled(case, rows)


def test_cfg2_full_tensor():
    # the benchmark configuration, every row of every head (the oracle needs some ten seconds on a many-core host)
    compare_full(inputs.make_prefill("cfg2_16k"))


def test_cfg2_general_kernel_sampled():
    case = inputs.make_prefill("cfg2_16k")
    compare_sampled(case, sample_rows(case.T, case.L, 8, seed=3), force_general=True)


def test_cfg4_256k_sampled():
    """262,144 tokens: chunks 0, 1, 2, 63, 126 and 127 compared in full (every row, every head), 64 seeded
    rows of every other chunk, plus the tile and chunk boundaries of `sample_rows`: 7.7 % of all rows."""
    case = inputs.make_prefill("cfg4_256k")
    rng = np.random.default_rng(case.seed + 1)
    full = (0, 1, 2, 63, 126, 127)
    parts = [np.arange(c * case.L, (c + 1) * case.L) for c in full]
    parts += [c * case.L + np.sort(rng.choice(case.L, size=64, replace=False)) for c in range(case.C) if c not in full]
    parts.append(sample_rows(case.T, case.L, 16, seed=case.seed))
    rows = np.unique(np.concatenate(parts)).astype(np.int32)
    assert rows.size >= 6 * case.L + 64 * (case.C - 6)
    compare_sampled(case, rows)


# ------------------------------------------------------------------ sliding chunk window + prefix
def run_gpu_window(case, *, force_general=False, validate=True):
    q, k, v = (to_gpu(x) for x in (case.q, case.k, case.v))
    ridx_t = torch.from_numpy(np.ascontiguousarray(case.retained_idx)).cuda() if case.R > 0 else None
    out, lse = vb.chunk_prefill_attn(q, k, v, case.L, ridx_t, scale=case.scale, return_lse=True,
                                     force_general=force_general, validate=validate, step=case.step,
                                     prefix_len=case.prefix_len)
    torch.cuda.synchronize()
    return out, lse


WINDOW = [
    # T_vis, L, step, prefix_len, R, Hq, Hkv, D
    (512, 256, 256, 37, 8, 4, 2, 128),       # prefix only (step = window): ragged prefix tile
    (768, 512, 256, 0, 16, 7, 1, 128),       # window of two steps, no prefix
    (1024, 512, 256, 100, 24, 4, 2, 128),    # both; the retained list ends inside a key tile
    (1536, 768, 256, 256, 0, 2, 1, 128),     # window of three steps, R = 0, prefix = two key tiles
    (320, 128, 64, 9, 5, 2, 1, 64),          # D = 64, steps shorter than a query tile pair
    (288, 96, 48, 150, 3, 3, 1, 64),         # step not a multiple of the tile, long prefix
    (2048, 1024, 512, 300, 64, 2, 1, 128),   # several tile pairs per step block
    (1536, 384, 128, 70, 12, 4, 2, 128),     # steps of one query tile: the pair's second tile is surplus
    (2304, 768, 384, 0, 40, 2, 1, 128),      # a step and a half pairs long
    (1920, 960, 320, 130, 16, 2, 2, 128),    # steps off the tile grid: general kernel
]


@pytest.mark.parametrize("force_general", [False, True])
@pytest.mark.parametrize("T_vis,L,step,prefix_len,R,Hq,Hkv,D", WINDOW)
def test_window_and_prefix(T_vis, L, step, prefix_len, R, Hq, Hkv, D, force_general):
    case = inputs.make_prefill_window(T_vis=T_vis, L=L, step=step, prefix_len=prefix_len, R=R, Hq=Hq, Hkv=Hkv,
                                      D=D, seed=T_vis + step + prefix_len, chunk_mean_std=0.5)
    out, lse = run_gpu_window(case, force_general=force_general)
    kind = vb.prefill_kernel_kind(B=1, T=case.T, Hq=Hq, Hkv=Hkv, D=D, chunk_len=L, R=R, force_general=force_general,
                                  step=step, prefix_len=prefix_len)
    fast = not force_general and (step == L or step % 128 == 0)
    assert kind == (1 if fast else 0)
    want, want_lse = ref.prefill_window(case.q, case.k, case.v, case.L, case.step, case.prefix_len,
                                        case.retained_idx, case.scale)
    check_close(out, want, f"{case.name} out")
    check_close(lse, want_lse, f"{case.name} lse", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)


def test_window_long_sequence_sampled():
    """64K visual tokens, window 2048 sliding by 1024, 512-token prefix: sampled rows against the oracle."""
    case = inputs.make_prefill_window(T_vis=65536, L=2048, step=1024, prefix_len=512, R=128, Hq=28, Hkv=4,
                                      D=128, seed=inputs.config_seed(3, 7), chunk_mean_std=0.5)
    out, lse = run_gpu_window(case, validate=False)
    rows = sample_rows(case.T - case.prefix_len, case.step, 48, seed=3) + case.prefix_len
    rows = np.unique(np.concatenate([rows, np.array([0, 1, 127, 128, 511], dtype=np.int32)])).astype(np.int32)
    want, want_lse = ref.prefill_window(case.q, case.k, case.v, case.L, case.step, case.prefix_len,
                                        case.retained_idx, case.scale, rows=rows)
    idx = torch.from_numpy(rows.astype(np.int64)).cuda()
    check_close(out[idx], want, "window 64k out[rows]")
    check_close(lse[idx], want_lse, "window 64k lse[rows]", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)
    assert torch.isfinite(out).all()


def test_prefix_only_sequence_and_batched_window():
    # no visual tokens at all: plain causal attention over the prefix, through both kernel choices
    case = inputs.make_prefill_window(T_vis=0, L=256, step=256, prefix_len=200, R=0, Hq=4, Hkv=2, D=128, seed=91)
    for fg in (False, True):
        out, lse = run_gpu_window(case, force_general=fg, validate=False)
        want, want_lse = ref.prefill_window(case.q, case.k, case.v, case.L, case.step, case.prefix_len,
                                            case.retained_idx, case.scale)
        check_close(out, want, "prefix only out")
        check_close(lse, want_lse, "prefix only lse", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)
    # two sequences with different data in one call, bf16 output
    a = inputs.make_prefill_window(T_vis=768, L=512, step=256, prefix_len=60, R=16, Hq=4, Hkv=2, D=128, seed=92)
    b = inputs.make_prefill_window(T_vis=768, L=512, step=256, prefix_len=60, R=16, Hq=4, Hkv=2, D=128, seed=93)
    q = torch.stack([to_gpu(a.q), to_gpu(b.q)])
    k = torch.stack([to_gpu(a.k), to_gpu(b.k)])
    v = torch.stack([to_gpu(a.v), to_gpu(b.v)])
    ridx = torch.from_numpy(a.retained_idx).cuda()
    out = vb.chunk_prefill_attn(q, k, v, a.L, ridx, scale=a.scale, step=a.step, prefix_len=a.prefix_len,
                                out_dtype=torch.bfloat16)
    torch.cuda.synchronize()
    for i, c in enumerate((a, b)):
        want, _ = ref.prefill_window(c.q, c.k, c.v, c.L, c.step, c.prefix_len, a.retained_idx, c.scale)
        check_close(out[i], want, f"batched window b{i}", max_err=2e-2, mean_err=2e-3)


def test_more_chunk_pairs_than_the_ranking_table_holds():
    """4,100 chunks of 256 tokens: the device-side ranking of work items is skipped and the items
    are walked in the fixed longest-first order instead."""
    case = inputs.make_prefill(T=4100 * 256, L=256, R=4, Hq=1, Hkv=1, D=128, seed=123)
    rows = sample_rows(case.T, case.L, 40, seed=9)
    compare_sampled(case, rows)


# ------------------------------------------------------------------ one call per chunk (block range)
def _nan_like(x):
    return torch.full_like(x, float("nan"))


@pytest.mark.parametrize("force_general", [False, True])
@pytest.mark.parametrize("T,L,R,Hq,Hkv,D,per_call", [(2048, 512, 48, 4, 2, 128, 1), (1536, 256, 100, 7, 1, 128, 2),
                                                    (640, 128, 8, 2, 1, 64, 1)])
def test_chunk_by_chunk_calls_equal_the_whole_call_and_read_nothing_ahead(T, L, R, Hq, Hkv, D, per_call, force_general):
    case = inputs.make_prefill(T=T, L=L, R=R, Hq=Hq, Hkv=Hkv, D=D, seed=91)
    q_all, k_all, v_all = (to_gpu(x)[None] for x in (case.q, case.k, case.v))
    ridx = torch.from_numpy(np.ascontiguousarray(case.retained_idx)).cuda()
    # the caller's buffers: tokens arrive chunk by chunk, everything not yet received is NaN
    q, k, v = _nan_like(q_all), _nan_like(k_all), _nan_like(v_all)
    out = torch.full((1, T, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full((1, T, Hq), float("nan"), dtype=torch.float32, device="cuda")
    ws = vb.prefill_workspace(B=1, T=T, Hq=Hq, Hkv=Hkv, D=D, chunk_len=L, R=R, device="cuda")
    C = T // L
    for c0 in range(0, C, per_call):
        n = min(per_call, C - c0)
        rows = slice(c0 * L, (c0 + n) * L)
        q[:, rows], k[:, rows], v[:, rows] = q_all[:, rows], k_all[:, rows], v_all[:, rows]
        vb.chunk_prefill_attn(q, k, v, L, ridx, scale=case.scale, out=out, lse=lse, return_lse=True, workspace=ws,
                              force_general=force_general, validate=True, block_begin=c0, block_count=n)
        torch.cuda.synchronize()
        assert vb.device_status(ws) == vb.VXL_OK
        assert torch.isfinite(out[:, :(c0 + n) * L]).all()                 # no NaN from rows not yet received
        assert torch.isnan(out[:, (c0 + n) * L:]).all()                    # rows after the range are untouched
    want, want_lse = ref.prefill(case.q, case.k, case.v, case.L, case.retained_idx, case.scale)
    check_close(out[0], want, "chunk-by-chunk out")
    check_close(lse[0], want_lse, "chunk-by-chunk lse", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)
    whole = vb.chunk_prefill_attn(q_all, k_all, v_all, L, ridx, scale=case.scale, force_general=force_general)
    assert torch.equal(whole, out)                                          # same kernels, same key order per row


def test_block_range_with_window_and_prefix():
    case = inputs.make_prefill_window(T_vis=2048, L=1024, step=512, prefix_len=300, R=64, Hq=2, Hkv=1, D=128, seed=92)
    q, k, v = (to_gpu(x)[None] for x in (case.q, case.k, case.v))
    ridx = torch.from_numpy(np.ascontiguousarray(case.retained_idx)).cuda()
    T = case.q.shape[0]
    out = torch.full((1, T, case.Hq, case.D), float("nan"), dtype=torch.float32, device="cuda")
    nblocks = (T - case.prefix_len) // case.step
    for c0 in (2, 0, 3, 1):                                                 # any order: the calls are independent
        vb.chunk_prefill_attn(q, k, v, case.L, ridx, scale=case.scale, out=out, step=case.step,
                              prefix_len=case.prefix_len, block_begin=c0, block_count=1)
        if c0 == 2:                                                         # the prefix belongs to the call that starts at block 0
            assert torch.isnan(out[:, :case.prefix_len]).all()
    assert nblocks == 4
    want, _ = ref.prefill_window(case.q, case.k, case.v, case.L, case.step, case.prefix_len, case.retained_idx, case.scale)
    check_close(out[0], want, "block range with window and prefix")


@pytest.mark.parametrize("B,out_dtype,per_call", [(1, torch.float32, 3), (2, torch.bfloat16, 1)])
def test_host_prefill_pipeline_equals_the_oracle_twice_in_a_row(B, out_dtype, per_call):
    """vxl_chunk_prefill_host: pinned host q/k/v in, pinned host out (and lse), the pipeline inside the library."""
    cases = [inputs.make_prefill(T=2048, L=256, R=32, Hq=4, Hkv=2, D=128, seed=93 + b) for b in range(B)]
    c0 = cases[0]
    pin = lambda arrs: torch.from_numpy(np.stack([np.ascontiguousarray(a).view(np.int16) for a in arrs])).pin_memory()
    hq, hk, hv = pin([c.q for c in cases]), pin([c.k for c in cases]), pin([c.v for c in cases])
    hridx = torch.from_numpy(np.ascontiguousarray(c0.retained_idx)).pin_memory()
    hout = torch.empty((B, c0.T, c0.Hq, c0.D), dtype=out_dtype).pin_memory()
    hlse = torch.empty((B, c0.T, c0.Hq), dtype=torch.float32).pin_memory()
    hp = vb.HostPrefill(c0.T, c0.Hq, c0.Hkv, c0.D, c0.L, c0.R, B=B, chunks_per_call=per_call, scale=c0.scale,
                        out_dtype=out_dtype, with_lse=True)
    tol = dict(max_err=2e-2, mean_err=2e-3) if out_dtype == torch.bfloat16 else {}
    for _ in range(2):
        hout.fill_(float("nan")); hlse.fill_(float("nan"))
        hp.run(hq, hk, hv, hridx, hout, hlse)
        torch.cuda.synchronize()
        assert vb.device_status(hp.ws) == vb.VXL_OK
        for b, c in enumerate(cases):
            want, want_lse = ref.prefill(c.q, c.k, c.v, c.L, c0.retained_idx, c.scale)
            check_close(hout[b].float(), want, f"host prefill pipeline b{b}", **tol)
            check_close(hlse[b], want_lse, "host prefill lse", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)
    # the device arrays hold the sequence afterwards: the KV cache a decoding call would read
    assert torch.equal(hp.k.cpu().view(torch.int16), hk) and torch.equal(hp.v.cpu().view(torch.int16), hv)


def test_ragged_chunks_batched_bf16_out_and_range_fallback():
    T, L, R, Hq, Hkv, D = 1158, 386, 40, 4, 2, 128
    cases = [inputs.make_prefill(T=T, L=L, R=R, Hq=Hq, Hkv=Hkv, D=D, seed=95 + b) for b in range(2)]
    q = torch.stack([to_gpu(c.q) for c in cases]); k = torch.stack([to_gpu(c.k) for c in cases])
    v = torch.stack([to_gpu(c.v) for c in cases])
    ridx = torch.from_numpy(np.ascontiguousarray(cases[0].retained_idx)).cuda()
    out, lse = vb.chunk_prefill_attn(q, k, v, L, ridx, scale=cases[0].scale, return_lse=True, out_dtype=torch.bfloat16)
    assert vb.prefill_kernel_kind(B=2, T=T, Hq=Hq, Hkv=Hkv, D=D, chunk_len=L, R=R) == 1
    for b, c in enumerate(cases):
        want, want_lse = ref.prefill(c.q, c.k, c.v, L, cases[0].retained_idx, c.scale)
        check_close(out[b].float(), want, f"ragged batched b{b}", max_err=2e-2, mean_err=2e-3)
        check_close(lse[b], want_lse, f"ragged batched lse b{b}", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)
    # a range of ragged chunks goes through the general kernel (nothing after the range may be read)
    out2 = torch.full((2, T, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
    k2, v2 = k.clone(), v.clone()
    k2[:, 2 * L:] = float("nan"); v2[:, 2 * L:] = float("nan")
    vb.chunk_prefill_attn(q, k2, v2, L, ridx, scale=cases[0].scale, out=out2, block_begin=1, block_count=1)
    want, _ = ref.prefill(cases[1].q, cases[1].k, cases[1].v, L, cases[0].retained_idx, cases[1].scale)
    check_close(out2[1, L:2 * L], want[L:2 * L], "ragged range call")
    assert torch.isnan(out2[:, :L]).all() and torch.isnan(out2[:, 2 * L:]).all()


@pytest.mark.parametrize("T,L,R,Hq,Hkv,D", [
    (16384, 2048, 128, 8, 2, 64),     # head dimension 64 over many work items per CTA
    (16384, 64, 8, 4, 2, 64),         # the tiny configuration's chunk shape, 256 chunks of it
    (24576, 192, 24, 7, 1, 128),      # 128 short ragged chunks, retained list of 127 x 24 rows
])
def test_head_dim_64_and_short_chunks_at_scale_sampled(T, L, R, Hq, Hkv, D):
    case = inputs.make_prefill(T=T, L=L, R=R, Hq=Hq, Hkv=Hkv, D=D, seed=T + L + D, chunk_mean_std=0.5)
    assert vb.prefill_kernel_kind(B=1, T=T, Hq=Hq, Hkv=Hkv, D=D, chunk_len=L, R=R) == 1
    rows = sample_rows(T, L, 96, seed=L)
    compare_sampled(case, rows)


def test_head_dim_64_batched_bf16_out_with_window():
    a = inputs.make_prefill_window(T_vis=1536, L=512, step=256, prefix_len=70, R=20, Hq=6, Hkv=2, D=64, seed=301)
    b = inputs.make_prefill_window(T_vis=1536, L=512, step=256, prefix_len=70, R=20, Hq=6, Hkv=2, D=64, seed=302)
    q = torch.stack([to_gpu(a.q), to_gpu(b.q)]); k = torch.stack([to_gpu(a.k), to_gpu(b.k)])
    v = torch.stack([to_gpu(a.v), to_gpu(b.v)])
    ridx = torch.from_numpy(a.retained_idx).cuda()
    assert vb.prefill_kernel_kind(B=2, T=a.T, Hq=6, Hkv=2, D=64, chunk_len=512, R=20, step=256, prefix_len=70) == 1
    out, lse = vb.chunk_prefill_attn(q, k, v, a.L, ridx, scale=a.scale, step=a.step, prefix_len=a.prefix_len,
                                     out_dtype=torch.bfloat16, return_lse=True)
    torch.cuda.synchronize()
    for i, c in enumerate((a, b)):
        want, want_lse = ref.prefill_window(c.q, c.k, c.v, c.L, c.step, c.prefix_len, a.retained_idx, c.scale)
        check_close(out[i], want, f"D=64 batched window b{i}", max_err=2e-2, mean_err=2e-3)
        check_close(lse[i], want_lse, "lse", max_err=LSE_ABS_ERR, mean_err=LSE_ABS_ERR)
