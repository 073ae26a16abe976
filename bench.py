#!/usr/bin/env python
"""Benchmark of the chunk-sparse attention hot path (one JSON line on stdout, rank 0).

A step = one pass of the whole path over one batch of seeded synthetic input:
  1. vxl_chunk_prefill_attn on the prefill workload (default: 262,144 tokens, 128 chunks x 2,048,
     128 retained rows per chunk, 28 query / 4 kv heads, head dim 128, fp32 output);
  2. vxl_bilevel_decode_attn (scores + top-k + mixed dense/sparse attention + combine) on a
     262,144-token cache, batch 8, k = 8 and then k = 16;
  3. the same at batch 1, once per sequence of that cache and per k (8 calls over 8 distinct caches,
     so that the 67-100 MB a call reads never sits in the 126 MB L2 from the call before).
`value` is prefill useful TFLOP/s (non-masked FLOPs / device time of the prefill calls); the decode
figures (us/token, GB/s of algorithmic bytes) sit in "decode" and, for the record a reader keeps,
in "roofline.decode".  Timing is CUDA events on the launching stream, max over ranks.  With
--gpus N every rank runs the same work on its own GPU (independent sequences, no collective on
the data path): weak scaling.

Every workload that is timed is also checked: a seeded sample of its outputs is compared with the
fp64 CPU oracle outside the timed region and the result is printed in "parity".

`--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2506_19225_b200 import inputs, replicas

NOMINAL_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
MAX_ERR, MEAN_ERR, LSE_ERR, NEAR_TIE = 1e-2, 1e-3, 2e-3, 1e-4
CSRC = os.path.join(ROOT, "paper_2506_19225_b200", "csrc")


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def kernel_source_digest(files):
    h = hashlib.sha256()
    for name in files:
        with open(os.path.join(CSRC, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def captured_traffic(key, units):
    """DRAM bytes per launch from the stored profiler counters, scaled to `units` (tokens or sequences)
    by the units of the capture; None when no capture exists or the kernel's source has changed since."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        rec = json.load(f).get(key)
    if rec is None or rec.get("source_digest") != kernel_source_digest(rec["source_files"]):
        return None
    return int((rec["dram_bytes_read"] + rec["dram_bytes_write"]) * units / rec["units"])


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            parts = [x.strip() for x in r.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        # "under load": the samples taken while kernels ran (an idle GPU drops far below half its maximum clock)
        busy = [x for x, m in zip(sm, mx) if x >= 0.5 * m]
        return {"sm_mhz": float(np.median(busy)) if busy else (float(np.median(sm)) if sm else None),
                "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "samples_under_load": len(busy)}


# ---------------------------------------------------------------------- synthetic inputs
def decode_bytes_per_seq(C, L, R, Hkv, D, topk):
    """Algorithmic K+V bytes one decode call reads per sequence in the one-pass design: the
    sparse level of every chunk (K and V) plus the dense rows of the k selected chunks."""
    row = Hkv * D * 2
    return (C * R + topk * L) * row * 2


def gen_decode(B, T, L, R, Hq, Hkv, D, seed, n_planted, device):
    """Decode recipe of inputs.make_decode drawn with torch's generator on `device`: N(0,1) bf16 cache,
    `n_planted` chunks per sequence whose keys align with the query (cos ~ 0.5)."""
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    C, G = T // L, Hq // Hkv
    q = torch.randn((B, Hq, D), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    u = q.float().view(B, Hkv, G, D).mean(2)
    u = u / u.norm(dim=-1, keepdim=True).clamp_min(1e-20)
    k = torch.empty((B, T, Hkv, D), dtype=torch.bfloat16, device=device)
    v = torch.empty((B, T, Hkv, D), dtype=torch.bfloat16, device=device)
    rng = np.random.default_rng(seed)
    planted = np.stack([np.sort(rng.choice(C, size=n_planted, replace=False)) for _ in range(B)])
    for b in range(B):
        kb = torch.randn((T, Hkv, D), generator=g, device=device, dtype=torch.float32)
        for c in planted[b]:
            kb[c * L:(c + 1) * L] = kb[c * L:(c + 1) * L] * (0.75 ** 0.5) + 0.5 * (D ** 0.5) * u[b][None]
        k[b] = kb.to(torch.bfloat16)
        del kb
        v[b] = torch.randn((T, Hkv, D), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    ridx = inputs.make_retained_idx(rng, C, L, R)
    off = (np.arange(C + 1, dtype=np.int64) * L).astype(np.int32)
    return q, k, v, off, ridx, planted


def gen_prefill(shape: inputs.PrefillCase, device, seed=None):
    """Prefill recipe of inputs.make_prefill drawn with torch's generator on `device`."""
    seed = shape.seed if seed is None else seed
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    rng = np.random.default_rng(seed)
    ridx = inputs.make_retained_idx(rng, shape.C, shape.L, shape.R)
    q = torch.empty((shape.T, shape.Hq, shape.D), dtype=torch.bfloat16, device=device)
    step = 1 << 15
    for s in range(0, shape.T, step):
        q[s:s + step] = torch.randn((min(step, shape.T - s), shape.Hq, shape.D), generator=g, device=device).to(torch.bfloat16)
    k = torch.randn((shape.T, shape.Hkv, shape.D), generator=g, device=device)
    if shape.chunk_mean_std > 0:
        mu = torch.randn((shape.C, shape.Hkv, shape.D), generator=g, device=device) * shape.chunk_mean_std
        k += mu.repeat_interleave(shape.L, dim=0)
    k = k.to(torch.bfloat16)
    v = torch.randn((shape.T, shape.Hkv, shape.D), generator=g, device=device).to(torch.bfloat16)
    return q, k, v, ridx


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor (any device) -> its bit patterns as a uint16 NumPy array."""
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def boundary_rows(T, L, n_random, seed):
    """Row sample with tile and chunk boundaries of the first, middle and last chunks plus random rows."""
    rng = np.random.default_rng(seed)
    C = T // L
    rows = set()
    for c in sorted({0, 1, C // 2, C - 1}):
        for r in (0, 127, 128, 255, 256, L // 2, L - 129, L - 128, L - 1):
            if 0 <= c < C and 0 <= r < L:
                rows.add(c * L + r)
    rows.update(int(x) for x in rng.integers(0, T, size=n_random))
    return np.array(sorted(rows), dtype=np.int32)


# ---------------------------------------------------------------------- oracle checks (outside the timed region)
def parity_prefill(sh, qb, kb, vb_, ridx, out, n_random, seed):
    """Sampled rows of a prefill output against the fp64 oracle on the same bytes."""
    from oracle import ref
    rows = boundary_rows(sh.T, sh.L, n_random, seed)
    want, _ = ref.prefill(qb, kb, vb_, sh.L, ridx, sh.scale, rows=rows)
    got = out[torch.from_numpy(rows.astype(np.int64)).to(out.device)].double().cpu().numpy()
    err = np.abs(got - want)
    ok = bool(np.isfinite(got).all() and err.max() <= MAX_ERR and err.mean() <= MEAN_ERR)
    return {"rows": int(rows.size), "of": sh.T, "max_err": float(err.max()), "mean_err": float(err.mean()), "ok": ok}


def parity_decode(seqs, q, k, v, off, ridx, scale, topk, got_out, got_topk, got_scores=None):
    """Whole outputs of the given sequences against the oracle (scores, selection, mixed attention)."""
    from oracle import ref
    mx, mn, ok, ties = 0.0, [], True, 0
    for b in seqs:
        qb, kb, vb_ = bits(q[b]), bits(k[b]), bits(v[b])
        _, sc = ref.scores(qb, kb, ridx, scale)
        idx, gap = ref.topk(sc, topk)
        sel = got_topk[b].cpu().numpy()
        if sel.tolist() != idx.tolist():
            ties += 1
            ok = ok and gap < NEAR_TIE and len(set(sel.tolist()) ^ set(idx.tolist())) == 2
        if got_scores is not None:
            ok = ok and float(np.abs(got_scores[b].double().cpu().numpy() - sc).max()) <= LSE_ERR
        want, _ = ref.decode(qb, kb, vb_, off, ridx, sel, scale)
        g = got_out[b].double().cpu().numpy()
        err = np.abs(g - want)
        mx = max(mx, float(err.max())); mn.append(float(err.mean()))
        ok = ok and bool(np.isfinite(g).all() and err.max() <= MAX_ERR and err.mean() <= MEAN_ERR)
    return {"sequences": list(int(b) for b in seqs), "outputs": "all", "max_err": mx, "mean_err": float(np.mean(mn)),
            "topk_sets_equal_or_reported_near_tie": ok, "near_ties": ties, "ok": bool(ok)}


# ---------------------------------------------------------------------- timing helpers
def timed_calls(fn, iters, stream, between=None):
    """Device milliseconds of each of `iters` calls of fn (one event pair per call)."""
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    for a, b in evs:
        if between is not None:
            between()
        a.record(stream)
        fn()
        b.record(stream)
    torch.cuda.synchronize()
    return np.array([a.elapsed_time(b) for a, b in evs])


def summary(ms):
    return {"median": float(np.median(ms)), "mean": float(np.mean(ms)), "min": float(np.min(ms)), "n": int(len(ms))}


# ---------------------------------------------------------------------- CPU oracle timings
def oracle_prefill_sample(sh, qb, kb, vb_, ridx, target_seconds):
    """Times the oracle on uniformly sampled rows of the workload; returns a result dict."""
    from oracle import ref
    rng = np.random.default_rng(123)
    per_row_flops = sh.useful_flops() / sh.T
    probe = np.sort(rng.choice(sh.T, size=32, replace=False)).astype(np.int32)
    t0 = time.perf_counter()
    ref.prefill(qb, kb, vb_, sh.L, ridx, sh.scale, rows=probe)
    t_probe = time.perf_counter() - t0
    n = int(max(32, min(sh.T, target_seconds / max(t_probe / 32, 1e-9))))
    rows = np.sort(rng.choice(sh.T, size=n, replace=False)).astype(np.int32)
    t0 = time.perf_counter()
    ref.prefill(qb, kb, vb_, sh.L, ridx, sh.scale, rows=rows)
    dt = time.perf_counter() - t0
    return {"value": per_row_flops * n / dt / 1e12, "unit": "TFLOP/s", "cores": ref.threads(),
            "kind": "oracle", "seconds": dt,
            "extrapolated_full_workload_seconds": dt * sh.T / n,
            "sample": f"{n} uniformly sampled query rows (all {sh.Hq} heads) of {sh.name}, fp64; "
                      "the full-workload time is extrapolated from the sample"}


def oracle_decode_full(qb, kb, vb_, off, ridx, scale, topk, bytes_seq, repeats=3):
    """The oracle's scores + top-k + mixed attention for one sequence of the decode workload, in full."""
    from oracle import ref
    ts = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        _, sc = ref.scores(qb, kb, ridx, scale)
        idx, _ = ref.topk(sc, topk)
        ref.decode(qb, kb, vb_, off, ridx, idx, scale)
        ts.append(time.perf_counter() - t0)
    dt = float(np.median(ts))
    return {"us_per_token": dt * 1e6, "gbs": bytes_seq / dt / 1e9, "cores": ref.threads(), "kind": "oracle",
            "sample": f"one full sequence (scores + top-k + mixed attention, k={topk}), median of {repeats}, fp64"}


def workload_config(sh, topks, dB):
    return {"workload": sh.name, "T": sh.T, "chunk_len": sh.L, "chunks": sh.C, "retained_per_chunk": sh.R,
            "Hq": sh.Hq, "Hkv": sh.Hkv, "D": sh.D, "out": "fp32",
            "decode_workload": f"cfg5: cache 262144 tok = 128 chunks x 2048, R=128, k in {list(topks)}, batch {dB} and batch 1",
            "l2": "no flush: every call's inputs exceed the 126 MB L2 (prefill q+k+v+out = %.1f GB, a batch decode call "
                  "reads 0.5-0.8 GB); batch-1 decode calls rotate over %d distinct caches" %
                  ((sh.T * sh.Hq * sh.D * 6 + 4 * sh.T * sh.Hkv * sh.D) / 1e9, dB)}


def cpu_inputs(sh):
    """The prefill workload drawn on the host cores (same recipe, torch's CPU generator)."""
    q, k, v, ridx = gen_prefill(sh, "cpu")
    return bits(q), bits(k), bits(v), ridx


def run_reference(args, rank):
    if rank != 0:
        return
    sh = inputs.prefill_shape(args.workload)
    qb, kb, vb_, ridx = cpu_inputs(sh)
    steps, warm = max(args.steps, 1), args.warmup
    per_step = max(2.0, min(20.0, 120.0 / (steps + warm)))
    for _ in range(warm):
        oracle_prefill_sample(sh, qb, kb, vb_, ridx, per_step / 4)
    vals, secs = [], []
    for _ in range(steps):
        r = oracle_prefill_sample(sh, qb, kb, vb_, ridx, per_step)
        vals.append(r["value"]); secs.append(r["seconds"])
    v = float(np.mean(vals))
    line = {"impl": "reference", "metric": "prefill_useful_tflops", "value": v, "unit": "TFLOP/s",
            "n_gpus": args.gpus, "steps": steps, "warmup": warm, "ms_per_step": float(np.mean(secs)) * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(sh, (8, 16), args.decode_batch),
            "cpu_baseline": {"value": v, "unit": "TFLOP/s", "cores": r["cores"], "kind": "oracle", "sample": r["sample"]},
            "e2e": {"value": v, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="vxl", choices=["vxl", "reference"])
    ap.add_argument("--workload", default="cfg4_256k", choices=sorted(inputs.PREFILL_SHAPES))
    ap.add_argument("--decode-batch", type=int, default=8)
    ap.add_argument("--no-extra", action="store_true", help="skip the other workloads (sweeps, variants)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-parity", action="store_true", help="skip the oracle checks of the timed workloads")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-to-host legs (profiling runs)")
    ap.add_argument("--force-general", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch the batch-1 decode calls eagerly")
    ap.add_argument("--only", default="all", choices=["all", "prefill", "decode"],
                    help="profiling aid: run only one half of the step (the JSON line is then partial)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    from paper_2506_19225_b200 import binding as vb
    vb.load()                                    # fails loudly if the CUDA library is missing
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    stream = torch.cuda.current_stream()
    peaks, peak_kind = load_peaks()
    do_prefill, do_decode = args.only != "decode", args.only != "prefill"
    profiling = args.only != "all"
    check = not args.no_parity and not profiling and rank == 0

    # ------------------------------------------------------------------ inputs
    sh = inputs.prefill_shape(args.workload)
    q, k, v, ridx_np = gen_prefill(sh, dev, replicas.rank_seed(sh.seed, rank))
    ridx = torch.from_numpy(ridx_np).to(dev)
    out = torch.empty((sh.T, sh.Hq, sh.D), dtype=torch.float32, device=dev)
    ws_p = vb.prefill_workspace(B=1, T=262144, Hq=28, Hkv=4, D=128, chunk_len=2048, R=256, device=dev)
    kind = vb.prefill_kernel_kind(B=1, T=sh.T, Hq=sh.Hq, Hkv=sh.Hkv, D=sh.D, chunk_len=sh.L, R=sh.R,
                                  force_general=args.force_general)

    dB, dT, dL, dR, dHq, dHkv, dD = args.decode_batch, 262144, 2048, 128, 28, 4, 128
    topks = (8, 16)
    dC = dT // dL
    if do_decode:
        dq, dk, dv, doff_np, dridx_np, planted = gen_decode(dB, dT, dL, dR, dHq, dHkv, dD, inputs.config_seed(5, rank), 4, dev)
        doff, dridx = torch.from_numpy(doff_np).to(dev), torch.from_numpy(dridx_np).to(dev)
        shape_d = vb._decode_shape(dq, dk, None, None, False)
        ws_d = {kk: vb.new_workspace(vb.workspace_bytes(vb.VXL_OP_DECODE, shape_d, dC, dR, kk, dL), dev) for kk in topks}
        dout = {kk: torch.empty((dB, dHq, dD), dtype=torch.float32, device=dev) for kk in topks}
        dout1 = {kk: torch.empty((dB, 1, dHq, dD), dtype=torch.float32, device=dev) for kk in topks}
        dsel = {kk: torch.empty((dB, kk), dtype=torch.int32, device=dev) for kk in topks}
        dsc = torch.empty((dB, dC), dtype=torch.float32, device=dev)
        # the sparse level is stored on its own once the cache exists (vxl_pack_retained), outside the step
        dks, dvs = vb.pack_retained(dk, dv, dridx)
    d_scale = 1.0 / float(np.sqrt(dD))

    def run_prefill():
        vb.chunk_prefill_attn(q, k, v, sh.L, ridx, scale=sh.scale, out=out, workspace=ws_p,
                              force_general=args.force_general)

    def decode_call(qq, kk_, vv, oo, kk, ks_, vs_, want_sel=False):
        lib_out = vb.bilevel_decode_attn(qq, kk_, vv, doff, dridx, kk, max_chunk_len=dL, out=oo, workspace=ws_d[kk],
                                         sparse=(ks_, vs_), return_scores=want_sel)
        return lib_out

    def run_decode_batch(kk):
        decode_call(dq, dk, dv, dout[kk], kk, dks, dvs)

    def run_decode_single(kk):
        for b in range(dB):
            decode_call(dq[b:b + 1], dk[b:b + 1], dv[b:b + 1], dout1[kk][b], kk, dks[b:b + 1], dvs[b:b + 1])

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def step_once(single):
        if do_prefill:
            run_prefill()
        if do_decode:
            for kk in topks:
                run_decode_batch(kk)
            for kk in topks:
                single(kk)

    # ------------------------------------------------------------------ warm-up
    for _ in range(args.warmup):
        step_once(run_decode_single)
    torch.cuda.synchronize()
    assert vb.device_status(ws_p) == vb.VXL_OK
    if do_decode:
        assert all(vb.device_status(w) == vb.VXL_OK for w in ws_d.values())
    # The batch-1 decode loop is launch bound on the host (one call is ~25 us of GPU work), so the
    # eight single-sequence calls of a step are captured once per k in a CUDA graph and replayed.
    graphs = {}
    if do_decode and not args.no_graph:
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            for kk in topks:
                graphs[kk] = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graphs[kk], stream=side):
                    run_decode_single(kk)
        stream.wait_stream(side)
        for kk in topks:
            graphs[kk].replay()
        torch.cuda.synchronize()

    def run_decode_single_step(kk):
        if kk in graphs:
            graphs[kk].replay()
        else:
            run_decode_single(kk)

    # ------------------------------------------------------------------ timed steps
    K = args.steps
    nev = 2 + 2 * len(topks)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(nev)] for _ in range(K)]
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    barrier()
    t_wall = time.perf_counter()
    for i in range(K):
        e = ev[i]
        e[0].record(stream)
        if do_prefill:
            run_prefill()
        e[1].record(stream)
        j = 1
        for kk in topks:
            if do_decode:
                run_decode_batch(kk)
            j += 1; e[j].record(stream)
        for kk in topks:
            if do_decode:
                run_decode_single_step(kk)
            j += 1; e[j].record(stream)
    barrier()
    t_wall = time.perf_counter() - t_wall
    seg = np.array([[ev[i][j].elapsed_time(ev[i][j + 1]) for j in range(nev - 1)] for i in range(K)])   # [K, segments]
    ms_step = float(np.mean([ev[i][0].elapsed_time(ev[i][nev - 1]) for i in range(K)]))
    ms_p = max(float(seg[:, 0].mean()), 1e-6)
    ms_db = {kk: max(float(seg[:, 1 + i].mean()), 1e-6) for i, kk in enumerate(topks)}
    ms_d1 = {kk: max(float(seg[:, 1 + len(topks) + i].mean()) / dB, 1e-6) for i, kk in enumerate(topks)}
    med_p = float(np.median(seg[:, 0]))
    # keep the clocks sampler alive over a longer stretch of the same work when the timed region is short
    t_end = time.perf_counter() + max(0.0, 1.5 - t_wall)
    while time.perf_counter() < t_end:
        step_once(run_decode_single_step)
        torch.cuda.synchronize()
    clocks = sampler.stop()
    assert vb.device_status(ws_p) == vb.VXL_OK
    flat = [ms_p, ms_step] + [ms_db[kk] for kk in topks] + [ms_d1[kk] for kk in topks]
    flat = replicas.max_over_ranks(flat, dist, dev)
    ms_p, ms_step = flat[0], flat[1]
    for i, kk in enumerate(topks):
        ms_db[kk], ms_d1[kk] = flat[2 + i], flat[2 + len(topks) + i]

    flops = sh.useful_flops()
    tflops = replicas.whole_job_rate(flops, world, ms_p) / 1e12
    bytes_seq = {kk: decode_bytes_per_seq(dC, dL, dR, dHkv, dD, kk) for kk in topks}
    peak_tf, peak_hbm = float(peaks["bf16_tflops"]), float(peaks["hbm_gbs"])

    # ------------------------------------------------------------------ the prefill call alone, on a rested GPU
    # Inside the timed steps the GPU sits at its power cap; the burst peak it is compared with was taken on short
    # GEMMs at boost clocks.  The like-for-like figure: one call after a second of idling, three times.
    isolated_ms = None
    if do_prefill and not profiling:
        iso = []
        for _ in range(3):
            torch.cuda.synchronize()
            time.sleep(1.0)
            iso.append(float(timed_calls(run_prefill, 1, stream)[0]))
        isolated_ms = replicas.max_over_ranks([float(np.median(iso))], dist, dev)[0]

    # ------------------------------------------------------------------ decode alone: medians over many calls
    decode = None
    if do_decode:
        decode = {"batch": dB, "in_step": {}, "decode_only_loop": {}}
        for kk in topks:
            gb, g1 = dB * bytes_seq[kk] / (ms_db[kk] * 1e-3) / 1e9, bytes_seq[kk] / (ms_d1[kk] * 1e-3) / 1e9
            decode["in_step"][f"k{kk}"] = {
                "us_per_step_batch": ms_db[kk] * 1e3, "gbs_batch": gb, "frac_hbm_measured_batch": gb / peak_hbm,
                "frac_hbm_nominal_batch": gb / NOMINAL_HBM_GBS, "us_per_token_b1": ms_d1[kk] * 1e3, "gbs_b1": g1,
                "frac_hbm_measured_b1": g1 / peak_hbm, "frac_hbm_nominal_b1": g1 / NOMINAL_HBM_GBS,
                "bytes_per_seq": bytes_seq[kk]}
        n_calls = 200 if not profiling else 10
        for kk in topks:
            # batch call: the 8 single-sequence calls of the other k run in between, so nothing of the batch's
            # 0.5-0.8 GB is left in L2; single calls rotate over the 8 caches
            other = topks[1] if kk == topks[0] else topks[0]
            msb = timed_calls(lambda: run_decode_batch(kk), n_calls, stream, between=lambda: run_decode_single_step(other))
            ms1 = timed_calls(lambda: run_decode_single_step(kk), max(n_calls // dB, 5), stream) / dB
            eager = timed_calls(lambda: run_decode_single(kk), max(n_calls // dB // 2, 3), stream) / dB
            gb, g1 = dB * bytes_seq[kk] / (np.median(msb) * 1e-3) / 1e9, bytes_seq[kk] / (np.median(ms1) * 1e-3) / 1e9
            decode["decode_only_loop"][f"k{kk}"] = {
                "us_per_step_batch": summary(msb * 1e3), "gbs_batch": float(gb), "frac_hbm_measured_batch": float(gb / peak_hbm),
                "frac_hbm_nominal_batch": float(gb / NOMINAL_HBM_GBS),
                "us_per_token_b1": summary(ms1 * 1e3), "gbs_b1": float(g1), "frac_hbm_measured_b1": float(g1 / peak_hbm),
                "frac_hbm_nominal_b1": float(g1 / NOMINAL_HBM_GBS),
                "us_per_token_b1_eager_launches": summary(eager * 1e3),
                "calls": {"batch": int(n_calls), "b1": int(max(n_calls // dB, 5) * dB)}}
        assert all(vb.device_status(w) == vb.VXL_OK for w in ws_d.values())

    # ------------------------------------------------------------------ parity of what was timed
    parity = {}
    host_bits = None
    if do_prefill and rank == 0 and (check or not args.no_cpu_baseline):
        host_bits = (bits(q), bits(k), bits(v))
    if check and do_prefill:
        parity[sh.name] = parity_prefill(sh, host_bits[0], host_bits[1], host_bits[2], ridx_np, out, 160, 11)
    if check and do_decode:
        seqs = sorted({0, dB - 1})
        for kk in topks:
            res = decode_call(dq, dk, dv, dout[kk], kk, dks, dvs, want_sel=True)
            torch.cuda.synchronize()
            parity[f"decode_B{dB}_k{kk}"] = parity_decode(seqs, dq, dk, dv, doff_np, dridx_np, d_scale, kk, res["out"],
                                                          res["topk"], res["scores"])
            run_decode_single_step(kk)                      # the graph replay's outputs, the same sequences
            torch.cuda.synchronize()
            single = dout1[kk][:, 0]
            p1 = parity_decode(seqs, dq, dk, dv, doff_np, dridx_np, d_scale, kk, single, res["topk"])
            p1["equal_to_batch_call"] = bool(torch.equal(single, res["out"]))
            parity[f"decode_B1_k{kk}"] = p1

    # ------------------------------------------------------------------ end to end (host buffers)
    e2e = None
    if do_prefill and not profiling and not args.no_e2e:
        hq, hk, hv = (x.view(torch.int16).cpu().pin_memory() for x in (q, k, v))
        hridx = torch.from_numpy(ridx_np).pin_memory()
        e2e_variants = {}
        for name, odt in (("fp32_out", torch.float32), ("bf16_out", torch.bfloat16)):
            hout = torch.empty((sh.T, sh.Hq, sh.D), dtype=odt).pin_memory()
            # vxl_chunk_prefill_host: one 2-D copy per tensor and chunk, one prefill call per chunk, three streams
            host_prefill = vb.HostPrefill(sh.T, sh.Hq, sh.Hkv, sh.D, sh.L, sh.R, device=dev, scale=sh.scale,
                                          out_dtype=odt, force_general=args.force_general)
            run_e2e = lambda: host_prefill.run(hq, hk, hv, hridx, hout)
            for _ in range(2):
                run_e2e()
            barrier()
            ms = float(np.mean(timed_calls(run_e2e, max(3, min(K, 5)), stream)))
            ms = replicas.max_over_ranks([ms], dist, dev)[0]
            e2e_variants[name] = {"ms": ms, "value": world * flops / (ms * 1e-3) / 1e12,
                                  "h2d_bytes_per_step": int(hq.numel() * 2 + hk.numel() * 2 + hv.numel() * 2 + hridx.numel() * 4),
                                  "d2h_bytes_per_step": int(hout.numel() * hout.element_size())}
            if check and name == "fp32_out":
                torch.cuda.synchronize()
                ri = torch.from_numpy(boundary_rows(sh.T, sh.L, 24, 5).astype(np.int64))
                e2e_variants[name]["equal_to_device_call_on_sampled_rows"] = bool(torch.equal(hout[ri], out[ri.to(dev)].cpu()))
            del host_prefill, hout
        e2e = {"value": e2e_variants["fp32_out"]["value"], "unit": "TFLOP/s", "ms": e2e_variants["fp32_out"]["ms"],
               "h2d_bytes_per_step": e2e_variants["fp32_out"]["h2d_bytes_per_step"],
               "d2h_bytes_per_step": e2e_variants["fp32_out"]["d2h_bytes_per_step"],
               "path": "vxl_chunk_prefill_host: pinned host q/k/v -> device (one copy per tensor and chunk) -> one prefill "
                       "call per chunk -> pinned host out, on three streams",
               "bf16_out": e2e_variants["bf16_out"]}
        del hq, hk, hv
    if do_decode and not profiling and not args.no_e2e:
        # decode from a pinned host query to a pinned host output: every call is followed by the copy back
        # and a synchronisation, as a token loop on the host would do
        hq1 = dq.cpu().pin_memory()
        e2e_dec = {}
        for B_, kk in ((1, 8), (dB, 8), (1, 16), (dB, 16)):
            qd = torch.empty((B_, dHq, dD), dtype=torch.bfloat16, device=dev)
            od = torch.empty((B_, dHq, dD), dtype=torch.float32, device=dev)
            ho = torch.empty((B_, dHq, dD), dtype=torch.float32).pin_memory()
            ts = []
            for it in range(203):
                b0 = it % dB if B_ == 1 else 0
                t0 = time.perf_counter()
                qd.copy_(hq1[b0:b0 + B_], non_blocking=True)
                vb.bilevel_decode_attn(qd, dk[b0:b0 + B_], dv[b0:b0 + B_], doff, dridx, kk, max_chunk_len=dL, out=od,
                                       workspace=ws_d[kk], sparse=(dks[b0:b0 + B_], dvs[b0:b0 + B_]))
                ho.copy_(od, non_blocking=True)
                torch.cuda.synchronize()
                ts.append(time.perf_counter() - t0)
            us = float(np.median(ts[3:])) * 1e6
            e2e_dec[f"B{B_}_k{kk}"] = {"us_per_step_host_to_host": us, "gbs": B_ * bytes_seq[kk] / us / 1e3,
                                       "h2d_bytes_per_step": int(qd.numel() * 2), "d2h_bytes_per_step": int(ho.numel() * 4),
                                       "calls": 200}
        if e2e is not None:
            e2e["decode"] = e2e_dec

    # ------------------------------------------------------------------ CPU oracle beside it
    cpu = None
    if world == 1 and rank == 0 and not args.no_cpu_baseline and not profiling:
        if do_prefill:
            cpu = oracle_prefill_sample(sh, host_bits[0], host_bits[1], host_bits[2], ridx_np, 12.0)
            cpu.pop("seconds", None)
        if do_decode and cpu is not None:
            qb, kb, vb_ = bits(dq[0]), bits(dk[0]), bits(dv[0])
            cpu["decode"] = {f"k{kk}": oracle_decode_full(qb, kb, vb_, doff_np, dridx_np, d_scale, kk, bytes_seq[kk]) for kk in topks}
            del qb, kb, vb_
    host_bits = None

    # ------------------------------------------------------------------ other workloads (sweeps and variants)
    extra, by_workload = {}, {}
    if not args.no_extra and rank == 0 and not profiling:
        del q, k, v, out
        torch.cuda.empty_cache()

        def time_prefill(name, n_iter, n_rows):
            s2 = inputs.prefill_shape(name)
            eq, ek, evv, eridx_np = gen_prefill(s2, dev)
            eridx = torch.from_numpy(eridx_np).to(dev)
            eo = torch.empty((s2.T, s2.Hq, s2.D), dtype=torch.float32, device=dev)
            fn = lambda: vb.chunk_prefill_attn(eq, ek, evv, s2.L, eridx, scale=s2.scale, out=eo, workspace=ws_p)
            for _ in range(3):
                fn()
            ms = timed_calls(fn, n_iter, stream)
            tf = s2.useful_flops() / (np.median(ms) * 1e-3) / 1e12
            rec = {"T": s2.T, "chunk_len": s2.L, "R": s2.R, "ms": summary(ms), "useful_tflops": float(tf),
                   "frac_of_measured_burst": float(tf / peak_tf), "frac_of_nominal": float(tf / NOMINAL_TFLOPS)}
            if check:
                rec["parity"] = parity_prefill(s2, bits(eq), bits(ek), bits(evv), eridx_np, eo, n_rows, 12)
            return rec

        # time against T (16K / 64K / 256K; the 256K line is the headline above) and against the chunk length at 64K
        for name, n_iter in (("cfg2_16k", 20), ("cfg3_64k", 20), ("sweep_L512", 20), ("sweep_L1024", 20),
                             ("sweep_L2048", 20), ("sweep_L4096", 20)):
            if name != sh.name:
                by_workload[name] = time_prefill(name, n_iter, 48)
        # sliding chunk window (window 2048 advancing by 1024) behind a 512-token prefix, 64K visual tokens
        wT, wL, wS, wP, wR = 65536, 2048, 1024, 512, 128
        g = torch.Generator(device=dev); g.manual_seed(inputs.config_seed(3, 7))
        wq = torch.randn((wP + wT, 28, 128), generator=g, device=dev).to(torch.bfloat16)
        wk = torch.randn((wP + wT, 4, 128), generator=g, device=dev).to(torch.bfloat16)
        wv = torch.randn((wP + wT, 4, 128), generator=g, device=dev).to(torch.bfloat16)
        wridx = torch.from_numpy(inputs.make_retained_idx(np.random.default_rng(1), wT // wS, wS, wR) + np.int32(wP)).to(dev)
        wo = torch.empty((wP + wT, 28, 128), dtype=torch.float32, device=dev)
        fn = lambda: vb.chunk_prefill_attn(wq, wk, wv, wL, wridx, out=wo, workspace=ws_p, step=wS, prefix_len=wP)
        fn(); fn()
        ms = float(np.median(timed_calls(fn, 5, stream)))
        wfl = inputs.window_useful_flops(wT, wL, wS, wP, wR, 28, 128)
        extra["window_64k_L2048_S1024_P512"] = {"ms": ms, "useful_tflops": wfl / (ms * 1e-3) / 1e12,
                                                "frac_of_measured_burst": wfl / (ms * 1e-3) / 1e12 / peak_tf}
        del wq, wk, wv, wo
        if do_decode:
            kk = topks[0]
            dx = {}
            # sparse rows gathered from the dense cache by index (no packed level)
            fn = lambda: vb.bilevel_decode_attn(dq, dk, dv, doff, dridx, kk, max_chunk_len=dL, out=dout[kk], workspace=ws_d[kk])
            fn(); fn()
            ms = float(np.median(timed_calls(fn, 10, stream)))
            dx[f"B{dB}_k{kk}_unpacked_sparse"] = {"us_per_step": ms * 1e3, "gbs": dB * bytes_seq[kk] / (ms * 1e-3) / 1e9}
            # sparse level by average pooling: one pass over the dense cache (K and V read once)
            fn = lambda: vb.pool_sparse(dk, dv, doff, dR)
            fn(); fn()
            ms = float(np.median(timed_calls(fn, 5, stream)))
            pool_bytes = 2 * dk.numel() * 2 + 2 * dB * dC * dR * dHkv * dD * 2
            dx["pool_sparse_level"] = {"ms": ms, "gbs": pool_bytes / (ms * 1e-3) / 1e9,
                                       "frac_hbm_measured": pool_bytes / (ms * 1e-3) / 1e9 / peak_hbm}
            pks, pvs = vb.pool_sparse(dk, dv, doff, dR)
            fn = lambda: vb.bilevel_decode_attn(dq, dk, dv, doff, None, kk, max_chunk_len=dL, out=dout[kk], workspace=ws_d[kk],
                                                sparse=(pks, pvs))
            fn(); fn()
            ms = float(np.median(timed_calls(fn, 10, stream)))
            dx[f"B{dB}_k{kk}_pooled_sparse_level"] = {"us_per_step": ms * 1e3, "gbs": dB * bytes_seq[kk] / (ms * 1e-3) / 1e9}
            del pks, pvs
            # dense level kept in pinned host memory, selected chunks reloaded over PCIe every step (2 sequences)
            oB = min(2, dB)
            kh, vh = dk[:oB].cpu().pin_memory(), dv[:oB].cpu().pin_memory()
            dec = vb.OfflineDecoder(kh, vh, doff.cpu(), (dks[:oB], dvs[:oB]), kk, dL, dHq)
            fn = lambda: dec.step(dq[:oB])
            fn(); fn()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for _ in range(5):
                fn()
            torch.cuda.synchronize()
            sec = (time.perf_counter() - t0) / 5               # the call synchronises inside: wall clock per step
            h2d_off = oB * kk * dL * dHkv * dD * 2 * 2
            dx[f"B{oB}_k{kk}_offline_dense_level"] = {"us_per_step": sec * 1e6, "h2d_bytes_per_step": h2d_off,
                                                      "h2d_gbs": h2d_off / sec / 1e9}
            del dec, kh, vh
            extra["decode"] = dx

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    ach = flops / (ms_p * 1e-3) / 1e12        # per launch, from the timed region's events
    kname = "prefill_tc_kernel" if kind == 1 else "prefill_general_kernel"
    # Denominator: the burst figure for a kernel timed alone, the sustained one for a kernel timed inside a long
    # step.  The kernel counts as "inside a long step" when the timed steps last a quarter of a second or more
    # and the clock samples taken meanwhile show the power cap at work; both fractions are printed either way.
    sustained_tf = float(peaks.get("bf16_tflops_sustained", peak_tf))
    long_step = (K * ms_step >= 250.0) and ("sw_power_cap" in clocks.get("reasons", []))
    roof_tf = sustained_tf if long_step else peak_tf
    roofline = {"bound": "tensor", "kernel": kname, "workload": sh.name,
                "achieved": ach, "peak": roof_tf, "unit": "TFLOP/s", "frac": ach / roof_tf,
                "peak_kind": (f"{peak_kind} " if peak_kind == "measured" else "fallback ") +
                             ("sustained bf16 (the timed steps last %.2f s under sw_power_cap)" % (K * ms_step * 1e-3) if long_step
                              else "burst bf16 (short timed region)"),
                "frac_of_burst": ach / peak_tf, "burst_peak": peak_tf,
                "frac_of_sustained": ach / sustained_tf, "sustained_peak": sustained_tf,
                "frac_of_nominal": ach / NOMINAL_TFLOPS, "nominal_peak": NOMINAL_TFLOPS,
                "useful_flops_per_launch": flops, "ms_per_launch": ms_p, "ms_per_launch_median": med_p,
                "traffic": captured_traffic("prefill_tc_kernel", sh.T) if kind == 1 else None}
    if isolated_ms is not None:
        roofline["isolated_call"] = {"ms": isolated_ms, "achieved": flops / (isolated_ms * 1e-3) / 1e12,
                                     "frac_of_burst": flops / (isolated_ms * 1e-3) / 1e12 / peak_tf,
                                     "frac_of_nominal": flops / (isolated_ms * 1e-3) / 1e12 / NOMINAL_TFLOPS,
                                     "how": "one call after 1 s of idling, median of 3 (boost clocks, as the burst peak was taken)"}
    if decode is not None:
        loop = decode["decode_only_loop"]
        roofline["decode"] = {
            "bound": "hbm", "kernel": "decode_stream_kernel (sparse and dense passes) + combine_two_pass_kernel",
            "peak": peak_hbm, "nominal_peak": NOMINAL_HBM_GBS, "unit": "GB/s",
            "traffic": captured_traffic("decode_stream_kernel", dB) if dB > 0 else None}
        for kk in topks:
            ins, lp = decode["in_step"][f"k{kk}"], loop[f"k{kk}"]
            roofline["decode"][f"k{kk}"] = {
                "bytes_per_seq": bytes_seq[kk],
                f"B{dB}": {"us_in_step": ins["us_per_step_batch"], "achieved_in_step": ins["gbs_batch"], "frac_in_step": ins["frac_hbm_measured_batch"],
                           "us": lp["us_per_step_batch"]["median"], "achieved": lp["gbs_batch"], "frac": lp["frac_hbm_measured_batch"],
                           "frac_of_nominal": lp["frac_hbm_nominal_batch"]},
                "B1": {"us_in_step": ins["us_per_token_b1"], "achieved_in_step": ins["gbs_b1"], "frac_in_step": ins["frac_hbm_measured_b1"],
                       "us": lp["us_per_token_b1"]["median"], "achieved": lp["gbs_b1"], "frac": lp["frac_hbm_measured_b1"],
                       "frac_of_nominal": lp["frac_hbm_nominal_b1"]}}
    if by_workload:
        roofline["by_workload"] = {n: {"ms": r["ms"]["median"], "useful_tflops": r["useful_tflops"], "frac": r["frac_of_measured_burst"],
                                       "frac_of_nominal": r["frac_of_nominal"],
                                       "parity_ok": r.get("parity", {}).get("ok")} for n, r in by_workload.items()}

    config = workload_config(sh, topks, dB)
    launches_prefill = (3 if sh.R > 0 and sh.C > 1 else 2) if kind == 1 else 1
    line = {
        "metric": "prefill_useful_tflops", "value": tflops, "unit": "TFLOP/s", "n_gpus": world,
        "steps": K, "warmup": args.warmup, "ms_per_step": ms_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "config": config,
        "notes": {"prefill_kernel": "tcgen05" if kind == 1 else "general(mma.sync)",
                  "decode": "stored sparse level streamed by TMA; batch-1 calls " + ("replayed from a CUDA graph" if graphs else "launched eagerly"),
                  "l2": "prefill q+k+v+out = %.0f MB; a batch decode call reads %.0f-%.0f MB (> 126 MB L2); batch-1 calls rotate over %d caches"
                        % ((sh.T * sh.Hq * sh.D * 6 + 4 * sh.T * sh.Hkv * sh.D) / 1e6, dB * bytes_seq[topks[0]] / 1e6,
                           dB * bytes_seq[topks[-1]] / 1e6, dB),
                  "inputs": "drawn on the device with the recipe of inputs.py; sampled outputs checked against the fp64 oracle (parity)",
                  "parallelism": f"replicas x{world}"},
        "ms_prefill": ms_p,
        "frac_of_nominal_bf16": tflops / world / NOMINAL_TFLOPS,
        "parity": parity if parity else None,
        "decode": decode,
        "roofline": roofline,
        "e2e": e2e,
        # per step: prefill = pack + rank + attention kernels (tcgen05 path) or one general kernel;
        # every decode call = sparse pass, dense pass (ranks the chunks itself), combine
        "gpu_launches": K * ((launches_prefill if do_prefill else 0) + (3 * len(topks) * (1 + dB) if do_decode else 0)),
        "clocks": clocks,
        "cpu_baseline": cpu,
        "prefill_by_workload": by_workload if by_workload else None,
        "extra": extra,
    }
    if profiling:
        line["partial"] = args.only
        if args.only == "decode":
            line["value"] = None; line["roofline"] = None; line["ms_prefill"] = None
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
