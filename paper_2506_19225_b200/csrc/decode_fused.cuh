// Bi-level decoding as ONE persistent kernel: relevance scores, top-k, sparse and dense split-KV
// attention and (for small batches) the final merge, with no launch between the steps.
//
// The separate stream passes of decode_stream.cuh each pay a launch, a ramp of the TMA pipeline and a
// tail; at batch 1 a call moves 67-100 MB, about 10-15 us of HBM time, and three such ramps cost as
// much again.  Here every CTA (one per SM) runs one continuous stream of 32-row tiles through its
// 3-stage TMA ring and the steps of the method are resolved inside that stream:
//
//   score sweep    K tiles of a chunk's sparse rows.  The consumer warp of a kv head reduces the chunk's
//                  log-sum-exp over its query heads, stores it (score_part) and counts the chunk as
//                  published for its sequence (release fence + atomic).
//   attend sweep   K and V tiles of the same sparse rows (K comes back from L2: it was read moments
//                  ago without an evict-first hint) -> the chunk's partial (m, l, o).  The score sweep
//                  of a CTA runs one chunk ahead of its attend sweep, so every score of a sequence is
//                  published while at least one attend sweep per CTA is still streaming.
//   ranking        before its first dense tile of a sequence, the producer warp waits (bounded) until
//                  all chunk scores of that sequence are published, ranks them (ties to the lower chunk
//                  id, ascending output) and resolves its dense items; the loads already in the ring
//                  keep the consumers busy meanwhile.
//   dense slices   rows of the selected chunks, dealt in contiguous blocks so that a CTA touches few
//                  sequences; the CTA that holds a sequence's first dense item also writes the selection,
//                  the flags and the scores for the merge and for the caller.
//   merge          when one round of merge tasks fits the grid (batch 1 with 28 heads), the CTAs meet at a
//                  counter (bounded wait) and merge the partials themselves; otherwise the combine kernel
//                  follows as its own launch.
//
// The producer describes every stage it fills in a small descriptor beside the ring (kind, sequence,
// head block, partial slot, valid rows, first / last tile of an item); the consumer warps know nothing
// about items or phases.
//
// CTAs of this grid wait for one another (score counters, the merge counter).  The grid never exceeds one
// CTA per SM and the kernel allows one CTA per SM, so all of them become resident, including when the
// launch overlaps the tail of an earlier kernel (whose CTAs do not depend on this one).  Every wait is
// bounded; on expiry the kernel records VXL_ERR_TIMEOUT, raises a grid-wide abort flag and winds down.
// The counters live in the workspace and are returned to zero by the last CTA to leave.
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "decode.cuh"
#include "decode_stream.cuh"

namespace vxl {

struct FusedMaps {
    CUtensorMap ks, vs;                  // sparse level [B*C*R, Hkv*D]
    CUtensorMap k, v;                    // dense cache [B*T, Hkv*D]
};

struct FusedParams {
    const __nv_bfloat16 *q;
    const int32_t *off;                  // [C+1]
    float *part_m, *part_l, *part_o;     // [B,Hq,P], [B,Hq,P], [B,Hq,P,D]
    float *score_part;                   // [B,C,Hkv]
    int32_t *sel, *flags;                // workspace [B,topk], [B,C]
    int32_t *topk_out;                   // caller's [B,topk] or null
    float *scores_out;                   // caller's [B,C] or null
    int32_t *seq_count;                  // workspace [B]: (chunk, kv head) scores published; zero between calls
    int32_t *sync;                       // workspace: [0] CTAs past their last item, [1] CTAs leaving, [2] abort
    WsHeader *hdr;
    void *out;
    float *lse;
    int64_t o_sb, o_sh;
    int64_t q_sb, q_sh;
    int B, T, Hq, Hkv, G, C, R, topk;
    int nslices, slice_rows, P, nhb;
    int nA, nB;                          // sparse items B*C*nhb, dense items B*topk*nslices*nhb
    int combine;                         // 1: merge the partials in this kernel
    int out_bf16;
    float scale_log2;
};

enum : int { kFuScore = 0, kFuSparse = 1, kFuDense = 2, kFuEnd = 3 };

__device__ __forceinline__ int ld_acquire_gpu(const int *p)
{
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Bounded wait for a counter written by other CTAs; gives up early when the grid has aborted.
__device__ __forceinline__ bool wait_count(const int *p, int target, const int *abort_flag)
{
    if (ld_acquire_gpu(p) >= target) return true;
    const long long start = clock64();
    for (int it = 0;; ++it) {
        if (ld_acquire_gpu(p) >= target) return true;
        if ((it & 15) == 15 && (ld_acquire_gpu(abort_flag) != 0 || clock64() - start > kWaitCycles)) return false;
        __nanosleep(20);
    }
}

// Running softmax state of one kv head's query group in the fragment layout of the warp-level MMA:
// rows g and g + 8 of the quad's lanes are query heads, the key tile sits on the N side.
template <int D>
struct GroupAcc {
    float o[D / 8][4];
    float m_lo, m_hi, l_lo, l_hi;

    __device__ __forceinline__ void reset()
    {
#pragma unroll
        for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
        m_lo = m_hi = -INFINITY;
        l_lo = l_hi = 0.f;
    }

    // One tile of TK = 32 keys: logits, online softmax and (WITH_V) P.V.  tK / tV: shared-memory address of
    // this kv head's first 128-byte panel of the K / V tile (128-byte swizzle, panels kPanel bytes apart).
    template <bool WITH_V>
    __device__ __forceinline__ void tile(uint32_t tK, uint32_t tV, uint32_t kPanel, int nvalid, const uint32_t (&qf)[D / 16][4],
                                         float scale_log2, int lane)
    {
        constexpr int TK = 32;
        const int t = lane & 3;
        float s[TK / 8][4];
#pragma unroll
        for (int i = 0; i < TK / 8; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
        for (int kb = 0; kb < D / 16; ++kb) {
#pragma unroll
            for (int kg = 0; kg < TK / 16; ++kg) {
                const int mi = lane >> 3, ri = lane & 7;
                const int key = kg * 16 + (mi >> 1) * 8 + ri;
                const int col = kb * 16 + (mi & 1) * 8;
                const uint32_t addr = tK + (col >> 6) * kPanel + key * 128 + ((((col & 63) >> 3) ^ (key & 7)) << 4);
                uint32_t b0, b1, b2, b3;
                ldsm_x4(addr, b0, b1, b2, b3);
                mma_bf16(s[2 * kg], qf[kb][0], qf[kb][1], qf[kb][2], qf[kb][3], b0, b1);
                mma_bf16(s[2 * kg + 1], qf[kb][0], qf[kb][1], qf[kb][2], qf[kb][3], b2, b3);
            }
        }
        float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
        for (int nb = 0; nb < TK / 8; ++nb)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int key = nb * 8 + 2 * t + (j & 1);
                const float x = (key < nvalid) ? s[nb][j] * scale_log2 : -INFINITY;
                s[nb][j] = x;
                if (j < 2) mx_lo = fmaxf(mx_lo, x); else mx_hi = fmaxf(mx_hi, x);
            }
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
        const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
        const bool moved = (mn_lo != m_lo) || (mn_hi != m_hi);
        if (__any_sync(0xffffffffu, moved)) {
            const float c_lo = fast_exp2(m_lo - mn_lo), c_hi = fast_exp2(m_hi - mn_hi);
            l_lo *= c_lo; l_hi *= c_hi;
            if (WITH_V) {
#pragma unroll
                for (int nd = 0; nd < D / 8; ++nd) {
                    o[nd][0] *= c_lo; o[nd][1] *= c_lo; o[nd][2] *= c_hi; o[nd][3] *= c_hi;
                }
            }
            m_lo = mn_lo; m_hi = mn_hi;
        }
#pragma unroll
        for (int nb = 0; nb < TK / 8; ++nb) {
            s[nb][0] = fast_exp2(s[nb][0] - m_lo); s[nb][1] = fast_exp2(s[nb][1] - m_lo);
            s[nb][2] = fast_exp2(s[nb][2] - m_hi); s[nb][3] = fast_exp2(s[nb][3] - m_hi);
            l_lo += s[nb][0] + s[nb][1];
            l_hi += s[nb][2] + s[nb][3];
        }
        if (WITH_V) {
#pragma unroll
            for (int kg = 0; kg < TK / 16; ++kg) {
                const uint32_t a0 = pack_bf16(s[2 * kg][0], s[2 * kg][1]), a1 = pack_bf16(s[2 * kg][2], s[2 * kg][3]);
                const uint32_t a2 = pack_bf16(s[2 * kg + 1][0], s[2 * kg + 1][1]);
                const uint32_t a3 = pack_bf16(s[2 * kg + 1][2], s[2 * kg + 1][3]);
#pragma unroll
                for (int nd2 = 0; nd2 < D / 16; ++nd2) {
                    const int mi = lane >> 3, ri = lane & 7;
                    const int key = kg * 16 + (mi & 1) * 8 + ri;
                    const int col = nd2 * 16 + (mi >> 1) * 8;
                    const uint32_t addr = tV + (col >> 6) * kPanel + key * 128 + ((((col & 63) >> 3) ^ (key & 7)) << 4);
                    uint32_t b0, b1, b2, b3;
                    ldsm_x4_t(addr, b0, b1, b2, b3);
                    if (nvalid < TK) {
                        // rows past the item's end hold whatever follows in memory; their probabilities are 0
                        // and 0 x NaN must not reach O: read those V rows as zeros
                        const int k0 = kg * 16 + 2 * t;
                        const uint32_t m0 = (k0 < nvalid ? 0xFFFFu : 0u) | (k0 + 1 < nvalid ? 0xFFFF0000u : 0u);
                        const uint32_t m1 = (k0 + 8 < nvalid ? 0xFFFFu : 0u) | (k0 + 9 < nvalid ? 0xFFFF0000u : 0u);
                        b0 &= m0; b2 &= m0; b1 &= m1; b3 &= m1;
                    }
                    mma_bf16(o[2 * nd2], a0, a1, a2, a3, b0, b1);
                    mma_bf16(o[2 * nd2 + 1], a0, a1, a2, a3, b2, b3);
                }
            }
        }
    }

    // A row's keys are spread over the four lanes of a quad: finish the sums.
    __device__ __forceinline__ void finish()
    {
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
    }
};

template <int D, int HPC>
__global__ void __launch_bounds__(StreamCfg<D, HPC>::kThreads, 1)
decode_fused_kernel(const __grid_constant__ FusedMaps maps, const FusedParams p)
{
    using Cfg = StreamCfg<D, HPC>;
    constexpr int TK = Cfg::TK, NS = Cfg::kStages, NT = Cfg::kThreads;
    extern __shared__ unsigned char smem_dyn[];
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char *gen = smem_dyn + (base - smem_u32(smem_dyn));
    const uint32_t bar0 = base + Cfg::kBarOff;
    volatile int *s_abort = reinterpret_cast<volatile int *>(gen + Cfg::kBarOff + 8 * 2 * NS);
    volatile int4 *s_desc = reinterpret_cast<volatile int4 *>(gen + Cfg::kBarOff + 64);
    float *s_score = reinterpret_cast<float *>(gen + Cfg::kSelOff);
    int *s_flag = reinterpret_cast<int *>(gen + Cfg::kSelOff + Cfg::kSelMaxChunks * 4);
    int *s_sel = reinterpret_cast<int *>(gen + Cfg::kSelOff + Cfg::kSelMaxChunks * 8);
    auto full = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto empty = [&](int s) { return bar0 + 8u * (uint32_t)(NS + s); };

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = (int)gridDim.x, x = (int)blockIdx.x;
    if (tid == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), HPC); }
        *s_abort = 0;
        mbar_fence_init();
    }
    __syncthreads();
    // Everything above overlaps the tail of the previous kernel in the stream; the workspace (counters,
    // partials) and the inputs are only touched below.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int *g_abort = p.sync + 2;

    if (warp == HPC) {
        // ------------------------------------------------------------------ producer
        int issued = 0;
        bool ok = true;
        const uint64_t once_policy = l2_evict_first_policy();
        // one stage: descriptor, then the loads (none for an empty item); with_v = 0 loads the K tile only
        auto issue = [&](int kind, bool first, bool last, int b, int hb, int slot, int nvalid, const CUtensorMap *mk,
                         const CUtensorMap *mv, int64_t y, bool with_v, bool once) -> bool {
            const int stage = issued % NS;
            const uint32_t ph = (issued / NS) & 1;
            if (!mbar_wait(empty(stage), ph ^ 1) || *s_abort) return false;
            if (lane == 0) {
                s_desc[stage].x = kind | (first ? 16 : 0) | (last ? 32 : 0) | (hb << 8);
                s_desc[stage].y = b;
                s_desc[stage].z = slot;
                s_desc[stage].w = nvalid;
                if (nvalid <= 0) {
                    mbar_arrive(full(stage));
                } else {
                    mbar_expect_tx(full(stage), with_v ? Cfg::kStageBytes : Cfg::kTileBytes);
                    const uint32_t dK = base + stage * Cfg::kStageBytes;
                    const int x0 = hb * HPC * D;
#pragma unroll
                    for (int pn = 0; pn < Cfg::PANELS; ++pn) {
                        if (once)
                            asm volatile(
                                "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;" ::"r"(dK + pn * Cfg::kPanelBytes),
                                "l"(mk), "r"(x0 + pn * 64), "r"((int)y), "r"(full(stage)), "l"(once_policy)
                                : "memory");
                        else
                            asm volatile(
                                "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dK + pn * Cfg::kPanelBytes),
                                "l"(mk), "r"(x0 + pn * 64), "r"((int)y), "r"(full(stage))
                                : "memory");
                        if (with_v)
                            asm volatile(
                                "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;" ::"r"(dK + Cfg::kTileBytes + pn * Cfg::kPanelBytes),
                                "l"(mv), "r"(x0 + pn * 64), "r"((int)y), "r"(full(stage)), "l"(once_policy)
                                : "memory");
                    }
                }
            }
            ++issued;
            return true;
        };
        // sparse rows of chunk item a: score sweep (keys only, kept in L2 for the attend sweep) or attend sweep
        auto sparse_item = [&](int a, int kind) -> bool {
            const int hb = a % p.nhb, it2 = a / p.nhb;
            const int b = it2 / p.C, c = it2 % p.C;
            const int64_t row0 = ((int64_t)b * p.C + c) * p.R;
            for (int r = 0; r < p.R; r += TK)
                if (!issue(kind, r == 0, r + TK >= p.R, b, hb, c, min(TK, p.R - r), &maps.ks, &maps.vs, row0 + r,
                           kind == kFuSparse, kind == kFuSparse))
                    return false;
            return true;
        };
        const int nA_mine = x < p.nA ? (p.nA - x + G - 1) / G : 0;
        for (int i = 0; i < nA_mine && ok; ++i) {
            ok = sparse_item(x + i * G, kFuScore);
            if (ok && i > 0) ok = sparse_item(x + (i - 1) * G, kFuSparse);
        }
        if (ok && nA_mine > 0) ok = sparse_item(x + (nA_mine - 1) * G, kFuSparse);

        // dense items: a contiguous block, dealt from the far end of the grid so that the CTAs with the fewest
        // sparse items take the first (earliest ranked) sequences
        const int ipc = (p.nB + G - 1) / G;
        const int lo_item = (G - 1 - x) * ipc, hi_item = min(p.nB, lo_item + ipc);
        const int per_b = p.topk * p.nslices * p.nhb;
        int ranked_b = -1, sel_b0 = lo_item < hi_item ? lo_item / per_b : 0;
        for (int item = lo_item; item < hi_item && ok; ++item) {
            const int hb = item % p.nhb, it2 = item / p.nhb;
            const int b = it2 / (p.topk * p.nslices), js = it2 % (p.topk * p.nslices);
            const int j = js / p.nslices, s = js % p.nslices;
            if (b != ranked_b) {
                // ---- every chunk score of sequence b must be in; then rank (the whole warp)
                if (!wait_count(p.seq_count + b, p.C * p.Hkv, g_abort)) { ok = false; break; }
                const bool owner = (b * per_b >= lo_item);                // this CTA holds the sequence's first dense item
                for (int c = lane; c < p.C; c += 32) {
                    const float *sp = p.score_part + ((int64_t)b * p.C + c) * p.Hkv;
                    float acc = 0.f;
                    for (int g2 = 0; g2 < p.Hkv; ++g2) acc += __ldcg(sp + g2);
                    const float sc = acc / (float)p.Hq;
                    s_score[c] = sc;
                    if (owner && p.scores_out != nullptr) p.scores_out[(int64_t)b * p.C + c] = sc;
                }
                __syncwarp();
                // rank of chunk c = number of chunks that beat it (larger score, or equal score and lower id)
                for (int c = lane; c < p.C; c += 32) {
                    const float sc = s_score[c];
                    int rank = 0;
#pragma unroll 8
                    for (int c2 = 0; c2 < p.C; ++c2) {
                        const float s2 = s_score[c2];
                        rank += (s2 > sc || (s2 == sc && c2 < c)) ? 1 : 0;
                    }
                    s_flag[c] = rank < p.topk ? 1 : 0;
                }
                __syncwarp();
                int before = 0;                                          // selected chunks with a lower id: ascending output
                for (int c0 = 0; c0 < p.C; c0 += 32) {
                    const int c = c0 + lane;
                    const int f = c < p.C ? s_flag[c] : 0;
                    const unsigned bal = __ballot_sync(0xffffffffu, f != 0);
                    const int pos = before + __popc(bal & ((1u << lane) - 1u));
                    if (c < p.C && owner) p.flags[(int64_t)b * p.C + c] = f;
                    if (f && pos < p.topk) {
                        s_sel[(b - sel_b0) * p.topk + pos] = c;
                        if (owner) {
                            p.sel[(int64_t)b * p.topk + pos] = c;
                            if (p.topk_out != nullptr) p.topk_out[(int64_t)b * p.topk + pos] = c;
                        }
                    }
                    before += __popc(bal);
                }
                __syncwarp();
                ranked_b = b;
            }
            const int chunk = s_sel[(b - sel_b0) * p.topk + j];
            int lo = 0, len = 0;
            if (chunk < 0 || chunk >= p.C) {
                if (lane == 0) raise_status(p.hdr, VXL_ERR_INVALID_INDEX, 150);
            } else {
                lo = p.off[chunk];
                len = p.off[chunk + 1] - lo;
                if (lo < 0 || len < 0 || lo + len > p.T) {
                    if (lane == 0) raise_status(p.hdr, VXL_ERR_INVALID_INDEX, 151);
                    lo = 0; len = 0;
                }
                if (len > p.nslices * p.slice_rows) {                     // max_chunk_len was not a bound
                    if (lane == 0) raise_status(p.hdr, VXL_ERR_INVALID_ARG, 152);
                    len = p.nslices * p.slice_rows;
                }
            }
            const int64_t row0 = (int64_t)b * p.T + lo + (int64_t)s * p.slice_rows;
            const int nrows = max(0, min(p.slice_rows, len - s * p.slice_rows));
            const int slot = p.C + js;
            if (nrows == 0) {
                ok = issue(kFuDense, true, true, b, hb, slot, 0, &maps.k, &maps.v, 0, true, true);   // an empty partial
                continue;
            }
            for (int r = 0; r < nrows && ok; r += TK)
                ok = issue(kFuDense, r == 0, r + TK >= nrows, b, hb, slot, min(TK, nrows - r), &maps.k, &maps.v, row0 + r,
                           true, true);
        }
        if (ok) {
            // end of the stream
            const int stage = issued % NS;
            if (mbar_wait(empty(stage), ((issued / NS) & 1) ^ 1) && !*s_abort) {
                if (lane == 0) { s_desc[stage].x = kFuEnd; mbar_arrive(full(stage)); }
                ++issued;
            } else {
                ok = false;
            }
        }
        if (!ok && lane == 0) {
            raise_status(p.hdr, VXL_ERR_TIMEOUT, 153);
            *s_abort = 1;
            atomicExch(p.sync + 2, 1);
        }
        for (int s = 0; s < NS && s < issued; ++s) {          // let the last copies land before the ring is reused
            const int i2 = issued - 1 - s;
            mbar_wait(full(i2 % NS), (i2 / NS) & 1);
        }
    } else {
        // ------------------------------------------------------------------ consumers: one warp per kv head
        const int hl = warp;
        const int g = lane >> 2, t = lane & 3;
        int consumed = 0;
        bool ok = true;
        int q_key = -1;
        uint32_t qf[D / 16][4];
        GroupAcc<D> acc;
        acc.reset();
        for (;;) {
            const int stage = consumed % NS;
            const uint32_t ph = (consumed / NS) & 1;
            if (!mbar_wait(full(stage), ph) || *s_abort) { ok = false; break; }
            ++consumed;
            const int dx = s_desc[stage].x, b = s_desc[stage].y, slot = s_desc[stage].z, nvalid = s_desc[stage].w;
            const int kind = dx & 15, hb = dx >> 8;
            if (kind == kFuEnd) break;
            const int kvh = hb * HPC + hl;
            if (dx & 16) {
                if (b * p.nhb + hb != q_key) {                        // query fragments: rows = heads of the kv group
                    q_key = b * p.nhb + hb;
                    const __nv_bfloat16 *qb = p.q + (int64_t)b * p.q_sb + (int64_t)kvh * p.G * p.q_sh;
#pragma unroll
                    for (int kb = 0; kb < D / 16; ++kb) {
                        const int c0 = kb * 16 + 2 * t;
                        qf[kb][0] = (g < p.G) ? *reinterpret_cast<const uint32_t *>(qb + (int64_t)g * p.q_sh + c0) : 0u;
                        qf[kb][1] = (g + 8 < p.G) ? *reinterpret_cast<const uint32_t *>(qb + (int64_t)(g + 8) * p.q_sh + c0) : 0u;
                        qf[kb][2] = (g < p.G) ? *reinterpret_cast<const uint32_t *>(qb + (int64_t)g * p.q_sh + c0 + 8) : 0u;
                        qf[kb][3] = (g + 8 < p.G) ? *reinterpret_cast<const uint32_t *>(qb + (int64_t)(g + 8) * p.q_sh + c0 + 8) : 0u;
                    }
                }
                acc.reset();
            }
            if (nvalid > 0) {
                const uint32_t tK = base + stage * Cfg::kStageBytes + hl * (D / 64) * Cfg::kPanelBytes;
                if (kind == kFuScore) acc.template tile<false>(tK, tK, Cfg::kPanelBytes, nvalid, qf, p.scale_log2, lane);
                else acc.template tile<true>(tK, tK + Cfg::kTileBytes, Cfg::kPanelBytes, nvalid, qf, p.scale_log2, lane);
            }
            if (dx & 32) {
                acc.finish();
                if (kind == kFuScore) {
                    // sum over this kv head's query heads of the chunk's log-sum-exp, then count the chunk in
                    float sc = 0.f;
                    if (t == 0) {
                        if (g < p.G) sc += (acc.m_lo + log2f(acc.l_lo)) * kLn2;
                        if (g + 8 < p.G) sc += (acc.m_hi + log2f(acc.l_hi)) * kLn2;
                    }
#pragma unroll
                    for (int o2 = 16; o2 > 0; o2 >>= 1) sc += __shfl_xor_sync(0xffffffffu, sc, o2);
                    if (lane == 0) {
                        p.score_part[((int64_t)b * p.C + slot) * p.Hkv + kvh] = sc;
                        __threadfence();
                        atomicAdd(p.seq_count + b, 1);
                    }
                } else {
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        const int r2 = g + 8 * half;
                        if (r2 >= p.G) continue;
                        const int h = kvh * p.G + r2;
                        const int64_t pi = ((int64_t)b * p.Hq + h) * p.P + slot;
#pragma unroll
                        for (int nd = 0; nd < D / 8; ++nd)
                            *reinterpret_cast<float2 *>(p.part_o + pi * D + nd * 8 + 2 * t) =
                                make_float2(acc.o[nd][2 * half], acc.o[nd][2 * half + 1]);
                        if (t == 0) {
                            p.part_m[pi] = half ? acc.m_hi : acc.m_lo;
                            p.part_l[pi] = half ? acc.l_hi : acc.l_lo;
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty(stage));
        }
        if (!ok && lane == 0) {
            raise_status(p.hdr, VXL_ERR_TIMEOUT, 154);
            *s_abort = 1;
            atomicExch(p.sync + 2, 1);
        }
    }

    // ------------------------------------------------------------------ merge of the partials (small batches)
    __syncthreads();
    if (p.combine) {
        __shared__ int s_go;
        if (tid == 0) {
            __threadfence();                                  // this CTA's partials, flags and selection before the count
            atomicAdd(p.sync + 0, 1);
            const bool ok = !*s_abort && wait_count(p.sync + 0, G, g_abort);
            if (!ok && !*s_abort) { raise_status(p.hdr, VXL_ERR_TIMEOUT, 155); atomicExch(p.sync + 2, 1); }
            s_go = ok ? 1 : 0;
        }
        __syncthreads();
        if (s_go) {
            // task = (sequence, head, 32 output columns); 8 lanes x (threads / 8) slot groups.  Each thread folds
            // its slots with a running maximum, eight loads in flight; the groups meet in shared memory.
            constexpr int LN = 8, SG = NT / LN, U = 8;
            float *s_m = reinterpret_cast<float *>(gen);                 // the ring is idle now
            float *s_l = s_m + SG;
            float4 *s_o = reinterpret_cast<float4 *>(gen + 1024);
            const int nparts = D / 32, ntasks = p.B * p.Hq * nparts;
            const int ln = tid % LN, sg = tid / LN;
            for (int task = x; task < ntasks; task += G) {
                const int part = task % nparts, bh = task / nparts;
                const int b = bh / p.Hq, h = bh % p.Hq;
                const int64_t pb = ((int64_t)b * p.Hq + h) * p.P;
                const int32_t *fl = p.flags + (int64_t)b * p.C;
                float M = -INFINITY, L = 0.f;
                float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int s0 = sg; s0 < p.P; s0 += SG * U) {
                    float m[U], l[U];
                    float4 v[U];
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const int s2 = s0 + u * SG;
                        const bool in = s2 < p.P;
                        const bool dense_elsewhere = in && s2 < p.C && __ldcg(fl + s2) != 0;
                        m[u] = in ? __ldcg(p.part_m + pb + s2) : -INFINITY;
                        l[u] = (in && !dense_elsewhere) ? __ldcg(p.part_l + pb + s2) : 0.f;
                        v[u] = in ? __ldcg(reinterpret_cast<const float4 *>(p.part_o + (pb + s2) * D + part * 32 + ln * 4))
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        if (!(l[u] > 0.f)) continue;
                        const float Mn = fmaxf(M, m[u]);
                        const float fo = fast_exp2(M - Mn), fn = fast_exp2(m[u] - Mn);
                        L = L * fo + l[u] * fn;
                        a.x = a.x * fo + v[u].x * fn; a.y = a.y * fo + v[u].y * fn;
                        a.z = a.z * fo + v[u].z * fn; a.w = a.w * fo + v[u].w * fn;
                        M = Mn;
                    }
                }
                if (ln == 0) { s_m[sg] = M; s_l[sg] = L; }
                s_o[sg * LN + ln] = a;
                __syncthreads();
                if (sg == 0) {
                    float Mt = -INFINITY;
                    for (int i = 0; i < SG; ++i) Mt = fmaxf(Mt, s_m[i]);
                    float Lt = 0.f;
                    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (int i = 0; i < SG; ++i) {
                        const float f = (s_m[i] == -INFINITY) ? 0.f : fast_exp2(s_m[i] - Mt);
                        Lt += s_l[i] * f;
                        const float4 vv = s_o[i * LN + ln];
                        r.x += vv.x * f; r.y += vv.y * f; r.z += vv.z * f; r.w += vv.w * f;
                    }
                    const float inv = Lt > 0.f ? 1.f / Lt : 0.f;
                    const int64_t ob = (int64_t)b * p.o_sb + (int64_t)h * p.o_sh + part * 32 + ln * 4;
                    if (p.out_bf16) {
                        uint2 pk;
                        pk.x = pack_bf16(r.x * inv, r.y * inv);
                        pk.y = pack_bf16(r.z * inv, r.w * inv);
                        *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(p.out) + ob) = pk;
                    } else {
                        *reinterpret_cast<float4 *>(reinterpret_cast<float *>(p.out) + ob) =
                            make_float4(r.x * inv, r.y * inv, r.z * inv, r.w * inv);
                    }
                    if (p.lse != nullptr && part == 0 && ln == 0)
                        p.lse[(int64_t)b * p.Hq + h] = Lt > 0.f ? (Mt + log2f(Lt)) * kLn2 : -INFINITY;
                }
                __syncthreads();
            }
        }
    }

    // ------------------------------------------------------------------ the last CTA to leave returns the counters to zero
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        if (atomicAdd(p.sync + 1, 1) == G - 1) {
            for (int b = 0; b < p.B; ++b) p.seq_count[b] = 0;
            p.sync[0] = 0;
            p.sync[2] = 0;
            __threadfence();
            p.sync[1] = 0;
        }
    }
}

}  // namespace vxl
