// Split-KV partial attention for bi-level decoding as a persistent HBM stream.
//
// Used when the rows a work item reads are contiguous in memory: dense slices of a selected
// chunk, and the sparse level once it has been packed (vxl_pack_retained).  K and V are then
// 2-D bf16 arrays [rows, Hkv*D] and whole tiles of TK rows are brought in by TMA (128-byte
// swizzle, one request per 128-byte column panel: 4 KB or more per request instead of one
// request per row), through a 3-stage ring of 64 KB stages that stays full across work items.
// One CTA per SM walks a static list of items (sequence, partial slot, row range); a producer
// warp issues the loads and one consumer warp per kv head runs the logits and P.V of all TK keys
// of a tile on the warp-level bf16 MMA, with the query heads of the kv group on the M side, keeps
// the running (m, l, o) in registers and writes one partial per item (no cross-warp merge).
// The dense pass of a decode call can also rank the chunks itself (see StreamParams).
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "decode.cuh"

namespace vxl {

struct StreamMaps {
    CUtensorMap k, v;
};

struct StreamParams {
    const __nv_bfloat16 *q;
    const int32_t *off;                  // [C+1]            (dense)
    const int32_t *sel;                  // [B,topk]         (dense)
    const int32_t *flags;                // [B,C] or null    (sparse: skip chunks read dense)
    float *part_m, *part_l, *part_o;
    float *score_part;                   // [B,C,Hkv] or null (sparse pass): sum over a kv head's query heads of the
                                         // chunk's log-sum-exp, so that top-k reads Hkv numbers per chunk, not 2*Hq
    WsHeader *hdr;
    int64_t q_sb, q_sh;
    int B, T, Hq, Hkv, G, C, R, topk;
    int nslices, slice_rows, P;
    int staged;                          // dense pass: > 0 = the selected chunks were copied into a staging
                                         // buffer [B, topk, staged rows, Hkv*D] (chunk j of a sequence at slot j)
    int n_items;                         // sparse: B*C ; dense: B*topk*nslices
    // Dense pass that selects for itself (sel_scores != null): every CTA ranks the chunks of the
    // sequences its items belong to from the per-kv-head score sums of the sparse pass, so no
    // separate top-k launch sits between the two passes.  Items are then dealt in contiguous
    // blocks (a CTA touches few sequences); the CTA that holds a sequence's first item also writes
    // the selection, the dense flags and the scores for the combine pass and the caller.
    const float *sel_scores;             // [B,C,Hkv] or null
    int32_t *sel_out, *flags_out, *topk_out;   // [B,topk], [B,C], [B,topk] or null
    float *scores_out;                   // [B,C] or null
    int nhb;                             // kv head blocks (Hkv / HPC)
    float scale_log2;
};

template <int D, int HPC>
struct StreamCfg {
    static constexpr int TK = 32;                              // rows per stage
    static constexpr int PANELS = HPC * D / 64;                // 128-byte column panels per row
    static constexpr uint32_t kPanelBytes = TK * 128;
    static constexpr uint32_t kTileBytes = PANELS * kPanelBytes;   // K (or V) of one stage
    static constexpr uint32_t kStageBytes = 2 * kTileBytes;
    static constexpr int kStages = 3;
    static constexpr uint32_t kBarOff = kStages * kStageBytes;
    static constexpr uint32_t kSelOff = kBarOff + 256;            // selection scratch of the self-selecting dense pass
    static constexpr int kSelMaxChunks = 1024, kSelMaxEntries = 1024;
    static constexpr uint32_t kSelBytes = kSelMaxChunks * 8 + kSelMaxEntries * 4;
    static constexpr uint32_t kSmemBytes = kSelOff + kSelBytes + 1024;  // + alignment slack
    static constexpr int kThreads = 32 * (HPC + 1);            // one consumer warp per kv head + producer
    static_assert(kPanelBytes % 1024 == 0, "panels must keep the swizzle atom alignment");
};

template <int D, int HPC, bool SPARSE, bool WITH_V>
__global__ void __launch_bounds__(StreamCfg<D, HPC>::kThreads, 1)
decode_stream_kernel(const __grid_constant__ StreamMaps maps, const StreamParams p)
{
    using Cfg = StreamCfg<D, HPC>;
    constexpr int TK = Cfg::TK, NS = Cfg::kStages;
    extern __shared__ unsigned char smem_dyn[];
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char *gen = smem_dyn + (base - smem_u32(smem_dyn));
    const uint32_t bar0 = base + Cfg::kBarOff;
    volatile int *s_abort = reinterpret_cast<volatile int *>(gen + Cfg::kBarOff + 8 * 2 * NS);
    auto full = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto empty = [&](int s) { return bar0 + 8u * (uint32_t)(NS + s); };

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), HPC); }
        *s_abort = 0;
        mbar_fence_init();
    }
    __syncthreads();
    // Everything above overlaps the tail of the previous kernel in the stream; its results
    // (partials, flags, selection) are only read below.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // Items of this CTA: round-robin over the grid, or one contiguous block when the pass selects itself.
    const bool self_select = !SPARSE && p.sel_scores != nullptr;
    int item_lo = blockIdx.x, item_hi = p.n_items, item_step = gridDim.x;
    float *s_score = reinterpret_cast<float *>(gen + Cfg::kSelOff);
    int *s_flag = reinterpret_cast<int *>(gen + Cfg::kSelOff + Cfg::kSelMaxChunks * 4);
    int *s_sel = reinterpret_cast<int *>(gen + Cfg::kSelOff + Cfg::kSelMaxChunks * 8);
    int sel_b0 = 0;
    if (self_select) {
        const int ipc = (p.n_items + (int)gridDim.x - 1) / (int)gridDim.x;
        item_lo = blockIdx.x * ipc;
        item_hi = min(p.n_items, item_lo + ipc);
        item_step = 1;
        if (item_lo < item_hi) {
            const int per_b = p.topk * p.nslices * p.nhb;
            sel_b0 = item_lo / per_b;
            const int b1 = (item_hi - 1) / per_b;
            for (int b = sel_b0; b <= b1; ++b) {
                const bool owner = (b * per_b >= item_lo);            // holds the sequence's first item
                for (int c = tid; c < p.C; c += blockDim.x) {
                    const float *sp = p.sel_scores + ((int64_t)b * p.C + c) * p.Hkv;
                    float acc = 0.f;
                    for (int g2 = 0; g2 < p.Hkv; ++g2) acc += sp[g2];
                    const float sc = acc / (float)p.Hq;
                    s_score[c] = sc;
                    if (owner && p.scores_out != nullptr) p.scores_out[(int64_t)b * p.C + c] = sc;
                }
                __syncthreads();
                // rank of chunk c = number of chunks that beat it (larger score, or equal score and lower id)
                for (int c = tid; c < p.C; c += blockDim.x) {
                    const float sc = s_score[c];
                    int rank = 0;
#pragma unroll 8
                    for (int c2 = 0; c2 < p.C; ++c2) {
                        const float s2 = s_score[c2];
                        rank += (s2 > sc || (s2 == sc && c2 < c)) ? 1 : 0;
                    }
                    s_flag[c] = rank < p.topk ? 1 : 0;
                }
                __syncthreads();
                for (int c = tid; c < p.C; c += blockDim.x) {
                    const int f = s_flag[c];
                    if (owner && p.flags_out != nullptr) p.flags_out[(int64_t)b * p.C + c] = f;
                    if (f) {
                        int pos = 0;
                        for (int c2 = 0; c2 < c; ++c2) pos += s_flag[c2];
                        if (pos < p.topk) {                          // selected chunks in ascending id order
                            s_sel[(b - sel_b0) * p.topk + pos] = c;
                            if (owner && p.sel_out != nullptr) p.sel_out[(int64_t)b * p.topk + pos] = c;
                            if (owner && p.topk_out != nullptr) p.topk_out[(int64_t)b * p.topk + pos] = c;
                        }
                    }
                }
                __syncthreads();
            }
        }
    }

    // item -> (b, hb, slot, first row in the 2-D view, rows)
    auto decode_item = [&](int item, int &b, int &hb, int &slot, int64_t &row0, int &nrows) {
        hb = item % p.nhb;
        const int it2 = item / p.nhb;
        if (SPARSE) {
            b = it2 / p.C;
            const int c = it2 % p.C;
            slot = c;
            row0 = ((int64_t)b * p.C + c) * p.R;
            nrows = p.R;
            if (p.flags != nullptr && p.flags[(int64_t)b * p.C + c] != 0) nrows = -1;   // read dense elsewhere
        } else {
            const int per_b = p.topk * p.nslices;
            b = it2 / per_b;
            const int js = it2 % per_b;
            const int j = js / p.nslices, s = js % p.nslices;
            slot = p.C + js;
            int chunk = self_select ? s_sel[(b - sel_b0) * p.topk + j] : p.sel[(int64_t)b * p.topk + j];
            int lo = 0, len = 0;
            if (chunk < 0 || chunk >= p.C) {
                if (tid == 0) raise_status(p.hdr, VXL_ERR_INVALID_INDEX, 140);
            } else {
                lo = p.off[chunk];
                len = p.off[chunk + 1] - lo;
                if (lo < 0 || len < 0 || lo + len > p.T) {
                    if (tid == 0) raise_status(p.hdr, VXL_ERR_INVALID_INDEX, 141);
                    lo = 0; len = 0;
                }
                if (len > p.nslices * p.slice_rows) {             // max_chunk_len was not a bound
                    if (tid == 0) raise_status(p.hdr, VXL_ERR_INVALID_ARG, 142);
                    len = p.nslices * p.slice_rows;
                }
            }
            row0 = p.staged > 0 ? ((int64_t)b * p.topk + j) * p.staged + (int64_t)s * p.slice_rows
                                : (int64_t)b * p.T + lo + (int64_t)s * p.slice_rows;
            nrows = min(p.slice_rows, len - s * p.slice_rows);
            if (nrows < 0) nrows = 0;
        }
    };

    if (warp == HPC) {
        // ------------------------------------------------------------------ producer
        int issued = 0;
        bool ok = true;
        // every row is read once per call: evict-first keeps the stream from displacing anything else in L2
        const uint64_t stream_policy = l2_evict_first_policy();
        for (int item = item_lo; item < item_hi && ok; item += item_step) {
            int b, hb, slot, nrows; int64_t row0;
            decode_item(item, b, hb, slot, row0, nrows);
            for (int r = 0; r < nrows; r += TK) {
                const int stage = issued % NS;
                const uint32_t ph = (issued / NS) & 1;
                if (!mbar_wait(empty(stage), ph ^ 1) || *s_abort) { ok = false; break; }
                if (lane == 0) {
                    mbar_expect_tx(full(stage), WITH_V ? Cfg::kStageBytes : Cfg::kTileBytes);
                    const uint32_t dK = base + stage * Cfg::kStageBytes;
                    const int x0 = hb * HPC * D;
                    const int y = (int)(row0 + r);
#pragma unroll
                    for (int pn = 0; pn < Cfg::PANELS; ++pn) {
                        asm volatile(
                            "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;" ::"r"(dK + pn * Cfg::kPanelBytes),
                            "l"(&maps.k), "r"(x0 + pn * 64), "r"(y), "r"(full(stage)), "l"(stream_policy)
                            : "memory");
                        if (WITH_V)
                            asm volatile(
                                "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;" ::"r"(dK + Cfg::kTileBytes + pn * Cfg::kPanelBytes),
                                "l"(&maps.v), "r"(x0 + pn * 64), "r"(y), "r"(full(stage)), "l"(stream_policy)
                                : "memory");
                    }
                }
                ++issued;
            }
        }
        if (!ok && lane == 0) { raise_status(p.hdr, VXL_ERR_TIMEOUT, 143); *s_abort = 1; }
        for (int s = 0; s < NS && s < issued; ++s) {          // let the last copies land before retiring
            const int i2 = issued - 1 - s;
            mbar_wait(full(i2 % NS), (i2 / NS) & 1);
        }
    } else {
        // ------------------------------------------------------------------ consumers
        // one warp per kv head: all TK keys of a tile, so no cross-warp merge is needed
        const int hl = warp;
        const int g = lane >> 2, t = lane & 3;
        int consumed = 0;
        bool ok = true;
        int q_b = -1, q_hb = -1;
        uint32_t qf[D / 16][4];
        for (int item = item_lo; item < item_hi; item += item_step) {
            int b, hb, slot, nrows; int64_t row0;
            decode_item(item, b, hb, slot, row0, nrows);
            if (nrows < 0) continue;                              // sparse slot of a dense chunk: unused
            const int kvh = hb * HPC + hl;
            if (b != q_b || hb != q_hb) {                         // query fragments: rows = heads of the kv group
                q_b = b; q_hb = hb;
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
            float o[D / 8][4];
#pragma unroll
            for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
            float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

            for (int r = 0; r < nrows && ok; r += TK) {
                const int nvalid = min(TK, nrows - r);
                const int stage = consumed % NS;
                const uint32_t ph = (consumed / NS) & 1;
                if (!mbar_wait(full(stage), ph) || *s_abort) { ok = false; break; }
                ++consumed;
                const uint32_t tK = base + stage * Cfg::kStageBytes + hl * (D / 64) * Cfg::kPanelBytes;
                const uint32_t tV = tK + Cfg::kTileBytes;
                float s[TK / 8][4];
#pragma unroll
                for (int i = 0; i < TK / 8; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
                for (int kb = 0; kb < D / 16; ++kb) {
#pragma unroll
                    for (int kg = 0; kg < TK / 16; ++kg) {
                        const int mi = lane >> 3, ri = lane & 7;
                        const int key = kg * 16 + (mi >> 1) * 8 + ri;
                        const int col = kb * 16 + (mi & 1) * 8;                       // element within the head
                        const uint32_t addr = tK + (col >> 6) * Cfg::kPanelBytes + key * 128 +
                                              ((((col & 63) >> 3) ^ (key & 7)) << 4);
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
                        const float x = (key < nvalid) ? s[nb][j] * p.scale_log2 : -INFINITY;
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
                            const uint32_t addr = tV + (col >> 6) * Cfg::kPanelBytes + key * 128 +
                                                  ((((col & 63) >> 3) ^ (key & 7)) << 4);
                            uint32_t b0, b1, b2, b3;
                            ldsm_x4_t(addr, b0, b1, b2, b3);
                            if (nvalid < TK) {
                                // Rows past the item's end are whatever follows in memory (the next chunk, unwritten
                                // cache capacity, a staging slot's leftovers): their probabilities are 0, and 0 x NaN
                                // must not reach O, so those V rows are read as zeros.  b0/b2 hold keys kg*16 + 2t, +1
                                // and b1/b3 keys kg*16 + 8 + 2t, +1 (low half first).
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
                __syncwarp();
                if (lane == 0) mbar_arrive(empty(stage));
            }
            if (!ok) break;
            l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
            l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
            l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
            l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int r2 = g + 8 * half;
                if (r2 >= p.G) continue;
                const int h = kvh * p.G + r2;
                const int64_t pi = ((int64_t)b * p.Hq + h) * p.P + slot;
                if (WITH_V) {
#pragma unroll
                    for (int nd = 0; nd < D / 8; ++nd)
                        *reinterpret_cast<float2 *>(p.part_o + pi * D + nd * 8 + 2 * t) =
                            make_float2(o[nd][2 * half], o[nd][2 * half + 1]);
                }
                if (t == 0) {
                    p.part_m[pi] = half ? m_hi : m_lo;
                    p.part_l[pi] = half ? l_hi : l_lo;
                }
            }
            if (SPARSE && p.score_part != nullptr) {
                // rows g (< G) and g + 8 (< G) of the quad's first lane hold the heads of this kv head
                float acc = 0.f;
                if (t == 0) {
                    if (g < p.G) acc += (m_lo + log2f(l_lo)) * kLn2;
                    if (g + 8 < p.G) acc += (m_hi + log2f(l_hi)) * kLn2;
                }
#pragma unroll
                for (int o2 = 16; o2 > 0; o2 >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o2);
                if (lane == 0) p.score_part[((int64_t)b * p.C + slot) * p.Hkv + kvh] = acc;
            }
        }
        if (!ok && lane == 0) { raise_status(p.hdr, VXL_ERR_TIMEOUT, 144); *s_abort = 1; }
    }
}

// ---------------------------------------------------------------------------------------
// Chunk relevance + top-k, parallel version: one warp per chunk gathers the per-head
// log-sum-exps (lanes = heads), then the ranking runs out of shared memory.
__global__ void __launch_bounds__(1024) topk_fast_kernel(const TopkParams p)
{
    extern __shared__ float s_score[];
    __shared__ int s_wcount[32];
    __shared__ int s_base;
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = blockDim.x >> 5;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // 8 threads per chunk, heads strided over them: every (m, l) load is independent
    for (int c0 = 0; c0 < p.C; c0 += (int)blockDim.x / 8) {
        const int c = c0 + tid / 8, sub = tid & 7;
        float acc = 0.f;
        if (c < p.C && p.score_part != nullptr) {
            // the sparse pass left one sum per kv head
            for (int g2 = sub; g2 < p.Hkv; g2 += 8) acc += p.score_part[((int64_t)b * p.C + c) * p.Hkv + g2];
        } else if (c < p.C) {
#pragma unroll 4
            for (int h = sub; h < p.Hq; h += 8) {
                const int64_t pi = ((int64_t)b * p.Hq + h) * p.P + c;
                acc += (p.part_m[pi] + log2f(p.part_l[pi])) * kLn2;
            }
        }
        acc += __shfl_xor_sync(0xffffffffu, acc, 1);
        acc += __shfl_xor_sync(0xffffffffu, acc, 2);
        acc += __shfl_xor_sync(0xffffffffu, acc, 4);
        if (c < p.C && sub == 0) {
            const float sc = acc / (float)p.Hq;
            s_score[c] = sc;
            if (p.scores_out != nullptr) p.scores_out[(int64_t)b * p.C + c] = sc;
        }
    }
    if (tid == 0) s_base = 0;
    __syncthreads();
    // rank of chunk c = number of chunks that beat it (larger score, or equal score and lower id)
    for (int c0 = 0; c0 < p.C; c0 += blockDim.x) {
        const int c = c0 + tid;
        int f = 0;
        if (c < p.C) {
            const float sc = s_score[c];
            int rank = 0;
#pragma unroll 8
            for (int c2 = 0; c2 < p.C; ++c2) {
                const float s2 = s_score[c2];
                rank += (s2 > sc || (s2 == sc && c2 < c)) ? 1 : 0;
            }
            f = rank < p.topk ? 1 : 0;
            p.flags[(int64_t)b * p.C + c] = f;
        }
        // ascending output position = number of selected chunks with a lower id
        const unsigned bal = __ballot_sync(0xffffffffu, f != 0);
        if (lane == 0) s_wcount[warp] = __popc(bal);
        __syncthreads();
        int pre = s_base;
        for (int w = 0; w < warp; ++w) pre += s_wcount[w];
        const int pos = pre + __popc(bal & ((1u << lane) - 1u));
        if (f && pos < p.topk) {
            if (p.sel_ws != nullptr) p.sel_ws[(int64_t)b * p.topk + pos] = c;
            if (p.topk_out != nullptr) p.topk_out[(int64_t)b * p.topk + pos] = c;
        }
        __syncthreads();
        if (tid == 0) { int tot = 0; for (int w = 0; w < nw; ++w) tot += s_wcount[w]; s_base += tot; }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------
// Combine, parallel version: 1024 threads = 32 slot groups x (D/4) float4 lanes (D = 128: 32).
// Each thread folds its slots with a running max (independent, unrolled loads), then the
// groups are merged through shared memory.  Sparse slots of chunks read dense are skipped.
template <int D>
__global__ void __launch_bounds__(1024) combine_fast_kernel(const CombineParams p)
{
    constexpr int DL = D / 4;
    constexpr int SG = 1024 / DL;
    __shared__ float s_m[SG], s_l[SG];
    __shared__ float4 s_o[SG][DL];
    const int h = blockIdx.x, b = blockIdx.y;
    const int tid = threadIdx.x, dl = tid % DL, sg = tid / DL;
    const int64_t base = ((int64_t)b * p.Hq + h) * p.P;
    const int32_t *fl = p.flags + (int64_t)b * p.C;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    float M = -INFINITY, Lsum = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
    for (int s = sg; s < p.P; s += SG) {
        const bool valid = !(s < p.C && fl[s] != 0);
        const float m = p.part_m[base + s];
        const float l = p.part_l[base + s];
        const float4 v = *reinterpret_cast<const float4 *>(p.part_o + (base + s) * D + dl * 4);
        if (valid && l > 0.f) {
            const float Mn = fmaxf(M, m);
            const float fo = fast_exp2(M - Mn), fn = fast_exp2(m - Mn);
            Lsum = Lsum * fo + l * fn;
            acc.x = acc.x * fo + v.x * fn; acc.y = acc.y * fo + v.y * fn;
            acc.z = acc.z * fo + v.z * fn; acc.w = acc.w * fo + v.w * fn;
            M = Mn;
        }
    }
    if (dl == 0) { s_m[sg] = M; s_l[sg] = Lsum; }
    s_o[sg][dl] = acc;
    __syncthreads();
    if (sg == 0) {
        float Mt = -INFINITY;
#pragma unroll
        for (int i = 0; i < SG; ++i) Mt = fmaxf(Mt, s_m[i]);
        float Lt = 0.f;
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
        for (int i = 0; i < SG; ++i) {
            const float f = (s_m[i] == -INFINITY) ? 0.f : fast_exp2(s_m[i] - Mt);
            Lt += s_l[i] * f;
            const float4 v = s_o[i][dl];
            a.x += v.x * f; a.y += v.y * f; a.z += v.z * f; a.w += v.w * f;
        }
        const float inv = Lt > 0.f ? 1.f / Lt : 0.f;
        const int64_t ob = (int64_t)b * p.o_sb + (int64_t)h * p.o_sh + dl * 4;
        if (p.out_bf16) {
            uint2 pk;
            pk.x = pack_bf16(a.x * inv, a.y * inv);
            pk.y = pack_bf16(a.z * inv, a.w * inv);
            *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(p.out) + ob) = pk;
        } else {
            *reinterpret_cast<float4 *>(reinterpret_cast<float *>(p.out) + ob) =
                make_float4(a.x * inv, a.y * inv, a.z * inv, a.w * inv);
        }
        if (p.lse != nullptr && dl == 0)
            p.lse[(int64_t)b * p.Hq + h] = Lt > 0.f ? (Mt + log2f(Lt)) * kLn2 : -INFINITY;
    }
}


// ---------------------------------------------------------------------------------------
// Combine without a serial dependency between slots (used while the slot weights fit in shared
// memory): pass A, one thread per slot, finds the largest partial maximum among the live slots and
// turns every slot into a weight 2^(m - max) (0 for empty slots and for sparse slots of chunks
// that were read dense); pass B sums weight * partial output with all loads of a thread in flight.
constexpr int kCombineMaxSlots = 8000;     // weights (4 B each) + 16.5 KB of static shared memory stay under 48 KB

template <int D>
__global__ void __launch_bounds__(1024) combine_two_pass_kernel(const CombineParams p)
{
    constexpr int DL = D / 4;
    constexpr int SG = 1024 / DL;
    extern __shared__ float s_w[];                       // P weights
    __shared__ float s_red[32];
    __shared__ float4 s_o[SG][DL];
    const int h = blockIdx.x, b = blockIdx.y;
    const int tid = threadIdx.x, dl = tid % DL, sg = tid / DL;
    const int64_t base = ((int64_t)b * p.Hq + h) * p.P;
    const int32_t *fl = p.flags + (int64_t)b * p.C;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // The first eight partial rows of this thread are requested before anything is known about their
    // weights (one memory round trip fewer; a slot nobody wrote may hold anything and gets weight 0).
    float4 v0[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const int s2 = sg + u * SG;
        v0[u] = (s2 < p.P) ? *reinterpret_cast<const float4 *>(p.part_o + (base + s2) * D + dl * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    float M = -INFINITY;
    float l_first = 0.f;                                  // part_l of this thread's first slot (the only one when P <= 1024)
    for (int s2 = tid; s2 < p.P; s2 += 1024) {
        const float l = p.part_l[base + s2];
        const float m = p.part_m[base + s2];
        if (s2 == tid) l_first = l;
        const bool valid = !(s2 < p.C && fl[s2] != 0) && l > 0.f;
        s_w[s2] = valid ? m : -INFINITY;
        M = valid ? fmaxf(M, m) : M;
    }
#pragma unroll
    for (int o2 = 16; o2 > 0; o2 >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o2));
    if ((tid & 31) == 0) s_red[tid >> 5] = M;
    __syncthreads();
    float Mt = -INFINITY;
#pragma unroll
    for (int i = 0; i < 32; ++i) Mt = fmaxf(Mt, s_red[i]);
    __syncthreads();
    float Lsum = 0.f;
    for (int s2 = tid; s2 < p.P; s2 += 1024) {
        const float m = s_w[s2];
        const float wgt = (m == -INFINITY) ? 0.f : fast_exp2(m - Mt);
        s_w[s2] = wgt;
        if (wgt != 0.f) Lsum += wgt * (s2 == tid ? l_first : p.part_l[base + s2]);
    }
#pragma unroll
    for (int o2 = 16; o2 > 0; o2 >>= 1) Lsum += __shfl_xor_sync(0xffffffffu, Lsum, o2);
    if ((tid & 31) == 0) s_red[tid >> 5] = Lsum;
    __syncthreads();
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const int s2 = sg + u * SG;
        const float wgt = (s2 < p.P) ? s_w[s2] : 0.f;
        if (wgt != 0.f) { acc.x += v0[u].x * wgt; acc.y += v0[u].y * wgt; acc.z += v0[u].z * wgt; acc.w += v0[u].w * wgt; }
    }
    for (int s0 = sg + 8 * SG; s0 < p.P; s0 += 8 * SG) {
        float4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int s2 = s0 + u * SG;
            v[u] = (s2 < p.P && s_w[s2] != 0.f) ? *reinterpret_cast<const float4 *>(p.part_o + (base + s2) * D + dl * 4)
                                                : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int s2 = s0 + u * SG;
            const float wgt = (s2 < p.P) ? s_w[s2] : 0.f;
            acc.x += v[u].x * wgt; acc.y += v[u].y * wgt; acc.z += v[u].z * wgt; acc.w += v[u].w * wgt;
        }
    }
    s_o[sg][dl] = acc;
    __syncthreads();
    if (sg == 0) {
        float Lt = 0.f;
#pragma unroll
        for (int i = 0; i < 32; ++i) Lt += s_red[i];
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int i = 0; i < SG; ++i) {
            const float4 v = s_o[i][dl];
            a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
        }
        const float inv = Lt > 0.f ? 1.f / Lt : 0.f;
        const int64_t ob = (int64_t)b * p.o_sb + (int64_t)h * p.o_sh + dl * 4;
        if (p.out_bf16) {
            uint2 pk;
            pk.x = pack_bf16(a.x * inv, a.y * inv);
            pk.y = pack_bf16(a.z * inv, a.w * inv);
            *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(p.out) + ob) = pk;
        } else {
            *reinterpret_cast<float4 *>(reinterpret_cast<float *>(p.out) + ob) =
                make_float4(a.x * inv, a.y * inv, a.z * inv, a.w * inv);
        }
        if (p.lse != nullptr && dl == 0)
            p.lse[(int64_t)b * p.Hq + h] = Lt > 0.f ? (Mt + log2f(Lt)) * kLn2 : -INFINITY;
    }
}

}  // namespace vxl
