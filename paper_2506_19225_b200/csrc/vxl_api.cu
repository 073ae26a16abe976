// C ABI of the vxl library: argument validation, workspace carving and kernel launches.
// Every step of the path runs in the CUDA kernels of this directory; there is no CPU path.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "../../include/vxl.h"
#include "common.cuh"
#include "decode.cuh"
#include "prefill_general.cuh"
#include "prefill_tc.cuh"
#include "decode_stream.cuh"

namespace {

using namespace vxl;

constexpr int kMaxDevices = 64;
constexpr int kSliceRows = 128;      // dense rows per split-KV CTA
constexpr int kMaxSlices = 64;       // per selected chunk; longer chunks loop inside the CTA
constexpr int kMaxChunks = 4096;     // top-k ranks chunks in shared memory with O(C^2) compares

inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }
inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool shape_ok(const vxl_shape *s)
{
    if (s == nullptr || s->struct_size != sizeof(vxl_shape)) return false;
    if (s->B <= 0 || s->T <= 0 || s->Hq <= 0 || s->Hkv <= 0 || s->D <= 0) return false;
    if (s->Hq % s->Hkv != 0 || s->Hq / s->Hkv > 16) return false;
    if (s->out_dtype != VXL_BF16 && s->out_dtype != VXL_F32) return false;
    if (s->score_mode != VXL_SCORE_LSE && s->score_mode != VXL_SCORE_MASS) return false;
    return true;
}

bool strides_ok(const vxl_shape *s, bool prefill)
{
    auto m8 = [](int64_t x) { return x >= 0 && (x % 8) == 0; };
    if (!m8(s->q_stride_b) || !m8(s->q_stride_h) || !m8(s->kv_stride_b) || !m8(s->kv_stride_t) ||
        !m8(s->kv_stride_h))
        return false;
    if (prefill && !m8(s->q_stride_t)) return false;
    if (s->q_stride_h < s->D || s->kv_stride_h < s->D && s->Hkv > 1) return false;
    if (s->kv_stride_t < s->D) return false;
    if (s->out_stride_b < 0 || s->out_stride_t < 0 || s->out_stride_h < 0) return false;
    if ((s->out_stride_b % 4) || (s->out_stride_t % 4) || (s->out_stride_h % 4)) return false;
    return true;
}

int heads_per_cta(int Hkv) { return (Hkv % 4 == 0) ? 4 : (Hkv % 2 == 0) ? 2 : 1; }

// Dense split: rows per slice (a multiple of 128, at least kSliceRows) and slices per chunk (they
// cover max_chunk_len).  The persistent dense pass deals its items (sequence, selected chunk, slice)
// round-robin to one CTA per SM, so its length is (items per CTA, rounded up) x (rows per item + a
// fixed cost per item for the query fragments and the partial it writes); the plan takes the slice
// length that makes this smallest, the longer slice on a tie (fewer partials for the combine).
struct SlicePlan { int slice_rows, nslices; };
SlicePlan plan_slices(int B, int topk, int max_chunk_len, int Hkv)
{
    constexpr int64_t kCtas = 148, kItemCostRows = 24;
    const int64_t units = (int64_t)B * (topk > 0 ? topk : 1) * (Hkv / heads_per_cta(Hkv));   // x kv head blocks
    const int64_t cap = ((int64_t)max_chunk_len + 127) / 128 * 128;
    int64_t best_rows = cap, best_cost = -1;
    for (int64_t rows = kSliceRows; rows <= cap; rows += 128) {
        const int64_t n = (max_chunk_len + rows - 1) / rows;
        if (n > kMaxSlices) continue;
        const int64_t waves = (units * n + kCtas - 1) / kCtas;
        const int64_t cost = waves * (rows + kItemCostRows);
        if (best_cost < 0 || cost <= best_cost) { best_cost = cost; best_rows = rows; }
    }
    int n = (int)((max_chunk_len + best_rows - 1) / best_rows);
    if (n < 1) n = 1;
    if (n > kMaxSlices) { n = kMaxSlices; best_rows = (((int64_t)max_chunk_len + n - 1) / n + 127) / 128 * 128; }
    return SlicePlan{(int)best_rows, n};
}


struct DecodeWs {
    WsHeader *hdr;
    float *part_m, *part_l, *part_o, *score_part;
    int32_t *sel, *flags;
    size_t bytes;
};

DecodeWs carve_decode(void *ws, const vxl_shape *s, int C, int topk, int nslices, bool with_o)
{
    DecodeWs w{};
    const size_t P = (size_t)C + (size_t)topk * nslices;
    const size_t nml = (size_t)s->B * s->Hq * P;
    size_t off = sizeof(WsHeader);
    char *base = static_cast<char *>(ws);
    w.hdr = reinterpret_cast<WsHeader *>(base);
    w.part_m = reinterpret_cast<float *>(base + off); off += align256(nml * sizeof(float));
    w.part_l = reinterpret_cast<float *>(base + off); off += align256(nml * sizeof(float));
    w.sel = reinterpret_cast<int32_t *>(base + off); off += align256((size_t)s->B * (topk > 0 ? topk : 1) * sizeof(int32_t));
    w.flags = reinterpret_cast<int32_t *>(base + off); off += align256((size_t)s->B * C * sizeof(int32_t));
    w.score_part = reinterpret_cast<float *>(base + off); off += align256((size_t)s->B * C * s->Hkv * sizeof(float));
    w.part_o = reinterpret_cast<float *>(base + off);
    if (with_o) off += align256(nml * s->D * sizeof(float));
    w.bytes = off;
    return w;
}

template <typename K>
cudaError_t ensure_smem(K kernel, size_t bytes, bool *done_flags)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (done_flags[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess) done_flags[dev] = true;
    return e;
}

template <int D, int HPC, bool SPARSE, bool WITH_V>
cudaError_t launch_partial(const DecodeParams &p, dim3 grid, cudaStream_t st)
{
    static bool done[kMaxDevices] = {};
    auto kern = decode_partial_kernel<D, HPC, SPARSE, WITH_V>;
    cudaError_t e = ensure_smem(kern, DecCfg<D, HPC>::kSmemBytes, done);
    if (e != cudaSuccess) return e;
    kern<<<grid, 32 * (kDecWarps + 1), DecCfg<D, HPC>::kSmemBytes, st>>>(p);
    return cudaGetLastError();
}

template <bool SPARSE, bool WITH_V>
cudaError_t dispatch_partial(int D, int HPC, const DecodeParams &p, dim3 grid, cudaStream_t st)
{
    if (D == 128) {
        if (HPC == 4) return launch_partial<128, 4, SPARSE, WITH_V>(p, grid, st);
        if (HPC == 2) return launch_partial<128, 2, SPARSE, WITH_V>(p, grid, st);
        return launch_partial<128, 1, SPARSE, WITH_V>(p, grid, st);
    }
    if (HPC == 4) return launch_partial<64, 4, SPARSE, WITH_V>(p, grid, st);
    if (HPC == 2) return launch_partial<64, 2, SPARSE, WITH_V>(p, grid, st);
    return launch_partial<64, 1, SPARSE, WITH_V>(p, grid, st);
}

// Launch with programmatic stream serialization: the kernel may start while the previous
// kernel of the stream drains; it orders itself with griddepcontrol.wait before reading.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, args...);
}

template <int D, int HPC, bool SPARSE, bool WITH_V>
cudaError_t launch_stream(const StreamMaps &maps, const StreamParams &sp, cudaStream_t st)
{
    static bool done[kMaxDevices] = {};
    auto kern = decode_stream_kernel<D, HPC, SPARSE, WITH_V>;
    cudaError_t e = ensure_smem(kern, StreamCfg<D, HPC>::kSmemBytes, done);
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    static int sm_count[kMaxDevices] = {};
    if (sm_count[dev] == 0) cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev);
    if (sm_count[dev] > 0) sms = sm_count[dev];
    const int grid = sp.n_items < sms ? sp.n_items : sms;
    if (grid <= 0) return cudaSuccess;
    return launch_pdl(kern, dim3(grid), dim3(StreamCfg<D, HPC>::kThreads), StreamCfg<D, HPC>::kSmemBytes, st, maps, sp);
}

template <bool SPARSE, bool WITH_V>
cudaError_t dispatch_stream(int D, int HPC, const StreamMaps &maps, const StreamParams &sp, cudaStream_t st)
{
    if (D == 128) {
        if (HPC == 4) return launch_stream<128, 4, SPARSE, WITH_V>(maps, sp, st);
        if (HPC == 2) return launch_stream<128, 2, SPARSE, WITH_V>(maps, sp, st);
        return launch_stream<128, 1, SPARSE, WITH_V>(maps, sp, st);
    }
    if (HPC == 4) return launch_stream<64, 4, SPARSE, WITH_V>(maps, sp, st);
    if (HPC == 2) return launch_stream<64, 2, SPARSE, WITH_V>(maps, sp, st);
    return launch_stream<64, 1, SPARSE, WITH_V>(maps, sp, st);
}

int stream_tile_rows(int) { return 32; }

// The TMA stream needs the rows of a sequence to be rows of one 2-D array [B*T, Hkv*D].
bool stream_layout_ok(const vxl_shape *s)
{
    if (s->kv_stride_h != s->D) return false;
    if (s->B > 1 && s->kv_stride_b != (int64_t)s->T * s->kv_stride_t) return false;
    return (int64_t)s->B * s->T < (1ll << 31);
}

void fill_stream_params(StreamParams &sp, const DecodeParams &p, int HPC, bool sparse)
{
    std::memset(&sp, 0, sizeof sp);
    sp.q = p.q; sp.off = p.off; sp.sel = p.sel; sp.flags = p.flags;
    sp.part_m = p.part_m; sp.part_l = p.part_l; sp.part_o = p.part_o; sp.hdr = p.hdr;
    sp.score_part = sparse ? p.score_part : nullptr;
    sp.q_sb = p.q_sb; sp.q_sh = p.q_sh;
    sp.B = p.B; sp.T = p.T; sp.Hq = p.Hq; sp.Hkv = p.Hkv; sp.G = p.G; sp.C = p.C; sp.R = p.R; sp.topk = p.topk;
    sp.nslices = p.nslices; sp.slice_rows = p.slice_rows; sp.P = p.P; sp.staged = p.staged;
    sp.nhb = p.Hkv / HPC;
    sp.n_items = sparse ? p.B * p.C * sp.nhb : p.B * p.topk * p.nslices * sp.nhb;
    sp.scale_log2 = p.scale_log2;
    if (!sparse) {
        sp.sel_scores = p.sel_scores; sp.sel_out = p.sel_out; sp.flags_out = p.flags_out;
        sp.topk_out = p.topk_out; sp.scores_out = p.scores_out;
    }
}


// The sparse pass streams the packed level (and leaves per-kv-head score sums) exactly when this holds.
bool sparse_pass_streams(const vxl_shape *s, const DecodeParams &p)
{
    return p.R > 0 && p.ks != nullptr && (int64_t)s->B * p.C * p.R < (1ll << 31);
}

// Sparse pass: packed level -> TMA stream, otherwise rows fetched by index.
template <bool WITH_V>
cudaError_t run_sparse_pass(const vxl_shape *s, const DecodeParams &p, int HPC, cudaStream_t st)
{
    if (p.R <= 0) {
        // nothing to read: the general kernel writes the empty partials
        return dispatch_partial<true, WITH_V>(s->D, HPC, p, dim3((unsigned)p.C, (unsigned)(s->Hkv / HPC), (unsigned)s->B), st);
    }
    if (p.ks != nullptr && (int64_t)s->B * p.C * p.R < (1ll << 31)) {
        StreamMaps maps;
        const uint64_t rows = (uint64_t)s->B * p.C * p.R, width = (uint64_t)s->Hkv * s->D;
        if (!tc_make_map(&maps.k, p.ks, width, rows, width, (uint32_t)stream_tile_rows(HPC))) return cudaErrorUnknown;
        if (WITH_V) { if (!tc_make_map(&maps.v, p.vs, width, rows, width, (uint32_t)stream_tile_rows(HPC))) return cudaErrorUnknown; }
        else maps.v = maps.k;
        StreamParams sp;
        fill_stream_params(sp, p, HPC, true);
        return dispatch_stream<true, WITH_V>(s->D, HPC, maps, sp, st);
    }
    if (p.ridx == nullptr) return cudaErrorInvalidValue;        // rows by index need the indices
    return dispatch_partial<true, WITH_V>(s->D, HPC, p, dim3((unsigned)p.C, (unsigned)(s->Hkv / HPC), (unsigned)s->B), st);
}

cudaError_t run_dense_pass(const vxl_shape *s, const DecodeParams &p, int HPC, cudaStream_t st)
{
    if (p.staged > 0 || stream_layout_ok(s)) {
        StreamMaps maps;
        // dense rows come from the cache, or from the contiguous staging buffer of the selected chunks
        const uint64_t width = (uint64_t)s->Hkv * s->D;
        const uint64_t rows = p.staged > 0 ? (uint64_t)s->B * p.topk * p.staged : (uint64_t)s->B * s->T;
        const uint64_t pitch = p.staged > 0 ? width : (uint64_t)s->kv_stride_t;
        if (!tc_make_map(&maps.k, p.k, width, rows, pitch, (uint32_t)stream_tile_rows(HPC)) ||
            !tc_make_map(&maps.v, p.v, width, rows, pitch, (uint32_t)stream_tile_rows(HPC)))
            return cudaErrorUnknown;
        StreamParams sp;
        fill_stream_params(sp, p, HPC, false);
        return dispatch_stream<false, true>(s->D, HPC, maps, sp, st);
    }
    return dispatch_partial<false, true>(s->D, HPC, p,
                                         dim3((unsigned)(p.topk * p.nslices), (unsigned)(s->Hkv / HPC), (unsigned)s->B), st);
}

float resolve_scale(const vxl_shape *s) { return s->scale > 0.f ? s->scale : 1.0f / std::sqrt((float)s->D); }

void fill_decode_params(DecodeParams &p, const vxl_shape *s, const void *q, const void *k, const void *v,
                        const int32_t *off, int C, const int32_t *ridx, int R, int64_t ridx_sb,
                        const vxl_sparse_level *sp, int topk, int nslices, int slice_rows, const DecodeWs &w)
{
    std::memset(&p, 0, sizeof p);
    p.q = static_cast<const __nv_bfloat16 *>(q);
    p.k = static_cast<const __nv_bfloat16 *>(k);
    p.v = static_cast<const __nv_bfloat16 *>(v);
    p.ks = sp ? static_cast<const __nv_bfloat16 *>(sp->k_sparse) : nullptr;
    p.vs = sp ? static_cast<const __nv_bfloat16 *>(sp->v_sparse) : nullptr;
    p.off = off; p.ridx = ridx; p.ridx_sb = ridx_sb;
    p.sel = w.sel; p.flags = nullptr;
    p.part_m = w.part_m; p.part_l = w.part_l; p.part_o = w.part_o; p.hdr = w.hdr;
    p.score_part = w.score_part;
    p.q_sb = s->q_stride_b; p.q_sh = s->q_stride_h;
    p.kv_sb = s->kv_stride_b; p.kv_st = s->kv_stride_t; p.kv_sh = s->kv_stride_h;
    p.B = s->B; p.T = s->T; p.Hq = s->Hq; p.Hkv = s->Hkv; p.G = s->Hq / s->Hkv;
    p.C = C; p.R = R; p.topk = topk; p.nslices = nslices; p.slice_rows = slice_rows;
    p.P = C + topk * nslices;
    p.scale_log2 = resolve_scale(s) * kLog2e;
}

vxl_status check_decode_common(const vxl_shape *s, const void *q, const void *k, const int32_t *off, int C,
                               const int32_t *ridx, int R, int64_t ridx_sb, const vxl_sparse_level *sp,
                               bool need_v)
{
    if (!shape_ok(s) || q == nullptr || k == nullptr || off == nullptr) return VXL_ERR_INVALID_ARG;
    if (C <= 0 || R < 0 || C > s->T) return VXL_ERR_INVALID_ARG;
    if (R > 0 && ridx == nullptr && sp == nullptr) return VXL_ERR_INVALID_ARG;   // a stored sparse level needs no indices
    if (ridx_sb != 0 && ridx_sb < (int64_t)C * R) return VXL_ERR_INVALID_ARG;
    if (s->D != 64 && s->D != 128) return VXL_ERR_UNSUPPORTED;
    if (!strides_ok(s, false) || !aligned16(q) || !aligned16(k)) return VXL_ERR_INVALID_ARG;
    if (sp != nullptr) {
        if (sp->k_sparse == nullptr || !aligned16(sp->k_sparse)) return VXL_ERR_INVALID_ARG;
        if (need_v && (sp->v_sparse == nullptr || !aligned16(sp->v_sparse))) return VXL_ERR_INVALID_ARG;
    }
    return VXL_OK;
}

// Host-side argument checks of vxl_chunk_scores (everything but the workspace).
vxl_status check_scores_args(const vxl_shape *s, const void *q, const void *k, const int32_t *off, int C,
                             const int32_t *ridx, int R, int64_t ridx_sb, const vxl_sparse_level *sp,
                             const float *scores, int topk)
{
    const vxl_status vs = check_decode_common(s, q, k, off, C, ridx, R, ridx_sb, sp, false);
    if (vs != VXL_OK) return vs;
    if (scores == nullptr || topk < 0 || topk > C) return VXL_ERR_INVALID_ARG;
    if (C > kMaxChunks) return VXL_ERR_UNSUPPORTED;
    if (R > 0 && ridx == nullptr && (sp == nullptr || (int64_t)s->B * C * R >= (1ll << 31))) return VXL_ERR_INVALID_ARG;
    return VXL_OK;
}

cudaError_t launch_validate(const int32_t *ridx, const int32_t *off, WsHeader *hdr, int64_t ridx_sb, int nb,
                            int C, int R, int L, int T, cudaStream_t st, int base = 0)
{
    if (R <= 0 && off == nullptr) return cudaSuccess;
    ValidateParams vp{ridx, off, hdr, ridx_sb, C, R, L, T, base};
    validate_idx_kernel<<<dim3(C, nb), 128, 0, st>>>(vp);
    return cudaGetLastError();
}

// Scratch of vxl_chunk_scores_static: lives in the library image, so every GPU that loads the
// library carries these bytes until the process exits.  Host code may only use the name to ask
// the runtime for the device address; it is not itself a device pointer.
constexpr size_t kStaticScratchBytes = VXL_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
void *g_static_scratch_ptr[kMaxDevices] = {};
std::mutex g_static_scratch_mu;

// Device address of the static scratch on the current device (looked up once per device).
void *static_scratch_address()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_static_scratch_mu);
    if (g_static_scratch_ptr[dev] == nullptr) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
            (void)cudaGetLastError();
            return nullptr;
        }
        g_static_scratch_ptr[dev] = ptr;
    }
    return g_static_scratch_ptr[dev];
}

// The dense pass can rank the chunks itself when it runs as the TMA stream after a streamed sparse
// pass (per-kv-head score sums exist), the ranking is small enough to repeat in every CTA and the
// selections of the sequences one CTA touches fit its scratch.
bool dense_pass_can_select(const vxl_shape *s, const DecodeParams &p, int C, int topk)
{
    if (s->score_mode != VXL_SCORE_LSE || topk <= 0 || C > 256) return false;
    if (!sparse_pass_streams(s, p) || !(p.staged > 0 || stream_layout_ok(s))) return false;
    return (int64_t)s->B * topk <= 1024;                     // selections of all sequences fit one CTA's scratch
}

// The passes of one decode call on stream st: (flags from a given selection,) sparse pass, (top-k,)
// dense pass, combine.  dense_ready: event the dense pass waits for (staged dense rows), or null.
vxl_status run_decode_passes(const vxl_shape *s, DecodeParams &p, const DecodeWs &w, int C, int R, int topk,
                             const int32_t *selected, void *out, float *lse, float *scores_out, int32_t *topk_out,
                             int HPC, cudaStream_t st, cudaEvent_t dense_ready)
{
    TopkParams tp{w.part_m, w.part_l, selected, scores_out, topk_out, w.sel, w.flags, w.hdr, s->B, s->Hq, C, p.P, topk,
                  sparse_pass_streams(s, p) ? w.score_part : nullptr, s->Hkv};
    if (selected != nullptr) {
        // externally chosen chunks: flags first, so the sparse pass can skip the dense chunks
        topk_kernel<<<s->B, 256, (size_t)C * 8, st>>>(tp);
        if (cudaGetLastError() != cudaSuccess) return VXL_ERR_CUDA;
        p.flags = w.flags;
    }
    if (R > 0 || selected == nullptr) {
        if (run_sparse_pass<true>(s, p, HPC, st) != cudaSuccess) return VXL_ERR_CUDA;
    }
    // With no selection given, the dense stream pass ranks the chunks itself where it can: one launch fewer.
    const bool self_select = selected == nullptr && dense_pass_can_select(s, p, C, topk);
    if (self_select) {
        p.sel_scores = w.score_part; p.sel_out = w.sel; p.flags_out = w.flags;
        p.topk_out = topk_out; p.scores_out = scores_out;
    }
    if (selected == nullptr && !self_select) {
        if (s->score_mode == VXL_SCORE_MASS) {
            topk_mass_kernel<<<s->B, 1024, (size_t)C * 8, st>>>(tp);
            if (cudaGetLastError() != cudaSuccess) return VXL_ERR_CUDA;
        } else if (launch_pdl(topk_fast_kernel, dim3(s->B), dim3(1024), (size_t)C * 8, st, tp) != cudaSuccess) {
            return VXL_ERR_CUDA;
        }
    }
    if (topk > 0) {
        p.flags = nullptr;
        if (dense_ready != nullptr && cudaStreamWaitEvent(st, dense_ready, 0) != cudaSuccess) return VXL_ERR_CUDA;
        if (run_dense_pass(s, p, HPC, st) != cudaSuccess) return VXL_ERR_CUDA;
    }
    CombineParams cp;
    std::memset(&cp, 0, sizeof cp);
    cp.part_m = w.part_m; cp.part_l = w.part_l; cp.part_o = w.part_o; cp.flags = w.flags;
    cp.out = out; cp.lse = lse;
    cp.o_sh = s->out_stride_h ? s->out_stride_h : s->D;
    cp.o_sb = s->out_stride_b ? s->out_stride_b : (int64_t)s->Hq * cp.o_sh;
    cp.B = s->B; cp.Hq = s->Hq; cp.C = C; cp.P = p.P; cp.D = s->D;
    cp.out_bf16 = (s->out_dtype == VXL_BF16);
    cudaError_t ce;
    if (p.P <= kCombineMaxSlots) {
        const size_t sm = (size_t)p.P * sizeof(float);
        ce = (s->D == 128) ? launch_pdl(combine_two_pass_kernel<128>, dim3(s->Hq, s->B), dim3(1024), sm, st, cp)
                           : launch_pdl(combine_two_pass_kernel<64>, dim3(s->Hq, s->B), dim3(1024), sm, st, cp);
    } else {
        ce = (s->D == 128) ? launch_pdl(combine_fast_kernel<128>, dim3(s->Hq, s->B), dim3(1024), 0, st, cp)
                           : launch_pdl(combine_fast_kernel<64>, dim3(s->Hq, s->B), dim3(1024), 0, st, cp);
    }
    return ce == cudaSuccess ? VXL_OK : VXL_ERR_CUDA;
}

// General kernel over the step blocks and the prefix (or the prefix alone).
vxl_status launch_prefill_general(const PrefillParams &p, const vxl_shape *s, cudaStream_t st, bool prefix_rows = true)
{
    // blockIdx.x beyond the step tiles addresses the prefix tiles: leave them out when another call owns the prefix
    const int64_t tiles = (p.prefix_only ? 0 : (int64_t)((p.S + kGenBM - 1) / kGenBM) * p.Cn) +
                          (prefix_rows ? (p.P0 + kGenBM - 1) / kGenBM : 0);
    if (tiles > 0x7fffffffLL || s->Hq > 65535 || s->B > 65535) return VXL_ERR_UNSUPPORTED;
    if (tiles == 0) return VXL_OK;
    dim3 grid((unsigned)tiles, (unsigned)s->Hq, (unsigned)s->B);
    cudaError_t e;
    if (s->D == 128) {
        static bool done[kMaxDevices] = {};
        e = ensure_smem(prefill_general_kernel<128>, GenSmem<128>::kBytes, done);
        if (e != cudaSuccess) return VXL_ERR_CUDA;
        prefill_general_kernel<128><<<grid, 128, GenSmem<128>::kBytes, st>>>(p);
    } else {
        static bool done[kMaxDevices] = {};
        e = ensure_smem(prefill_general_kernel<64>, GenSmem<64>::kBytes, done);
        if (e != cudaSuccess) return VXL_ERR_CUDA;
        prefill_general_kernel<64><<<grid, 128, GenSmem<64>::kBytes, st>>>(p);
    }
    return cudaGetLastError() == cudaSuccess ? VXL_OK : VXL_ERR_CUDA;
}

// One warp waits, with the kernels' own bounded wait, on a barrier that nothing will ever complete.
__global__ void bounded_wait_probe_kernel(WsHeader *hdr, long long limit_cycles)
{
    __shared__ __align__(8) uint64_t bar;
    if (threadIdx.x == 0) { mbar_init(smem_u32(&bar), 1); mbar_fence_init(); }
    __syncthreads();
    const bool ok = mbar_wait(smem_u32(&bar), 0, limit_cycles);
    if (!ok && threadIdx.x == 0) raise_status(hdr, VXL_ERR_TIMEOUT, 900);
}

}  // namespace

extern "C" {

vxl_status vxl_selftest_bounded_wait(void *workspace, int64_t limit_cycles, void *cuda_stream)
{
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return VXL_ERR_WORKSPACE;
    if (limit_cycles <= 0 || limit_cycles > 200000000ll) return VXL_ERR_INVALID_ARG;     // a tenth of a second at most
    bounded_wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(static_cast<WsHeader *>(workspace),
                                                                                   (long long)limit_cycles);
    return cudaGetLastError() == cudaSuccess ? VXL_OK : VXL_ERR_CUDA;
}


const char *vxl_status_str(vxl_status s)
{
    switch (s) {
        case VXL_OK: return "ok";
        case VXL_ERR_INVALID_ARG: return "invalid argument";
        case VXL_ERR_UNSUPPORTED: return "unsupported shape";
        case VXL_ERR_INVALID_INDEX: return "invalid index (device)";
        case VXL_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case VXL_ERR_CUDA: return "CUDA call failed";
        case VXL_ERR_TIMEOUT: return "bounded device wait expired";
    }
    return "unknown status";
}

size_t vxl_workspace_bytes(int32_t op, const vxl_shape *shape, int32_t C, int32_t R, int32_t topk,
                           int32_t max_chunk_len)
{
    (void)R;
    if (!shape_ok(shape) || C < 0 || topk < 0) return 0;
    switch (op) {
        case VXL_OP_PREFILL: return sizeof(WsHeader) + prefill_tc_workspace_bytes(shape, C, R);
        case VXL_OP_SCORES: return carve_decode(nullptr, shape, C, 0, 1, false).bytes;
        case VXL_OP_DECODE: return carve_decode(nullptr, shape, C, topk, plan_slices(shape->B, topk, max_chunk_len > 0 ? max_chunk_len : 1, shape->Hkv).nslices, true).bytes;
        default: return 0;
    }
}

int32_t vxl_prefill_kernel_kind(const vxl_shape *s, int32_t chunk_len, int32_t R)
{
    const int step = s != nullptr && s->prefill_step > 0 ? s->prefill_step : chunk_len;
    if (!shape_ok(s) || chunk_len <= 0 || step <= 0 || s->prefix_len < 0 || s->prefix_len > s->T ||
        chunk_len % step != 0 || (s->T - s->prefix_len) % step != 0 || R < 0)
        return -1;
    if (s->force_general) return 0;
    return prefill_tc_supported(s, chunk_len, R) ? 1 : 0;
}

vxl_status vxl_chunk_prefill_attn(const void *q, const void *k, const void *v, int32_t chunk_len,
                                  const int32_t *retained_idx, int32_t R, void *out, float *lse,
                                  const vxl_shape *s, void *workspace, size_t ws_bytes, void *cuda_stream)
{
    if (!shape_ok(s) || q == nullptr || k == nullptr || v == nullptr || out == nullptr) return VXL_ERR_INVALID_ARG;
    // sliding chunk window: blocks of `step` tokens after a prefix; the plain form is step = chunk_len, no prefix
    const int step = s->prefill_step > 0 ? s->prefill_step : chunk_len;
    const int P0 = s->prefix_len;
    if (chunk_len <= 0 || step <= 0 || P0 < 0 || P0 > s->T || chunk_len % step != 0 || (s->T - P0) % step != 0 ||
        R < 0 || R > step)
        return VXL_ERR_INVALID_ARG;
    const int C = (s->T - P0) / step;                    // rows of retained_idx
    if (R > 0 && C > 1 && retained_idx == nullptr) return VXL_ERR_INVALID_ARG;
    if (s->block_begin < 0 || s->block_count < 0 || s->block_begin > C || s->block_count > C - s->block_begin)
        return VXL_ERR_INVALID_ARG;
    const int c0 = s->block_begin;
    const int Cn = s->block_count > 0 ? s->block_count : C - c0;
    const bool with_prefix = (c0 == 0);                  // the prefix rows belong to the call that starts at block 0
    if (s->D != 64 && s->D != 128) return VXL_ERR_UNSUPPORTED;
    if (!strides_ok(s, true) || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out))
        return VXL_ERR_INVALID_ARG;
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        ws_bytes < vxl_workspace_bytes(VXL_OP_PREFILL, s, C, R, 0, chunk_len))
        return VXL_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    WsHeader *hdr = static_cast<WsHeader *>(workspace);

    PrefillParams p;
    std::memset(&p, 0, sizeof p);
    p.q = static_cast<const __nv_bfloat16 *>(q);
    p.k = static_cast<const __nv_bfloat16 *>(k);
    p.v = static_cast<const __nv_bfloat16 *>(v);
    p.out = out; p.lse = lse; p.ridx = retained_idx; p.hdr = hdr;
    p.q_sb = s->q_stride_b; p.q_st = s->q_stride_t; p.q_sh = s->q_stride_h;
    p.kv_sb = s->kv_stride_b; p.kv_st = s->kv_stride_t; p.kv_sh = s->kv_stride_h;
    p.o_sh = s->out_stride_h ? s->out_stride_h : s->D;
    p.o_st = s->out_stride_t ? s->out_stride_t : (int64_t)s->Hq * p.o_sh;
    p.o_sb = s->out_stride_b ? s->out_stride_b : (int64_t)s->T * p.o_st;
    p.B = s->B; p.T = s->T; p.Hq = s->Hq; p.Hkv = s->Hkv; p.G = s->Hq / s->Hkv;
    p.L = chunk_len; p.C = C; p.R = (C > 1) ? R : 0;
    p.S = step; p.P0 = P0; p.prefix_only = 0;
    p.c0 = c0; p.Cn = Cn;
    p.out_bf16 = (s->out_dtype == VXL_BF16);
    p.scale_log2 = resolve_scale(s) * kLog2e;

    if (s->validate && R > 0) {
        if (launch_validate(retained_idx, nullptr, hdr, 0, 1, C, R, step, s->T, st, P0) != cudaSuccess)
            return VXL_ERR_CUDA;
    }
    if (!s->force_general && prefill_tc_supported(s, chunk_len, R)) {
        char *order_ws = static_cast<char *>(workspace) + sizeof(WsHeader);
        char *ks = order_ws + prefill_tc_order_bytes();
        char *vs = ks + prefill_tc_packed_bytes(s, C, R);
        p.gather4 = s->prefill_gather4 ? 1 : 0;
        if (!p.gather4 && p.R > 0) {
            // the sparse level of this call: retained rows of every chunk, contiguous
            PackParams pp;
            std::memset(&pp, 0, sizeof pp);
            pp.k = p.k; pp.v = p.v;
            pp.ks = reinterpret_cast<__nv_bfloat16 *>(ks); pp.vs = reinterpret_cast<__nv_bfloat16 *>(vs);
            pp.ridx = retained_idx; pp.ridx_sb = 0;
            pp.kv_sb = p.kv_sb; pp.kv_st = p.kv_st; pp.kv_sh = p.kv_sh;
            pp.B = s->B; pp.T = s->T; pp.Hkv = s->Hkv; pp.D = s->D; pp.CR = C * R;
            // the last block of the range sees the retained rows of the blocks before it; whole key tiles are
            // loaded, so the rest of the last tile is zero-filled rather than taken from rows that a caller
            // working chunk by chunk has not written yet
            pp.n_valid = (c0 + Cn - 1) * R;
            pp.n_rows = (pp.n_valid + 127) / 128 * 128;
            if (pp.n_rows > pp.CR) pp.n_rows = pp.CR;
            if (Cn == 0) pp.n_valid = pp.n_rows = 0;
            const int64_t total = (int64_t)s->B * pp.n_rows * (s->Hkv * s->D / 8);
            int blocks = (int)((total + 255) / 256);
            if (blocks > 148 * 16) blocks = 148 * 16;
            if (blocks > 0) {
                pack_retained_kernel<<<blocks, 256, 0, st>>>(pp);
                if (cudaGetLastError() != cudaSuccess) return VXL_ERR_CUDA;
            }
        }
        if (Cn > 0) {
            const vxl_status r = prefill_tc_launch(p, s->D, order_ws, ks, vs, st);
            if (r != VXL_OK || P0 == 0 || !with_prefix) return r;
        }
        if (!with_prefix) return VXL_OK;
        // the prefix rows (causal among themselves, any length) go through the general kernel
        p.prefix_only = 1;
        return launch_prefill_general(p, s, st);
    }
    if (!with_prefix) return Cn == 0 ? VXL_OK : launch_prefill_general(p, s, st, false);

    return launch_prefill_general(p, s, st);
}

// Events that order the three streams of vxl_chunk_prefill_host: a pool per device, grown on demand and
// kept until the process exits.  A wait enqueued on a stream refers to the event's state at that
// moment, so a later call may record the same events again; the mutex only serialises the enqueueing.
struct HostPrefillEvents {
    std::mutex mu;
    cudaEvent_t *ev = nullptr;
    int n = 0;
};
HostPrefillEvents g_hp_events[kMaxDevices];

bool hp_reserve_events(HostPrefillEvents &pool, int need)
{
    if (need <= pool.n) return true;
    cudaEvent_t *grown = static_cast<cudaEvent_t *>(std::realloc(pool.ev, sizeof(cudaEvent_t) * (size_t)need));
    if (grown == nullptr) return false;
    pool.ev = grown;
    while (pool.n < need) {
        if (cudaEventCreateWithFlags(&pool.ev[pool.n], cudaEventDisableTiming) != cudaSuccess) return false;
        ++pool.n;
    }
    return true;
}

vxl_status vxl_chunk_prefill_host(const void *q_host, const void *k_host, const void *v_host, int32_t chunk_len,
                                  const int32_t *retained_idx_host, int32_t R, void *out_host, float *lse_host,
                                  void *q_dev, void *k_dev, void *v_dev, int32_t *retained_idx_dev, void *out_dev,
                                  float *lse_dev, int32_t chunks_per_call, const vxl_shape *s, void *workspace,
                                  size_t ws_bytes, void *cuda_stream, void *h2d_stream, void *d2h_stream)
{
    if (!shape_ok(s) || q_host == nullptr || k_host == nullptr || v_host == nullptr || out_host == nullptr ||
        q_dev == nullptr || k_dev == nullptr || v_dev == nullptr || out_dev == nullptr)
        return VXL_ERR_INVALID_ARG;
    if ((lse_host == nullptr) != (lse_dev == nullptr)) return VXL_ERR_INVALID_ARG;
    if (chunk_len <= 0 || s->T % chunk_len != 0 || R < 0 || R > chunk_len || chunks_per_call < 0) return VXL_ERR_INVALID_ARG;
    // plain chunks over back-to-back rows: the host and device arrays share one contiguous layout
    if (s->prefill_step != 0 && s->prefill_step != chunk_len) return VXL_ERR_UNSUPPORTED;
    if (s->prefix_len != 0 || s->block_begin != 0 || s->block_count != 0) return VXL_ERR_UNSUPPORTED;
    const int64_t qrow = (int64_t)s->Hq * s->D, kvrow = (int64_t)s->Hkv * s->D;
    if (s->q_stride_h != s->D || s->q_stride_t != qrow || s->q_stride_b != (int64_t)s->T * qrow ||
        s->kv_stride_h != s->D || s->kv_stride_t != kvrow || s->kv_stride_b != (int64_t)s->T * kvrow)
        return VXL_ERR_UNSUPPORTED;
    if ((s->out_stride_h != 0 && s->out_stride_h != s->D) || (s->out_stride_t != 0 && s->out_stride_t != qrow) ||
        (s->out_stride_b != 0 && s->out_stride_b != (int64_t)s->T * qrow))
        return VXL_ERR_UNSUPPORTED;
    const int C = s->T / chunk_len;
    if (R > 0 && C > 1 && (retained_idx_host == nullptr || retained_idx_dev == nullptr)) return VXL_ERR_INVALID_ARG;
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        ws_bytes < vxl_workspace_bytes(VXL_OP_PREFILL, s, C, R, 0, chunk_len))
        return VXL_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream), sin = static_cast<cudaStream_t>(h2d_stream),
                 sout = static_cast<cudaStream_t>(d2h_stream);
    if (sin == st || sout == st || sin == sout) return VXL_ERR_INVALID_ARG;     // the overlap needs three streams

    const int per = chunks_per_call > 0 ? chunks_per_call : 1;
    const int groups = (C + per - 1) / per;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return VXL_ERR_CUDA;
    HostPrefillEvents &pool = g_hp_events[dev];
    std::lock_guard<std::mutex> lock(pool.mu);
    if (!hp_reserve_events(pool, 2 * groups + 2)) return VXL_ERR_CUDA;
    cudaEvent_t *ev_in = pool.ev, *ev_done = pool.ev + groups;
    cudaEvent_t ev_begin = pool.ev[2 * groups], ev_end = pool.ev[2 * groups + 1];

    // the copy streams start after whatever the caller's stream still does with the device arrays
    if (cudaEventRecord(ev_begin, st) != cudaSuccess || cudaStreamWaitEvent(sin, ev_begin, 0) != cudaSuccess ||
        cudaStreamWaitEvent(sout, ev_begin, 0) != cudaSuccess)
        return VXL_ERR_CUDA;
    if (R > 0 && C > 1 &&
        cudaMemcpyAsync(retained_idx_dev, retained_idx_host, sizeof(int32_t) * (size_t)C * R, cudaMemcpyHostToDevice, sin) != cudaSuccess)
        return VXL_ERR_CUDA;
    const size_t esz = sizeof(__nv_bfloat16), osz = (s->out_dtype == VXL_BF16) ? 2 : 4;
    // one copy per tensor and chunk group: the rows of the group in every sequence (a 2-D copy whose
    // pitch is one sequence)
    auto copy_rows = [&](void *dst, const void *src, int64_t row_elems, size_t elem, int row0, int nrows,
                         cudaMemcpyKind kind, cudaStream_t cs) {
        const size_t pitch = (size_t)s->T * row_elems * elem, off = (size_t)row0 * row_elems * elem;
        return cudaMemcpy2DAsync(static_cast<char *>(dst) + off, pitch, static_cast<const char *>(src) + off, pitch,
                                 (size_t)nrows * row_elems * elem, (size_t)s->B, kind, cs);
    };
    for (int g = 0; g < groups; ++g) {
        const int c0 = g * per, n = (C - c0 < per) ? C - c0 : per;
        const int row0 = c0 * chunk_len, nrows = n * chunk_len;
        if (copy_rows(q_dev, q_host, qrow, esz, row0, nrows, cudaMemcpyHostToDevice, sin) != cudaSuccess ||
            copy_rows(k_dev, k_host, kvrow, esz, row0, nrows, cudaMemcpyHostToDevice, sin) != cudaSuccess ||
            copy_rows(v_dev, v_host, kvrow, esz, row0, nrows, cudaMemcpyHostToDevice, sin) != cudaSuccess ||
            cudaEventRecord(ev_in[g], sin) != cudaSuccess)
            return VXL_ERR_CUDA;
    }
    vxl_shape sub = *s;
    for (int g = 0; g < groups; ++g) {
        const int c0 = g * per, n = (C - c0 < per) ? C - c0 : per;
        if (cudaStreamWaitEvent(st, ev_in[g], 0) != cudaSuccess) return VXL_ERR_CUDA;
        sub.block_begin = c0; sub.block_count = n;
        const vxl_status r = vxl_chunk_prefill_attn(q_dev, k_dev, v_dev, chunk_len, retained_idx_dev, R, out_dev, lse_dev, &sub,
                                                    workspace, ws_bytes, cuda_stream);
        if (r != VXL_OK) return r;
        if (cudaEventRecord(ev_done[g], st) != cudaSuccess) return VXL_ERR_CUDA;
    }
    for (int g = 0; g < groups; ++g) {
        const int c0 = g * per, n = (C - c0 < per) ? C - c0 : per;
        const int row0 = c0 * chunk_len, nrows = n * chunk_len;
        if (cudaStreamWaitEvent(sout, ev_done[g], 0) != cudaSuccess ||
            copy_rows(out_host, out_dev, qrow, osz, row0, nrows, cudaMemcpyDeviceToHost, sout) != cudaSuccess)
            return VXL_ERR_CUDA;
        if (lse_host != nullptr &&
            copy_rows(lse_host, lse_dev, s->Hq, sizeof(float), row0, nrows, cudaMemcpyDeviceToHost, sout) != cudaSuccess)
            return VXL_ERR_CUDA;
    }
    // later work on the caller's stream comes after the last copy back
    if (cudaEventRecord(ev_end, sout) != cudaSuccess || cudaStreamWaitEvent(st, ev_end, 0) != cudaSuccess) return VXL_ERR_CUDA;
    return VXL_OK;
}

vxl_status vxl_chunk_scores(const void *q, const void *k_cache, const int32_t *chunk_offsets, int32_t C,
                            const int32_t *retained_idx, int32_t R, int64_t ridx_stride_b,
                            const vxl_sparse_level *sparse, float *scores, int32_t topk, int32_t *topk_idx,
                            const vxl_shape *s, void *workspace, size_t ws_bytes, void *cuda_stream)
{
    vxl_status vs = check_scores_args(s, q, k_cache, chunk_offsets, C, retained_idx, R, ridx_stride_b, sparse, scores, topk);
    if (vs != VXL_OK) return vs;
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        ws_bytes < vxl_workspace_bytes(VXL_OP_SCORES, s, C, R, 0, 0))
        return VXL_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    DecodeWs w = carve_decode(workspace, s, C, 0, 1, false);
    if (s->validate &&
        launch_validate(retained_idx, chunk_offsets, w.hdr, ridx_stride_b, ridx_stride_b ? s->B : 1, C,
                        retained_idx ? R : 0, 0, s->T, st) != cudaSuccess)
        return VXL_ERR_CUDA;
    DecodeParams p;
    fill_decode_params(p, s, q, k_cache, nullptr, chunk_offsets, C, retained_idx, R, ridx_stride_b, sparse, 0, 1, kSliceRows, w);
    const int HPC = heads_per_cta(s->Hkv);
    if (run_sparse_pass<false>(s, p, HPC, st) != cudaSuccess) return VXL_ERR_CUDA;
    TopkParams tp{w.part_m, w.part_l, nullptr, scores, topk_idx, nullptr, w.flags, w.hdr, s->B, s->Hq, C, p.P,
                  topk_idx ? topk : 0, sparse_pass_streams(s, p) ? w.score_part : nullptr, s->Hkv};
    if (s->score_mode == VXL_SCORE_MASS) {
        topk_mass_kernel<<<s->B, 1024, (size_t)C * 8, st>>>(tp);
        return cudaGetLastError() == cudaSuccess ? VXL_OK : VXL_ERR_CUDA;
    }
    if (launch_pdl(topk_fast_kernel, dim3(s->B), dim3(1024), (size_t)C * 8, st, tp) != cudaSuccess) return VXL_ERR_CUDA;
    return VXL_OK;
}

vxl_status vxl_topk_select(const float *scores, int32_t B, int32_t C, int32_t topk, int32_t *topk_idx, void *cuda_stream)
{
    if (scores == nullptr || topk_idx == nullptr || B <= 0 || C <= 0 || topk < 0 || topk > C) return VXL_ERR_INVALID_ARG;
    if (C > kMaxChunks) return VXL_ERR_UNSUPPORTED;
    if (topk == 0) return VXL_OK;
    topk_scores_kernel<<<B, 1024, (size_t)C * 8, static_cast<cudaStream_t>(cuda_stream)>>>(scores, topk_idx, C, topk);
    return cudaGetLastError() == cudaSuccess ? VXL_OK : VXL_ERR_CUDA;
}

vxl_status vxl_chunk_scores_multi(const void *q, int32_t n_query_tokens, const void *k_cache,
                                  const int32_t *chunk_offsets, int32_t C, const int32_t *retained_idx, int32_t R,
                                  int64_t ridx_stride_b, const vxl_sparse_level *sparse, float *scores, int32_t topk,
                                  int32_t *topk_idx, const vxl_shape *s, void *workspace, size_t ws_bytes,
                                  void *cuda_stream)
{
    vxl_status vs = check_decode_common(s, q, k_cache, chunk_offsets, C, retained_idx, R, ridx_stride_b, sparse, false);
    if (vs != VXL_OK) return vs;
    if (scores == nullptr || topk < 0 || topk > C || n_query_tokens <= 0) return VXL_ERR_INVALID_ARG;
    if (n_query_tokens > 1 && (s->q_stride_t <= 0 || s->q_stride_t % 8 != 0)) return VXL_ERR_INVALID_ARG;
    if (C > kMaxChunks) return VXL_ERR_UNSUPPORTED;
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        ws_bytes < vxl_workspace_bytes(VXL_OP_SCORES, s, C, R, 0, 0))
        return VXL_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    DecodeWs w = carve_decode(workspace, s, C, 0, 1, false);
    if (s->validate &&
        launch_validate(retained_idx, chunk_offsets, w.hdr, ridx_stride_b, ridx_stride_b ? s->B : 1, C,
                        retained_idx ? R : 0, 0, s->T, st) != cudaSuccess)
        return VXL_ERR_CUDA;
    const int HPC = heads_per_cta(s->Hkv);
    for (int t = 0; t < n_query_tokens; ++t) {
        // one sparse-level pass (keys only) per query token, then its share of the mean
        const __nv_bfloat16 *qt = static_cast<const __nv_bfloat16 *>(q) + (int64_t)t * s->q_stride_t;
        DecodeParams p;
        fill_decode_params(p, s, qt, k_cache, nullptr, chunk_offsets, C, retained_idx, R, ridx_stride_b, sparse, 0, 1,
                           kSliceRows, w);
        if (run_sparse_pass<false>(s, p, HPC, st) != cudaSuccess) return VXL_ERR_CUDA;
        ScoreAccumParams ap{w.part_m, w.part_l, scores, s->B, s->Hq, C, p.P, 1.0f / (float)n_query_tokens, t == 0 ? 1 : 0};
        score_accum_kernel<<<dim3((unsigned)((C * 4 + 255) / 256), (unsigned)s->B), 256, 0, st>>>(ap);
        if (cudaGetLastError() != cudaSuccess) return VXL_ERR_CUDA;
    }
    if (topk_idx != nullptr && topk > 0) return vxl_topk_select(scores, s->B, C, topk, topk_idx, cuda_stream);
    return VXL_OK;
}

vxl_status vxl_chunk_scores_static(const void *q, const void *k_cache, const int32_t *chunk_offsets, int32_t C,
                                   const int32_t *retained_idx, int32_t R, int64_t ridx_stride_b,
                                   const vxl_sparse_level *sparse, float *scores, int32_t topk, int32_t *topk_idx,
                                   int32_t *device_status_out, const vxl_shape *s, void *cuda_stream)
{
    // Every host-side check comes first: a call that is refused has touched neither the stream nor the
    // shared array (whose status word an earlier call's status copy may not have read yet).
    if (!shape_ok(s) || C <= 0 || R < 0) return VXL_ERR_INVALID_ARG;
    const size_t need = vxl_workspace_bytes(VXL_OP_SCORES, s, C, R, 0, 0);
    if (need == 0) return VXL_ERR_INVALID_ARG;
    if (need > kStaticScratchBytes) return VXL_ERR_WORKSPACE;
    const vxl_status pre = check_scores_args(s, q, k_cache, chunk_offsets, C, retained_idx, R, ridx_stride_b, sparse, scores, topk);
    if (pre != VXL_OK) return pre;
    void *scratch = static_scratch_address();
    if (scratch == nullptr) return VXL_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // The array keeps whatever the previous call left.  Only the status word has to start at
    // zero; partials, flags and the selection are fully rewritten before they are read.
    if (cudaMemsetAsync(scratch, 0, sizeof(WsHeader), st) != cudaSuccess) return VXL_ERR_CUDA;
    const vxl_status rc = vxl_chunk_scores(q, k_cache, chunk_offsets, C, retained_idx, R, ridx_stride_b, sparse,
                                           scores, topk, topk_idx, s, scratch, kStaticScratchBytes, cuda_stream);
    if (rc != VXL_OK) return rc;
    if (device_status_out != nullptr &&
        cudaMemcpyAsync(device_status_out, scratch, sizeof(int32_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return VXL_ERR_CUDA;
    return VXL_OK;
}

vxl_status vxl_bilevel_decode_attn(const void *q, const void *k_cache, const void *v_cache,
                                   const int32_t *chunk_offsets, int32_t C, int32_t max_chunk_len,
                                   const int32_t *retained_idx, int32_t R, int64_t ridx_stride_b,
                                   const vxl_sparse_level *sparse, int32_t topk, const int32_t *selected,
                                   void *out, float *lse, float *scores_out, int32_t *topk_out,
                                   const vxl_shape *s, void *workspace, size_t ws_bytes, void *cuda_stream)
{
    vxl_status vs = check_decode_common(s, q, k_cache, chunk_offsets, C, retained_idx, R, ridx_stride_b, sparse, true);
    if (vs != VXL_OK) return vs;
    if (v_cache == nullptr || out == nullptr || !aligned16(v_cache) || !aligned16(out)) return VXL_ERR_INVALID_ARG;
    if (topk < 0 || topk > C || max_chunk_len <= 0) return VXL_ERR_INVALID_ARG;
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        ws_bytes < vxl_workspace_bytes(VXL_OP_DECODE, s, C, R, topk, max_chunk_len))
        return VXL_ERR_WORKSPACE;
    if (C > kMaxChunks) return VXL_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const SlicePlan plan = plan_slices(s->B, topk, max_chunk_len, s->Hkv);
    const int nslices = plan.nslices;
    DecodeWs w = carve_decode(workspace, s, C, topk, nslices, true);
    if (s->validate &&
        launch_validate(retained_idx, chunk_offsets, w.hdr, ridx_stride_b, ridx_stride_b ? s->B : 1, C,
                        retained_idx ? R : 0, 0, s->T, st) != cudaSuccess)
        return VXL_ERR_CUDA;
    DecodeParams p;
    fill_decode_params(p, s, q, k_cache, v_cache, chunk_offsets, C, retained_idx, R, ridx_stride_b, sparse, topk,
                       nslices, plan.slice_rows, w);
    const int HPC = heads_per_cta(s->Hkv);
    return run_decode_passes(s, p, w, C, R, topk, selected, out, lse, scores_out, topk_out, HPC, st, nullptr);
}

vxl_status vxl_bilevel_decode_offline(const void *q, const void *k_host, const void *v_host,
                                      const int32_t *chunk_offsets, const int32_t *chunk_offsets_host, int32_t C,
                                      int32_t max_chunk_len, const vxl_sparse_level *sparse, int32_t R, int32_t topk,
                                      void *k_stage, void *v_stage, int32_t *topk_host, void *out, float *lse,
                                      float *scores_out, int32_t *topk_out, const vxl_shape *s, void *workspace,
                                      size_t ws_bytes, void *cuda_stream, void *copy_stream)
{
    if (!shape_ok(s) || q == nullptr || k_host == nullptr || v_host == nullptr || chunk_offsets == nullptr ||
        chunk_offsets_host == nullptr || sparse == nullptr || sparse->k_sparse == nullptr || sparse->v_sparse == nullptr ||
        k_stage == nullptr || v_stage == nullptr || topk_host == nullptr || out == nullptr || scores_out == nullptr ||
        topk_out == nullptr)
        return VXL_ERR_INVALID_ARG;
    if (C <= 0 || C > s->T || R <= 0 || topk <= 0 || topk > C || max_chunk_len <= 0) return VXL_ERR_INVALID_ARG;
    if (s->D != 64 && s->D != 128) return VXL_ERR_UNSUPPORTED;
    if (C > kMaxChunks || (int64_t)s->B * C * R >= (1ll << 31) || (int64_t)s->B * topk * max_chunk_len >= (1ll << 31))
        return VXL_ERR_UNSUPPORTED;
    // whole token rows are copied: the host cache must hold a token's kv heads contiguously
    if (s->kv_stride_h != s->D || s->kv_stride_t != (int64_t)s->Hkv * s->D) return VXL_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k_stage) || !aligned16(v_stage) || !aligned16(out)) return VXL_ERR_INVALID_ARG;
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        ws_bytes < vxl_workspace_bytes(VXL_OP_DECODE, s, C, R, topk, max_chunk_len))
        return VXL_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream), cs = static_cast<cudaStream_t>(copy_stream);

    // 1. relevance and top-k from the sparse level, which stays on the device
    vxl_status vs = vxl_chunk_scores(q, sparse->k_sparse, chunk_offsets, C, nullptr, R, 0, sparse, scores_out, topk, topk_out,
                                     s, workspace, ws_bytes, cuda_stream);
    if (vs != VXL_OK) return vs;
    // 2. the selection comes to the host (this call synchronises the stream here)
    if (cudaMemcpyAsync(topk_host, topk_out, sizeof(int32_t) * (size_t)s->B * topk, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return VXL_ERR_CUDA;
    // 3. reload: dense rows of the selected chunks, host -> staging slots, on the copy stream
    const size_t row_bytes = (size_t)s->Hkv * s->D * sizeof(__nv_bfloat16);
    for (int b = 0; b < s->B; ++b) {
        for (int j = 0; j < topk; ++j) {
            const int c = topk_host[(size_t)b * topk + j];
            if (c < 0 || c >= C) return VXL_ERR_INVALID_INDEX;
            const int lo = chunk_offsets_host[c], len = chunk_offsets_host[c + 1] - lo;
            if (lo < 0 || len < 0 || lo + len > s->T || len > max_chunk_len) return VXL_ERR_INVALID_INDEX;
            const size_t src = ((size_t)b * (size_t)s->kv_stride_b + (size_t)lo * (size_t)s->kv_stride_t) * sizeof(__nv_bfloat16);
            const size_t dst = ((size_t)b * topk + j) * (size_t)max_chunk_len * row_bytes;
            if (len > 0 &&
                (cudaMemcpyAsync(static_cast<char *>(k_stage) + dst, static_cast<const char *>(k_host) + src,
                                 (size_t)len * row_bytes, cudaMemcpyHostToDevice, cs) != cudaSuccess ||
                 cudaMemcpyAsync(static_cast<char *>(v_stage) + dst, static_cast<const char *>(v_host) + src,
                                 (size_t)len * row_bytes, cudaMemcpyHostToDevice, cs) != cudaSuccess))
                return VXL_ERR_CUDA;
        }
    }
    static cudaEvent_t copies_done[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return VXL_ERR_CUDA;
    if (copies_done[dev] == nullptr && cudaEventCreateWithFlags(&copies_done[dev], cudaEventDisableTiming) != cudaSuccess)
        return VXL_ERR_CUDA;
    if (cudaEventRecord(copies_done[dev], cs) != cudaSuccess) return VXL_ERR_CUDA;
    // 4. sparse pass of the other chunks while the copies run, then the dense pass over the staging slots
    const SlicePlan plan = plan_slices(s->B, topk, max_chunk_len, s->Hkv);
    DecodeWs w = carve_decode(workspace, s, C, topk, plan.nslices, true);
    DecodeParams p;
    fill_decode_params(p, s, q, k_stage, v_stage, chunk_offsets, C, nullptr, R, 0, sparse, topk, plan.nslices,
                       plan.slice_rows, w);
    p.staged = max_chunk_len;
    return run_decode_passes(s, p, w, C, R, topk, topk_out, out, lse, nullptr, nullptr, heads_per_cta(s->Hkv), st,
                             copies_done[dev]);
}

vxl_status vxl_pack_retained(const void *k_cache, const void *v_cache, const int32_t *retained_idx, int32_t C,
                             int32_t R, int64_t ridx_stride_b, void *k_sparse, void *v_sparse,
                             const vxl_shape *s, void *cuda_stream)
{
    if (!shape_ok(s) || k_cache == nullptr || v_cache == nullptr || k_sparse == nullptr || v_sparse == nullptr)
        return VXL_ERR_INVALID_ARG;
    if (C <= 0 || R < 0 || (R > 0 && retained_idx == nullptr)) return VXL_ERR_INVALID_ARG;
    if (ridx_stride_b != 0 && ridx_stride_b < (int64_t)C * R) return VXL_ERR_INVALID_ARG;
    if (s->D % 8 != 0) return VXL_ERR_UNSUPPORTED;
    if (!strides_ok(s, false) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(k_sparse) ||
        !aligned16(v_sparse))
        return VXL_ERR_INVALID_ARG;
    if (R == 0) return VXL_OK;
    PackParams pp;
    std::memset(&pp, 0, sizeof pp);
    pp.k = static_cast<const __nv_bfloat16 *>(k_cache);
    pp.v = static_cast<const __nv_bfloat16 *>(v_cache);
    pp.ks = static_cast<__nv_bfloat16 *>(k_sparse);
    pp.vs = static_cast<__nv_bfloat16 *>(v_sparse);
    pp.ridx = retained_idx; pp.ridx_sb = ridx_stride_b;
    pp.kv_sb = s->kv_stride_b; pp.kv_st = s->kv_stride_t; pp.kv_sh = s->kv_stride_h;
    pp.B = s->B; pp.T = s->T; pp.Hkv = s->Hkv; pp.D = s->D; pp.CR = C * R;
    pp.n_valid = pp.n_rows = C * R;
    const int64_t total = (int64_t)s->B * C * R * (s->Hkv * s->D / 8);
    int blocks = (int)((total + 255) / 256);
    if (blocks > 148 * 16) blocks = 148 * 16;
    pack_retained_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(pp);
    return cudaGetLastError() == cudaSuccess ? VXL_OK : VXL_ERR_CUDA;
}

vxl_status vxl_pool_sparse(const void *k_cache, const void *v_cache, const int32_t *chunk_offsets, int32_t C,
                           int32_t R, void *k_sparse, void *v_sparse, const vxl_shape *s, void *cuda_stream)
{
    if (!shape_ok(s) || k_cache == nullptr || v_cache == nullptr || k_sparse == nullptr || v_sparse == nullptr ||
        chunk_offsets == nullptr)
        return VXL_ERR_INVALID_ARG;
    if (C <= 0 || R < 0 || C > s->T) return VXL_ERR_INVALID_ARG;
    if (s->D % 8 != 0) return VXL_ERR_UNSUPPORTED;
    if (!strides_ok(s, false) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(k_sparse) ||
        !aligned16(v_sparse))
        return VXL_ERR_INVALID_ARG;
    if (R == 0) return VXL_OK;
    PoolParams pp;
    std::memset(&pp, 0, sizeof pp);
    pp.k = static_cast<const __nv_bfloat16 *>(k_cache);
    pp.v = static_cast<const __nv_bfloat16 *>(v_cache);
    pp.ks = static_cast<__nv_bfloat16 *>(k_sparse);
    pp.vs = static_cast<__nv_bfloat16 *>(v_sparse);
    pp.off = chunk_offsets;
    pp.kv_sb = s->kv_stride_b; pp.kv_st = s->kv_stride_t; pp.kv_sh = s->kv_stride_h;
    pp.B = s->B; pp.T = s->T; pp.Hkv = s->Hkv; pp.D = s->D; pp.C = C; pp.R = R;
    const int64_t total = (int64_t)s->B * C * R * (s->Hkv * s->D / 8);
    int blocks = (int)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
    pool_sparse_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(pp);
    return cudaGetLastError() == cudaSuccess ? VXL_OK : VXL_ERR_CUDA;
}

vxl_status vxl_device_status(void *workspace, void *cuda_stream)
{
    if (workspace == nullptr) return VXL_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int host[2] = {0, 0};
    if (cudaMemcpyAsync(host, workspace, sizeof host, cudaMemcpyDeviceToHost, st) != cudaSuccess) return VXL_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return VXL_ERR_CUDA;
    if (host[0] != 0) {
        if (cudaMemsetAsync(workspace, 0, sizeof host, st) != cudaSuccess) return VXL_ERR_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return VXL_ERR_CUDA;
    }
    if (host[0] < 0 || host[0] > VXL_ERR_TIMEOUT) return VXL_ERR_CUDA;
    return static_cast<vxl_status>(host[0]);
}

}  // extern "C"
