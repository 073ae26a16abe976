// Chunk-sparse prefill on the 5th-generation tensor cores (sm_100a): tcgen05.mma with TMEM
// accumulators, K/V tiles staged in shared memory by TMA; retained rows come from the packed
// sparse level as plain tiles, or by index with TMA gather4 (four rows per request).
//
// Persistent kernel, one CTA per SM.  A work item = two adjacent 128-row query tiles of one chunk
// (rows [256p, 256p+256)) for one query head.  Its key list is: the c*R retained rows of the
// preceding chunks (no mask, in tiles of 128 rows), then the chunk's own 128-row tiles 0 .. 2p+1
// (causal mask on each query tile's diagonal tile only; the last tile is read by the second query
// tile only).  Items are ranked by length on the device and dealt to the CTAs in a fixed order.
//
// Warp roles (384 threads = three warpgroups, so that registers can move between them):
//   warps 0-3   softmax / correction / epilogue for query tile 0 (one thread per row)
//   warps 4-7   the same for query tile 1
//   warp  8     MMA issuer (one thread), owns the TMEM allocation
//   warp  9     TMA producer: Q per item; K and V tiles in units (V_j with K_{j+1}) through a ring
//               of 64 KB pair slots that runs on into the next item while the current one finishes
//   warps 10-11 idle; the third warpgroup hands most of its registers to the softmax warps
// TMEM (512 columns x 128 lanes, fp32): S0 [0,128) S1 [128,256) O0 [256,256+D) O1 [384,384+D);
// P (bf16, two per column) overwrites the first 64 columns of its S.
// The two query tiles ping-pong: while the softmax warps of one tile work on S_j, the tensor
// pipe runs the other tile's P.V and the next Q.K^T.  Across items the pipeline keeps going: the
// epilogue of an item (O from TMEM through a swizzled staging block to coalesced global stores)
// overlaps the first key tiles of the next one.
// Every mbarrier wait is bounded; on expiry the kernel records VXL_ERR_TIMEOUT and winds down.
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "prefill_general.cuh"

namespace vxl {

constexpr int kTcThreads = 384;                          // three warpgroups (the last one has two idle warps)
#ifndef VXL_TC_STAGES
#define VXL_TC_STAGES 4
#endif
constexpr int kTcStages = VXL_TC_STAGES;               // K/V ring slots of 32 KB
constexpr int kTcPairs = kTcStages / 2;                  // pair slots of 64 KB (V tile + K tile)
static_assert(kTcStages % 2 == 0, "the ring is used in pairs of tiles");
constexpr uint32_t kTcTileBytes = 128 * 128 * 2;        // room of one tile in shared memory (128 rows x 128 columns of bf16)
template <int D> constexpr uint32_t kTcTileLoad = 128u * D * 2u;   // bytes a 128-row tile of head dimension D brings in
constexpr uint32_t kTcPanelBytes = 128 * 64 * 2;        // 64 columns (128 B) x 128 rows
constexpr uint32_t kTcSmemQ = 0;
constexpr uint32_t kTcSmemKV = 2 * kTcTileBytes;
constexpr uint32_t kTcSmemStage = kTcSmemKV + kTcStages * kTcTileBytes;   // epilogue staging: 8 warps x 4 KB
constexpr uint32_t kTcSmemBar = kTcSmemStage + 8 * 4096;
constexpr uint32_t kTcSmemBytes = kTcSmemBar + 256 + 1024;   // + slack for 1024-byte alignment
constexpr int kTcMaxOrder = 4096;                        // (chunk, pair) entries ranked on the device
constexpr float kTcRescaleThreshold = 8.0f;              // log2 units: keep a stale max up to 2^8

struct TcMaps {
    CUtensorMap q, k, v, kg, vg;
    CUtensorMap o;        // fp32 output as [rows, Hq*128], boxes of 32 columns x 32 rows (valid when tma_out)
};

// barrier indices inside the barrier block
enum : int {
    kBarFull = 0,                       // [pairs used of stages] K/V unit landed (TMA -> MMA)
    kBarEmpty = kBarFull + kTcStages,   // [pairs used of stages] K/V unit consumed (MMA -> TMA)
    kBarQ = kBarEmpty + kTcStages,      // Q tiles landed
    kBarS = kBarQ + 1,                  // [2] S_t ready (MMA -> softmax)
    kBarP = kBarS + 2,                  // [2] keys 0-63 of P_t written, O_t rescaled (softmax -> MMA)
    kBarP2 = kBarP + 2,                 // [2] keys 64-127 of P_t written
    kBarO = kBarP2 + 2,                 // [2] O_t final (MMA -> epilogue)
    kBarOFree = kBarO + 2,              // [2] O_t read out of tensor memory (epilogue -> MMA)
    kBarQFree = kBarOFree + 2,          // last S = Q.K^T of the item done (MMA -> TMA)
    kBarCount = kBarQFree + 1
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap *map, int x, int y0, int y1, int y2,
                                            int y3, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, "
        "%4, %5, %6}], [%7];" ::"r"(dst),
        "l"(map), "r"(x), "r"(y0), "r"(y1), "r"(y2), "r"(y3), "r"(bar)
        : "memory");
}
// One staged 32 x 32 fp32 box from shared memory to the output (bulk async group of the issuing thread).
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, int x, int y, uint32_t src)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];" ::"l"(map), "r"(x), "r"(y),
                 "r"(src)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float *r)
{
    uint32_t *u = reinterpret_cast<uint32_t *>(r);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]),
          "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15]), "=r"(u[16]),
          "=r"(u[17]), "=r"(u[18]), "=r"(u[19]), "=r"(u[20]), "=r"(u[21]), "=r"(u[22]), "=r"(u[23]), "=r"(u[24]),
          "=r"(u[25]), "=r"(u[26]), "=r"(u[27]), "=r"(u[28]), "=r"(u[29]), "=r"(u[30]), "=r"(u[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t *u)
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),
        "r"(u[0]), "r"(u[1]), "r"(u[2]), "r"(u[3]), "r"(u[4]), "r"(u[5]), "r"(u[6]), "r"(u[7]), "r"(u[8]), "r"(u[9]),
        "r"(u[10]), "r"(u[11]), "r"(u[12]), "r"(u[13]), "r"(u[14]), "r"(u[15]), "r"(u[16]), "r"(u[17]), "r"(u[18]),
        "r"(u[19]), "r"(u[20]), "r"(u[21]), "r"(u[22]), "r"(u[23]), "r"(u[24]), "r"(u[25]), "r"(u[26]), "r"(u[27]),
        "r"(u[28]), "r"(u[29]), "r"(u[30]), "r"(u[31])
        : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (SWIZZLE_128B, version 1): 14-bit fields in 16-byte units.
__device__ __forceinline__ uint64_t tc_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (2ull << 61);
}
// Low / high 32-bit words of that descriptor, for code that steps the address field itself.
__device__ __forceinline__ uint32_t tc_desc_lo(uint32_t saddr, uint32_t lbo_bytes)
{
    return ((saddr >> 4) & 0x3FFFu) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}
__host__ __device__ constexpr uint32_t tc_desc_hi(uint32_t sbo_bytes)
{
    return ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);
}
// One S = Q.K^T tile: eight k = 16 steps issued from one asm block.  a_lo / b_lo are the low
// descriptor words of the Q and K tiles (address and leading offset fields); a step only moves
// the 14-bit address field, by constants, so each MMA costs two adds.
__device__ __forceinline__ void tc_qk8(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc)
{
    asm volatile(
        "{\n\t"
        ".reg .pred pf, pt;\n\t.reg .b64 da, db;\n\t.reg .b32 al, bl;\n\t"
        "setp.ne.b32 pf, %0, %0;\n\tsetp.eq.b32 pt, %0, %0;\n\t"
        "add.u32 al, %1, 0;\n\tadd.u32 bl, %2, 0;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pf;\n\t"
        "add.u32 al, %1, 2;\n\tadd.u32 bl, %2, 2;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
        "add.u32 al, %1, 4;\n\tadd.u32 bl, %2, 4;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
        "add.u32 al, %1, 6;\n\tadd.u32 bl, %2, 6;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
        "add.u32 al, %1, 1024;\n\tadd.u32 bl, %2, 1024;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
        "add.u32 al, %1, 1026;\n\tadd.u32 bl, %2, 1026;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
        "add.u32 al, %1, 1028;\n\tadd.u32 bl, %2, 1028;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
        "add.u32 al, %1, 1030;\n\tadd.u32 bl, %2, 1030;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
        "}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc)
        : "memory");
}
// The same for a head dimension of 64: four k = 16 steps inside the one 64-column panel.
__device__ __forceinline__ void tc_qk4(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc)
{
    asm volatile(
        "{\n\t"
        ".reg .pred pf, pt;\n\t.reg .b64 da, db;\n\t.reg .b32 al, bl;\n\t"
        "setp.ne.b32 pf, %0, %0;\n\tsetp.eq.b32 pt, %0, %0;\n\t"
        "add.u32 al, %1, 0;\n\tadd.u32 bl, %2, 0;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pf;\n\t"
        "add.u32 al, %1, 2;\n\tadd.u32 bl, %2, 2;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
        "add.u32 al, %1, 4;\n\tadd.u32 bl, %2, 4;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
        "add.u32 al, %1, 6;\n\tadd.u32 bl, %2, 6;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
        "}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc)
        : "memory");
}
// Half of one O += P.V tile: four k = 16 steps (64 keys).  p_tmem is the TMEM address of the
// first P column of the half, b_lo the low descriptor word of the first V row block of the half;
// `acc` = 0 makes the first step overwrite O.
__device__ __forceinline__ void tc_pv4(uint32_t d_tmem, uint32_t p_tmem, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                       uint32_t acc)
{
    asm volatile(
        "{\n\t"
        ".reg .pred pa, pt;\n\t.reg .b64 db;\n\t.reg .b32 al, bl;\n\t"
        "setp.ne.b32 pa, %5, 0;\n\tsetp.eq.b32 pt, %0, %0;\n\t"
        "add.u32 al, %1, 0;\n\tadd.u32 bl, %2, 0;\n\tmov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [al], db, %4, pa;\n\t"
        "add.u32 al, %1, 8;\n\tadd.u32 bl, %2, 128;\n\tmov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [al], db, %4, pt;\n\t"
        "add.u32 al, %1, 16;\n\tadd.u32 bl, %2, 256;\n\tmov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [al], db, %4, pt;\n\t"
        "add.u32 al, %1, 24;\n\tadd.u32 bl, %2, 384;\n\tmov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [al], db, %4, pt;\n\t"
        "}" ::"r"(d_tmem), "r"(p_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc)
        : "memory");
}
// Instruction descriptor for kind::f16: bf16 x bf16 -> fp32, M = 128, N = n (128 keys for S, the head dimension for O).
__host__ __device__ constexpr uint32_t tc_idesc(bool b_mn_major, uint32_t n = 128u)
{
    return (1u << 4)                      // D format: F32
           | (1u << 7)                    // A format: BF16
           | (1u << 10)                   // B format: BF16
           | ((b_mn_major ? 1u : 0u) << 16)
           | ((n >> 3) << 17)             // N
           | ((128u >> 4) << 24);         // M
}

// Probabilities of columns [LO, HI) of one score row: p = 2^(s*scale - m), packed to bf16 pairs,
// with two running partial sums.
#ifndef VXL_TC_SPEC
#define VXL_TC_SPEC 32
#endif
constexpr int kTcSpec = VXL_TC_SPEC;                      // columns exponentiated ahead of the row max
template <int LO, int HI>
__device__ __forceinline__ void tc_exp_block(const float (&s)[128], uint32_t (&pk)[64], float scale_log2, float neg_m,
                                             float &sum0, float &sum1)
{
#pragma unroll
    for (int i = LO; i < HI; i += 2) {
        const float p0 = fast_exp2(fmaf(s[i], scale_log2, neg_m));
        const float p1 = fast_exp2(fmaf(s[i + 1], scale_log2, neg_m));
        sum0 += p0;
        sum1 += p1;
        pk[i >> 1] = pack_bf16(p0, p1);
    }
}

// ------------------------------------------------------------------ work order
// (chunk, pair) entries sorted by number of key tiles, longest first, so that the tail of the
// grid is made of short items.  Rank sort in one CTA; n <= kTcMaxOrder.
// Key tiles of entry (block c, pair pr) that vary with the entry: retained tiles + window tiles
// before the pair (S = rows per block, L = window length; S == L for plain chunks).
__device__ __forceinline__ int tc_entry_cost(int c, int pr, int R, int S, int L)
{
    const int ws = max(0, (c + 1) * S - L);
    return ((ws / S) * R + 127) / 128 + (c * S - ws) / 128 + 2 * pr;
}
__global__ void __launch_bounds__(1024) prefill_tc_order_kernel(int2 *order, int c0, int Cn, int pairs, int R, int S, int L)
{
    __shared__ int s_cost[kTcMaxOrder];
    const int n = Cn * pairs;                             // blocks c0 .. c0 + Cn - 1
    for (int e = threadIdx.x; e < n; e += blockDim.x) s_cost[e] = tc_entry_cost(c0 + e / pairs, e % pairs, R, S, L);
    __syncthreads();
    for (int e = threadIdx.x; e < n; e += blockDim.x) {
        const int cost = s_cost[e];
        int rank = 0;
#pragma unroll 8
        for (int e2 = 0; e2 < n; ++e2) {
            const int cost2 = s_cost[e2];
            rank += (cost2 > cost || (cost2 == cost && e2 < e)) ? 1 : 0;
        }
        order[rank] = make_int2(c0 + e / pairs, e % pairs);
    }
}

// Work item of the persistent kernel: (chunk, pair of query tiles, sequence, head).
struct TcItem {
    int c, pr, b, h, kvh;     // c = block of S rows after the prefix (a chunk in the plain form)
    int n_r, n_ret, n;        // retained rows visible, tiles of them, key tiles of query tile 1
    int n_pre;                // prefix tiles (after the retained tiles, before the window tiles)
    int win_row0;             // first row of the window, sequence-relative
    int row_base, q_row0;
};

// Items are numbered in cost order (longest first); CTA x of G takes item k*G + x on even
// rounds k and k*G + (G-1-x) on odd rounds, so every CTA gets a like mix of long and short ones.
__device__ __forceinline__ bool tc_item(const PrefillParams &p, const int2 *__restrict__ order, int pairs, int k, TcItem &it)
{
    const int G = (int)gridDim.x, x = (int)blockIdx.x;
    // 32-bit arithmetic on purpose (the host refuses shapes with 2^31 items or more): a 64-bit
    // division here is a called routine, and its presence alone slowed the main loops by a tenth.
    const int total = p.Cn * pairs * p.B * p.Hq;
    if (k > (total - 1) / G) return false;
    const int id = k * G + ((k & 1) ? (G - 1 - x) : x);
    if (id >= total) return false;
    const int BH = p.B * p.Hq;
    const int cp = id / BH, bh = id % BH;
    it.b = bh / p.Hq; it.h = bh % p.Hq;
    if (order != nullptr) { const int2 o = order[cp]; it.c = o.x; it.pr = o.y; }
    else { it.c = p.c0 + p.Cn - 1 - cp / pairs; it.pr = pairs - 1 - cp % pairs; }
    it.kvh = it.h / p.G;
    const int ws = max(0, (it.c + 1) * p.S - p.L);         // window start, in tokens after the prefix
    it.n_r = (ws / p.S) * p.R;                              // blocks wholly before the window
    it.n_ret = (it.n_r + 127) >> 7;
    it.n_pre = (p.P0 + 127) >> 7;
    it.n = it.n_ret + it.n_pre + (it.c * p.S - ws) / 128 + 2 * it.pr + 2;
    it.row_base = it.b * p.T;
    it.win_row0 = p.P0 + ws;
    it.q_row0 = p.P0 + it.c * p.S + it.pr * 256;
    return true;
}

template <int D>
__global__ void __launch_bounds__(kTcThreads, 1)
prefill_tc_kernel(const __grid_constant__ TcMaps maps, const PrefillParams p, const int2 *__restrict__ order, const int pairs,
                  const int tma_out)
{
    extern __shared__ unsigned char smem_dyn[];
    const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char *smem_gen = smem_dyn + (smem_base - smem_u32(smem_dyn));
    const uint32_t bar_base = smem_base + kTcSmemBar;
    volatile uint32_t *s_tmem = reinterpret_cast<volatile uint32_t *>(smem_gen + kTcSmemBar + kBarCount * 8);
    volatile int *s_abort = reinterpret_cast<volatile int *>(smem_gen + kTcSmemBar + kBarCount * 8 + 4);
    auto bar = [&](int i) { return bar_base + 8u * (uint32_t)i; };

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    if (tid == 0) {
        for (int i = 0; i < kBarCount; ++i) {
            const bool four = (i >= kBarP && i < kBarP + 4) || (i >= kBarOFree && i < kBarOFree + 2);
            mbar_init(bar(i), four ? 4u : 1u);
        }
        *s_abort = 0;
        mbar_fence_init();
    }
    if (warp == 8) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void *)s_tmem)),
                     "r"(512u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *s_tmem;

    // Register hand-over (per warpgroup): the softmax threads hold a 128-entry score row plus the
    // packed probabilities; the issuer and producer need little.  Each role executes its own
    // setmaxnreg so that the compiler sees one limit per branch.
    if (warp >= 10) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 88;" ::: "memory");     // idle
    } else if (warp == 9) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 88;" ::: "memory");
        // =============================================================== TMA producer
        // K/V tiles travel in units that share one full / empty barrier pair: unit 0 of an item is K_0
        // alone, unit u >= 1 is V_{u-1} together with K_u (the last unit has no K).  A unit occupies one
        // 64 KB pair slot: V in its first half, K in its second.  Fewer barriers for the issuer to poll.
        int un = 0;                                      // units issued so far (all items)
        int q_loads = 0;
        bool ok = true;
        const bool gather4 = (p.gather4 != 0);
        TcItem w, wn;
        bool have = tc_item(p, order, pairs, 0, w);
        for (int k = 0; ok && have; ++k) {
            const bool have_next = tc_item(p, order, pairs, k + 1, wn);
            // Q of this item: its shared memory is free once the last S = Q.K^T of the previous item is done
            if (k > 0 && (!mbar_wait(bar(kBarQFree), (k - 1) & 1) || *s_abort)) { ok = false; break; }
            if (lane == 0) {
                mbar_expect_tx(bar(kBarQ), 2 * kTcTileLoad<D>);
#pragma unroll
                for (int t = 0; t < 2; ++t)
#pragma unroll
                    for (int pn = 0; pn < D / 64; ++pn)
                        tma_load_2d(smem_base + kTcSmemQ + t * kTcTileBytes + pn * kTcPanelBytes, &maps.q,
                                    w.h * D + pn * 64, w.row_base + w.q_row0 + t * 128, bar(kBarQ));
            }
            ++q_loads;
            const int pk_row0 = w.b * p.C * p.R;         // this sequence's rows in the packed sparse level
            // one K (kv = 0) or V (kv = 1) tile of key tile j into dst, completion on fb
            auto load_tile = [&](int kv, int j, uint32_t dst, uint32_t fb) {
                if (gather4 && j < w.n_ret) {
                    // rows past the end of the list repeat the last valid row; their columns are masked
                    const int e = j * 128 + lane * 4;
                    const int y0 = w.row_base + p.ridx[min(e + 0, w.n_r - 1)], y1 = w.row_base + p.ridx[min(e + 1, w.n_r - 1)];
                    const int y2 = w.row_base + p.ridx[min(e + 2, w.n_r - 1)], y3 = w.row_base + p.ridx[min(e + 3, w.n_r - 1)];
                    const CUtensorMap *m = kv ? &maps.vg : &maps.kg;
                    tma_gather4(dst + lane * 512, m, w.kvh * D, y0, y1, y2, y3, fb);
                    if (D == 128) tma_gather4(dst + kTcPanelBytes + lane * 512, m, w.kvh * D + 64, y0, y1, y2, y3, fb);
                } else if (lane == 0) {
                    // retained tiles come from the packed sparse level (rows past this chunk's
                    // prefix belong to later chunks or are out of range: masked / zero filled)
                    const bool ret = j < w.n_ret;
                    const CUtensorMap *m = ret ? (kv ? &maps.vg : &maps.kg) : (kv ? &maps.v : &maps.k);
                    const int jp = j - w.n_ret;                  // prefix tiles first, then the window
                    const int y = ret ? pk_row0 + j * 128
                                      : (jp < w.n_pre ? w.row_base + jp * 128 : w.row_base + w.win_row0 + (jp - w.n_pre) * 128);
                    tma_load_2d(dst, m, w.kvh * D, y, fb);
                    if (D == 128) tma_load_2d(dst + kTcPanelBytes, m, w.kvh * D + 64, y, fb);
                }
            };
            for (int u = 0; u <= w.n && ok; ++u, ++un) {
                const int slot = un % kTcPairs;
                const uint32_t ph = (un / kTcPairs) & 1;
                if (!mbar_wait(bar(kBarEmpty + slot), ph ^ 1) || *s_abort) { ok = false; break; }
                const uint32_t dst = smem_base + kTcSmemKV + slot * 2 * kTcTileBytes;
                const bool has_v = (u > 0), has_k = (u < w.n);
                if (lane == 0) mbar_expect_tx(bar(kBarFull + slot), (has_v && has_k) ? 2 * kTcTileLoad<D> : kTcTileLoad<D>);
                __syncwarp();
                if (has_v) load_tile(1, u - 1, dst, bar(kBarFull + slot));
                if (has_k) load_tile(0, u, dst + kTcTileBytes, bar(kBarFull + slot));
            }
            w = wn;
            have = have_next;
        }
        if (!ok && lane == 0) { raise_status(p.hdr, VXL_ERR_TIMEOUT, 200); *s_abort = 1; }
        // Do not retire while copies into this CTA's shared memory may still be in flight.
        for (int s2 = 0; s2 < kTcPairs && s2 < un; ++s2) {
            const int i2 = un - 1 - s2;
            mbar_wait(bar(kBarFull + i2 % kTcPairs), (i2 / kTcPairs) & 1);
        }
        if (q_loads > 0) mbar_wait(bar(kBarQ), (q_loads - 1) & 1);
    } else if (warp == 8) {
        // =============================================================== MMA issuer
        asm volatile("setmaxnreg.dec.sync.aligned.u32 88;" ::: "memory");
        if (lane == 0) {
            constexpr uint32_t idesc_qk = tc_idesc(false, 128u), idesc_pv = tc_idesc(true, (uint32_t)D);
            constexpr uint32_t desc_hi = tc_desc_hi(1024);
            bool ok = true;
            int ub = 0;                                  // K/V units consumed before this item
            int pc0 = 0, pc1 = 0;                        // P tiles consumed per query tile (all items)
            auto issue_qk = [&](int t, uint32_t ka) {
                if (D == 128)
                    tc_qk8(tmem + t * 128, tc_desc_lo(smem_base + kTcSmemQ + t * kTcTileBytes, 16), tc_desc_lo(ka, 16), desc_hi, idesc_qk);
                else
                    tc_qk4(tmem + t * 128, tc_desc_lo(smem_base + kTcSmemQ + t * kTcTileBytes, 16), tc_desc_lo(ka, 16), desc_hi, idesc_qk);
            };
            // P.V in two halves of 64 keys: the first runs while the softmax still works on the second
            auto issue_pv = [&](int t, uint32_t va, bool acc, int pc) -> bool {
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    if (!mbar_wait(bar((half ? kBarP2 : kBarP) + t), pc & 1)) return false;
                    tc_fence_after();
                    tc_pv4(tmem + 256 + t * 128, tmem + t * 128 + half * 32, tc_desc_lo(va + half * 8192, kTcPanelBytes),
                           desc_hi, idesc_pv, (acc || half) ? 1u : 0u);
                }
                return true;
            };
            auto wait_full = [&](int u) { return mbar_wait(bar(kBarFull + u % kTcPairs), (u / kTcPairs) & 1); };
            auto unit_base = [&](int u) { return smem_base + kTcSmemKV + (uint32_t)(u % kTcPairs) * 2 * kTcTileBytes; };
            // the next item's descriptor is worked out while this one runs (see the softmax warps)
            TcItem w, wn;
            bool have = tc_item(p, order, pairs, 0, w);
            for (int k = 0; ok && have; ++k) {
                const int n = w.n;
                const bool have_next = tc_item(p, order, pairs, k + 1, wn);
                if (!(ok = mbar_wait(bar(kBarQ), k & 1))) break;
                if (!(ok = wait_full(ub))) break;
                tc_fence_after();
                // S of the new item may be written at once: the P.V products of the previous item
                // that read the same columns precede these MMAs in the pipe.
                issue_qk(0, unit_base(ub) + kTcTileBytes); tc_commit(bar(kBarS + 0));
                issue_qk(1, unit_base(ub) + kTcTileBytes); tc_commit(bar(kBarS + 1));
                tc_commit(bar(kBarEmpty + ub % kTcPairs));
                for (int j = 0; j < n && ok; ++j) {
                    const int u = ub + 1 + j;            // unit: V_j in the first half, K_{j+1} in the second
                    const uint32_t va = unit_base(u), ka = va + kTcTileBytes;
                    const bool has_next = (j + 1 < n);
                    if (!(ok = wait_full(u))) break;
                    if (j < n - 1) {
                        // the first P.V of an item overwrites O: the previous item's O must have been read out
                        if (j == 0 && k > 0 && !(ok = mbar_wait(bar(kBarOFree + 0), (k - 1) & 1))) break;
                        if (!(ok = issue_pv(0, va, j > 0, pc0))) break;
                        ++pc0;
                        if (j + 1 < n - 1) {
                            issue_qk(0, ka); tc_commit(bar(kBarS + 0));
                        } else {
                            tc_commit(bar(kBarO + 0));              // tile 0 has seen its last key tile
                        }
                    }
                    if (j == 0 && k > 0 && !(ok = mbar_wait(bar(kBarOFree + 1), (k - 1) & 1))) break;
                    if (!(ok = issue_pv(1, va, j > 0, pc1))) break;
                    ++pc1;
                    if (has_next) {
                        issue_qk(1, ka); tc_commit(bar(kBarS + 1));
                        if (j == n - 2) tc_commit(bar(kBarQFree));  // last use of this item's Q
                    } else {
                        tc_commit(bar(kBarO + 1));
                    }
                    tc_commit(bar(kBarEmpty + u % kTcPairs));
                }
                ub += n + 1;
                w = wn;
                have = have_next;
            }
            if (!ok) { raise_status(p.hdr, VXL_ERR_TIMEOUT, 201); *s_abort = 1; }
        }
    } else {
        // =============================================================== softmax / epilogue
        asm volatile("setmaxnreg.inc.sync.aligned.u32 208;" ::: "memory");
        const int t = warp >> 2;                        // query tile
        const int row = (warp & 3) * 32 + lane;         // row within the tile = TMEM lane
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + lane_addr + t * 128;
        const uint32_t tO = tmem + lane_addr + 256 + t * 128;
        const uint32_t stage = smem_base + kTcSmemStage + warp * 4096;   // 32 rows x 128 B, private to the warp
        bool ok = true;
        int sc = 0;                                     // S tiles consumed (all items)
        float s[128];
        // The descriptor of the next item (integer divisions and a load from the ranking table) is worked
        // out at the start of the current one, off the path between two items.
        TcItem w, wn;
        bool have = tc_item(p, order, pairs, 0, w);
        for (int k = 0; ok && have; ++k) {
            const bool have_next = tc_item(p, order, pairs, k + 1, wn);
            const int nj = w.n - 1 + t;
            const int diag = w.n - 2 + t;                   // this tile's diagonal key tile
            const int tail_valid = w.n_r - (w.n_ret - 1) * 128;   // valid columns of the last gathered tile
            const int pre_last = w.n_ret + w.n_pre - 1;     // last prefix tile: rows past the prefix are masked
            const int pre_valid = p.P0 - (w.n_pre - 1) * 128;
            float m_run = -INFINITY, l_run = 0.f;
            for (int j = 0; j < nj; ++j, ++sc) {
                if (!mbar_wait(bar(kBarS + t), sc & 1) || *s_abort) { ok = false; break; }
                tc_fence_after();
                tc_ld32(tS + 0, s + 0);
                tc_ld32(tS + 32, s + 32);
                tc_ld32(tS + 64, s + 64);
                tc_ld32(tS + 96, s + 96);
                tc_wait_ld();
                if (j == diag) {
#pragma unroll
                    for (int i = 0; i < 128; ++i) s[i] = (i > row) ? -INFINITY : s[i];
                } else if (j == w.n_ret - 1 && tail_valid < 128) {
#pragma unroll
                    for (int i = 0; i < 128; ++i) s[i] = (i >= tail_valid) ? -INFINITY : s[i];
                } else if (j == pre_last && w.n_pre > 0 && pre_valid < 128) {
#pragma unroll
                    for (int i = 0; i < 128; ++i) s[i] = (i >= pre_valid) ? -INFINITY : s[i];
                }
                // The first kTcSpec probabilities are computed against the running max of the previous
                // tiles while the row max of this tile is still being reduced: the max is then off the
                // critical path (it moves rarely after the first tiles); a row whose max does move
                // recomputes that block.
                uint32_t pk[64];
                float sp0 = 0.f, sp1 = 0.f;
                tc_exp_block<0, kTcSpec>(s, pk, p.scale_log2, -m_run, sp0, sp1);
                float mx0 = s[0], mx1 = s[1], mx2 = s[2], mx3 = s[3];
#pragma unroll
                for (int i = 4; i < 128; i += 4) {
                    mx0 = fmaxf(mx0, s[i]); mx1 = fmaxf(mx1, s[i + 1]);
                    mx2 = fmaxf(mx2, s[i + 2]); mx3 = fmaxf(mx3, s[i + 3]);
                }
                const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * p.scale_log2;
                // Lazy rescale: keep the running max unless the new one exceeds it by more than the
                // threshold, so O is rarely touched after the first tiles.
                const bool grow = !((mx - m_run) <= kTcRescaleThreshold);   // also true on the first tile (m_run = -inf)
                if (__any_sync(0xffffffffu, grow)) {
                    float alpha = 1.f;
                    if (grow) {
                        alpha = fast_exp2(m_run - mx);      // 0 on the first tile
                        m_run = mx;
                        l_run *= alpha;
                        sp0 = 0.f; sp1 = 0.f;
                        tc_exp_block<0, kTcSpec>(s, pk, p.scale_log2, -m_run, sp0, sp1);
                    }
                    if (j > 0) {
                        // PV of tile j-1 has completed (S_j was committed after it), so O is stable.
                        float o[32];
#pragma unroll 1
                        for (int cb = 0; cb < D / 32; ++cb) {
                            tc_ld32(tO + cb * 32, o);
                            tc_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] *= alpha;
                            tc_st32(tO + cb * 32, reinterpret_cast<const uint32_t *>(o));
                        }
                    }
                }
                const float neg_m = -m_run;
                float sum0 = 0.f, sum1 = 0.f;
                // keys 0-63 are handed to the tensor pipe before keys 64-127 are exponentiated
                auto publish = [&](int half) {
                    tc_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar((half ? kBarP2 : kBarP) + t));
                };
                tc_exp_block<kTcSpec, 64>(s, pk, p.scale_log2, neg_m, sum0, sum1);
                tc_st32(tS + 0, pk);
                tc_exp_block<64, 80>(s, pk, p.scale_log2, neg_m, sum0, sum1);
                publish(0);
                tc_exp_block<80, 128>(s, pk, p.scale_log2, neg_m, sum0, sum1);
                l_run += (sum0 + sum1) + (sp0 + sp1);
                tc_st32(tS + 32, pk + 32);
                publish(1);
            }
            if (!ok) break;
            // ---- epilogue of the item: O / l -> global, 32 columns at a time through a swizzled
            // staging block, so that a store instruction writes four rows of 128 contiguous bytes
            if (!mbar_wait(bar(kBarO + t), k & 1) || *s_abort) { ok = false; break; }
            tc_fence_after();
            const float inv = 1.f / l_run;
            const int tok0 = w.q_row0 + t * 128 + (warp & 3) * 32;            // first token of this warp's rows
            const int vrows = p.S - (w.pr * 256 + t * 128 + (warp & 3) * 32);  // rows of this warp inside the block (may be <= 0 or >= 32)
            const int64_t obase = (int64_t)w.b * p.o_sb + (int64_t)w.h * p.o_sh;
            // element offsets of the rows this lane stores (row i*4 + lane/8, 16-byte piece lane%8), once per item
            int64_t erow[8];
#pragma unroll
            for (int i = 0; i < 8; ++i)
                erow[i] = obase + (int64_t)(tok0 + i * 4 + (lane >> 3)) * p.o_st + (lane & 7) * 4;
            // all of O into the registers of the dead score row at once: one load latency instead of
            // four, and the tensor memory is handed back before the stores start
            tc_ld32(tO + 0, s + 0);
            tc_ld32(tO + 32, s + 32);
            if (D == 128) {
                tc_ld32(tO + 64, s + 64);
                tc_ld32(tO + 96, s + 96);
            }
            tc_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarOFree + t));
            // Whole boxes of 32 rows leave as TMA stores from the staging block (the swizzle is the TMA's own
            // 128-byte pattern); a warp whose rows end inside the box (ragged last tile pair) or an output
            // layout without a tensor map stores row pieces itself.
            const bool box_store = tma_out != 0 && vrows >= 32;
            if (box_store && p.out_bf16) {
                // bf16 output: a box is 32 rows x 64 columns (128 bytes a row, the same swizzle), two per warp
#pragma unroll
                for (int cb = 0; cb < D / 64; ++cb) {
                    if (lane == 0) tma_store_wait_read();
                    __syncwarp();
#pragma unroll
                    for (int c8 = 0; c8 < 8; ++c8) {
                        const uint32_t a = stage + lane * 128 + ((c8 ^ (lane & 7)) << 4);
                        const float *sv = s + cb * 64 + 8 * c8;
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(pack_bf16(sv[0] * inv, sv[1] * inv)),
                                     "r"(pack_bf16(sv[2] * inv, sv[3] * inv)), "r"(pack_bf16(sv[4] * inv, sv[5] * inv)),
                                     "r"(pack_bf16(sv[6] * inv, sv[7] * inv))
                                     : "memory");
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) tma_store_2d(&maps.o, w.h * D + cb * 64, w.row_base + tok0, stage);
                }
            } else
#pragma unroll
            for (int cb = 0; cb < D / 32; ++cb) {
                if (tma_out != 0) {
                    if (lane == 0) tma_store_wait_read();             // the previous box has left the staging block
                    __syncwarp();
                }
#pragma unroll
                for (int c8 = 0; c8 < 8; ++c8) {
                    const uint32_t a = stage + lane * 128 + ((c8 ^ (lane & 7)) << 4);
                    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(a), "f"(s[cb * 32 + 4 * c8] * inv),
                                 "f"(s[cb * 32 + 4 * c8 + 1] * inv), "f"(s[cb * 32 + 4 * c8 + 2] * inv),
                                 "f"(s[cb * 32 + 4 * c8 + 3] * inv)
                                 : "memory");
                }
                if (box_store) {
                    fence_proxy_async_smem();                         // generic-proxy writes -> visible to the TMA
                    __syncwarp();
                    if (lane == 0) tma_store_2d(&maps.o, w.h * D + cb * 32, w.row_base + tok0, stage);
                    continue;
                }
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = i * 4 + (lane >> 3), c8 = lane & 7;
                    float4 v;
                    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                                 : "r"(stage + r * 128 + ((c8 ^ (r & 7)) << 4)));
                    const int64_t e = erow[i] + cb * 32;
                    if (r >= vrows) continue;                             // a row of the next chunk: not ours to write
                    if (p.out_bf16)
                        *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(p.out) + e) =
                            make_uint2(pack_bf16(v.x, v.y), pack_bf16(v.z, v.w));
                    else
                        *reinterpret_cast<float4 *>(reinterpret_cast<float *>(p.out) + e) = v;
                }
                __syncwarp();
            }
            if (p.lse != nullptr && lane < vrows)
                p.lse[((int64_t)w.b * p.T + tok0 + lane) * p.Hq + w.h] = (m_run + log2f(l_run)) * kLn2;
            w = wn;
            have = have_next;
        }
        if (!ok && lane == 0) { raise_status(p.hdr, VXL_ERR_TIMEOUT, 202); *s_abort = 1; }
        if (tma_out != 0 && lane == 0) tma_store_wait_all();          // no store may outlive the CTA's shared memory
    }

    // ---- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 8) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

// ------------------------------------------------------------------ host side
// Workspace after the header: [order table][packed retained K][packed retained V].
inline size_t prefill_tc_order_bytes() { return (size_t)kTcMaxOrder * sizeof(int2); }
inline size_t prefill_tc_packed_bytes(const vxl_shape *s, int C, int R)
{
    const size_t b = (size_t)s->B * C * R * s->Hkv * s->D * sizeof(__nv_bfloat16);
    return (b + 255) & ~(size_t)255;
}
inline size_t prefill_tc_workspace_bytes(const vxl_shape *s, int C, int R)
{
    return prefill_tc_order_bytes() + 2 * prefill_tc_packed_bytes(s, C, R);
}

inline bool prefill_tc_supported(const vxl_shape *s, int L, int R)
{
    (void)R;
    const int step = s->prefill_step > 0 ? s->prefill_step : L;
    if (s->D != 128 && s->D != 64) return false;
    if (step == L) {
        // Plain chunks of any length from 256 rows: the last pair of query tiles may reach past the chunk.
        // Its surplus rows are computed on whatever follows (the next chunk's rows, zero fill past the
        // array) and never stored; for the rows that count, every key past the chunk is also past the
        // diagonal.  A call over a range of chunks must read nothing after the range, so there the
        // chunk has to end on a key-tile boundary.
        if ((s->block_begin > 0 || s->block_count > 0) && L % 128 != 0) return false;
    } else {
        // Sliding window: the key tiles are laid from the window start, the query tiles from the block
        // start; the two grids must coincide for every block, the first ones included, whose window
        // is cut off at the start of the sequence: every block starts a whole number of tiles in.
        if (step % 128 != 0) return false;
    }
    if (s->q_stride_h != s->D || s->kv_stride_h != s->D) return false;
    if (s->B > 1 && (s->q_stride_b != (int64_t)s->T * s->q_stride_t || s->kv_stride_b != (int64_t)s->T * s->kv_stride_t))
        return false;
    if ((int64_t)s->B * s->T >= (1ll << 31)) return false;
    if ((int64_t)s->B * s->Hq * ((int64_t)s->T / 256 + s->T / step + 1) >= (1ll << 31)) return false;
    return true;
}

typedef CUresult (*tc_encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                 const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline tc_encode_fn tc_get_encode()
{
    static tc_encode_fn fn = nullptr;
    if (fn == nullptr) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<tc_encode_fn>(sym);
    }
    return fn;
}

// 2-D bf16 view [rows, width] with a row pitch in elements; box = 64 columns x box_rows.
inline bool tc_make_map(CUtensorMap *m, const void *base, uint64_t width, uint64_t rows, uint64_t pitch_elems,
                        uint32_t box_rows)
{
    tc_encode_fn enc = tc_get_encode();
    if (enc == nullptr) return false;
    const cuuint64_t dims[2] = {width, rows};
    const cuuint64_t strides[1] = {pitch_elems * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// ks/vs: packed sparse level [B*C*R, Hkv, 128] (built by the caller of this function with
// pack_retained_kernel), or null when p.gather4 selects TMA gather4 straight from K/V.
template <int D>
inline vxl_status prefill_tc_launch_d(const PrefillParams &p, void *order_ws, const void *ks, const void *vs,
                                      cudaStream_t st)
{
    TcMaps maps;
    const uint64_t rows = (uint64_t)p.B * p.T;
    const uint64_t prow = (uint64_t)p.B * p.C * p.R;
    const bool need_sparse = p.R > 0 && p.C > 1;
    if (!tc_make_map(&maps.q, p.q, (uint64_t)p.Hq * D, rows, (uint64_t)p.q_st, 128) ||
        !tc_make_map(&maps.k, p.k, (uint64_t)p.Hkv * D, rows, (uint64_t)p.kv_st, 128) ||
        !tc_make_map(&maps.v, p.v, (uint64_t)p.Hkv * D, rows, (uint64_t)p.kv_st, 128))
        return VXL_ERR_CUDA;
    if (p.gather4 || !need_sparse) {
        if (!tc_make_map(&maps.kg, p.k, (uint64_t)p.Hkv * D, rows, (uint64_t)p.kv_st, 1) ||
            !tc_make_map(&maps.vg, p.v, (uint64_t)p.Hkv * D, rows, (uint64_t)p.kv_st, 1))
            return VXL_ERR_CUDA;
    } else {
        if (!tc_make_map(&maps.kg, ks, (uint64_t)p.Hkv * D, prow, (uint64_t)p.Hkv * D, 128) ||
            !tc_make_map(&maps.vg, vs, (uint64_t)p.Hkv * D, prow, (uint64_t)p.Hkv * D, 128))
            return VXL_ERR_CUDA;
    }
    // output with heads side by side and sequences back to back: boxes leave by TMA store
    int tma_out = 0;
    const int o_esz = p.out_bf16 ? 2 : 4;
    if (p.o_sh == D && (p.B == 1 || p.o_sb == (int64_t)p.T * p.o_st) &&
        (reinterpret_cast<uintptr_t>(p.out) & 15u) == 0 && (p.o_st * o_esz) % 16 == 0) {
        tc_encode_fn enc = tc_get_encode();
        const cuuint64_t dims[2] = {(cuuint64_t)p.Hq * D, rows};
        const cuuint64_t strides[1] = {(cuuint64_t)p.o_st * o_esz};
        const cuuint32_t box[2] = {p.out_bf16 ? 64u : 32u, 32};      // 128 bytes a row either way
        const cuuint32_t estr[2] = {1, 1};
        if (enc != nullptr &&
            enc(&maps.o, p.out_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, p.out, dims, strides,
                box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS)
            tma_out = 1;
    }
    if (!tma_out) std::memset(&maps.o, 0, sizeof maps.o);
    static bool smem_done[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return VXL_ERR_CUDA;
    if (!smem_done[dev]) {
        if (cudaFuncSetAttribute(prefill_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcSmemBytes) != cudaSuccess)
            return VXL_ERR_CUDA;
        smem_done[dev] = true;
    }
    const int pairs = (p.S + 255) / 256;
    const int entries = p.Cn * pairs;
    int2 *order = nullptr;
    if (entries <= kTcMaxOrder) {
        order = static_cast<int2 *>(order_ws);
        prefill_tc_order_kernel<<<1, 1024, 0, st>>>(order, p.c0, p.Cn, pairs, p.R, p.S, p.L);
        if (cudaGetLastError() != cudaSuccess) return VXL_ERR_CUDA;
    }
    // persistent: one CTA per SM walks its share of the items
    static int sm_count[64] = {};
    if (sm_count[dev] == 0 &&
        (cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sm_count[dev] <= 0))
        sm_count[dev] = 148;
    const int64_t items = (int64_t)entries * p.B * p.Hq;
    const unsigned grid = (unsigned)(items < sm_count[dev] ? items : sm_count[dev]);
    prefill_tc_kernel<D><<<grid, kTcThreads, kTcSmemBytes, st>>>(maps, p, order, pairs, tma_out);
    return cudaGetLastError() == cudaSuccess ? VXL_OK : VXL_ERR_CUDA;
}

inline vxl_status prefill_tc_launch(const PrefillParams &p, int D, void *order_ws, const void *ks, const void *vs,
                                    cudaStream_t st)
{
    return D == 128 ? prefill_tc_launch_d<128>(p, order_ws, ks, vs, st) : prefill_tc_launch_d<64>(p, order_ws, ks, vs, st);
}

}  // namespace vxl
