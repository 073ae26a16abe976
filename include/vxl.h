/*
 * vxl — chunk-structured sparse attention for task-aware KV sparsification (Video-XL-2),
 * C ABI of the CUDA (sm_100a) library.
 *
 * The calls follow the two steps of the paper's "Efficiency Optimization" subsection:
 *   - chunk-based pre-filling   -> vxl_chunk_prefill_attn
 *   - bi-level KV decoding      -> vxl_chunk_scores (relevance + top-k),
 *                                  vxl_bilevel_decode_attn (mixed dense/sparse attention),
 *                                  vxl_pack_retained (the sparse level stored on its own)
 *
 * Conventions shared by every call
 *   Pointers   q/k/v/out/lse/scores/indices/workspace are DEVICE pointers owned by the caller;
 *              `shape` and the returned strings are HOST memory.  Nothing is retained after
 *              the call returns except a small host-side cache of TMA descriptors.
 *   Layout     the head dimension D is contiguous; all other strides are given in elements in
 *              `vxl_shape`.  Data pointers must be 16-byte aligned, strides multiples of 8.
 *   Types      q, k, v are bf16.  `out` is fp32 (VXL_F32) or bf16 (VXL_BF16); lse / scores are
 *              fp32; indices and offsets are int32.
 *   Stream     `cuda_stream` is a cudaStream_t (NULL = legacy default stream).  Calls only
 *              enqueue work; they never synchronise, except vxl_device_status and
 *              vxl_bilevel_decode_offline (which needs the selection on the host).
 *              vxl_chunk_prefill_host takes HOST arrays beside the device ones (stated there).
 *   Workspace  caller-allocated scratch of at least vxl_workspace_bytes(...) bytes, 256-byte
 *              aligned, zero-filled once before its first use (cudaMemset).  Its first word is
 *              a sticky device status (0 = ok).  Calls that run concurrently on different
 *              streams need different workspaces.
 *   Errors     host-detectable problems return a code and launch nothing.  Problems seen on
 *              the device (bad index under `validate`, a bounded wait that ran out) set the
 *              status word; kernels then finish cleanly with unspecified output.  The library
 *              never aborts, throws or traps.
 *   Indices    retained_idx[c][r] is an ABSOLUTE token position inside chunk c, distinct within
 *              a row; any order is accepted.  Out-of-range entries are clamped or read as
 *              zero rows (never a fault) and are reported only when `validate` is set.
 */
#ifndef VXL_H_
#define VXL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    VXL_OK = 0,
    VXL_ERR_INVALID_ARG = 1,   /* null pointer, bad size, misalignment                       */
    VXL_ERR_UNSUPPORTED = 2,   /* legal but not built (e.g. D not in {64,128})               */
    VXL_ERR_INVALID_INDEX = 3, /* device-side: retained_idx / chunk_offsets / selected       */
    VXL_ERR_WORKSPACE = 4,     /* workspace missing, too small or misaligned                 */
    VXL_ERR_CUDA = 5,          /* a CUDA runtime / driver call failed                        */
    VXL_ERR_TIMEOUT = 6        /* device-side: a bounded barrier wait ran out                */
} vxl_status;

typedef enum { VXL_BF16 = 0, VXL_F32 = 1 } vxl_dtype;

/* Relevance score of a chunk (Bi-level KVs Decoding paragraph: the paper lists an attention-score
 * rule among several possible ones and gives no formula).
 * VXL_SCORE_LSE   mean over query heads of ln sum_{p in sparse(c)} exp(scale * q.k_p)   (default)
 * VXL_SCORE_MASS  mean over query heads of the share of the head's softmax over the whole sparse
 *                 level that falls on the chunk: exp(lse[h,c]) / sum_c' exp(lse[h,c'])
 * The mean of the logits over a chunk's rows is VXL_SCORE_LSE over a sparse level with one
 * pooled row per chunk (vxl_pool_sparse with R = 1). */
typedef enum { VXL_SCORE_LSE = 0, VXL_SCORE_MASS = 1 } vxl_score_mode;

typedef enum {
    VXL_OP_PREFILL = 0,
    VXL_OP_SCORES = 1,
    VXL_OP_DECODE = 2
} vxl_op;

/* Problem shape shared by all calls.  struct_size = sizeof(vxl_shape) (ABI growth). */
typedef struct vxl_shape {
    uint32_t struct_size;
    int32_t B;                 /* sequences                                                   */
    int32_t T;                 /* tokens per sequence (prefill: q and kv; decode: cache)      */
    int32_t Hq, Hkv;           /* query heads, kv heads; Hq % Hkv == 0; Hq/Hkv <= 16          */
    int32_t D;                 /* head dim: 64 or 128                                         */
    int64_t q_stride_b, q_stride_t, q_stride_h;     /* elements; q_stride_t unused by decode  */
    int64_t kv_stride_b, kv_stride_t, kv_stride_h;  /* elements, same for k and v             */
    int64_t out_stride_b, out_stride_t, out_stride_h; /* elements of out dtype; 0 = contiguous */
    float scale;               /* softmax scale; <= 0 means 1/sqrt(D)                         */
    int32_t out_dtype;         /* vxl_dtype                                                   */
    int32_t validate;          /* 1: also run the index-validation kernel                     */
    int32_t force_general;     /* 1: prefill uses the general (mma.sync) kernel for any shape */
    int32_t prefill_gather4;   /* 1: tcgen05 prefill fetches retained rows with TMA gather4
                                  straight from k/v instead of packing them first (slower)    */
    int32_t prefill_step;      /* sliding chunk window: step in tokens (a divisor of chunk_len);
                                  0 or chunk_len = disjoint chunks                            */
    int32_t prefix_len;        /* prefill: the first prefix_len tokens (system prompt) are
                                  visible to every later token; 0 = none                      */
    int32_t block_begin;       /* prefill: compute only the rows of the chunks (step blocks, with a window)  */
    int32_t block_count;       /* [block_begin, block_begin + block_count); count 0 = from block_begin to the
                                  end.  Rows outside the range are neither read as queries nor written; keys
                                  and retained rows after the range are not read either, so a caller that
                                  receives its tokens chunk by chunk can run one call per chunk over the
                                  same buffers.  The prefix rows belong to the call whose range starts at 0 */
    int32_t score_mode;        /* vxl_score_mode, used by vxl_chunk_scores and by
                                  vxl_bilevel_decode_attn when it selects itself              */
} vxl_shape;

/* The sparse level stored on its own (Bi-level KVs Decoding paragraph: both levels of every
 * chunk are kept after prefill): k_sparse/v_sparse are [B, C*R, Hkv, D] bf16, contiguous, row c*R+r = the KV row
 * retained_idx[c][r].  Built by vxl_pack_retained.  Optional everywhere it appears. */
typedef struct vxl_sparse_level {
    const void *k_sparse;
    const void *v_sparse;
} vxl_sparse_level;

/* Bytes of workspace the given operation needs (0 on bad arguments).  C = number of chunks,
 * R = retained rows per chunk, topk = dense chunks per sequence and max_chunk_len = longest
 * chunk (both used by VXL_OP_DECODE only).  Host-only; launches nothing. */
size_t vxl_workspace_bytes(int32_t op, const vxl_shape *shape, int32_t C, int32_t R, int32_t topk,
                           int32_t max_chunk_len);

/*
 * Chunk-based pre-filling (paper: "Chunk-based Pre-filling" paragraph, Fig. 2).
 * Plain form (shape->prefill_step = 0, shape->prefix_len = 0).  For token i in chunk
 * c = i / chunk_len and query head h (kv head h / (Hq/Hkv)):
 *   keys(i) = { j : c*chunk_len <= j <= i }  U  retained_idx[c'] for all c' < c
 *   out[b,i,h,:] = softmax_j( scale * q[b,i,h].k[b,j,g] ) . v[b,j,g,:]
 *   lse[b,i,h]   = ln sum_j exp( scale * q.k )                (optional)
 * q [B,T,Hq,D], k/v [B,T,Hkv,D] by the strides in `shape`; retained_idx [C,R] int32, C =
 * T/chunk_len, shared by all sequences (row C-1 is never read); out [B,T,Hq,D]; lse [B,T,Hq]
 * contiguous, may be NULL.  Requires T % chunk_len == 0; R may be 0 (retained_idx may then be
 * NULL).  bf16 products, fp32 accumulation and softmax.
 *
 * Sliding chunk window and prefix (same paragraph and Fig. 2 right: the window advances by a
 * step smaller than its length, and the system prompt stays visible).  With S = shape->prefill_step (a divisor of
 * chunk_len) and P0 = shape->prefix_len, the tokens after the prefix form blocks of S; a window
 * of chunk_len tokens advances by S, and the tokens it covers for the first time see the rest of
 * it.  For i >= P0, u = (i - P0) / S, ws = max(0, (u+1)*S - chunk_len):
 *   keys(i) = { j < P0 }  U  { P0 + ws <= j <= i }  U  retained_idx[u'] for (u'+1)*S <= ws
 * and keys(i) = { j <= i } for a prefix token.  retained_idx is then [C,R] with
 * C = (T - P0) / S, row u' inside block u' (absolute positions).  Requires (T - P0) % S == 0.
 */
vxl_status vxl_chunk_prefill_attn(const void *q, const void *k, const void *v,
                                  int32_t chunk_len, const int32_t *retained_idx, int32_t R,
                                  void *out, float *lse, const vxl_shape *shape,
                                  void *workspace, size_t ws_bytes, void *cuda_stream);

/*
 * Chunk-based pre-filling of sequences whose tokens live in HOST memory (Chunk-based Pre-filling
 * paragraph: the long input is encoded one chunk after the other, each step touching only the
 * current chunk and the few retained KVs before it).  The call runs the chunks as a pipeline over
 * three streams: the rows of chunk group g travel host -> device on h2d_stream, group g is attended
 * on cuda_stream by vxl_chunk_prefill_attn restricted to its blocks (nothing after the group is
 * read), and its output rows travel device -> host on d2h_stream, so copies in both directions
 * overlap the kernels and each other.  One 2-D copy per tensor and group (its rows in every
 * sequence).  Same result as vxl_chunk_prefill_attn over the same data.
 *   q_host [B,T,Hq,D], k_host/v_host [B,T,Hkv,D] bf16, retained_idx_host [C,R] int32, out_host
 *   [B,T,Hq,D] of shape->out_dtype, lse_host [B,T,Hq] fp32 or NULL: HOST memory, contiguous; pin it
 *   (cudaHostAlloc / cudaHostRegister), or the copies will not overlap anything.
 *   q_dev, k_dev, v_dev, retained_idx_dev, out_dev, lse_dev (NULL iff lse_host is): DEVICE arrays of
 *   the same shapes, caller-owned, overwritten; they hold the sequence afterwards (k_dev/v_dev are
 *   the KV cache the decoding calls read).
 *   chunks_per_call: chunks per pipeline step (0 = 1).  The strides in `shape` must describe the
 *   contiguous layout; plain chunks only (no window, prefix or block range).
 * The three streams must differ.  On return everything is enqueued; work submitted to cuda_stream
 * afterwards is ordered after the last copy back, and the host arrays may be read once
 * cuda_stream (or d2h_stream) has been synchronised.  The library keeps a pool of CUDA events per
 * device for this call (created on first use, never during stream capture).
 */
vxl_status vxl_chunk_prefill_host(const void *q_host, const void *k_host, const void *v_host,
                                  int32_t chunk_len, const int32_t *retained_idx_host, int32_t R,
                                  void *out_host, float *lse_host,
                                  void *q_dev, void *k_dev, void *v_dev, int32_t *retained_idx_dev,
                                  void *out_dev, float *lse_dev, int32_t chunks_per_call,
                                  const vxl_shape *shape, void *workspace, size_t ws_bytes,
                                  void *cuda_stream, void *h2d_stream, void *d2h_stream);

/*
 * Per-chunk relevance and top-k selection (paper: "Bi-level KVs Decoding" paragraph: a
 * relevance score per chunk, dense KVs for the few most relevant chunks).  The paper
 * leaves the scoring rule open; this library implements the attention-score form on the
 * sparse level:
 *   scores[b,c] = (1/Hq) * sum_h  ln sum_{p in retained_idx[c]} exp( scale * q[b,h].k[b,p,g] )
 * and, if topk_idx != NULL, the `topk` chunks with the largest score per sequence (equal
 * scores: lower chunk id first), written as ascending chunk ids [B,topk].
 * q [B,Hq,D]; k_cache [B,T,Hkv,D]; chunk_offsets [C+1] increasing, off[0] = 0, off[C] <= T;
 * retained_idx [C,R] (ridx_stride_b = 0) or [B,C,R] (ridx_stride_b = C*R); `sparse` may be
 * NULL (rows gathered from k_cache by index) or a packed sparse level; scores [B,C] fp32.
 */
vxl_status vxl_chunk_scores(const void *q, const void *k_cache,
                            const int32_t *chunk_offsets, int32_t C,
                            const int32_t *retained_idx, int32_t R, int64_t ridx_stride_b,
                            const vxl_sparse_level *sparse,
                            float *scores, int32_t topk, int32_t *topk_idx,
                            const vxl_shape *shape, void *workspace, size_t ws_bytes,
                            void *cuda_stream);

/*
 * Relevance for a query of several tokens (Bi-level KVs Decoding paragraph: chunks are scored
 * against the text of the task query; how the tokens' scores are pooled is not stated).  This call takes
 * the arithmetic mean over the n_query_tokens tokens and the query heads of the same
 * log-sum-exp as vxl_chunk_scores:
 *   scores[b,c] = 1/(Tq*Hq) * sum_t sum_h ln sum_{p in sparse(c)} exp( scale * q[b,t,h].k[b,p,g] )
 * q [B,Tq,Hq,D] with token stride shape->q_stride_t (elements); everything else as for
 * vxl_chunk_scores (one sparse-level pass over the keys per token).
 */
vxl_status vxl_chunk_scores_multi(const void *q, int32_t n_query_tokens, const void *k_cache,
                                  const int32_t *chunk_offsets, int32_t C,
                                  const int32_t *retained_idx, int32_t R, int64_t ridx_stride_b,
                                  const vxl_sparse_level *sparse,
                                  float *scores, int32_t topk, int32_t *topk_idx,
                                  const vxl_shape *shape, void *workspace, size_t ws_bytes,
                                  void *cuda_stream);

/*
 * Selection from relevance scores computed elsewhere (Bi-level KVs Decoding paragraph: the scorer
 * is left open, e.g. an embedding model or a pipeline of the user's own): the `topk` chunks
 * with the largest score per sequence, equal scores going to the lower chunk id, written as
 * ascending chunk ids.  scores [B,C] fp32 and topk_idx [B,topk] int32 are device memory; the
 * result can be passed as `selected` to vxl_bilevel_decode_attn.  C <= 4096.
 */
vxl_status vxl_topk_select(const float *scores, int32_t B, int32_t C, int32_t topk,
                           int32_t *topk_idx, void *cuda_stream);

/*
 * vxl_chunk_scores for callers that cannot allocate device memory.  (The paper has no
 * counterpart to this call; it exists for deployment reasons only.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a plug-in inside a host
 * application that owns the whole device heap and hands out no scratch, a real-time loop
 * whose memory budget is frozen after start-up, or a stage that must not touch the allocator
 * because an allocation may synchronise the device or fail late.  Such a caller still owns
 * its inputs and outputs but has nowhere to put the (m, l) partials, flags and status word
 * that vxl_chunk_scores keeps in its workspace.  Here they live in a fixed array of
 * VXL_STATIC_SCRATCH_BYTES inside the library image; every GPU that loads the library holds
 * that array until the process exits.
 *
 * Same arguments and results as vxl_chunk_scores, minus the workspace, plus
 * device_status_out: optional DEVICE int32 that receives the device status word of this call
 * (0 = ok) in stream order, since there is no workspace to hand to vxl_device_status.
 *
 * Limits and rules
 *   - Problems whose scratch need, vxl_workspace_bytes(VXL_OP_SCORES, ...), exceeds
 *     VXL_STATIC_SCRATCH_BYTES are refused with VXL_ERR_WORKSPACE and nothing is launched
 *     (1 MiB covers B*Hq*C up to about 120,000, e.g. B = 8, Hq = 28, C = 512).
 *   - The call itself performs no cudaMalloc / cudaFree and calls no allocating library
 *     routine.  The first call on each device looks up the array's device address (with that
 *     device current); make that first call outside of any stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's contents.
 *     The call clears the status word itself; everything else is rewritten before it is read.
 *     Two calls that overlap on the GPU (different streams) race on the array: serialise them.
 */
#define VXL_STATIC_SCRATCH_BYTES (1u << 20)
vxl_status vxl_chunk_scores_static(const void *q, const void *k_cache,
                                   const int32_t *chunk_offsets, int32_t C,
                                   const int32_t *retained_idx, int32_t R, int64_t ridx_stride_b,
                                   const vxl_sparse_level *sparse,
                                   float *scores, int32_t topk, int32_t *topk_idx,
                                   int32_t *device_status_out,
                                   const vxl_shape *shape, void *cuda_stream);

/*
 * Bi-level KV decoding attention (paper: "Bi-level KVs Decoding" paragraph, Fig. 3): one
 * query token per sequence attends over the mixed KV set = all rows
 * [off[c], off[c+1]) of the selected chunks plus the rows retained_idx[c] of every other
 * chunk (a chunk is read at one level only):
 *   out[b,h,:] = softmax over that set of scale * q[b,h].k  applied to v ;  lse[b,h] optional.
 * `selected` [B,topk] chunk ids (any order) chooses the dense chunks; NULL makes the call
 * score the chunks and pick the top-k itself (same rule as vxl_chunk_scores), in which case
 * scores_out [B,C] and topk_out [B,topk] receive them when non-NULL.  topk may be 0..C.
 * max_chunk_len must bound every selected chunk: it sizes the launch and the workspace; a selected
 * chunk that is longer is cut off there and sets the status word to VXL_ERR_INVALID_ARG.
 * out [B,Hq,D] (out strides of `shape`, out_stride_t unused).
 */
vxl_status vxl_bilevel_decode_attn(const void *q, const void *k_cache, const void *v_cache,
                                   const int32_t *chunk_offsets, int32_t C, int32_t max_chunk_len,
                                   const int32_t *retained_idx, int32_t R, int64_t ridx_stride_b,
                                   const vxl_sparse_level *sparse,
                                   int32_t topk, const int32_t *selected,
                                   void *out, float *lse, float *scores_out, int32_t *topk_out,
                                   const vxl_shape *shape, void *workspace, size_t ws_bytes,
                                   void *cuda_stream);

/*
 * Bi-level KV decoding with the dense level kept off the device (Bi-level KVs Decoding paragraph:
 * both levels are parked in memory outside the accelerator and reloaded per query, dense KVs for
 * the relevant chunks, sparse KVs for the rest).  Here the sparse level
 * lives on the device and the dense cache in pinned host memory; one call
 *   1. scores the chunks on the sparse level and picks the top-k (as vxl_chunk_scores),
 *   2. brings the selection to the host -- THIS CALL SYNCHRONISES cuda_stream at that point --
 *   3. copies the dense rows of the selected chunks host -> device into staging slots on
 *      copy_stream (one cudaMemcpyAsync per chunk and per K / V),
 *   4. runs the sparse pass of the other chunks on cuda_stream while the copies run, then the
 *      dense pass over the staging slots and the combine.
 * The result is that of vxl_bilevel_decode_attn over the same data.
 *   k_host, v_host      pinned HOST memory, [B,T,Hkv,D] bf16 by shape->kv_stride_b, with
 *                       kv_stride_t = Hkv*D and kv_stride_h = D (whole token rows are copied)
 *   chunk_offsets       [C+1] on the device, chunk_offsets_host the same values on the host
 *   sparse, R           stored sparse level on the device (required), R rows per chunk
 *   k_stage, v_stage    device, [B, topk, max_chunk_len, Hkv, D] bf16, contents overwritten
 *   topk_host           pinned HOST memory, [B,topk] int32, receives the selection
 *   scores_out [B,C], topk_out [B,topk]   device, both required
 * Workspace as for vxl_bilevel_decode_attn.  The call keeps one CUDA event per device.
 */
vxl_status vxl_bilevel_decode_offline(const void *q, const void *k_host, const void *v_host,
                                      const int32_t *chunk_offsets, const int32_t *chunk_offsets_host,
                                      int32_t C, int32_t max_chunk_len,
                                      const vxl_sparse_level *sparse, int32_t R, int32_t topk,
                                      void *k_stage, void *v_stage, int32_t *topk_host,
                                      void *out, float *lse, float *scores_out, int32_t *topk_out,
                                      const vxl_shape *shape, void *workspace, size_t ws_bytes,
                                      void *cuda_stream, void *copy_stream);

/*
 * Retained-index layout in HBM (paper: the sparse KVs are obtained per chunk from the dense
 * ones and both levels are stored): copies the rows named by retained_idx out of the dense
 * cache into a contiguous sparse level, k_sparse/v_sparse [B, C*R, Hkv, D] bf16.
 */
vxl_status vxl_pack_retained(const void *k_cache, const void *v_cache,
                             const int32_t *retained_idx, int32_t C, int32_t R,
                             int64_t ridx_stride_b, void *k_sparse, void *v_sparse,
                             const vxl_shape *shape, void *cuda_stream);

/*
 * Sparse level by pooling (Bi-level KVs Decoding paragraph: each chunk's sparse KVs come from a
 * pooling step over its dense ones).  The paper does not name the pooling; this
 * call averages: pooled row r of chunk c is the mean of the dense rows
 * [off[c] + r*len/R, off[c] + (r+1)*len/R) (integer division, len = off[c+1] - off[c]; an empty
 * window gives a zero row), summed and divided in fp64 and rounded once to bf16.
 * k_cache/v_cache [B,T,Hkv,D]; chunk_offsets [C+1] (device); k_sparse/v_sparse [B, C*R, Hkv, D]
 * bf16, contiguous: a vxl_sparse_level for vxl_chunk_scores / vxl_bilevel_decode_attn, which
 * then read R pooled rows for a chunk that is not selected (retained_idx may be NULL there).
 */
vxl_status vxl_pool_sparse(const void *k_cache, const void *v_cache,
                           const int32_t *chunk_offsets, int32_t C, int32_t R,
                           void *k_sparse, void *v_sparse,
                           const vxl_shape *shape, void *cuda_stream);

/* Synchronises `cuda_stream`, reads the workspace status word and clears it.  Returns VXL_OK,
 * the device-side error recorded since the last clear, or VXL_ERR_CUDA. */
vxl_status vxl_device_status(void *workspace, void *cuda_stream);

/* Self-test of the failure path every kernel of this library shares (the paper has no counterpart).  All
 * device-side waits are bounded: when one runs out, the kernel records VXL_ERR_TIMEOUT in the workspace's
 * status word and returns, and the context stays usable.  This call launches one warp that waits, with that
 * same bounded wait and a limit of limit_cycles SM clocks (1 .. 200,000,000), on a barrier that nothing
 * completes; vxl_device_status(workspace) must then report VXL_ERR_TIMEOUT, and the next call on the same
 * workspace must work.  workspace: at least 256 bytes, 256-byte aligned, device memory. */
vxl_status vxl_selftest_bounded_wait(void *workspace, int64_t limit_cycles, void *cuda_stream);

/* Static, NUL-terminated description of a status code (host memory, never freed). */
const char *vxl_status_str(vxl_status s);

/* Which prefill kernel the shape would use: 1 = tcgen05/TMA kernel, 0 = general kernel,
 * -1 = invalid.  Host-only; launches nothing.  The tcgen05 kernel takes D = 64 or 128 with head
 * stride D, sequences laid out back to back, and either plain chunks (any length; a multiple of 128
 * when the call covers a range of chunks) or a sliding window whose prefill_step is a multiple of
 * 128.  Chunks shorter than 256 rows run there too, with the unused rows of their tile pair
 * computed and dropped. */
int32_t vxl_prefill_kernel_kind(const vxl_shape *shape, int32_t chunk_len, int32_t R);

#ifdef __cplusplus
}
#endif
#endif /* VXL_H_ */
