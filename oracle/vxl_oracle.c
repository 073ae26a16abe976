/*
 * fp64 CPU oracle for chunk-structured sparse attention (TEST INFRASTRUCTURE ONLY).
 *
 * This file is the plain definition of what the hot path computes, written for checking by
 * eye against the paper, not for speed.  It is used by the tests, by the smoke check and by
 * the CPU-baseline leg of the benchmark; the product path never calls it and shares no code
 * with it.
 *
 * What it follows (Efficiency Optimization subsection of the paper):
 *   - Chunk-based pre-filling paragraph and Fig. 2 (left): a token of chunk c attends to the
 *     tokens of its own chunk (causally, since the language model is decoder-only) and to the
 *     retained KVs (the KVs of the timestamp tokens met so far) of every preceding chunk.
 *   - Bi-level KVs decoding paragraph and Fig. 3: every chunk has a dense level (all its KVs)
 *     and a sparse level (a sub-sampled set of them); a relevance score is computed per chunk;
 *     the most relevant chunks are read dense, the others sparse; the rows read are
 *     concatenated into one mixed KV set over which the query attends.
 * Given the key set, the result is ordinary softmax attention, so each function below is that
 * definition written out: explicit mask row / explicit score table / explicit mixed row list,
 * softmax by max-subtraction, all sums in double.  Inputs are bf16 bit patterns widened
 * exactly to double.
 *
 * Readings where the paper is silent (relevance score = mean over query heads of the
 * log-sum-exp of the scaled logits over the chunk's sparse keys; ties in top-k go to the lower
 * chunk index) are stated at the functions that use them.
 *
 * Parity pins: every function here is pinned by tests that compare it with textbook dense /
 * causal attention, closed forms, a hand-computed fixture and an independent brute-force twin.
 * The choice of the score formula itself is a reading of the paper, not a printed fact.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_f64(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int vxl_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Softmax attention of one query vector over an explicit list of key rows.
 *   qrow  : D bf16 values
 *   k, v  : [T, Hkv, D] bf16, kv head g
 *   rows  : n token positions (the key set, any order)
 * Writes out[D] and *lse = m + ln(sum exp(x - m)).  n == 0 gives out = 0, lse = -inf.
 */
static void attend_rows(const uint16_t *qrow, const uint16_t *k, const uint16_t *v,
                        int Hkv, int D, int g, const int32_t *rows, int64_t n, double scale,
                        double *logit_buf, double *out, double *lse)
{
    double m = -INFINITY;
    for (int64_t a = 0; a < n; ++a) {
        const uint16_t *krow = k + ((int64_t)rows[a] * Hkv + g) * D;
        double dot = 0.0;
        for (int d = 0; d < D; ++d) dot += bf16_to_f64(qrow[d]) * bf16_to_f64(krow[d]);
        logit_buf[a] = scale * dot;
        if (logit_buf[a] > m) m = logit_buf[a];
    }
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    if (n == 0) { *lse = -INFINITY; return; }
    double l = 0.0;
    for (int64_t a = 0; a < n; ++a) {
        double p = exp(logit_buf[a] - m);
        l += p;
        const uint16_t *vrow = v + ((int64_t)rows[a] * Hkv + g) * D;
        for (int d = 0; d < D; ++d) out[d] += p * bf16_to_f64(vrow[d]);
    }
    for (int d = 0; d < D; ++d) out[d] /= l;
    *lse = m + log(l);
}

/*
 * Chunk-based pre-filling (paragraph "Chunk-based Pre-filling", Fig. 2 left).
 *
 * For each requested token i (chunk c = i / L) the allowed-key mask row M[i, 0..T) is built
 * explicitly:  M[i, j] = 1 for c*L <= j <= i, and M[i, p] = 1 for every p in
 * retained_idx[c'] with c' < c.  Then out[i, h] = softmax(scale * q[i,h].K[M])V[M] with kv
 * head g = h / (Hq/Hkv).
 *
 *   q [T,Hq,D], k/v [T,Hkv,D] bf16 bits; retained_idx [C,R] absolute positions
 *   rows[n_rows] token indices to compute (NULL = all T tokens, n_rows ignored)
 *   out [n_rows,Hq,D], lse [n_rows,Hq] doubles
 * Returns 0, or -1 on bad arguments / allocation failure.
 */
int vxl_oracle_prefill(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                       int T, int Hq, int Hkv, int D, int L,
                       const int32_t *retained_idx, int R, double scale,
                       const int32_t *rows, int64_t n_rows, double *out, double *lse)
{
    if (T <= 0 || L <= 0 || T % L || Hkv <= 0 || Hq % Hkv || R < 0) return -1;
    const int G = Hq / Hkv;
    const int64_t n = rows ? n_rows : T;
    int fail = 0;
#pragma omp parallel
    {
        uint8_t *mask = (uint8_t *)malloc((size_t)T);
        int32_t *list = (int32_t *)malloc(sizeof(int32_t) * (size_t)T);
        double *buf = (double *)malloc(sizeof(double) * (size_t)T);
        if (!mask || !list || !buf) {
#pragma omp atomic write
            fail = 1;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (int64_t a = 0; a < n; ++a) {
                const int i = rows ? rows[a] : (int)a;
                const int c = i / L;
                memset(mask, 0, (size_t)T);
                for (int j = c * L; j <= i; ++j) mask[j] = 1;
                for (int cp = 0; cp < c; ++cp)
                    for (int r = 0; r < R; ++r) mask[retained_idx[(int64_t)cp * R + r]] = 1;
                int64_t cnt = 0;
                for (int j = 0; j < T; ++j)
                    if (mask[j]) list[cnt++] = j;
                for (int h = 0; h < Hq; ++h) {
                    const uint16_t *qrow = q + ((int64_t)i * Hq + h) * D;
                    attend_rows(qrow, k, v, Hkv, D, h / G, list, cnt, scale, buf,
                                out + ((int64_t)a * Hq + h) * D, lse + (int64_t)a * Hq + h);
                }
            }
        }
        free(mask); free(list); free(buf);
    }
    return fail ? -1 : 0;
}

/*
 * Chunk-based pre-filling with a sliding chunk window and an always-visible prefix (Chunk-based
 * Pre-filling paragraph and Fig. 2 right: besides itself and the earlier timestamp tokens, the
 * current chunk sees the system prompt, and because the window moves by a step shorter than the
 * window it also sees the dense tokens of the part of the previous chunk that it overlaps).
 *
 * Reading (the paper gives no formula): the first P0 tokens are the prefix.  The other tokens are
 * cut into step blocks of S tokens.  A window of L tokens (L a multiple of S) slides by S; the
 * tokens a window covers for the first time are the ones computed in it, and they see the rest
 * of that window densely.  So for token i >= P0, with iv = i - P0, u = iv / S and window start
 * ws = max(0, (u + 1) * S - L) (both in visual coordinates):
 *   M[i, j] = 1  for j < P0                                   (prefix)
 *   M[i, j] = 1  for P0 + ws <= j <= i                        (own window, causal)
 *   M[i, p] = 1  for p in retained_idx[u'] with (u' + 1) * S <= ws   (blocks wholly before the window)
 * and for a prefix token i < P0: M[i, j] = 1 for j <= i.
 * retained_idx [Cs, R] holds absolute token positions (prefix included), row u' inside block u',
 * Cs = (T - P0) / S.  S == L and P0 == 0 is the plain chunked form above.
 */
int vxl_oracle_prefill_window(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                              int T, int Hq, int Hkv, int D, int L, int S, int P0,
                              const int32_t *retained_idx, int R, double scale,
                              const int32_t *rows, int64_t n_rows, double *out, double *lse)
{
    if (T <= 0 || L <= 0 || S <= 0 || L % S || P0 < 0 || P0 > T || (T - P0) % S || Hkv <= 0 || Hq % Hkv || R < 0)
        return -1;
    const int G = Hq / Hkv;
    const int64_t n = rows ? n_rows : T;
    int fail = 0;
#pragma omp parallel
    {
        uint8_t *mask = (uint8_t *)malloc((size_t)T);
        int32_t *list = (int32_t *)malloc(sizeof(int32_t) * (size_t)T);
        double *buf = (double *)malloc(sizeof(double) * (size_t)T);
        if (!mask || !list || !buf) {
#pragma omp atomic write
            fail = 1;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (int64_t a = 0; a < n; ++a) {
                const int i = rows ? rows[a] : (int)a;
                memset(mask, 0, (size_t)T);
                if (i < P0) {
                    for (int j = 0; j <= i; ++j) mask[j] = 1;
                } else {
                    const int u = (i - P0) / S;
                    const int ws = (u + 1) * S - L > 0 ? (u + 1) * S - L : 0;
                    for (int j = 0; j < P0; ++j) mask[j] = 1;
                    for (int j = P0 + ws; j <= i; ++j) mask[j] = 1;
                    for (int up = 0; (up + 1) * S <= ws; ++up)
                        for (int r = 0; r < R; ++r) mask[retained_idx[(int64_t)up * R + r]] = 1;
                }
                int64_t cnt = 0;
                for (int j = 0; j < T; ++j)
                    if (mask[j]) list[cnt++] = j;
                for (int h = 0; h < Hq; ++h) {
                    const uint16_t *qrow = q + ((int64_t)i * Hq + h) * D;
                    attend_rows(qrow, k, v, Hkv, D, h / G, list, cnt, scale, buf,
                                out + ((int64_t)a * Hq + h) * D, lse + (int64_t)a * Hq + h);
                }
            }
        }
        free(mask); free(list); free(buf);
    }
    return fail ? -1 : 0;
}

/*
 * Per-chunk relevance (Bi-level KVs Decoding paragraph: every video chunk gets a
 * relevance score for the query; the attention-score form is one of the options the paper lists and
 * the formula is this build's reading):
 *   lse_hc[h, c] = ln sum_{p in retained_idx[c]} exp(scale * q[h].k[p, g(h)])
 *   scores[c]    = (1/Hq) * sum_h lse_hc[h, c]
 * One sequence: q [Hq,D], k [T,Hkv,D]; retained_idx [C,R] absolute positions.
 * R == 0 gives -inf everywhere.
 */
int vxl_oracle_scores(const uint16_t *q, const uint16_t *k, int T, int Hq, int Hkv, int D,
                      int C, const int32_t *retained_idx, int R, double scale,
                      double *lse_hc, double *scores)
{
    if (Hkv <= 0 || Hq % Hkv || R < 0 || C < 0) return -1;
    (void)T;
    const int G = Hq / Hkv;
    double *x = (double *)malloc(sizeof(double) * (size_t)(R > 0 ? R : 1));
    if (!x) return -1;
    for (int h = 0; h < Hq; ++h) {
        const int g = h / G;
        for (int c = 0; c < C; ++c) {
            double m = -INFINITY;
            for (int r = 0; r < R; ++r) {
                const uint16_t *krow = k + ((int64_t)retained_idx[(int64_t)c * R + r] * Hkv + g) * D;
                double dot = 0.0;
                for (int d = 0; d < D; ++d)
                    dot += bf16_to_f64(q[(int64_t)h * D + d]) * bf16_to_f64(krow[d]);
                x[r] = scale * dot;
                if (x[r] > m) m = x[r];
            }
            double l = 0.0;
            for (int r = 0; r < R; ++r) l += exp(x[r] - m);
            lse_hc[(int64_t)h * C + c] = (R > 0) ? m + log(l) : -INFINITY;
        }
    }
    for (int c = 0; c < C; ++c) {
        double s = 0.0;
        for (int h = 0; h < Hq; ++h) s += lse_hc[(int64_t)h * C + c];
        scores[c] = s / Hq;
    }
    free(x);
    return 0;
}

/*
 * Top-k chunk selection (Bi-level KVs Decoding paragraph: the few most relevant chunks are read dense).
 * The k largest scores; equal scores go to the lower chunk index (a reading: the paper gives
 * no tie rule).  Selection by repeated arg-max so the rule is visible; output ascending chunk
 * ids.  *gap = (k-th largest) - ((k+1)-th largest), +inf if k == 0 or k == C.
 */
int vxl_oracle_topk(const double *scores, int C, int k, int32_t *idx_out, double *gap)
{
    if (k < 0 || k > C) return -1;
    uint8_t *taken = (uint8_t *)calloc((size_t)(C > 0 ? C : 1), 1);
    if (!taken) return -1;
    double kth = INFINITY, next = -INFINITY;
    for (int a = 0; a <= k && a < C; ++a) {
        int best = -1;
        for (int c = 0; c < C; ++c) {
            if (taken[c]) continue;
            if (best < 0 || scores[c] > scores[best]) best = c;   /* strict: lower index wins ties */
        }
        if (a < k) { taken[best] = 1; kth = scores[best]; }
        else next = scores[best];
    }
    int n = 0;
    for (int c = 0; c < C; ++c)
        if (taken[c]) idx_out[n++] = c;
    if (gap) *gap = (k == 0 || k == C) ? INFINITY : kth - next;
    free(taken);
    return 0;
}

/*
 * Mixed-KV decode attention (Bi-level KVs Decoding paragraph: dense KVs for the selected
 * chunks, sparse KVs for the others, joined into one mixed KV set that replaces the full cache).
 * The explicit row list is built chunk by chunk: all rows [off[c], off[c+1]) when c is in
 * `selected`, else the rows retained_idx[c].  A chunk is read at one level only.
 * One sequence: q [Hq,D], k/v [T,Hkv,D].  mixed_rows_out (nullable) receives the list,
 * capacity T; *n_mixed its length.
 */
int vxl_oracle_decode(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                      int T, int Hq, int Hkv, int D, int C, const int32_t *chunk_offsets,
                      const int32_t *retained_idx, int R,
                      const int32_t *selected, int n_selected, double scale,
                      double *out, double *lse, int32_t *mixed_rows_out, int64_t *n_mixed)
{
    if (Hkv <= 0 || Hq % Hkv || R < 0 || C < 0) return -1;
    const int G = Hq / Hkv;
    int32_t *list = (int32_t *)malloc(sizeof(int32_t) * (size_t)(T > 0 ? T : 1));
    uint8_t *is_sel = (uint8_t *)calloc((size_t)(C > 0 ? C : 1), 1);
    if (!list || !is_sel) { free(list); free(is_sel); return -1; }
    for (int a = 0; a < n_selected; ++a) {
        if (selected[a] < 0 || selected[a] >= C) { free(list); free(is_sel); return -1; }
        is_sel[selected[a]] = 1;
    }
    int64_t cnt = 0;
    for (int c = 0; c < C; ++c) {
        if (is_sel[c]) {
            for (int j = chunk_offsets[c]; j < chunk_offsets[c + 1]; ++j) list[cnt++] = j;
        } else {
            for (int r = 0; r < R; ++r) list[cnt++] = retained_idx[(int64_t)c * R + r];
        }
    }
    int fail = 0;
#pragma omp parallel
    {
        double *hbuf = (double *)malloc(sizeof(double) * (size_t)(cnt > 0 ? cnt : 1));
        if (!hbuf) {
#pragma omp atomic write
            fail = 1;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (int h = 0; h < Hq; ++h)
                attend_rows(q + (int64_t)h * D, k, v, Hkv, D, h / G, list, cnt, scale, hbuf,
                            out + (int64_t)h * D, lse + h);
        }
        free(hbuf);
    }
    if (fail) { free(list); free(is_sel); return -1; }
    if (mixed_rows_out) memcpy(mixed_rows_out, list, sizeof(int32_t) * (size_t)cnt);
    if (n_mixed) *n_mixed = cnt;
    free(list); free(is_sel);
    return 0;
}

/*
 * Sparse level by pooling (Bi-level KVs Decoding paragraph: the sparse KVs of a chunk are made by
 * pooling its dense KVs; the kind of pooling is not named).  Reading: average
 * pooling, R pooled rows per chunk; pooled row r of chunk c is the arithmetic mean of the dense
 * rows [lo + floor(r*len/R), lo + floor((r+1)*len/R)) with lo = chunk_offsets[c] and
 * len = chunk_offsets[c+1] - lo (equal windows of len/R rows when R divides len; an empty window
 * gives a zero row).  The mean is taken in double and stored as the nearest bf16 (ties to even),
 * because the sparse level is a KV cache of the same type as the dense one.
 *   x [T,Hkv,D] bf16 bits (K or V) -> pooled [C*R,Hkv,D] bf16 bits.
 */
static uint16_t f64_to_bf16_rne(double x)
{
    /* double -> float is exact enough here only if it does not double-round: round once, by hand */
    if (x == 0.0) return 0;
    if (isnan(x)) return 0x7fc0;
    if (isinf(x)) return x > 0 ? 0x7f80 : 0xff80;
    const int neg = x < 0;
    double a = fabs(x);
    int e;
    double m = frexp(a, &e);                 /* a = m * 2^e, 0.5 <= m < 1 */
    /* bf16 normal: 8 significant bits; value = (m * 256) * 2^(e - 8) */
    int bexp = e - 1 + 127;                  /* biased exponent of the leading bit */
    if (bexp <= 0) {                         /* subnormal range of bf16: fixed scale 2^-133 per unit */
        double q = nearbyint(ldexp(a, 133)); /* round to nearest even in the current (default) mode */
        uint16_t bits = (uint16_t)q;         /* may carry into the smallest normal: the encoding is continuous */
        return (uint16_t)(bits | (neg ? 0x8000 : 0));
    }
    double sig = nearbyint(ldexp(m, 8));     /* 128..256 */
    if (sig == 256.0) { sig = 128.0; ++bexp; }
    if (bexp >= 255) return (uint16_t)((neg ? 0x8000 : 0) | 0x7f80);
    return (uint16_t)((neg ? 0x8000 : 0) | (bexp << 7) | ((int)sig - 128));
}

int vxl_oracle_pool(const uint16_t *x, int T, int Hkv, int D, int C, const int32_t *chunk_offsets,
                    int R, uint16_t *pooled)
{
    if (T <= 0 || Hkv <= 0 || D <= 0 || C < 0 || R < 0) return -1;
    const int64_t W = (int64_t)Hkv * D;
    for (int c = 0; c < C; ++c) {
        const int lo = chunk_offsets[c], len = chunk_offsets[c + 1] - lo;
        if (lo < 0 || len < 0 || lo + len > T) return -1;
        for (int r = 0; r < R; ++r) {
            const int a = lo + (int)(((int64_t)r * len) / R), b = lo + (int)(((int64_t)(r + 1) * len) / R);
            for (int64_t e = 0; e < W; ++e) {
                double s = 0.0;
                for (int j = a; j < b; ++j) s += bf16_to_f64(x[(int64_t)j * W + e]);
                pooled[((int64_t)c * R + r) * W + e] = (b > a) ? f64_to_bf16_rne(s / (double)(b - a)) : 0;
            }
        }
    }
    return 0;
}

/*
 * Bi-level decoding with a sparse level stored on its own (pooled rows are not rows of the dense
 * cache): the mixed KV set is, chunk by chunk, all dense rows of a selected chunk or the R rows
 * c*R .. c*R+R-1 of the sparse level.  Written as an explicit row list over the concatenation
 * [dense rows 0..T) ; sparse rows T..T+C*R).
 *   k, v [T,Hkv,D]; ks, vs [C*R,Hkv,D] (bf16 bits); out [Hq,D], lse [Hq].
 */
int vxl_oracle_decode_levels(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                             const uint16_t *ks, const uint16_t *vs,
                             int T, int Hq, int Hkv, int D, int C, const int32_t *chunk_offsets, int R,
                             const int32_t *selected, int n_selected, double scale, double *out, double *lse)
{
    if (T <= 0 || Hkv <= 0 || Hq % Hkv || R < 0 || C < 0) return -1;
    const int G = Hq / Hkv;
    const int64_t W = (int64_t)Hkv * D, n_all = (int64_t)T + (int64_t)C * R;
    uint16_t *kc = (uint16_t *)malloc(sizeof(uint16_t) * (size_t)(n_all * W));
    uint16_t *vc = (uint16_t *)malloc(sizeof(uint16_t) * (size_t)(n_all * W));
    int32_t *list = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_all);
    uint8_t *is_sel = (uint8_t *)calloc((size_t)(C > 0 ? C : 1), 1);
    if (!kc || !vc || !list || !is_sel) { free(kc); free(vc); free(list); free(is_sel); return -1; }
    memcpy(kc, k, sizeof(uint16_t) * (size_t)((int64_t)T * W));
    memcpy(vc, v, sizeof(uint16_t) * (size_t)((int64_t)T * W));
    if (C * R > 0) {
        memcpy(kc + (int64_t)T * W, ks, sizeof(uint16_t) * (size_t)((int64_t)C * R * W));
        memcpy(vc + (int64_t)T * W, vs, sizeof(uint16_t) * (size_t)((int64_t)C * R * W));
    }
    int bad = 0;
    for (int a = 0; a < n_selected; ++a) {
        if (selected[a] < 0 || selected[a] >= C) bad = 1; else is_sel[selected[a]] = 1;
    }
    int64_t cnt = 0;
    for (int c = 0; c < C && !bad; ++c) {
        if (is_sel[c]) {
            for (int j = chunk_offsets[c]; j < chunk_offsets[c + 1]; ++j) list[cnt++] = j;
        } else {
            for (int r = 0; r < R; ++r) list[cnt++] = T + c * R + r;
        }
    }
    double *buf = (double *)malloc(sizeof(double) * (size_t)(cnt > 0 ? cnt : 1));
    if (!buf) bad = 1;
    for (int h = 0; h < Hq && !bad; ++h)
        attend_rows(q + (int64_t)h * D, kc, vc, Hkv, D, h / G, list, cnt, scale, buf, out + (int64_t)h * D, lse + h);
    free(kc); free(vc); free(list); free(is_sel); free(buf);
    return bad ? -1 : 0;
}

/*
 * Relevance for a query of several tokens (the paper scores chunks against the text of the task
 * query, i.e. more than one token; how token scores are pooled is not stated).  Reading: the
 * score of a chunk is the arithmetic mean, over the query tokens and the query heads, of the
 * same log-sum-exp as above.
 *   q [Tq,Hq,D]; scores [C].  Tq == 1 is vxl_oracle_scores.
 */
int vxl_oracle_scores_multi(const uint16_t *q, int Tq, const uint16_t *k, int T, int Hq, int Hkv, int D,
                            int C, const int32_t *retained_idx, int R, double scale, double *scores)
{
    if (Tq <= 0 || C < 0) return -1;
    double *lse_hc = (double *)malloc(sizeof(double) * (size_t)((int64_t)Hq * (C > 0 ? C : 1)));
    double *one = (double *)malloc(sizeof(double) * (size_t)(C > 0 ? C : 1));
    if (!lse_hc || !one) { free(lse_hc); free(one); return -1; }
    for (int c = 0; c < C; ++c) scores[c] = 0.0;
    int rc = 0;
    for (int t = 0; t < Tq && rc == 0; ++t) {
        rc = vxl_oracle_scores(q + (int64_t)t * Hq * D, k, T, Hq, Hkv, D, C, retained_idx, R, scale, lse_hc, one);
        for (int c = 0; c < C; ++c) scores[c] += one[c];
    }
    for (int c = 0; c < C; ++c) scores[c] /= Tq;
    free(lse_hc); free(one);
    return rc;
}

/*
 * Relevance as attention mass (another attention-score reading of the paper's
 * relevance oracle): the share of the query's softmax attention over the whole sparse level that
 * falls on the chunk's sparse rows, averaged over the query heads:
 *   mass[h, c] = sum_{p in sparse(c)} exp(x_hp) / sum_{all sparse p'} exp(x_hp')
 *              = exp( lse_hc[h, c] - ln sum_c' exp(lse_hc[h, c']) )
 *   scores[c]  = (1/Hq) * sum_h mass[h, c]                       (they sum to 1 over the chunks)
 * Same arguments as vxl_oracle_scores.
 */
int vxl_oracle_scores_mass(const uint16_t *q, const uint16_t *k, int T, int Hq, int Hkv, int D,
                           int C, const int32_t *retained_idx, int R, double scale, double *scores)
{
    if (C <= 0 || R <= 0) return -1;
    double *lse_hc = (double *)malloc(sizeof(double) * (size_t)((int64_t)Hq * C));
    double *tmp = (double *)malloc(sizeof(double) * (size_t)C);
    if (!lse_hc || !tmp) { free(lse_hc); free(tmp); return -1; }
    int rc = vxl_oracle_scores(q, k, T, Hq, Hkv, D, C, retained_idx, R, scale, lse_hc, tmp);
    for (int c = 0; c < C; ++c) scores[c] = 0.0;
    for (int h = 0; h < Hq && rc == 0; ++h) {
        double m = -INFINITY, l = 0.0;
        for (int c = 0; c < C; ++c) if (lse_hc[(int64_t)h * C + c] > m) m = lse_hc[(int64_t)h * C + c];
        for (int c = 0; c < C; ++c) l += exp(lse_hc[(int64_t)h * C + c] - m);
        for (int c = 0; c < C; ++c) scores[c] += exp(lse_hc[(int64_t)h * C + c] - m) / l;
    }
    for (int c = 0; c < C; ++c) scores[c] /= Hq;
    free(lse_hc); free(tmp);
    return rc;
}
