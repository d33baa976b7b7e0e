/*
 * qf_oracle.c -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, fp64 CPU statement of what the Q-First cache-side decode
 * path computes: softmax attention of one query per request over a set of
 * cached positions, returned as the mergeable pair (O, log Z), and the merge
 * of such pairs.  Only tests, the smoke check and the benchmark's CPU-baseline
 * leg may build, load or call this file.  It shares no code, header, table or
 * helper with the CUDA library and must never be reachable from it.
 *
 * Every function is the definition written out (two passes over the scores:
 * max, then sums).  There is no tiling, fusion or reordering; the only loop
 * parallelism is OpenMP over independent (request, head[, shard]) outputs,
 * which does not change any output's arithmetic.
 *
 * Pins (tests, CPU only): single key, identical keys, constant values,
 * sharded == unsharded, pairwise fold == n-way merge, overflow cases at
 * log Z = 100, shift invariance, d(out)/d(v_j) = A_j, paging invariance,
 * SciPy / PyTorch fp64 library routines, exact-rational brute force on tiny
 * inputs; the two "pick" entry points (selected outputs only) against the rows of
 * the full set, bit for bit, and against a NumPy statement of the definition.  The projection pair at the end of the file (u' = z + W_o a,
 * q = W_q N_1(u')) has its own pins: one-hot inputs that read out weight
 * columns, exact row sums under a constant stream, power-of-two equivariance,
 * PyTorch fp64 matmul and rms_norm, exact rational brute force, nearest-bf16
 * checks of every rounding.  Nothing here is "parity unpinned".
 *
 * Conventions where the paper is silent (stated again in the design notes):
 *   - q, K, V are bf16 bit patterns, widened exactly to fp64.
 *   - KV pool layout: element (page, kv_head, slot, d) at
 *     ((page*Hkv + kv_head)*page_size + slot)*D + d; logical token i of
 *     request b lives in page block_table[b*max_pages_per_req + i/page_size],
 *     slot i % page_size.  block_table == NULL means the identity table.
 *   - query head h reads kv head h / G, G = Hq / Hkv.
 *   - the sweep covers cached positions only: [0, seq_lens[b]).
 *   - natural logarithm; scale applied to the finished dot product.
 *   - an empty set gives log Z = m = -inf and O = 0.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct qfo_shape {
    int32_t batch;
    int32_t num_q_heads;
    int32_t num_kv_heads;
    int32_t head_dim;
    int32_t page_size;
    int32_t max_pages_per_req;
    int32_t max_shards;
    double  sm_scale; /* <= 0 means 1/sqrt(head_dim) */
} qfo_shape;

/* bf16 -> fp64, exact: a bf16 is the top 16 bits of an IEEE binary32. */
static double bf16_to_f64(uint16_t bits)
{
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static double scale_of(const qfo_shape *sh)
{
    return sh->sm_scale > 0.0 ? sh->sm_scale : 1.0 / sqrt((double)sh->head_dim);
}

/* Address of row (token i, kv head c) of request b in a paged pool. */
static const uint16_t *kv_row(const uint16_t *pool, const int32_t *block_table,
                              const qfo_shape *sh, int b, int c, int64_t i)
{
    int64_t lp = i / sh->page_size;
    int64_t slot = i % sh->page_size;
    int64_t phys = block_table
        ? (int64_t)block_table[(int64_t)b * sh->max_pages_per_req + lp]
        : (int64_t)b * sh->max_pages_per_req + lp;
    int64_t off = ((phys * sh->num_kv_heads + c) * sh->page_size + slot) * sh->head_dim;
    return pool + off;
}

int qfo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void qfo_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/*
 * One query head against the token set [beg, end) of request b (Section 5:
 * Z(S) = sum e^{s_i}, W(S) = sum e^{s_i} v_i, O(S) = W/Z; Section 2:
 * s = q.k/sqrt(d)).  The caller has already clamped the range.
 *
 *   o[D]      O(S) = W(S)/Z(S)                      (0 when S is empty)
 *   *m        max_i s_i                             (-inf when empty)
 *   *lse      log Z(S) = m + log sum_i e^{s_i - m}  (-inf when empty)
 *   w_rel[D]  optional: sum_i e^{s_i - m} v_i, the accumulator relative to m,
 *             so that o = w_rel / e^{lse - m}
 *   scores    optional: s_i for i in [beg, end), length end-beg
 */
void qfo_attend_range(const uint16_t *q, const uint16_t *k_cache, const uint16_t *v_cache,
                      const int32_t *block_table, const qfo_shape *sh,
                      int b, int h, int64_t beg, int64_t end,
                      double *o, double *m, double *lse, double *w_rel, double *scores)
{
    const int D = sh->head_dim;
    const int G = sh->num_q_heads / sh->num_kv_heads;
    const int c = h / G;
    const double scale = scale_of(sh);
    const int64_t n = end > beg ? end - beg : 0;

    for (int d = 0; d < D; ++d) o[d] = 0.0;
    if (w_rel) for (int d = 0; d < D; ++d) w_rel[d] = 0.0;
    if (n == 0) {
        *m = -INFINITY;
        *lse = -INFINITY;
        return;
    }

    double *qd = (double *)malloc(sizeof(double) * (size_t)D);
    double *s = scores ? scores : (double *)malloc(sizeof(double) * (size_t)n);
    const uint16_t *qrow = q + ((int64_t)b * sh->num_q_heads + h) * D;
    for (int d = 0; d < D; ++d) qd[d] = bf16_to_f64(qrow[d]);

    /* scores and their maximum */
    double mx = -INFINITY;
    for (int64_t i = 0; i < n; ++i) {
        const uint16_t *kr = kv_row(k_cache, block_table, sh, b, c, beg + i);
        double dot = 0.0;
        for (int d = 0; d < D; ++d) dot += qd[d] * bf16_to_f64(kr[d]);
        s[i] = dot * scale;
        if (s[i] > mx) mx = s[i];
    }

    /* Z and W relative to the maximum */
    double z = 0.0;
    double *w = (double *)calloc((size_t)D, sizeof(double));
    for (int64_t i = 0; i < n; ++i) {
        double e = exp(s[i] - mx);
        const uint16_t *vr = kv_row(v_cache, block_table, sh, b, c, beg + i);
        z += e;
        for (int d = 0; d < D; ++d) w[d] += e * bf16_to_f64(vr[d]);
    }

    for (int d = 0; d < D; ++d) o[d] = w[d] / z;
    if (w_rel) for (int d = 0; d < D; ++d) w_rel[d] = w[d];
    *m = mx;
    *lse = mx + log(z);

    free(w);
    free(qd);
    if (!scores) free(s);
}

static void clamp_range(int64_t beg, int64_t end, int64_t len, int64_t *b0, int64_t *e0)
{
    if (beg < 0) beg = 0;
    if (end > len) end = len;
    if (end < beg) end = beg;
    *b0 = beg;
    *e0 = end;
}

/*
 * Per-shard partial states: for every (b, s, h) the pair (O, log Z) of the
 * shard's token range [shard_ranges[b][s][0], shard_ranges[b][s][1]) clamped
 * to [0, seq_lens[b]], plus the running max m.
 *   o_part [B][S][Hq][D], m_part/lse_part [B][S][Hq]  (fp64)
 */
int qfo_decode_partial(const uint16_t *q, const uint16_t *k_cache, const uint16_t *v_cache,
                       const int32_t *block_table, const int32_t *seq_lens,
                       const int32_t *shard_ranges, const qfo_shape *sh,
                       double *o_part, double *m_part, double *lse_part)
{
    const int B = sh->batch, S = sh->max_shards, H = sh->num_q_heads, D = sh->head_dim;
    if (sh->num_q_heads % sh->num_kv_heads) return -1;
    const int64_t total = (int64_t)B * S * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t idx = 0; idx < total; ++idx) {
        int h = (int)(idx % H);
        int s = (int)((idx / H) % S);
        int b = (int)(idx / ((int64_t)H * S));
        int64_t beg, end;
        clamp_range(shard_ranges[((int64_t)b * S + s) * 2], shard_ranges[((int64_t)b * S + s) * 2 + 1],
                    seq_lens[b], &beg, &end);
        qfo_attend_range(q, k_cache, v_cache, block_table, sh, b, h, beg, end,
                         o_part + idx * D, m_part + idx, lse_part + idx, NULL, NULL);
    }
    return 0;
}

/*
 * The unsharded result: one sweep over [0, seq_lens[b]) for every (b, h).
 * If n_pick > 0 only the listed (b, h) pairs pick[2*i], pick[2*i+1] are
 * computed and written to out[i][D], lse[i]; otherwise all B*Hq in order.
 */
int qfo_decode_full(const uint16_t *q, const uint16_t *k_cache, const uint16_t *v_cache,
                    const int32_t *block_table, const int32_t *seq_lens, const qfo_shape *sh,
                    const int32_t *pick, int64_t n_pick, double *out, double *lse)
{
    const int H = sh->num_q_heads, D = sh->head_dim;
    if (sh->num_q_heads % sh->num_kv_heads) return -1;
    const int64_t total = n_pick > 0 ? n_pick : (int64_t)sh->batch * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t idx = 0; idx < total; ++idx) {
        int b = n_pick > 0 ? pick[2 * idx] : (int)(idx / H);
        int h = n_pick > 0 ? pick[2 * idx + 1] : (int)(idx % H);
        double mx;
        qfo_attend_range(q, k_cache, v_cache, block_table, sh, b, h, 0, seq_lens[b],
                         out + idx * D, &mx, lse + idx, NULL, NULL);
    }
    return 0;
}

/*
 * Partial states of selected (b, s, h) triples only (pick[3*i..3*i+2]), for
 * spot checks at sizes where the full set would take too long.
 */
int qfo_decode_partial_pick(const uint16_t *q, const uint16_t *k_cache, const uint16_t *v_cache,
                            const int32_t *block_table, const int32_t *seq_lens,
                            const int32_t *shard_ranges, const qfo_shape *sh,
                            const int32_t *pick, int64_t n_pick,
                            double *o_part, double *m_part, double *lse_part)
{
    const int S = sh->max_shards, D = sh->head_dim;
    if (sh->num_q_heads % sh->num_kv_heads) return -1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t idx = 0; idx < n_pick; ++idx) {
        int b = pick[3 * idx], s = pick[3 * idx + 1], h = pick[3 * idx + 2];
        int64_t beg, end;
        clamp_range(shard_ranges[((int64_t)b * S + s) * 2], shard_ranges[((int64_t)b * S + s) * 2 + 1],
                    seq_lens[b], &beg, &end);
        qfo_attend_range(q, k_cache, v_cache, block_table, sh, b, h, beg, end,
                         o_part + idx * D, m_part + idx, lse_part + idx, NULL, NULL);
    }
    return 0;
}

/*
 * n-way merge of shard states (Section 5 with the weights written relative
 * to the largest log Z, which is the n-way form of 1/(1+e^{-x})):
 *   M = max_s lse_s;  w_s = e^{lse_s - M};
 *   out = sum_s w_s O_s / sum_s w_s;  lse = M + log sum_s w_s.
 * A shard whose lse is -inf is skipped and its vector never read.  All
 * shards empty: out = 0, lse = -inf.  shard_counts == NULL means max_shards.
 *   o_part [B][S][Hq][D], lse_part [B][S][Hq]; out [B][Hq][D], lse [B][Hq].
 */
int qfo_combine(const double *o_part, const double *lse_part, const int32_t *shard_counts,
                const qfo_shape *sh, double *out, double *lse)
{
    const int B = sh->batch, S = sh->max_shards, H = sh->num_q_heads, D = sh->head_dim;
    for (int b = 0; b < B; ++b) {
        int ns = shard_counts ? shard_counts[b] : S;
        if (ns > S) ns = S;
        for (int h = 0; h < H; ++h) {
            double *o = out + ((int64_t)b * H + h) * D;
            double M = -INFINITY;
            for (int s = 0; s < ns; ++s) {
                double l = lse_part[((int64_t)b * S + s) * H + h];
                if (l > M) M = l;
            }
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            if (M == -INFINITY) {
                lse[(int64_t)b * H + h] = -INFINITY;
                continue;
            }
            double wsum = 0.0;
            for (int s = 0; s < ns; ++s) {
                double l = lse_part[((int64_t)b * S + s) * H + h];
                if (l == -INFINITY) continue;
                double w = exp(l - M);
                const double *os = o_part + (((int64_t)b * S + s) * H + h) * D;
                wsum += w;
                for (int d = 0; d < D; ++d) o[d] += w * os[d];
            }
            for (int d = 0; d < D; ++d) o[d] /= wsum;
            lse[(int64_t)b * H + h] = M + log(wsum);
        }
    }
    return 0;
}

/* sigma(x) = 1/(1+e^{-x}): the overflow-safe weight of Section 2. */
static double sigmoid(double x) { return 1.0 / (1.0 + exp(-x)); }

/* Stabilised log(e^a + e^b) for finite a, b. */
static double logaddexp(double a, double b)
{
    double hi = a > b ? a : b, lo = a > b ? b : a;
    return hi + log1p(exp(lo - hi));
}

/*
 * The paper's pairwise merge, folded left to right over the shards in the
 * order given by perm (NULL = 0,1,2,...):
 *   O(A u B)     = lerp(O(B), O(A), sigma(log Z(A) - log Z(B)))
 *   log Z(A u B) = logaddexp(log Z(A), log Z(B)),   lerp(x,y,t) = (1-t)x + ty
 * with an explicit skip of empty (-inf) operands.
 */
int qfo_combine_fold(const double *o_part, const double *lse_part, const int32_t *shard_counts,
                     const int32_t *perm, const qfo_shape *sh, double *out, double *lse)
{
    const int B = sh->batch, S = sh->max_shards, H = sh->num_q_heads, D = sh->head_dim;
    for (int b = 0; b < B; ++b) {
        int ns = shard_counts ? shard_counts[b] : S;
        if (ns > S) ns = S;
        for (int h = 0; h < H; ++h) {
            double *oa = out + ((int64_t)b * H + h) * D; /* state A */
            double la = -INFINITY;
            for (int d = 0; d < D; ++d) oa[d] = 0.0;
            for (int j = 0; j < ns; ++j) {
                int s = perm ? perm[j] : j;
                double lb = lse_part[((int64_t)b * S + s) * H + h];
                const double *ob = o_part + (((int64_t)b * S + s) * H + h) * D;
                if (lb == -INFINITY) continue;
                if (la == -INFINITY) {
                    for (int d = 0; d < D; ++d) oa[d] = ob[d];
                    la = lb;
                    continue;
                }
                double t = sigmoid(la - lb);
                for (int d = 0; d < D; ++d) oa[d] = (1.0 - t) * ob[d] + t * oa[d];
                la = logaddexp(la, lb);
            }
            lse[(int64_t)b * H + h] = la;
        }
    }
    return 0;
}

/*
 * The accelerator-side finish of a decode step (Section 2; the fold stated in
 * the appendix on the combine): the cached positions act as one pseudo-token
 * of score lse_prev and value o_prev, and the current token (k_new, v_new) is
 * appended to it:
 *     s_jj = q . k_new / sqrt(d)
 *     out  = lerp(v_new, o_prev, sigma(lse_prev - s_jj)),  lerp(x,y,t) = (1-t)x + ty
 *     lse  = logaddexp(lse_prev, s_jj)
 * with sigma(x) = 1/(1+e^{-x}).  An empty cache (lse_prev = -inf) gives out = v_new,
 * lse = s_jj.  Query head h uses the new key/value of KV head h / G.
 *   o_prev [B][Hq][D], lse_prev [B][Hq] (fp64); q [B][Hq][D], k_new/v_new [B][Hkv][D] (bf16 bits)
 *   out [B][Hq][D], lse [B][Hq], s_self [B][Hq] (optional)
 */
int qfo_self_fold(const double *o_prev, const double *lse_prev, const uint16_t *q, const uint16_t *k_new,
                  const uint16_t *v_new, const qfo_shape *sh, double *out, double *lse, double *s_self)
{
    const int B = sh->batch, H = sh->num_q_heads, D = sh->head_dim;
    if (sh->num_q_heads % sh->num_kv_heads) return -1;
    const int G = H / sh->num_kv_heads;
    const double scale = scale_of(sh);
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < H; ++h) {
            const int c = h / G;
            const uint16_t *qr = q + ((int64_t)b * H + h) * D;
            const uint16_t *kr = k_new + ((int64_t)b * sh->num_kv_heads + c) * D;
            const uint16_t *vr = v_new + ((int64_t)b * sh->num_kv_heads + c) * D;
            double dot = 0.0;
            for (int d = 0; d < D; ++d) dot += bf16_to_f64(qr[d]) * bf16_to_f64(kr[d]);
            const double sjj = dot * scale;
            const double lp = lse_prev[(int64_t)b * H + h];
            double *o = out + ((int64_t)b * H + h) * D;
            const double *op = o_prev + ((int64_t)b * H + h) * D;
            if (s_self) s_self[(int64_t)b * H + h] = sjj;
            if (lp == -INFINITY) {
                for (int d = 0; d < D; ++d) o[d] = bf16_to_f64(vr[d]);
                lse[(int64_t)b * H + h] = sjj;
                continue;
            }
            const double t = sigmoid(lp - sjj);
            for (int d = 0; d < D; ++d) o[d] = (1.0 - t) * bf16_to_f64(vr[d]) + t * op[d];
            lse[(int64_t)b * H + h] = logaddexp(lp, sjj);
        }
    }
    return 0;
}


/* ------------------------------------------------------------------------
 * The cache side's projection pair at a layer boundary (Section 4,
 * placement: W_q and W_o live with the cache; the stage's contract ends in
 * u' = z + W_o a, and the next stage opens with q = W_q N_1(u'); the appendix
 * paragraph on batching at the cache side makes it a product over the co-resident
 * requests of a batch).
 *
 * The paper fixes bf16 weights and a bf16 residual stream (its per-layer byte
 * counts) and leaves the rest open; the reading taken here, stated again in
 * the design notes:
 *   - a  [M][n_q]      fp32, the attention output of the layer (what the merge
 *                      returns), rounded to bf16 before the product;
 *   - z  [M][d_model]  bf16, the residual stream after the feed-forward;
 *   - w_o [d_model][n_q], w_q [n_q][d_model], g [d_model]  bf16;
 *   - N_1 is the root-mean-square normalisation with gain g:
 *         N_1(u)_i = g_i u_i / sqrt(mean_j u_j^2 + eps);
 *   - u' is rounded to bf16 (it is the stream that goes on the wire) and the
 *     normalisation reads the rounded stream; x = N_1(u') is rounded to bf16
 *     (it is the operand of the second product); q is rounded to bf16 (it is
 *     what the sweep consumes).
 * Every rounding is value -> nearest binary32 -> nearest bf16, ties to even,
 * the two steps a kernel with an fp32 accumulator takes; the sums themselves
 * are exact products of bf16 values accumulated in fp64.
 *   u_out [M][d_model], q_out [M][n_q]   bf16 bit patterns
 *   u_exact, q_exact (optional, fp64)    the values before their last rounding
 * ------------------------------------------------------------------------ */
static uint16_t f64_to_bf16_via_f32(double x)
{
    float f = (float)x; /* round to nearest even (default rounding mode) */
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40u); /* NaN stays NaN */
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

int qfo_project_pair(int32_t M, int32_t d_model, int32_t n_q, const float *a, const uint16_t *z,
                     const uint16_t *w_o, const uint16_t *g, double eps, const uint16_t *w_q,
                     uint16_t *u_out, uint16_t *q_out, double *u_exact, double *q_exact)
{
    if (M <= 0 || d_model <= 0 || n_q <= 0) return -1;
    double *ab = (double *)malloc(sizeof(double) * (size_t)M * (size_t)n_q);
    double *x = (double *)malloc(sizeof(double) * (size_t)M * (size_t)d_model);
    if (!ab || !x) { free(ab); free(x); return -2; }
    for (int64_t i = 0; i < (int64_t)M * n_q; ++i) ab[i] = bf16_to_f64(f64_to_bf16_via_f32((double)a[i]));

    /* u' = z + W_o a */
#pragma omp parallel for schedule(static)
    for (int64_t idx = 0; idx < (int64_t)M * d_model; ++idx) {
        const int64_t m = idx / d_model, o = idx % d_model;
        double acc = 0.0;
        for (int k = 0; k < n_q; ++k) acc += bf16_to_f64(w_o[o * (int64_t)n_q + k]) * ab[m * (int64_t)n_q + k];
        const double u = bf16_to_f64(z[idx]) + acc;
        if (u_exact) u_exact[idx] = u;
        u_out[idx] = f64_to_bf16_via_f32(u);
    }
    /* x = N_1(u') on the rounded stream */
    for (int m = 0; m < M; ++m) {
        double ss = 0.0;
        for (int i = 0; i < d_model; ++i) {
            const double u = bf16_to_f64(u_out[(int64_t)m * d_model + i]);
            ss += u * u;
        }
        const double rstd = 1.0 / sqrt(ss / (double)d_model + eps);
        for (int i = 0; i < d_model; ++i) {
            const double u = bf16_to_f64(u_out[(int64_t)m * d_model + i]);
            x[(int64_t)m * d_model + i] = bf16_to_f64(f64_to_bf16_via_f32(bf16_to_f64(g[i]) * u * rstd));
        }
    }
    /* q = W_q x */
#pragma omp parallel for schedule(static)
    for (int64_t idx = 0; idx < (int64_t)M * n_q; ++idx) {
        const int64_t m = idx / n_q, o = idx % n_q;
        double acc = 0.0;
        for (int k = 0; k < d_model; ++k) acc += bf16_to_f64(w_q[o * (int64_t)d_model + k]) * x[m * (int64_t)d_model + k];
        if (q_exact) q_exact[idx] = acc;
        q_out[idx] = f64_to_bf16_via_f32(acc);
    }
    free(ab);
    free(x);
    return 0;
}
