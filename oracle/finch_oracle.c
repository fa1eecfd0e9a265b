/*
 * finch_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, fp64 CPU statement of prompt-guided KV-cache compression
 * (Finch, arXiv 2408.00167, Section "Method"): score every candidate key by the
 * softmax attention the prompt's queries give it, keep the top-r candidates,
 * gather their K/V rows.  It exists so that the CUDA library can be checked
 * against something written directly from the paper.  It shares no code,
 * header, table or helper with the CUDA path; only tests, the smoke check and
 * the benchmark's CPU-baseline leg may load it.
 *
 * Every function follows the paper's own order of operations:
 *
 *   logits      s_{h,p,j} = scale * q_{h,p} . k_{kv(h),j}      (Background, the attention equation)
 *   softmax     A_{h,p,j} = exp(s_{h,p,j} - lse_{h,p}), over the candidate keys j
 *   sum heads   A^sum_{p,j} = sum_h A_{h,p,j}                  (Method, bullet "Sum over heads")
 *   submatrix   rows = prompt tokens, columns = cache then chunk (bullet "Extract prompt-guided submatrix");
 *               only this submatrix is ever formed here
 *   normalise   A^norm = A^cont * count(A^cont != 0) / (m + c) (bullet "Normalization"; optional, see flag)
 *   aggregate   A^agg_j = sum_p A^norm_{p,j}                   (bullet "Selection of top r position")
 *   top-r       t = top-r(A^agg, r)                            (same bullet)
 *   cache       keep K,V at the selected positions             (paragraph "Managing the Cache")
 *
 * Readings taken where the paper is silent: the softmax runs over the candidate
 * keys only (rows sum to 1) unless the caller supplies, per prompt row, the
 * log-sum-exp of the row's logits against the prompt's own keys -- in the full
 * forward pass a prompt row also attends to the prompt ("N = m + n^que + c",
 * Method, bullet "Extract prompt-guided submatrix"), and with that term the
 * denominator is the full row's; query rows may be given a visibility limit
 * (row i attends to the first limit[i] candidates only: the causal mask of
 * rows that are themselves document tokens, Method, the positional-bias
 * paragraph), and then the normalisation can be taken per row: a row's
 * weights times the fraction of the candidates it sees, which takes the
 * "score of 1" of a token that only sees itself down to 1/(m+c);
 * ties go to the lower candidate index; kept rows
 * are written in ascending candidate order (a flag gives the paper's rank order
 * of its worked example instead); a NaN score ranks below every number.
 *
 * Pins (tests/test_oracle_pins.py): closed forms (N=1, N=2 logistic, uniform
 * keys), row-sum and shift invariants, a numpy restatement, exact-Fraction
 * brute force over all subsets for the selection, the paper's worked cache
 * example.  Parity with the authors' own code is unpinned (not available).
 *
 * Tensors are dense and packed:
 *   q        [L][Hq ][total_q    ][d]   request b owns rows q_off[b]   .. q_off[b+1]
 *   cache_k  [L][Hkv][total_cache][d]   request b owns rows cache_off[b] .. +cache_len[b] (capacity to cache_off[b+1])
 *   chunk_k  [L][Hkv][total_chunk][d]   request b owns rows chunk_off[b] .. chunk_off[b+1]
 *   scores   [L][G][total_cache + total_chunk], request b at cache_off[b] + chunk_off[b]
 *   kept_idx [L][G][total_cache],               request b at cache_off[b]
 * dtype 0 = IEEE binary32, 1 = bfloat16 (upper 16 bits of a binary32); both widen exactly to fp64.
 * group_mode 0: one selection group per KV head (G = Hkv); 1: one per layer (G = 1, the paper's sum over all H).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double widen(const void *base, int dtype, int64_t i)
{
    if (dtype == 0)
        return (double)((const float *)base)[i];
    uint32_t bits = ((uint32_t)((const uint16_t *)base)[i]) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

static int64_t elem_bytes(int dtype) { return dtype == 0 ? 4 : 2; }

int finch_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ scoring */

/* One selection unit: layer l, group G, request b.  Writes A^agg (length N) to
 * out_scores and, when row_lse != NULL, the log-sum-exp of each (head, prompt row). */
static void score_unit(int dtype, const void *q, const void *cache_k, const void *chunk_k,
                       int Hq, int Hkv, int d, int group_mode, double scale,
                       int64_t total_q, int64_t total_cache, int64_t total_chunk,
                       int l, int G, int64_t q0, int n_q, int64_t cache0, int c, int64_t chunk0, int m,
                       int apply_norm, const double *self_lse, const int32_t *row_limit, int row_norm,
                       double *out_scores, double *row_lse)
{
    const int N = c + m;
    const int heads_per_kv = Hq / Hkv;
    const int h_begin = group_mode == 0 ? G * heads_per_kv : 0;
    const int h_end = group_mode == 0 ? (G + 1) * heads_per_kv : Hq;
    if (N == 0)
        return;

    /* A^cont: prompt rows x candidate columns, summed over the heads of the group. */
    double *A = (double *)calloc((size_t)n_q * (size_t)N, sizeof(double));
    double *s = (double *)malloc((size_t)N * sizeof(double));

    for (int h = h_begin; h < h_end; ++h) {
        const int kvh = h / heads_per_kv;
        for (int p = 0; p < n_q; ++p) {
            const int64_t qrow = (((int64_t)l * Hq + h) * total_q + q0 + p) * d;
            for (int j = 0; j < N; ++j) {
                /* candidate j: cache rows first, then the chunk's rows */
                const void *kbase = j < c ? cache_k : chunk_k;
                const int64_t krow = j < c ? (((int64_t)l * Hkv + kvh) * total_cache + cache0 + j) * d
                                           : (((int64_t)l * Hkv + kvh) * total_chunk + chunk0 + (j - c)) * d;
                double dot = 0.0;
                for (int t = 0; t < d; ++t)
                    dot += widen(q, dtype, qrow + t) * widen(kbase, dtype, krow + t);
                s[j] = scale * dot;
            }
            /* the candidates this row attends to: all of them, or the first row_limit[p] (causal rows) */
            int vis = N;
            if (row_limit) {
                vis = row_limit[q0 + p];
                if (vis > N)
                    vis = N;
                if (vis <= 0) {
                    if (row_lse)
                        row_lse[(size_t)(h - h_begin) * n_q + p] = -INFINITY;
                    continue; /* a row that sees nothing gives nothing */
                }
            }
            double mx = s[0];
            for (int j = 1; j < vis; ++j)
                if (s[j] > mx)
                    mx = s[j];
            double Z = 0.0;
            for (int j = 0; j < vis; ++j)
                Z += exp(s[j] - mx);
            double lse = mx + log(Z);
            if (self_lse) {
                /* the row's keys are the candidates and the prompt's own keys: add the prompt's share,
                 * exp(self), to the denominator */
                const double extra = self_lse[(((int64_t)l * Hq + h) * total_q + q0 + p)];
                const double top = extra > lse ? extra : lse;
                if (extra > -INFINITY)
                    lse = top + log(exp(lse - top) + exp(extra - top));
            }
            if (row_lse)
                row_lse[(size_t)(h - h_begin) * n_q + p] = lse;
            /* per-row reading of the normalisation: count(row != 0) / (m + c) = vis / N */
            const double row_factor = row_norm ? (double)vis / (double)N : 1.0;
            for (int j = 0; j < vis; ++j)
                A[(size_t)p * N + j] += exp(s[j] - lse) * row_factor;
        }
    }

    if (apply_norm) {
        /* A^norm = A^cont * count(A^cont != 0) / (m + c), the count taken over the whole submatrix. */
        int64_t nonzero = 0;
        for (size_t i = 0; i < (size_t)n_q * (size_t)N; ++i)
            if (A[i] != 0.0)
                ++nonzero;
        const double factor = (double)nonzero / (double)N;
        for (size_t i = 0; i < (size_t)n_q * (size_t)N; ++i)
            A[i] *= factor;
    }

    for (int j = 0; j < N; ++j) {
        double agg = 0.0;
        for (int p = 0; p < n_q; ++p)
            agg += A[(size_t)p * N + j];
        out_scores[j] = agg;
    }
    free(s);
    free(A);
}

static int n_groups(int Hkv, int group_mode) { return group_mode == 0 ? Hkv : 1; }

/* scores [L][G][total_cache+total_chunk] fp64; row_lse (nullable) [L][Hq][total_q] fp64. */
int finch_oracle_score(int dtype, const void *q, const void *cache_k, const void *chunk_k,
                       int L, int Hq, int Hkv, int d, int group_mode, double scale,
                       int batch, const int32_t *q_off, const int32_t *chunk_off, const int32_t *cache_off,
                       const int32_t *cache_len, int apply_norm, const double *prompt_self_lse,
                       const int32_t *row_limit, int row_norm, double *scores, double *row_lse, int threads)
{
    if (L < 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || d <= 0 || batch < 0)
        return 1;
    const int Gn = n_groups(Hkv, group_mode);
    const int64_t total_q = q_off[batch], total_cache = cache_off[batch], total_chunk = chunk_off[batch];
    const int64_t total_cand = total_cache + total_chunk;
    const int heads_per_group = Hq / Gn;
    const int64_t n_units = (int64_t)L * Gn * batch;
    if (threads <= 0)
        threads = 1;
#pragma omp parallel for schedule(dynamic, 1) num_threads(threads)
    for (int64_t u = 0; u < n_units; ++u) {
        const int b = (int)(u % batch);
        const int G = (int)((u / batch) % Gn);
        const int l = (int)(u / batch / Gn);
        const int n_q = q_off[b + 1] - q_off[b];
        const int m = chunk_off[b + 1] - chunk_off[b];
        const int c = cache_len[b];
        double *lse_unit = NULL;
        if (row_lse && n_q > 0)
            lse_unit = (double *)malloc((size_t)heads_per_group * n_q * sizeof(double));
        score_unit(dtype, q, cache_k, chunk_k, Hq, Hkv, d, group_mode, scale, total_q, total_cache, total_chunk,
                   l, G, q_off[b], n_q, cache_off[b], c, chunk_off[b], m, apply_norm, prompt_self_lse,
                   row_limit, row_norm, scores + ((int64_t)l * Gn + G) * total_cand + cache_off[b] + chunk_off[b], lse_unit);
        if (lse_unit) {
            if (c + m > 0)
                for (int hh = 0; hh < heads_per_group; ++hh)
                    for (int p = 0; p < n_q; ++p)
                        row_lse[((int64_t)l * Hq + (int64_t)G * heads_per_group + hh) * total_q + q_off[b] + p] =
                            lse_unit[(size_t)hh * n_q + p];
            free(lse_unit);
        }
    }
    return 0;
}

/* ---------------------------------------------------------------- selection */

typedef struct {
    double score;
    int32_t idx;
} ranked;

/* Total order: higher score first; equal scores: lower index first.  NaN ranks
 * below every number (two NaNs compare by index). */
static int rank_cmp(const void *pa, const void *pb)
{
    const ranked *a = (const ranked *)pa, *b = (const ranked *)pb;
    const int an = isnan(a->score), bn = isnan(b->score);
    if (an != bn)
        return an ? 1 : -1;
    if (!an) {
        if (a->score > b->score)
            return -1;
        if (a->score < b->score)
            return 1;
    }
    return a->idx < b->idx ? -1 : (a->idx > b->idx ? 1 : 0);
}

static int idx_cmp(const void *pa, const void *pb)
{
    const int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    return a < b ? -1 : (a > b ? 1 : 0);
}

/* t = top-r(A^agg, r) for one unit.  Returns r' = min(r, N) and writes r' candidate
 * indices: ascending when rank_order == 0, in order of decreasing score otherwise. */
int finch_oracle_select_unit(const double *scores, int N, int r, int rank_order, int32_t *kept)
{
    if (r > N)
        r = N;
    if (r <= 0)
        return 0;
    ranked *v = (ranked *)malloc((size_t)N * sizeof(ranked));
    for (int j = 0; j < N; ++j) {
        v[j].score = scores[j];
        v[j].idx = j;
    }
    qsort(v, (size_t)N, sizeof(ranked), rank_cmp);
    for (int i = 0; i < r; ++i)
        kept[i] = v[i].idx;
    if (!rank_order)
        qsort(kept, (size_t)r, sizeof(int32_t), idx_cmp);
    free(v);
    return r;
}

/* Batched: scores [L][G][total_cand] fp64 -> kept_idx [L][G][total_cache], out_len [batch].
 * cand_len[b] = cache_len[b] + chunk_len[b]; budget[b] must not exceed the request's cache capacity. */
int finch_oracle_select(const double *scores, int L, int Gn, int batch,
                        const int32_t *chunk_off, const int32_t *cache_off, const int32_t *cache_len,
                        const int32_t *budget, int rank_order, int32_t *kept_idx, int32_t *out_len)
{
    const int64_t total_cache = cache_off[batch], total_chunk = chunk_off[batch];
    const int64_t total_cand = total_cache + total_chunk;
    for (int b = 0; b < batch; ++b) {
        const int N = cache_len[b] + (chunk_off[b + 1] - chunk_off[b]);
        const int r = budget[b] < N ? budget[b] : N;
        if (r > cache_off[b + 1] - cache_off[b])
            return 2;
        out_len[b] = r < 0 ? 0 : r;
    }
    for (int l = 0; l < L; ++l)
        for (int G = 0; G < Gn; ++G)
            for (int b = 0; b < batch; ++b) {
                const int N = cache_len[b] + (chunk_off[b + 1] - chunk_off[b]);
                finch_oracle_select_unit(scores + ((int64_t)l * Gn + G) * total_cand + cache_off[b] + chunk_off[b], N,
                                         budget[b], rank_order,
                                         kept_idx + ((int64_t)l * Gn + G) * total_cache + cache_off[b]);
            }
    return 0;
}

/* --------------------------------------------------------------- compaction */

/* Round a double to the storage type (round to nearest, ties to even) and store it at element i. */
static void narrow_store(void *base, int dtype, int64_t i, double x)
{
    if (dtype == 0) {
        ((float *)base)[i] = (float)x;
        return;
    }
    /* bfloat16: 8 significant bits.  Scale the significand to an integer, round it, scale back; the result is
     * exactly representable in binary32, whose upper half is then the bfloat16 pattern. */
    float f = 0.0f;
    if (x != 0.0 && isfinite(x)) {
        int e;
        const double sig = frexp(x, &e);          /* |sig| in [0.5, 1) */
        f = (float)ldexp(rint(ldexp(sig, 8)), e - 8);
    } else {
        f = (float)x;
    }
    uint32_t bits;
    memcpy(&bits, &f, sizeof bits);
    ((uint16_t *)base)[i] = (uint16_t)(bits >> 16);
}

/* Rotary position embedding moved by `delta` positions (Managing the Cache: a kept key that moves from position j
 * to slot i is rotated by the cosine and sine of the position difference).  RoFormer's rotation acts on pairs of
 * coordinates (x, y) with angle delta * theta^(-2t/d) for pair t:  x' = x cos - y sin,  y' = y cos + x sin.
 * pairing 0: pair t = coordinates (t, t + d/2), the layout of the Llama implementation the paper uses;
 * pairing 1: pair t = coordinates (2t, 2t + 1), RoFormer's own. */
static void rerotate_row(int dtype, const void *src, int64_t src_elem, void *dst, int64_t dst_elem, int d,
                         double theta, int pairing, int delta)
{
    for (int t = 0; t < d / 2; ++t) {
        const int ix = pairing == 0 ? t : 2 * t, iy = pairing == 0 ? t + d / 2 : 2 * t + 1;
        const double angle = (double)delta * pow(theta, -2.0 * (double)t / (double)d);
        const double x = widen(src, dtype, src_elem + ix), y = widen(src, dtype, src_elem + iy);
        narrow_store(dst, dtype, dst_elem + ix, x * cos(angle) - y * sin(angle));
        narrow_store(dst, dtype, dst_elem + iy, y * cos(angle) + x * sin(angle));
    }
}

/* out_k/out_v [L][Hkv][total_cache][d] (same dtype as the inputs), out_pos [L][G][total_cache];
 * cache_pos [L][G][total_cache], chunk_pos [total_chunk].  V rows and, with rope_theta == 0, K rows are bit copies.
 * With rope_theta > 0 the K rows are taken to carry rotary embeddings at their candidate index (the cache's rows at
 * their slots, the chunk's rows after them) and are re-rotated to the slot they land in: delta = i - kept[i]. */
int finch_oracle_compact(int dtype, const int32_t *kept_idx, const int32_t *out_len,
                         const void *cache_k, const void *cache_v, const int32_t *cache_pos,
                         const void *chunk_k, const void *chunk_v, const int32_t *chunk_pos,
                         int L, int Hkv, int d, int group_mode, int batch,
                         const int32_t *chunk_off, const int32_t *cache_off, const int32_t *cache_len,
                         double rope_theta, int rope_pairing, void *out_k, void *out_v, int32_t *out_pos)
{
    const int Gn = n_groups(Hkv, group_mode);
    const int kv_per_group = Hkv / Gn;
    const int64_t total_cache = cache_off[batch], total_chunk = chunk_off[batch];
    const int64_t row = (int64_t)d * elem_bytes(dtype);
    for (int l = 0; l < L; ++l)
        for (int G = 0; G < Gn; ++G)
            for (int b = 0; b < batch; ++b) {
                const int c = cache_len[b];
                const int32_t *kept = kept_idx + ((int64_t)l * Gn + G) * total_cache + cache_off[b];
                for (int i = 0; i < out_len[b]; ++i) {
                    const int j = kept[i];
                    const int64_t slot = ((int64_t)l * Gn + G) * total_cache + cache_off[b] + i;
                    out_pos[slot] = j < c ? cache_pos[((int64_t)l * Gn + G) * total_cache + cache_off[b] + j]
                                          : chunk_pos[chunk_off[b] + (j - c)];
                    for (int kk = 0; kk < kv_per_group; ++kk) {
                        const int kvh = G * kv_per_group + kk;
                        const int64_t dst = (((int64_t)l * Hkv + kvh) * total_cache + cache_off[b] + i) * row;
                        const int64_t src = j < c
                                                ? (((int64_t)l * Hkv + kvh) * total_cache + cache_off[b] + j) * row
                                                : (((int64_t)l * Hkv + kvh) * total_chunk + chunk_off[b] + (j - c)) * row;
                        if (rope_theta > 0.0)
                            rerotate_row(dtype, j < c ? cache_k : chunk_k, src / elem_bytes(dtype), out_k,
                                         dst / elem_bytes(dtype), d, rope_theta, rope_pairing, i - j);
                        else
                            memcpy((char *)out_k + dst, (const char *)(j < c ? cache_k : chunk_k) + src, (size_t)row);
                        memcpy((char *)out_v + dst, (const char *)(j < c ? cache_v : chunk_v) + src, (size_t)row);
                    }
                }
            }
    return 0;
}

/* ------------------------------------------------------------ the whole step */

/* score -> select -> compact, as one call (what the benchmark's CPU leg times).
 * scores_ws: caller's fp64 buffer [L][G][total_cand]. */
int finch_oracle_step(int dtype, const void *q, const void *cache_k, const void *cache_v, const int32_t *cache_pos,
                      const void *chunk_k, const void *chunk_v, const int32_t *chunk_pos,
                      int L, int Hq, int Hkv, int d, int group_mode, double scale, int batch,
                      const int32_t *q_off, const int32_t *chunk_off, const int32_t *cache_off,
                      const int32_t *cache_len, const int32_t *budget,
                      void *out_k, void *out_v, int32_t *out_pos, int32_t *kept_idx, int32_t *out_len,
                      double *scores_ws, int threads)
{
    int rc = finch_oracle_score(dtype, q, cache_k, chunk_k, L, Hq, Hkv, d, group_mode, scale, batch, q_off, chunk_off,
                                cache_off, cache_len, 0, NULL, NULL, 0, scores_ws, NULL, threads);
    if (rc)
        return rc;
    rc = finch_oracle_select(scores_ws, L, n_groups(Hkv, group_mode), batch, chunk_off, cache_off, cache_len, budget, 0,
                             kept_idx, out_len);
    if (rc)
        return rc;
    return finch_oracle_compact(dtype, kept_idx, out_len, cache_k, cache_v, cache_pos, chunk_k, chunk_v, chunk_pos, L,
                                Hkv, d, group_mode, batch, chunk_off, cache_off, cache_len, 0.0, 0, out_k, out_v, out_pos);
}
