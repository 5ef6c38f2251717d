/*
 * CPU oracle for the batched token sampler -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded restatement of what the sampling task (T4, paper
 * section 2.1; "core sampling computation", section 6.1 step 3) computes for each row
 * of the (s x v) logits matrix, with every feature of section 8.1 (Workload) enabled:
 * repetition / presence / frequency penalties from the request's token history,
 * temperature, top-k, min-p, top-p, a softmax with log-probability output (the
 * probability is appended to the sequence with the token, Appendix A "update
 * sequence"), and a seeded draw that is a pure function of (seed, global row, step,
 * token id) so that any partition of the rows over workers gives the same tokens
 * (section 6.2, deterministic random number generation).
 *
 * The paper fixes none of the arithmetic; the readings taken are listed in the
 * repository's design notes.  In short, per row:
 *   1. widen logits to fp32 (bf16 -> fp32 and fp16 -> fp32 are exact);
 *   2. count history occurrences per token id (ids outside [0,V) ignored);
 *   3. for tokens with count > 0: a = x>0 ? x/r : x*r ; a -= f*count ; a -= p
 *      (each step one rounded fp32 operation);
 *      with the history split into prompt and generated output (`out_start`: where the output begins
 *      in the row's history) the repetition penalty looks at both parts, the frequency and presence
 *      penalties at the output alone: a = rep(x) for a token seen anywhere; a -= f*c_out; and
 *      a -= p only if c_out > 0 (c_out: occurrences in the output);
 *   4. T == 0 (or < 0): greedy == top_k 1 with no scaling; else z = a * (1/T) in fp32;
 *   5. sort all ids by (order-preserving key of z descending, id ascending);
 *   6. top-k: keep the first min(k, #finite) -- or, in the keep-ties mode, every score not below
 *      the k-th largest (what masking "logits < k-th value" gives);
 *   7. min-p: keep z - zmax >= ln(min_p);
 *   8. top-p: smallest prefix whose mass >= top_p * (mass of the survivors);
 *   9. softmax over the survivors in fp64 -> log-probabilities;
 *  10. exponential race: Philox4x32-10 word per token -> E ~ Exp(1);
 *      token = argmax (z - zmax) - ln E.  (With pre-generated random numbers, the scheme of
 *      section 6.2, E is read from a caller-supplied [B, V] fp32 table of Exp(1) variates instead.)
 * Reductions are fp64 in sorted order.  No blocking, fusion or reordering.
 *
 * Nothing here is shared with the CUDA library, and only tests, the smoke check and
 * the benchmark's CPU-baseline leg may call it.
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -shared -fPIC (see oracle/albireo_oracle.py)
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_F32 0
#define ORACLE_BF16 1
#define ORACLE_F16 2      /* IEEE binary16, the precision of the paper's models (section 8.1) */

typedef struct {
    int32_t token;        /* sampled token id                                   */
    int32_t n_fin;        /* number of finite z in the row                      */
    int32_t n_topk;       /* kept after step 6 (top-k stage)                    */
    int32_t n_minp;       /* kept after step 7                                  */
    int32_t n_keep;       /* kept after step 8 (final kept set)                 */
    int32_t greedy;       /* 1 if the row was treated as greedy                 */
    double logprob;       /* log-probability of `token` in the final kept set   */
    double z_max;         /* largest z (as double)                              */
    double S;             /* normaliser of the log-probabilities: sum of exp(z - zmax) over the final
                             kept set (over all finite scores in the full-vocabulary mode)      */
    double race_gap;      /* best - second best race score (+inf if n_keep==1)  */
    double minp_margin;   /* min_j |d_j - ln(min_p)| over the step-6 set (+inf if off) */
    double topp_margin;   /* distance of top_p*S' to the nearest cumulative sum, / S' (+inf if off) */
} albireo_oracle_row_t;

/* ------------------------------------------------------------------ small helpers */

static float bits_to_f32(uint32_t b) { float f; memcpy(&f, &b, 4); return f; }
static uint32_t f32_to_bits(float f) { uint32_t b; memcpy(&b, &f, 4); return b; }

/* order-preserving map fp32 -> uint32 (larger float <=> larger key; -0 < +0) */
static uint32_t order_key(float z)
{
    uint32_t b = f32_to_bits(z);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

uint32_t albireo_oracle_order_key(float z) { return order_key(z); }

static float load_logit(const void *logits, int32_t dtype, int64_t pos)
{
    if (dtype == ORACLE_BF16) {
        uint16_t h = ((const uint16_t *)logits)[pos];
        return bits_to_f32(((uint32_t)h) << 16);
    }
    if (dtype == ORACLE_F16) {
        /* IEEE binary16 -> fp32, exact: 1 sign, 5 exponent (bias 15), 10 fraction bits */
        uint16_t h = ((const uint16_t *)logits)[pos];
        int sign = (h >> 15) & 1, ex = (h >> 10) & 0x1F, fr = h & 0x3FF;
        float v;
        if (ex == 0) v = ldexpf((float)fr, -24);                      /* zero and subnormals: fr * 2^-24 */
        else if (ex == 31) v = fr ? NAN : INFINITY;
        else v = ldexpf((float)(fr | 0x400), ex - 25);                /* (1024 + fr) * 2^(ex-15-10) */
        return sign ? -v : v;
    }
    return ((const float *)logits)[pos];
}

/* Philox4x32-10 (Salmon et al., "Parallel random numbers: as easy as 1, 2, 3"). */
void albireo_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)M0 * c0;
        uint64_t p1 = (uint64_t)M1 * c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;          /* the bump after the last round is unused */
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* the 32-bit word that belongs to token `id` of global row R at `step` under `seed` */
static uint32_t race_word(uint64_t seed, uint32_t R, uint64_t step, int32_t id)
{
    uint32_t ctr[4] = { (uint32_t)id >> 2, R, (uint32_t)(step & 0xFFFFFFFFu), (uint32_t)(step >> 32) };
    uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    uint32_t out[4];
    albireo_oracle_philox4x32_10(ctr, key, out);
    return out[id & 3];
}

/* Exp(1) variate from a 32-bit word: v = (w + 1/2) 2^-32 in (0,1), E = -log1p(-v) */
static double exp1_from_word(uint32_t w)
{
    double v = ((double)w + 0.5) * (1.0 / 4294967296.0);
    return -log1p(-v);
}

double albireo_oracle_exp1_from_word(uint32_t w) { return exp1_from_word(w); }

typedef struct { uint32_t key; int32_t id; } sort_item_t;

static int cmp_items(const void *pa, const void *pb)
{
    const sort_item_t *a = (const sort_item_t *)pa, *b = (const sort_item_t *)pb;
    if (a->key != b->key) return (a->key > b->key) ? -1 : 1;   /* key descending */
    if (a->id != b->id) return (a->id < b->id) ? -1 : 1;       /* id ascending   */
    return 0;
}

/* ------------------------------------------------------------------ one row */

typedef struct {
    float T, top_p, min_p, r, p, f;
    int32_t top_k;
    uint64_t seed;
} row_params_t;

/*
 * Steps 1-5 for one row: fills z[V] and the fully sorted order[V].  `counts` is a
 * caller-provided zeroed int32[V] scratch and is returned zeroed.
 * Returns 1 if the row is greedy.
 */
static int row_scores_and_order(const void *logits, int32_t dtype, int64_t row_pos, int32_t V,
                                const int32_t *hist, int32_t hist_len, int32_t out_start,
                                const row_params_t *rp,
                                int32_t *counts, float *z, sort_item_t *order)
{
    if (out_start < 0) out_start = 0;
    if (out_start > hist_len) out_start = hist_len;
    /* 1. widen */
    for (int32_t i = 0; i < V; ++i) z[i] = load_logit(logits, dtype, row_pos + i);
    /* 2. counts: counts[t] = occurrences in the output part; a token seen only in the prompt is
       marked with -1 (seen, zero output occurrences) */
    for (int32_t j = out_start; j < hist_len; ++j) {
        int32_t t = hist[j];
        if (t >= 0 && t < V) counts[t] += 1;
    }
    for (int32_t j = 0; j < out_start; ++j) {
        int32_t t = hist[j];
        if (t >= 0 && t < V && counts[t] == 0) counts[t] = -1;
    }
    /* 3. penalties, one rounded fp32 operation per line */
    for (int32_t i = 0; i < V; ++i) {
        if (counts[i] != 0) {
            int32_t c_out = counts[i] > 0 ? counts[i] : 0;
            float a = z[i];
            if (a > 0.0f) a = a / rp->r; else a = a * rp->r;
            float t = rp->f * (float)c_out;
            a = a - t;
            if (c_out > 0) a = a - rp->p;
            z[i] = a;
        }
    }
    for (int32_t j = 0; j < hist_len; ++j) {
        int32_t t = hist[j];
        if (t >= 0 && t < V) counts[t] = 0;
    }
    /* 4. temperature */
    int greedy = !(rp->T > 0.0f);
    if (!greedy) {
        float inv_T = 1.0f / rp->T;
        for (int32_t i = 0; i < V; ++i) z[i] = z[i] * inv_T;
    }
    /* 5. total order */
    for (int32_t i = 0; i < V; ++i) { order[i].key = order_key(z[i]); order[i].id = i; }
    qsort(order, (size_t)V, sizeof(sort_item_t), cmp_items);
    return greedy;
}

/*
 * Steps 6-10 given the sorted order.  ln_min_p_shift / top_p_shift perturb the two
 * real-valued cut parameters (used only to enumerate results inside the backward-error
 * band of a cut; both 0 for the primary result).
 */
static void row_cut_and_draw(const float *z, const sort_item_t *order, int32_t V, int greedy,
                             const row_params_t *rp, uint32_t R, uint64_t step,
                             const float *exp1_row /* NULL: Philox */, int keep_ties, int full_vocab,
                             double ln_min_p_shift, double top_p_shift,
                             albireo_oracle_row_t *out, double *e /* scratch [V] */)
{
    const double zmax = (double)z[order[0].id];
    int32_t n_fin = 0;
    for (int32_t j = 0; j < V; ++j) if (isfinite(z[order[j].id])) ++n_fin;
    /* finite values form a contiguous block of the order: +inf (contract violation) first, -inf last */
    int32_t top_k = greedy ? 1 : rp->top_k;
    double top_p = greedy ? 1.0 : (double)rp->top_p + top_p_shift;
    float min_p = greedy ? 0.0f : rp->min_p;

    /* 6. top-k */
    int32_t L = n_fin;
    if (top_k >= 1 && top_k < V && top_k < L) {
        L = top_k;
        /* keep-ties mode: everything equal to the k-th largest score stays (equal scores have equal keys) */
        if (keep_ties && !greedy)
            while (L < n_fin && order[L].key == order[L - 1].key) ++L;
    }
    if (L < 1) L = 1;
    out->n_fin = n_fin;
    out->n_topk = L;

    /* 7. min-p */
    out->minp_margin = INFINITY;
    if (min_p > 0.0f) {
        const double thr = log((double)min_p) + ln_min_p_shift;
        int32_t cnt = 0;
        for (int32_t j = 0; j < L; ++j) {
            double d = (double)z[order[j].id] - zmax;
            if (d >= thr) ++cnt;
            double m = fabs(d - thr);
            if (m < out->minp_margin) out->minp_margin = m;
        }
        L = cnt < 1 ? 1 : cnt;
    }
    out->n_minp = L;

    /* 8. top-p on the mass of the survivors */
    for (int32_t j = 0; j < L; ++j) e[j] = exp((double)z[order[j].id] - zmax);
    out->topp_margin = INFINITY;
    if (top_p < 1.0) {
        double Sp = 0.0;
        for (int32_t j = 0; j < L; ++j) Sp += e[j];
        const double target = top_p * Sp;
        double C = 0.0, Cprev = 0.0;
        int32_t keep = L;
        for (int32_t j = 0; j < L; ++j) {
            Cprev = C;
            C += e[j];
            if (C >= target) { keep = j + 1; break; }
        }
        double m1 = (C - target) / Sp, m2 = (keep > 1) ? (target - Cprev) / Sp : INFINITY;
        out->topp_margin = m1 < m2 ? m1 : m2;
        L = keep;
    }
    out->n_keep = L;

    /* 9. softmax over the final kept set -- or, in the full-vocabulary mode, over every finite score of
          the row (the cuts then decide what may be drawn, not what the probabilities are relative to) */
    double S = 0.0;
    if (full_vocab) {
        for (int32_t j = 0; j < V; ++j) {
            double zj = (double)z[order[j].id];
            if (isfinite(zj)) S += exp(zj - zmax);
        }
    } else {
        for (int32_t j = 0; j < L; ++j) S += e[j];
    }
    out->S = S;
    out->z_max = zmax;
    const double lnS = log(S);

    /* 10. exponential race */
    int32_t best = -1; double gbest = -INFINITY, gsecond = -INFINITY; int32_t jbest = 0;
    for (int32_t j = 0; j < L; ++j) {
        int32_t id = order[j].id;
        double E = exp1_row ? (double)exp1_row[id] : exp1_from_word(race_word(rp->seed, R, step, id));
        double g = ((double)z[id] - zmax) - log(E);
        if (best < 0 || g > gbest || (g == gbest && id < best)) {
            if (best >= 0) gsecond = gbest;
            gbest = g; best = id; jbest = j;
        } else if (g > gsecond) {
            gsecond = g;
        }
    }
    out->token = best;
    out->logprob = ((double)z[order[jbest].id] - zmax) - lnS;
    out->race_gap = (L > 1) ? gbest - gsecond : INFINITY;
    out->greedy = greedy;
}

static void load_params(int32_t b, const float *temperature, const int32_t *top_k, const float *top_p,
                        const float *min_p, const float *rep, const float *pres, const float *freq,
                        const uint64_t *seeds, row_params_t *rp)
{
    rp->T = temperature ? temperature[b] : 1.0f;
    rp->top_k = top_k ? top_k[b] : 0;
    rp->top_p = top_p ? top_p[b] : 1.0f;
    rp->min_p = min_p ? min_p[b] : 0.0f;
    rp->r = rep ? rep[b] : 1.0f;
    rp->p = pres ? pres[b] : 0.0f;
    rp->f = freq ? freq[b] : 0.0f;
    rp->seed = seeds ? seeds[b] : 0;
}

/* ------------------------------------------------------------------ batch entry */

/*
 * Samples rows [row_begin, row_end) of a [B, V] batch.  All pointers are host memory.
 * Optional outputs (may be NULL / 0):
 *   topk_ids  [B, topk_cap]  the step-6 kept ids in sorted order, -1 padded
 *   kept_ids  [B, kept_cap]  the final kept ids in sorted order, -1 padded
 *   top_ids / top_logprobs [B, num_top]  first min(num_top, n_keep) (id, logprob), padded (-1, -inf)
 * Returns 0, or -1 on allocation failure / bad arguments.
 */
int albireo_oracle_sample(const void *logits, int32_t B, int32_t V, int32_t dtype, int64_t row_stride,
                          const float *temperature, const int32_t *top_k, const float *top_p,
                          const float *min_p, const float *rep, const float *pres, const float *freq,
                          const int32_t *hist_ids, const int32_t *hist_off,
                          const uint64_t *seeds, uint64_t step, uint32_t row_base,
                          const float *exp1 /* [B, V] Exp(1) variates, or NULL */,
                          const int32_t *out_start /* [B] where the output begins in each history, or NULL: 0 */,
                          uint32_t flags /* value 2: top-k keeps ties; value 4: log-probabilities relative to the full vocabulary */,
                          int32_t row_begin, int32_t row_end,
                          albireo_oracle_row_t *rows_out,
                          int32_t topk_cap, int32_t *topk_ids,
                          int32_t kept_cap, int32_t *kept_ids,
                          int32_t num_top, int32_t *top_ids, double *top_logprobs)
{
    if (!logits || !rows_out || V < 1 || B < 0 || row_begin < 0 || row_end > B) return -1;
    if (dtype != ORACLE_F32 && dtype != ORACLE_BF16 && dtype != ORACLE_F16) return -1;
    float *z = (float *)malloc(sizeof(float) * (size_t)V);
    sort_item_t *order = (sort_item_t *)malloc(sizeof(sort_item_t) * (size_t)V);
    int32_t *counts = (int32_t *)calloc((size_t)V, sizeof(int32_t));
    double *e = (double *)malloc(sizeof(double) * (size_t)V);
    if (!z || !order || !counts || !e) { free(z); free(order); free(counts); free(e); return -1; }

    for (int32_t b = row_begin; b < row_end; ++b) {
        row_params_t rp;
        load_params(b, temperature, top_k, top_p, min_p, rep, pres, freq, seeds, &rp);
        const int32_t *h = NULL; int32_t hl = 0;
        if (hist_ids && hist_off) { h = hist_ids + hist_off[b]; hl = hist_off[b + 1] - hist_off[b]; }
        int greedy = row_scores_and_order(logits, dtype, (int64_t)b * row_stride, V, h, hl,
                                          out_start ? out_start[b] : 0, &rp, counts, z, order);
        albireo_oracle_row_t *o = &rows_out[b];
        row_cut_and_draw(z, order, V, greedy, &rp, row_base + (uint32_t)b, step,
                         exp1 ? exp1 + (int64_t)b * V : NULL, (flags & 2u) != 0, (flags & 4u) != 0, 0.0, 0.0, o, e);

        if (topk_ids) for (int32_t j = 0; j < topk_cap; ++j)
            topk_ids[(int64_t)b * topk_cap + j] = (j < o->n_topk) ? order[j].id : -1;
        if (kept_ids) for (int32_t j = 0; j < kept_cap; ++j)
            kept_ids[(int64_t)b * kept_cap + j] = (j < o->n_keep) ? order[j].id : -1;
        if (top_ids && top_logprobs) {
            const double lnS = log(o->S);
            /* the list runs over the final kept set; in the full-vocabulary mode over every finite score */
            const int32_t list_len = (flags & 4u) ? o->n_fin : o->n_keep;
            for (int32_t j = 0; j < num_top; ++j) {
                int64_t q = (int64_t)b * num_top + j;
                if (j < list_len) {
                    top_ids[q] = order[j].id;
                    top_logprobs[q] = ((double)z[order[j].id] - o->z_max) - lnS;
                } else {
                    top_ids[q] = -1;
                    top_logprobs[q] = -INFINITY;
                }
            }
        }
    }
    free(z); free(order); free(counts); free(e);
    return 0;
}

/*
 * One row again, with the two real-valued cut parameters shifted: the result the
 * definition gives for ln(min_p) + ln_min_p_shift and top_p + top_p_shift.  Used by the
 * parity tests to enumerate the results that are acceptable inside a cut's
 * backward-error band.  Optionally returns the sorted ids and z (length V).
 */
int albireo_oracle_row_shifted(const void *logits, int32_t B, int32_t V, int32_t dtype, int64_t row_stride,
                               const float *temperature, const int32_t *top_k, const float *top_p,
                               const float *min_p, const float *rep, const float *pres, const float *freq,
                               const int32_t *hist_ids, const int32_t *hist_off,
                               const uint64_t *seeds, uint64_t step, uint32_t row_base,
                               const float *exp1, const int32_t *out_start, uint32_t flags,
                               int32_t b, double ln_min_p_shift, double top_p_shift,
                               albireo_oracle_row_t *row_out, int32_t *sorted_ids, float *sorted_z,
                               double *sorted_g)
{
    if (!logits || !row_out || V < 1 || b < 0 || b >= B) return -1;
    float *z = (float *)malloc(sizeof(float) * (size_t)V);
    sort_item_t *order = (sort_item_t *)malloc(sizeof(sort_item_t) * (size_t)V);
    int32_t *counts = (int32_t *)calloc((size_t)V, sizeof(int32_t));
    double *e = (double *)malloc(sizeof(double) * (size_t)V);
    if (!z || !order || !counts || !e) { free(z); free(order); free(counts); free(e); return -1; }
    row_params_t rp;
    load_params(b, temperature, top_k, top_p, min_p, rep, pres, freq, seeds, &rp);
    const int32_t *h = NULL; int32_t hl = 0;
    if (hist_ids && hist_off) { h = hist_ids + hist_off[b]; hl = hist_off[b + 1] - hist_off[b]; }
    int greedy = row_scores_and_order(logits, dtype, (int64_t)b * row_stride, V, h, hl,
                                      out_start ? out_start[b] : 0, &rp, counts, z, order);
    const float *exp1_row = exp1 ? exp1 + (int64_t)b * V : NULL;
    row_cut_and_draw(z, order, V, greedy, &rp, row_base + (uint32_t)b, step, exp1_row, (flags & 2u) != 0, (flags & 4u) != 0,
                     ln_min_p_shift, top_p_shift, row_out, e);
    const double zmax = (double)z[order[0].id];
    for (int32_t j = 0; j < V; ++j) {
        int32_t id = order[j].id;
        if (sorted_ids) sorted_ids[j] = id;
        if (sorted_z) sorted_z[j] = z[id];
        if (sorted_g) {
            double E = exp1_row ? (double)exp1_row[id] : exp1_from_word(race_word(rp.seed, row_base + (uint32_t)b, step, id));
            sorted_g[j] = ((double)z[id] - zmax) - log(E);
        }
    }
    free(z); free(order); free(counts); free(e);
    return 0;
}

/* the penalised, temperature-scaled scores z of one row (steps 1-4), for pins */
int albireo_oracle_row_scores(const void *logits, int32_t V, int32_t dtype,
                              float T, float r, float p, float f,
                              const int32_t *hist, int32_t hist_len, int32_t out_start, float *z_out)
{
    if (!logits || !z_out || V < 1) return -1;
    sort_item_t *order = (sort_item_t *)malloc(sizeof(sort_item_t) * (size_t)V);
    int32_t *counts = (int32_t *)calloc((size_t)V, sizeof(int32_t));
    if (!order || !counts) { free(order); free(counts); return -1; }
    row_params_t rp; memset(&rp, 0, sizeof rp);
    rp.T = T; rp.r = r; rp.p = p; rp.f = f; rp.top_p = 1.0f;
    row_scores_and_order(logits, dtype, 0, V, hist, hist_len, out_start, &rp, counts, z_out, order);
    free(order); free(counts);
    return 0;
}

uint32_t albireo_oracle_race_word(uint64_t seed, uint32_t R, uint64_t step, int32_t id)
{
    return race_word(seed, R, step, id);
}
