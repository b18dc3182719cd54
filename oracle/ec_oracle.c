/*
 * CPU oracle for importance-driven KV-cache merging (Elastic Cache, arXiv 2407.18121).
 *
 * TEST INFRASTRUCTURE ONLY. This file is the slow, plain statement of what the method
 * computes, in fp64, written from the paper's definitions. It shares no code with the
 * CUDA library and must never be reached from the product path; only tests, the smoke
 * check and the benchmark's CPU-baseline leg may call it.
 *
 * Inputs that the GPU path receives as bf16 are received here as the same bf16 bit
 * patterns (uint16) and widened exactly to double; all arithmetic after that is double.
 * A "unit" is one (problem, head) pair; units are independent (OpenMP runs them in
 * parallel, which changes no result).
 *
 * Readings of the paper taken here:
 *  - Eq. 1: ordinary causal softmax, the denominator runs over keys m' <= m, so every
 *    row of A sums to one. An explicit `scale` multiplies the dot product.
 *  - Positions are 0-based, 0..T-1; Eq. 2's last bucket ends at T-1 and every bucket
 *    after the first starts one past the previous bucket's end (a partition).
 *  - A token half-way between two anchors goes to the earlier anchor (floor in Eq. 2).
 *  - Anchors: the C highest scores, equal scores resolved toward the lower position.
 *  - Eq. 3: plain mean over the bucket, the anchor's own vector included.
 *  - Fixed-point elimination: after appending the new row, the row that has exactly
 *    `offset` rows behind it is deleted (Algorithm 1's fix_idx with P = -offset).
 *  - Mean, maximum and moving-average importance (named in Sec. 3.2 without formulas): the
 *    definitions written above eco_importance_statistic.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_double(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Widen n bf16 values. */
void eco_widen_bf16(const uint16_t *src, int64_t n, double *dst)
{
    for (int64_t i = 0; i < n; ++i) dst[i] = bf16_to_double(src[i]);
}

/* Round double to bf16, nearest, ties to even, in one rounding (normal range only;
 * magnitudes below 2^-126 go through float, which is exact enough for a zero check). */
static uint16_t double_to_bf16(double x)
{
    if (x != x) return 0x7FC0;
    double ax = fabs(x);
    if (ax < 1.1754943508222875e-38) { /* below the smallest normal float */
        float f = (float)x;
        uint32_t u;
        memcpy(&u, &f, 4);
        uint32_t r = (u + 0x7FFFu + ((u >> 16) & 1u)) >> 16;
        return (uint16_t)r;
    }
    uint64_t b;
    memcpy(&b, &x, 8);
    uint64_t sign = b >> 63;
    int64_t e = (int64_t)((b >> 52) & 0x7FF) - 1023 + 127; /* float-biased exponent */
    uint64_t mant = b & 0xFFFFFFFFFFFFFull;               /* 52 bits */
    uint64_t keep = mant >> 45;                            /* top 7 bits */
    uint64_t rem = mant & ((1ull << 45) - 1);
    uint64_t half = 1ull << 44;
    if (rem > half || (rem == half && (keep & 1ull))) {
        keep += 1;
        if (keep == 128) { keep = 0; e += 1; }
    }
    if (e >= 255) return (uint16_t)((sign << 15) | 0x7F80u); /* overflow to inf */
    return (uint16_t)((sign << 15) | ((uint64_t)e << 7) | keep);
}

void eco_round_bf16(const double *src, int64_t n, uint16_t *dst)
{
    for (int64_t i = 0; i < n; ++i) dst[i] = double_to_bf16(src[i]);
}

/* Algorithm 1 computes the number of removed entries as int(seq_len - n*(1 - r)) where
 * (1 - r) is the retained fraction; at the prompt call n = seq_len = T, so
 * int(T - T*ratio) rows are merged away and the rest are kept. */
int eco_keep_count(int T, double ratio)
{
    int del = (int)((double)T - (double)T * ratio);
    if (del < 0) del = 0;
    int keep = T - del;
    if (keep < 1) keep = 1;
    if (keep > T) keep = T;
    return keep;
}

/*
 * Sec. 3.3 "Instruction Encoding", Eq. 1 and the importance definition that follows it:
 * A[m][n] = softmax over n <= m of scale*<q_m,k_n>;  I[n] = sum_m A[m][n].
 * Q, K: bf16 [U, T, D].  scores: [U, T].  lse (nullable): [U, T], the natural-log
 * normaliser of each query row.
 */
void eco_importance(const uint16_t *Q, const uint16_t *K, int U, int T, int D, double scale,
                    double *scores, double *lse)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < U; ++u) {
        double *q = (double *)malloc(sizeof(double) * (size_t)T * D);
        double *k = (double *)malloc(sizeof(double) * (size_t)T * D);
        double *s = (double *)malloc(sizeof(double) * (size_t)T);
        eco_widen_bf16(Q + (size_t)u * T * D, (int64_t)T * D, q);
        eco_widen_bf16(K + (size_t)u * T * D, (int64_t)T * D, k);
        double *I = scores + (size_t)u * T;
        for (int n = 0; n < T; ++n) I[n] = 0.0;
        for (int m = 0; m < T; ++m) {
            double mx = -INFINITY;
            for (int n = 0; n <= m; ++n) {
                double dot = 0.0;
                for (int c = 0; c < D; ++c) dot += q[(size_t)m * D + c] * k[(size_t)n * D + c];
                s[n] = scale * dot;
                if (s[n] > mx) mx = s[n];
            }
            double Z = 0.0;
            for (int n = 0; n <= m; ++n) Z += exp(s[n] - mx);
            for (int n = 0; n <= m; ++n) I[n] += exp(s[n] - mx) / Z;
            if (lse) lse[(size_t)u * T + m] = mx + log(Z);
        }
        free(q);
        free(k);
        free(s);
    }
}

/*
 * The same definition when the queries are only the LAST Tq tokens of a sequence of P + Tq keys
 * (a new instruction encoded on top of P rows that are already in the cache, Sec. 3.1: the
 * instruction stage also covers chat history): query m sees keys n <= m + P, and
 * I[n] = sum over the Tq queries of A[m][n]. P = 0 is eco_importance.
 * Q: bf16 [U, Tq, D]; K: bf16 [U, P+Tq, D]; scores [U, P+Tq]; lse (nullable) [U, Tq].
 */
void eco_importance_prefix(const uint16_t *Q, const uint16_t *K, int U, int Tq, int P, int D, double scale,
                           double *scores, double *lse)
{
    const int Tk = P + Tq;
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < U; ++u) {
        double *q = (double *)malloc(sizeof(double) * (size_t)Tq * D);
        double *k = (double *)malloc(sizeof(double) * (size_t)Tk * D);
        double *s = (double *)malloc(sizeof(double) * (size_t)Tk);
        eco_widen_bf16(Q + (size_t)u * Tq * D, (int64_t)Tq * D, q);
        eco_widen_bf16(K + (size_t)u * Tk * D, (int64_t)Tk * D, k);
        double *I = scores + (size_t)u * Tk;
        for (int n = 0; n < Tk; ++n) I[n] = 0.0;
        for (int m = 0; m < Tq; ++m) {
            const int last = m + P;
            double mx = -INFINITY;
            for (int n = 0; n <= last; ++n) {
                double dot = 0.0;
                for (int c = 0; c < D; ++c) dot += q[(size_t)m * D + c] * k[(size_t)n * D + c];
                s[n] = scale * dot;
                if (s[n] > mx) mx = s[n];
            }
            double Z = 0.0;
            for (int n = 0; n <= last; ++n) Z += exp(s[n] - mx);
            for (int n = 0; n <= last; ++n) I[n] += exp(s[n] - mx) / Z;
            if (lse) lse[(size_t)u * Tq + m] = mx + log(Z);
        }
        free(q);
        free(k);
        free(s);
    }
}

/*
 * The forward pass whose attention Algorithm 1 takes as its input ("Input: ... attn"): the causal
 * attention output of the prompt tokens, out[m] = sum_{n <= m+P} A[m][n] * v_n with A as in Eq. 1,
 * together with each row's natural-log normaliser. Same geometry as eco_importance_prefix.
 * Q: bf16 [U, Tq, D]; K, V: bf16 [U, P+Tq, D]; out: [U, Tq, D]; lse (nullable): [U, Tq].
 */
void eco_attention_prefix(const uint16_t *Q, const uint16_t *K, const uint16_t *V, int U, int Tq, int P, int D,
                          double scale, double *out, double *lse)
{
    const int Tk = P + Tq;
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < U; ++u) {
        double *q = (double *)malloc(sizeof(double) * (size_t)Tq * D);
        double *k = (double *)malloc(sizeof(double) * (size_t)Tk * D);
        double *v = (double *)malloc(sizeof(double) * (size_t)Tk * D);
        double *s = (double *)malloc(sizeof(double) * (size_t)Tk);
        eco_widen_bf16(Q + (size_t)u * Tq * D, (int64_t)Tq * D, q);
        eco_widen_bf16(K + (size_t)u * Tk * D, (int64_t)Tk * D, k);
        eco_widen_bf16(V + (size_t)u * Tk * D, (int64_t)Tk * D, v);
        for (int m = 0; m < Tq; ++m) {
            const int last = m + P;
            double mx = -INFINITY;
            for (int n = 0; n <= last; ++n) {
                double dot = 0.0;
                for (int c = 0; c < D; ++c) dot += q[(size_t)m * D + c] * k[(size_t)n * D + c];
                s[n] = scale * dot;
                if (s[n] > mx) mx = s[n];
            }
            double Z = 0.0;
            for (int n = 0; n <= last; ++n) Z += exp(s[n] - mx);
            double *o = out + ((size_t)u * Tq + m) * D;
            for (int c = 0; c < D; ++c) o[c] = 0.0;
            for (int n = 0; n <= last; ++n) {
                const double a = exp(s[n] - mx) / Z;
                for (int c = 0; c < D; ++c) o[c] += a * v[(size_t)n * D + c];
            }
            if (lse) lse[(size_t)u * Tq + m] = mx + log(Z);
        }
        free(q);
        free(k);
        free(v);
        free(s);
    }
}

/*
 * Other statistics of the attention a key receives (Sec. 3.2 "Importance Metrics" lists summation,
 * moving average, maximum value and mean; the ablation on the importance metric compares moving
 * average, mean and sum). The paper prints no formulas for them; the readings taken here:
 *   stat 0  sum             I[n] = sum_m A[m][n]                            (eco_importance_prefix)
 *   stat 1  mean            I[n] = (sum_m A[m][n]) / #{queries m that can see key n}
 *   stat 2  maximum         I[n] = max_m A[m][n]
 *   stat 3  moving average  E starts at zero; after each query m, in order,
 *                           E[n] <- beta*E[n] + (1-beta)*A[m][n] for every key n
 *                           (A[m][n] = 0 for keys the query cannot see); I = E after the last query
 * Same geometry as eco_importance_prefix: Tq queries, P + Tq keys, query m sees keys n <= m + P.
 * Q: bf16 [U, Tq, D]; K: bf16 [U, P+Tq, D]; scores [U, P+Tq]. beta is read for stat 3 only.
 * Returns 0, or -1 for an unknown stat.
 */
int eco_importance_statistic(const uint16_t *Q, const uint16_t *K, int U, int Tq, int P, int D, double scale,
                             int stat, double beta, double *scores)
{
    if (stat < 0 || stat > 3) return -1;
    const int Tk = P + Tq;
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < U; ++u) {
        double *q = (double *)malloc(sizeof(double) * (size_t)Tq * D);
        double *k = (double *)malloc(sizeof(double) * (size_t)Tk * D);
        double *a = (double *)malloc(sizeof(double) * (size_t)Tk);
        eco_widen_bf16(Q + (size_t)u * Tq * D, (int64_t)Tq * D, q);
        eco_widen_bf16(K + (size_t)u * Tk * D, (int64_t)Tk * D, k);
        double *I = scores + (size_t)u * Tk;
        for (int n = 0; n < Tk; ++n) I[n] = 0.0;
        for (int m = 0; m < Tq; ++m) {
            const int last = m + P;
            /* row m of A (Eq. 1), zero past the causal limit */
            double mx = -INFINITY;
            for (int n = 0; n <= last; ++n) {
                double dot = 0.0;
                for (int c = 0; c < D; ++c) dot += q[(size_t)m * D + c] * k[(size_t)n * D + c];
                a[n] = scale * dot;
                if (a[n] > mx) mx = a[n];
            }
            double Z = 0.0;
            for (int n = 0; n <= last; ++n) Z += exp(a[n] - mx);
            for (int n = 0; n <= last; ++n) a[n] = exp(a[n] - mx) / Z;
            for (int n = last + 1; n < Tk; ++n) a[n] = 0.0;
            /* fold the row into the statistic */
            for (int n = 0; n < Tk; ++n) {
                if (stat == 0 || stat == 1) I[n] += a[n];
                else if (stat == 2) { if (a[n] > I[n]) I[n] = a[n]; }
                else I[n] = beta * I[n] + (1.0 - beta) * a[n];
            }
        }
        if (stat == 1)
            for (int n = 0; n < Tk; ++n) {
                int seen_by = 0;                         /* queries m with n <= m + P */
                for (int m = 0; m < Tq; ++m) if (n <= m + P) ++seen_by;
                I[n] /= (double)seen_by;
            }
        free(q);
        free(k);
        free(a);
    }
    return 0;
}

/* Layer-wise population: the mean over the heads of a layer. scores [N, H, T] -> out [N, T]. */
void eco_layer_mean(const double *scores, int N, int H, int T, double *out)
{
    for (int n = 0; n < N; ++n)
        for (int t = 0; t < T; ++t) {
            double acc = 0.0;
            for (int h = 0; h < H; ++h) acc += scores[((size_t)n * H + h) * T + t];
            out[(size_t)n * T + t] = acc / (double)H;
        }
}

/* Population shared by `share` consecutive units (Sec. 3.2 "population types"; ablation on the
 * importance population): share = 1 is head-wise, share = H is layer-wise, share = L*H makes one
 * score vector per sequence ("identical" for all layers). scores [G*share, T] -> out [G, T]. */
void eco_group_mean(const double *scores, int G, int share, int T, double *out)
{
    for (int g = 0; g < G; ++g)
        for (int t = 0; t < T; ++t) {
            double acc = 0.0;
            for (int j = 0; j < share; ++j) acc += scores[((size_t)g * share + j) * T + t];
            out[(size_t)g * T + t] = acc / (double)share;
        }
}

/* Eviction instead of merging (the ablation's "cache eviction" row): the kept rows are the
 * anchors' own rows, everything else is dropped. X: bf16 [U, T, D]; anchors [U, C]; out [U, C, D]. */
void eco_gather(const uint16_t *X, int U, int T, int D, const int32_t *anchors, int C, double *out)
{
    for (int u = 0; u < U; ++u)
        for (int k = 0; k < C; ++k)
            for (int c = 0; c < D; ++c)
                out[((size_t)u * C + k) * D + c] = bf16_to_double(X[((size_t)u * T + anchors[(size_t)u * C + k]) * D + c]);
}

typedef struct {
    double score;
    int32_t pos;
} eco_ranked;

static int eco_rank_cmp(const void *a, const void *b)
{
    const eco_ranked *x = (const eco_ranked *)a, *y = (const eco_ranked *)b;
    if (x->score > y->score) return -1;
    if (x->score < y->score) return 1;
    return (x->pos > y->pos) - (x->pos < y->pos);
}

static int eco_int_cmp(const void *a, const void *b)
{
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

/*
 * Anchor selection: the C positions with the highest importance, listed in ascending
 * position order (the indices t_k of Sec. 3.3). With protect_ends the first and the last
 * prompt position are always anchors (the implementation detail of Sec. 4.1); when
 * C == 1 only position 0 is forced.
 * scores [U, T] -> anchors [U, C].
 */
void eco_select(const double *scores, int U, int T, int C, int protect_ends, int32_t *anchors)
{
    for (int u = 0; u < U; ++u) {
        eco_ranked *r = (eco_ranked *)malloc(sizeof(eco_ranked) * (size_t)T);
        for (int t = 0; t < T; ++t) {
            r[t].score = scores[(size_t)u * T + t];
            r[t].pos = t;
        }
        if (protect_ends) {
            r[0].score = INFINITY;
            if (C >= 2) r[T - 1].score = INFINITY;
        }
        qsort(r, (size_t)T, sizeof(eco_ranked), eco_rank_cmp);
        int32_t *a = anchors + (size_t)u * C;
        for (int k = 0; k < C; ++k) a[k] = r[k].pos;
        qsort(a, (size_t)C, sizeof(int32_t), eco_int_cmp);
        free(r);
    }
}

/*
 * Eq. 2: bucket k covers positions lo[k]..hi[k] (inclusive); hi[k] is the floor of the
 * midpoint between anchor k and anchor k+1, the first bucket starts at 0 and the last
 * ends at T-1. anchors [U, C] ascending -> lo, hi [U, C].
 */
void eco_buckets(const int32_t *anchors, int U, int T, int C, int32_t *lo, int32_t *hi)
{
    for (int u = 0; u < U; ++u) {
        const int32_t *t = anchors + (size_t)u * C;
        int32_t *l = lo + (size_t)u * C, *h = hi + (size_t)u * C;
        for (int k = 0; k < C; ++k) {
            l[k] = (k == 0) ? 0 : (t[k - 1] + t[k]) / 2 + 1;
            h[k] = (k == C - 1) ? T - 1 : (t[k] + t[k + 1]) / 2;
        }
    }
}

/*
 * Eq. 3: each kept row is the mean of the rows of its bucket.
 * X: bf16 [U, T, D] (K or V); lo, hi [U, C]; out: double [U, C, D].
 */
void eco_merge(const uint16_t *X, int U, int T, int D, const int32_t *lo, const int32_t *hi, int C,
               double *out)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < U; ++u) {
        for (int k = 0; k < C; ++k) {
            int a = lo[(size_t)u * C + k], b = hi[(size_t)u * C + k];
            double *o = out + ((size_t)u * C + k) * D;
            for (int c = 0; c < D; ++c) {
                double acc = 0.0;
                for (int t = a; t <= b; ++t) acc += bf16_to_double(X[((size_t)u * T + t) * D + c]);
                o[c] = acc / (double)(b - a + 1);
            }
        }
    }
}

/*
 * One generation step for U independent units that share the cache length
 * (Sec. 3.3 "Output Generation"; Algorithm 1's last branch).
 *
 * Kl, Vl: double [U, cap, D], rows 0..*len-1 valid, in queue order.
 * ids:    int64 [cap], the identity of each queue position (shared by all units: the
 *         eviction rule looks only at positions, never at contents).
 * q, k_new, v_new: bf16 [U, D].
 * Steps: (i) append (k_new, v_new) at the tail with identity new_id; (ii) out =
 * softmax(scale * q K^T) V over all *len+1 rows; (iii) eviction:
 *   policy 0 (fixed budget): if the length exceeds `budget`, delete one row;
 *   policy 1 (retention ratio): Algorithm 1 is called after the forward pass, so its
 *            seq_len is the cache length with the new row in it, and its n ("number of
 *            tokens") counts every token processed so far, the new one included, just as
 *            at the prompt call n = seq_len = T counts the whole prompt. With n_seen the
 *            tokens processed before this step: del = int(length - (n_seen + 1)*ratio),
 *            `ratio` being the retained fraction (Alg. 1's 1 - r); one row is deleted only
 *            when del >= 1, otherwise the cache keeps the new row and grows.
 * The deleted queue position is length - 1 - offset (0-based), so `offset` rows stay
 * behind it. Rows after it move up by one, as the concatenation of the two slices does.
 * Returns the deleted queue position, or -1 when nothing was deleted. *evicted_id gets
 * the identity of the deleted row (or -1).
 */
int eco_decode_step(double *Kl, double *Vl, int64_t *ids, int U, int cap, int D, int *len,
                    const uint16_t *q, const uint16_t *k_new, const uint16_t *v_new, double scale,
                    int64_t new_id, int policy, int budget, int offset, double ratio, int64_t n_seen,
                    double *out, int64_t *evicted_id)
{
    int L = *len;
    if (L + 1 > cap) return -2;
    ids[L] = new_id;
    int Lp = L + 1;
#pragma omp parallel for schedule(static)
    for (int u = 0; u < U; ++u) {
        double *Ku = Kl + (size_t)u * cap * D, *Vu = Vl + (size_t)u * cap * D;
        for (int c = 0; c < D; ++c) {
            Ku[(size_t)L * D + c] = bf16_to_double(k_new[(size_t)u * D + c]);
            Vu[(size_t)L * D + c] = bf16_to_double(v_new[(size_t)u * D + c]);
        }
        double *s = (double *)malloc(sizeof(double) * (size_t)Lp);
        double mx = -INFINITY;
        for (int j = 0; j < Lp; ++j) {
            double dot = 0.0;
            for (int c = 0; c < D; ++c) dot += bf16_to_double(q[(size_t)u * D + c]) * Ku[(size_t)j * D + c];
            s[j] = scale * dot;
            if (s[j] > mx) mx = s[j];
        }
        double Z = 0.0;
        for (int j = 0; j < Lp; ++j) Z += exp(s[j] - mx);
        double *o = out + (size_t)u * D;
        for (int c = 0; c < D; ++c) o[c] = 0.0;
        for (int j = 0; j < Lp; ++j) {
            double p = exp(s[j] - mx) / Z;
            for (int c = 0; c < D; ++c) o[c] += p * Vu[(size_t)j * D + c];
        }
        free(s);
    }
    int del;
    if (policy == 0) {
        del = (Lp > budget) ? 1 : 0;
    } else {
        const int64_t n = n_seen + 1;                       /* this step's token is counted */
        del = (int)floor((double)Lp - (double)n * ratio);
        if (del < 0) del = 0;
    }
    if (del < 1) {
        *len = Lp;
        *evicted_id = -1;
        return -1;
    }
    int fix = Lp - 1 - offset;
    if (fix < 0) fix = 0;
    *evicted_id = ids[fix];
    for (int j = fix; j < Lp - 1; ++j) ids[j] = ids[j + 1];
    for (int u = 0; u < U; ++u) {
        double *Ku = Kl + (size_t)u * cap * D, *Vu = Vl + (size_t)u * cap * D;
        memmove(Ku + (size_t)fix * D, Ku + (size_t)(fix + 1) * D, sizeof(double) * (size_t)(Lp - 1 - fix) * D);
        memmove(Vu + (size_t)fix * D, Vu + (size_t)(fix + 1) * D, sizeof(double) * (size_t)(Lp - 1 - fix) * D);
    }
    *len = Lp - 1;
    return fix;
}

int eco_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = (int)omp_get_num_threads();
    }
#endif
    return n;
}
