/*
 * R-KV compression step -- CPU oracle (TEST INFRASTRUCTURE, not a product path).
 *
 * A plain, slow, double-precision restatement of what one firing of the
 * decode-time KV-cache compression computes for one (sequence, KV head):
 * Section 3.1 (sizes), Eq. 1-3 (attention of the observation queries, max
 * pooled over the GQA group before one softmax), Eq. 4 (sliding max, mean
 * over the alpha queries), Eq. 5 (cosine similarity of keys, zero diagonal),
 * the "retention of recent tokens" rule of Section 3.3, Eq. 6 (mean
 * similarity, softmax), Eq. 7 (joint score), per-head top-k selection and the
 * gather/concatenate of Algorithm 1.
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call
 * this file.  It shares no code with the CUDA library.  No blocking, no
 * fusion, no reordering: every step is the formula written out, so that it
 * can be checked against the paper by eye.
 *
 * Readings taken where the paper is silent or inconsistent:
 *  - kept tokens per head = B_budget in total: k = B_budget - alpha candidates
 *    plus the alpha observation tokens (Section 3.1; Algorithm 1 would keep
 *    B_budget + alpha).
 *  - selection is per KV head (Section 3.4), not on a head-averaged score.
 *  - GQA: max over the G query heads on the scaled logits, then ONE softmax
 *    over the candidate keys (Eq. 2-3).
 *  - Eq. 4 as printed: window {i-W, ..., i+W-1} clipped to [0, n), max per
 *    query row, then the mean over rows.  W = 0 means no pooling.
 *  - "beta most recent" = the beta largest positions j among {j: S[j][i] > T}.
 *  - equal scores: the later position wins.
 *  - kept candidate positions are emitted in ascending order, followed by the
 *    alpha observation positions.
 * Parity unpinned: the VALUES of W, T and beta (the paper prints none); their
 * semantics are pinned by the tests.
 *
 * Floating point: inputs arrive as float (bf16 widened exactly, or fp32); all
 * arithmetic here is double.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* ---- Eq. 2-3 (Eq. 1 when G == 1): attention weights A[alpha][n] ---------- */
static void attention_weights(const float *K, const float *Q, int n, int d,
                              int G, int alpha, int mean_pool, double *A)
{
    const double root_d = sqrt((double)d);
    for (int j = 0; j < alpha; ++j) {
        /* Eq. 2: scaled logits of each query head g; Eq. 3: max over g.
         * mean_pool (a variant, off by default): the mean over g instead, the
         * pooling the paper's appendix ascribes to earlier work; read as Eq. 3
         * with the max replaced, i.e. still on the logits and before the one
         * softmax. */
        for (int i = 0; i < n; ++i) {
            double pooled = -INFINITY, total = 0.0;
            for (int g = 0; g < G; ++g) {
                const float *q = Q + ((size_t)g * alpha + j) * d;
                const float *k = K + (size_t)i * d;
                double dot = 0.0;
                for (int c = 0; c < d; ++c)
                    dot += (double)q[c] * (double)k[c];
                double logit = dot / root_d;
                if (logit > pooled)
                    pooled = logit;
                total += logit;
            }
            A[(size_t)j * n + i] = mean_pool ? total / (double)G : pooled;
        }
        /* Eq. 3: softmax along the key dimension */
        double top = -INFINITY;
        for (int i = 0; i < n; ++i)
            if (A[(size_t)j * n + i] > top)
                top = A[(size_t)j * n + i];
        double denom = 0.0;
        for (int i = 0; i < n; ++i)
            denom += exp(A[(size_t)j * n + i] - top);
        for (int i = 0; i < n; ++i)
            A[(size_t)j * n + i] = exp(A[(size_t)j * n + i] - top) / denom;
    }
}

/* ---- Eq. 4: sliding max over keys per query row, then mean over rows ---- */
static void importance_scores(const double *A, int n, int alpha, int W,
                              double *I)
{
    for (int i = 0; i < n; ++i) {
        double acc = 0.0;
        for (int j = 0; j < alpha; ++j) {
            double best = A[(size_t)j * n + i];
            if (W > 0) {
                int lo = i - W, hi = i + W - 1;
                if (lo < 0)
                    lo = 0;
                if (hi > n - 1)
                    hi = n - 1;
                for (int t = lo; t <= hi; ++t)
                    if (A[(size_t)j * n + t] > best)
                        best = A[(size_t)j * n + t];
            }
            acc += best;
        }
        I[i] = acc / (double)alpha;
    }
}

/* ---- Algorithm 1's ordering of the same two steps (a variant, off by default):
 * mean over the alpha query rows first, then the 1-D pooling.  The algorithm box
 * names neither the pooling's kind nor its size; it is read as the max pooling
 * of Eq. 4 over the same window {i-W, ..., i+W-1}. ---------------------------- */
static void importance_scores_mean_first(const double *A, int n, int alpha,
                                         int W, double *I)
{
    double *mean = (double *)malloc((size_t)n * sizeof(double));
    for (int i = 0; i < n; ++i) {
        double acc = 0.0;
        for (int j = 0; j < alpha; ++j)
            acc += A[(size_t)j * n + i];
        mean[i] = acc / (double)alpha;
    }
    for (int i = 0; i < n; ++i) {
        double best = mean[i];
        if (W > 0) {
            int lo = i - W, hi = i + W - 1;
            if (lo < 0)
                lo = 0;
            if (hi > n - 1)
                hi = n - 1;
            for (int t = lo; t <= hi; ++t)
                if (mean[t] > best)
                    best = mean[t];
        }
        I[i] = best;
    }
    free(mean);
}

/* ---- Eq. 5: S = Kbar Kbar^T with zero diagonal ---------------------------- */
static void cosine_matrix(const float *K, int n, int d, double eps, double *S)
{
    double *Kbar = (double *)malloc((size_t)n * d * sizeof(double));
    for (int i = 0; i < n; ++i) {
        double sq = 0.0;
        for (int c = 0; c < d; ++c)
            sq += (double)K[(size_t)i * d + c] * (double)K[(size_t)i * d + c];
        double denom = sqrt(sq) + eps;
        for (int c = 0; c < d; ++c)
            Kbar[(size_t)i * d + c] = (double)K[(size_t)i * d + c] / denom;
    }
    for (int i = 0; i < n; ++i)
        for (int j = 0; j < n; ++j) {
            double dot = 0.0;
            for (int c = 0; c < d; ++c)
                dot += Kbar[(size_t)i * d + c] * Kbar[(size_t)j * d + c];
            S[(size_t)i * n + j] = dot;
        }
    for (int i = 0; i < n; ++i)
        S[(size_t)i * n + i] = 0.0;
    free(Kbar);
}

/* ---- Section 3.3, retention of recent tokens: for each token i, among the
 * partners {j : S[j][i] > T} zero the entries of the (up to) beta largest j.
 * Column i's rule reads and writes column i only. ------------------------- */
static void retain_recent(double *S, int n, double T, int beta)
{
    for (int i = 0; i < n; ++i) {
        int zeroed = 0;
        for (int j = n - 1; j >= 0 && zeroed < beta; --j)
            if (S[(size_t)j * n + i] > T) {
                S[(size_t)j * n + i] = 0.0;
                ++zeroed;
            }
    }
}

/* ---- Eq. 6: column means and their softmax -------------------------------- */
static void redundancy_scores(const double *S, int n, double *Sbar, double *R)
{
    for (int i = 0; i < n; ++i) {
        double acc = 0.0;
        for (int j = 0; j < n; ++j)
            acc += S[(size_t)j * n + i];
        Sbar[i] = acc / (double)n;
    }
    double top = -INFINITY;
    for (int i = 0; i < n; ++i)
        if (Sbar[i] > top)
            top = Sbar[i];
    double denom = 0.0;
    for (int i = 0; i < n; ++i)
        denom += exp(Sbar[i] - top);
    for (int i = 0; i < n; ++i)
        R[i] = exp(Sbar[i] - top) / denom;
}

/* ---- selection: the k largest Z, later position first among equals ------- */
typedef struct {
    double z;
    int pos;
} scored_t;

static int by_score_then_recency(const void *a, const void *b)
{
    const scored_t *x = (const scored_t *)a, *y = (const scored_t *)b;
    if (x->z > y->z)
        return -1;
    if (x->z < y->z)
        return 1;
    return (x->pos > y->pos) ? -1 : (x->pos < y->pos);
}

static int ascending_int(const void *a, const void *b)
{
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

/* the k candidates with the largest score (later position first among equals),
 * ascending, then the alpha observation positions n .. n + alpha - 1 */
static int select_kept(const double *z, int n, int k, int alpha, int32_t *idx)
{
    scored_t *order = (scored_t *)malloc((size_t)n * sizeof(scored_t));
    if (!order)
        return -1;
    for (int i = 0; i < n; ++i) {
        order[i].z = z[i];
        order[i].pos = i;
    }
    qsort(order, (size_t)n, sizeof(scored_t), by_score_then_recency);
    for (int j = 0; j < k; ++j)
        idx[j] = order[j].pos;
    qsort(idx, (size_t)k, sizeof(int32_t), ascending_int);
    for (int j = 0; j < alpha; ++j) /* observation tokens, always kept */
        idx[k + j] = n + j;
    free(order);
    return 0;
}

/*
 * One (sequence, KV head).
 *   K      [L][d]            keys as float
 *   Q      [G][alpha][d]     observation-window queries of the head's group
 *   idx    [budget]          out: kept positions (see file header)
 *   A, I, Sbar, R, Z         optional outputs ([alpha][n] and [n]); may be NULL
 *   S_raw, S_mod             optional [n][n] dumps of Eq. 5's matrix before and
 *                            after the retention rule; may be NULL
 *   variant                  0 = the method as the equations state it; bit 0 =
 *                            Algorithm 1's order for the importance (mean, then pool);
 *                            bit 2 = mean instead of max over the query heads of a
 *                            group in Eq. 3
 * Returns 1 if the head was compressed, 0 if L <= budget (nothing to do:
 * idx = 0..L-1 then -1), -1 on bad arguments.
 */
int rkv_oracle_head(const float *K, const float *Q, int L, int d, int G,
                    int alpha, int budget, int W, int beta, double T,
                    double eps, double lambda, int32_t *idx, double *A,
                    double *I, double *Sbar, double *R, double *Z,
                    double *S_raw, double *S_mod, int variant)
{
    if (L < 0 || d < 1 || G < 1 || alpha < 1 || budget <= alpha || W < 0 ||
        beta < 0)
        return -1;
    if (L <= budget) { /* Algorithm 1's "not enough candidates" guard */
        for (int j = 0; j < budget; ++j)
            idx[j] = (j < L) ? j : -1;
        return 0;
    }
    const int n = L - alpha;      /* candidates: Section 3.1 */
    const int k = budget - alpha; /* candidates kept */

    double *A_ = (double *)malloc((size_t)alpha * n * sizeof(double));
    double *I_ = (double *)malloc((size_t)n * sizeof(double));
    double *S_ = (double *)malloc((size_t)n * n * sizeof(double));
    double *Sbar_ = (double *)malloc((size_t)n * sizeof(double));
    double *R_ = (double *)malloc((size_t)n * sizeof(double));
    scored_t *order = (scored_t *)malloc((size_t)n * sizeof(scored_t));
    if (!A_ || !I_ || !S_ || !Sbar_ || !R_ || !order) {
        free(A_); free(I_); free(S_); free(Sbar_); free(R_); free(order);
        return -1;
    }

    attention_weights(K, Q, n, d, G, alpha, (variant & 4) != 0, A_);
    if (variant & 1) /* RKV_ORACLE_MEAN_THEN_POOL */
        importance_scores_mean_first(A_, n, alpha, W, I_);
    else
        importance_scores(A_, n, alpha, W, I_);
    cosine_matrix(K, n, d, eps, S_);
    if (S_raw)
        memcpy(S_raw, S_, (size_t)n * n * sizeof(double));
    retain_recent(S_, n, T, beta);
    if (S_mod)
        memcpy(S_mod, S_, (size_t)n * n * sizeof(double));
    redundancy_scores(S_, n, Sbar_, R_);

    for (int i = 0; i < n; ++i) { /* Eq. 7 */
        order[i].z = lambda * I_[i] - (1.0 - lambda) * R_[i];
        order[i].pos = i;
        if (Z)
            Z[i] = order[i].z;
    }
    qsort(order, (size_t)n, sizeof(scored_t), by_score_then_recency);
    for (int j = 0; j < k; ++j)
        idx[j] = order[j].pos;
    qsort(idx, (size_t)k, sizeof(int32_t), ascending_int);
    for (int j = 0; j < alpha; ++j) /* observation tokens, always kept */
        idx[k + j] = n + j;

    if (A) memcpy(A, A_, (size_t)alpha * n * sizeof(double));
    if (I) memcpy(I, I_, (size_t)n * sizeof(double));
    if (Sbar) memcpy(Sbar, Sbar_, (size_t)n * sizeof(double));
    if (R) memcpy(R, R_, (size_t)n * sizeof(double));
    free(A_); free(I_); free(S_); free(Sbar_); free(R_); free(order);
    return 1;
}

/*
 * Algorithm 1's gather: out[j] = in[idx[j]] for j < count, row_bytes each,
 * byte for byte (out and in are distinct buffers here).
 */
void rkv_oracle_gather(const uint8_t *in, const int32_t *idx, int count,
                       size_t row_bytes, uint8_t *out)
{
    for (int j = 0; j < count; ++j)
        if (idx[j] >= 0)
            memcpy(out + (size_t)j * row_bytes,
                   in + (size_t)idx[j] * row_bytes, row_bytes);
}

/*
 * A batch of head-problems, OpenMP over (sequence, KV head).
 *   K   [B][Hkv][cap][d] float, Q [B][Hq][alpha][d] float (query head q
 *   belongs to KV head q / G), seq_lens [B], idx [B][Hkv][budget].
 *   scores: optional [4][B][Hkv][cap] doubles = I, Sbar, R, Z (first n used).
 *   compressed: optional [B] flags.
 *   variant: bits 0 and 2 as in rkv_oracle_head; bit 1 = one kept set per sequence
 *   from the head-averaged score (Algorithm 1) instead of one per KV head.
 * Returns the number of OpenMP threads used, or -1 on bad arguments.
 */
int rkv_oracle_batch(const float *K, const float *Q, const int32_t *seq_lens,
                     int B, int Hkv, int Hq, int cap, int d, int alpha,
                     int budget, int W, int beta, double T, double eps,
                     double lambda, int32_t *idx, double *scores,
                     int32_t *compressed, int variant)
{
    if (Hkv < 1 || Hq % Hkv != 0)
        return -1;
    const int G = Hq / Hkv;
    int bad = 0, threads = 1;
    const size_t plane = (size_t)B * Hkv * cap;
    /* variant bit 1: Algorithm 1's aggregated selection needs every head's Z */
    double *zown = NULL;
    if ((variant & 2) && !scores) {
        zown = (double *)malloc(plane * sizeof(double));
        if (!zown)
            return -1;
    }
    double *zall = scores ? scores + 3 * plane : zown;
#ifdef _OPENMP
    threads = omp_get_max_threads();
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int p = 0; p < B * Hkv; ++p) {
        const int b = p / Hkv, h = p % Hkv;
        const int L = seq_lens[b];
        if (L > cap) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
            bad = 1;
            continue;
        }
        const float *Kp = K + (size_t)p * cap * d;
        const float *Qp = Q + ((size_t)b * Hq + (size_t)h * G) * alpha * d;
        double *sc = scores ? scores + (size_t)p * cap : NULL;
        int r = rkv_oracle_head(Kp, Qp, L, d, G, alpha, budget, W, beta, T,
                                eps, lambda, idx + (size_t)p * budget, NULL,
                                sc, sc ? sc + plane : NULL,
                                sc ? sc + 2 * plane : NULL,
                                zall ? zall + (size_t)p * cap : NULL, NULL, NULL,
                                variant);
        if (r < 0) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
            bad = 1;
        }
        if (compressed && h == 0)
            compressed[b] = (r == 1);
    }
    if ((variant & 2) && !bad) {
        /* Algorithm 1's aggregated selection (a variant, off by default): the
         * scores of a sequence's KV heads are averaged, AggScore_i = mean_h Z_i^h,
         * and ONE set of positions is kept for all of its heads. */
        for (int b = 0; b < B; ++b) {
            const int L = seq_lens[b];
            if (L <= budget)
                continue;
            const int n = L - alpha, k = budget - alpha;
            double *zbar = (double *)malloc((size_t)n * sizeof(double));
            for (int i = 0; i < n; ++i) {
                double acc = 0.0;
                for (int h = 0; h < Hkv; ++h)
                    acc += zall[((size_t)b * Hkv + h) * cap + i];
                zbar[i] = acc / (double)Hkv;
            }
            int32_t *first = idx + (size_t)b * Hkv * budget;
            if (select_kept(zbar, n, k, alpha, first) < 0)
                bad = 1;
            for (int h = 1; h < Hkv; ++h)
                memcpy(first + (size_t)h * budget, first,
                       (size_t)budget * sizeof(int32_t));
            free(zbar);
        }
    }
    free(zown);
    return bad ? -1 : threads;
}

/*
 * Section 3.1's decode step on the cache as it stands (retained tokens plus the
 * buffer): the new token's query of every query head attends over the cached
 * keys of its KV head, Eq. 1 with a single query row,
 *   out[b][q] = sum_j softmax_j( q . K[b][q / G][j] / sqrt(d) ) V[b][q / G][j],
 *   j < seq_lens[b].
 * K, V [B][Hkv][cap][d] float, Qn [B][Hq][d] float, out [B][Hq][d] double.
 * A sequence with no cached token gives a zero row.  Returns 0, or -1 on bad
 * arguments.
 */
int rkv_oracle_decode_attention(const float *K, const float *V, const float *Qn,
                                const int32_t *seq_lens, int B, int Hkv, int Hq,
                                int cap, int d, double *out)
{
    if (B < 1 || Hkv < 1 || Hq % Hkv != 0 || d < 1 || cap < 1)
        return -1;
    const int G = Hq / Hkv;
    int bad = 0;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int bq = 0; bq < B * Hq; ++bq) {
        const int b = bq / Hq, q = bq % Hq, h = q / G;
        const int L = seq_lens[b];
        double *o = out + (size_t)bq * d;
        for (int c = 0; c < d; ++c)
            o[c] = 0.0;
        if (L < 0 || L > cap) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
            bad = 1;
            continue;
        }
        if (L == 0)
            continue;
        const float *Kh = K + ((size_t)b * Hkv + h) * cap * d;
        const float *Vh = V + ((size_t)b * Hkv + h) * cap * d;
        const float *qv = Qn + (size_t)bq * d;
        double *w = (double *)malloc((size_t)L * sizeof(double));
        double mx = -INFINITY;
        for (int j = 0; j < L; ++j) {
            double dot = 0.0;
            for (int c = 0; c < d; ++c)
                dot += (double)qv[c] * (double)Kh[(size_t)j * d + c];
            w[j] = dot / sqrt((double)d);
            if (w[j] > mx)
                mx = w[j];
        }
        double sum = 0.0;
        for (int j = 0; j < L; ++j) {
            w[j] = exp(w[j] - mx);
            sum += w[j];
        }
        for (int j = 0; j < L; ++j) {
            const double a = w[j] / sum;
            for (int c = 0; c < d; ++c)
                o[c] += a * (double)Vh[(size_t)j * d + c];
        }
        free(w);
    }
    return bad ? -1 : 0;
}
