/*
 * CPU oracle for Dodo's compressed-context inference path (arXiv 2310.02409).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain definition of what the
 * path computes, written out in fp64 with no blocking, fusion or reordering,
 * so that a reader can check it against the paper by eye.  It shares no code,
 * header, table or helper with the CUDA library and must never be called from
 * the product path.  Only the tests, the smoke check and the benchmark's CPU
 * baseline leg may load it.
 *
 * What each function follows:
 *   oracle_num_nuggets  k = ceil(n / r)                       Sec. 2.3, text before Eq. 14
 *   oracle_score        s_i = Scorer(x_i), linear form         Eq. 6, Eq. 15
 *   oracle_score_mlp    s_i = Scorer(x_i), two-layer form      Eq. 6, App. B.3 / Table 5 (d -> d -> 1)
 *   oracle_select       TopK(x_{1:n}, s_{1:n}, k)              Eq. 14 (+ its footnote)
 *   oracle_select_threshold   alpha_i = 1{s_i > Lambda}        Eq. 8
 *   oracle_estimate_threshold Lambda from sampled scores       Sec. 2.5, text after Eq. 8
 *   oracle_gather       {z_j} = {x_i : alpha_i = 1}            Eq. 5
 *   oracle_attend       Attn(x_t, [z_{1:k} ; x_{t-tau:t}])     Eq. 4, Eq. 9, Eq. 13, Eq. 16
 *   oracle_pool         mean of every even chunk of r tokens   Sec. 5.1 (the Compressive baseline, mean pooling)
 *
 * Parity pins (tests/test_oracle_pins.py): every function above is pinned to
 * something outside this file -- printed values of k, brute-force subset
 * enumeration for TopK, a library stable argsort, for the two-layer Scorer its
 * reduction to the linear Scorer (identity first layer) and a library matrix
 * product, for the threshold rule its
 * agreement with TopK when Lambda is the (k+1)-th largest score and a library
 * sort for the estimate, byte equality for the gather, and for attention the r = 1 reduction to full causal attention
 * computed by an independent library routine plus closed-form cases; the pooling against a library mean, its r = 1
 * identity and constant segments.
 *
 * Floating-point inputs are stored either as IEEE fp32 or as bf16 (the upper
 * 16 bits of an fp32); both convert to fp64 exactly.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };
enum { ORACLE_FORCE_LAST = 1u };

static double load_elem(const void *base, int dtype, size_t i) {
    if (dtype == ORACLE_F32) {
        return (double)((const float *)base)[i];
    } else {
        uint32_t bits = (uint32_t)((const uint16_t *)base)[i] << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
}

/* k = ceil(n / r), integer arithmetic (n tokens, compression ratio r >= 1). */
int oracle_num_nuggets(int n, int r) {
    int k = n / r;
    if (k * r < n) k += 1;
    return k;
}

/*
 * Linear Scorer: s_i = sum_c x[i][c] * w[c] + bias, summed in index order in
 * fp64.  X is [rows, d] row-major in `dtype`; w is [d] in the same dtype.
 */
void oracle_score(const void *X, int dtype, long rows, int d, const void *w,
                  double bias, double *s_out) {
    long i;
#pragma omp parallel for schedule(static)
    for (i = 0; i < rows; ++i) {
        double acc = 0.0;
        for (int c = 0; c < d; ++c)
            acc += load_elem(X, dtype, (size_t)i * (size_t)d + (size_t)c) *
                   load_elem(w, dtype, (size_t)c);
        s_out[i] = acc + bias;
    }
}

enum { ORACLE_ACT_IDENTITY = 0, ORACLE_ACT_RELU = 1, ORACLE_ACT_GELU_TANH = 2 };

static double activation(double v, int act) {
    if (act == ORACLE_ACT_RELU) return v > 0.0 ? v : 0.0;
    if (act == ORACLE_ACT_GELU_TANH)
        return 0.5 * v * (1.0 + tanh(0.7978845608028654 * (v + 0.044715 * v * v * v)));
    return v;
}

/*
 * Two-layer Scorer (Eq. 6 with the feed-forward network of App. B.3, whose parameter count in
 * Table 5 fits d*d + d + d + 1): h = act(W1 x_i + b1), s_i = w2 . h + b2, in fp64, sums in
 * index order.  X is [rows, d], W1 is [dh, d] (one row per hidden unit), b1 and w2 are [dh];
 * X, W1 and w2 are in `dtype`, b1 is fp32, b2 a scalar.  The paper does not name the
 * activation: it is a parameter (identity, ReLU, tanh-form GELU).
 */
void oracle_score_mlp(const void *X, int dtype, long rows, int d, const void *W1, const float *b1,
                      const void *w2, double b2, int dh, int act, double *s_out) {
    long i;
#pragma omp parallel for schedule(static)
    for (i = 0; i < rows; ++i) {
        double s = 0.0;
        for (int n = 0; n < dh; ++n) {
            double h = 0.0;
            for (int c = 0; c < d; ++c)
                h += load_elem(X, dtype, (size_t)i * (size_t)d + (size_t)c) *
                     load_elem(W1, dtype, (size_t)n * (size_t)d + (size_t)c);
            s += activation(h + (double)b1[n], act) * load_elem(w2, dtype, (size_t)n);
        }
        s_out[i] = s + b2;
    }
}

/*
 * Ranking rule for TopK: a ranks strictly before b when a is the larger
 * score.  +0 and -0 compare equal.  NaN ranks after every number (below
 * -inf) and all NaNs tie with each other.
 */
static int ranks_before(double a, double b) {
    if (isnan(a)) return 0;
    if (isnan(b)) return 1;
    return a > b;
}

/* Stable top-down merge sort of positions by descending score. */
static void merge_sort_desc(const double *s, int32_t *order, int32_t *tmp, int lo, int hi) {
    if (hi - lo < 2) return;
    int mid = lo + (hi - lo) / 2;
    merge_sort_desc(s, order, tmp, lo, mid);
    merge_sort_desc(s, order, tmp, mid, hi);
    int a = lo, b = mid, o = lo;
    while (a < mid && b < hi) {
        /* take the right element only when it ranks strictly before the left
           one: equal scores keep their original (ascending position) order */
        if (ranks_before(s[order[b]], s[order[a]])) tmp[o++] = order[b++];
        else tmp[o++] = order[a++];
    }
    while (a < mid) tmp[o++] = order[a++];
    while (b < hi) tmp[o++] = order[b++];
    for (o = lo; o < hi; ++o) order[o] = tmp[o];
}

static int cmp_i32(const void *a, const void *b) {
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

/*
 * TopK over one sequence: sort all positions by descending score with a
 * stable sort (ties therefore go to the lower position), keep the first k,
 * return them in ascending position order.  With ORACLE_FORCE_LAST the last
 * position n-1 is always kept and the remaining k-1 come from positions
 * 0..n-2.  Requires 0 <= k <= n.  Returns 0, or -1 on bad arguments.
 */
int oracle_select(const double *s, int n, int k, unsigned flags, int32_t *idx) {
    if (n < 0 || k < 0 || k > n) return -1;
    if (k == 0) return 0;
    int m = n, kk = k;
    if (flags & ORACLE_FORCE_LAST) { m = n - 1; kk = k - 1; }
    int32_t *order = (int32_t *)malloc(sizeof(int32_t) * (size_t)(m > 0 ? m : 1));
    int32_t *tmp = (int32_t *)malloc(sizeof(int32_t) * (size_t)(m > 0 ? m : 1));
    if (!order || !tmp) { free(order); free(tmp); return -1; }
    for (int i = 0; i < m; ++i) order[i] = i;
    merge_sort_desc(s, order, tmp, 0, m);
    for (int j = 0; j < kk; ++j) idx[j] = order[j];
    qsort(idx, (size_t)kk, sizeof(int32_t), cmp_i32);
    if (flags & ORACLE_FORCE_LAST) idx[k - 1] = n - 1;
    free(order);
    free(tmp);
    return 0;
}

/*
 * Threshold selection over one sequence (Eq. 8): position i is kept iff its
 * score is strictly above Lambda.  Positions come out ascending; the count is
 * returned.  IEEE comparison: a NaN score is never above anything, a NaN
 * Lambda keeps nothing, -0 and +0 compare equal.  `idx` needs room for n.
 */
int oracle_select_threshold(const double *s, int n, double lambda, int32_t *idx) {
    int count = 0;
    for (int i = 0; i < n; ++i)
        if (s[i] > lambda) idx[count++] = i;
    return count;
}

static int cmp_desc_nan_last(const void *a, const void *b) {
    const double x = *(const double *)a, y = *(const double *)b;
    if (ranks_before(x, y)) return -1;
    if (ranks_before(y, x)) return 1;
    return 0;
}

/*
 * Lambda from m sampled scores for compression ratio r (Sec. 2.5: run the
 * Scorer on sampled tokens and set Lambda so that about one token in r is
 * kept).  Reading: with k = ceil(m / r), Lambda is the (k+1)-th largest
 * sample score, so that exactly k of m distinct sample scores pass the
 * strict test of Eq. 8; when k >= m every score must pass and Lambda is -inf.
 * Scores are ranked as in oracle_select (NaN below -inf).
 */
double oracle_estimate_threshold(const double *s, int m, int r) {
    if (m <= 0 || r < 1) return -INFINITY;
    const int k = (m + r - 1) / r;
    if (k >= m) return -INFINITY;
    double *t = (double *)malloc(sizeof(double) * (size_t)m);
    if (!t) return NAN;
    memcpy(t, s, sizeof(double) * (size_t)m);
    qsort(t, (size_t)m, sizeof(double), cmp_desc_nan_last);
    const double lambda = t[k];
    free(t);
    return lambda;
}

/*
 * Nugget gather for one sequence and one of K or V: the rows idx[0..k) of
 * `src` ([n, row_bytes] bytes) are appended to the cache region `cache`
 * ([capacity, row_bytes]) after the `len` rows already there; the absolute
 * position pos_base + idx[j] of each is recorded when cache_pos is non-NULL.
 * Returns the new length, or -1 if the region would overflow.
 */
int oracle_gather(const unsigned char *src, size_t row_bytes, const int32_t *idx, int k,
                  int pos_base, unsigned char *cache, int32_t *cache_pos, int len,
                  int capacity) {
    if (len + k > capacity) return -1;
    for (int j = 0; j < k; ++j) {
        memcpy(cache + (size_t)(len + j) * row_bytes, src + (size_t)idx[j] * row_bytes,
               row_bytes);
        if (cache_pos) cache_pos[len + j] = pos_base + idx[j];
    }
    return len + k;
}

/*
 * Mean pooling of even chunks (the comparison system of Sec. 5.1: the text is cut evenly into segments and the
 * states of each segment are pooled into one vector; the paper uses the mean).  The n rows of `src` ([n, width]
 * elements of `dtype`) are cut into k = ceil(n / r) segments of r consecutive rows (the last one may be shorter);
 * out[j] is the fp64 mean of segment j, summed in row order, and pos[j] = pos_base + the position of the segment's
 * last row (a pooled state stands for everything up to there).  Returns k.
 */
int oracle_pool(const void *src, int dtype, int n, int width, int r, int pos_base, double *out, int32_t *pos) {
    const int k = oracle_num_nuggets(n, r);
    for (int j = 0; j < k; ++j) {
        const int first = j * r;
        const int last = (first + r < n ? first + r : n) - 1;
        for (int c = 0; c < width; ++c) {
            double sum = 0.0;
            for (int i = first; i <= last; ++i) sum += load_elem(src, dtype, (size_t)i * (size_t)width + (size_t)c);
            out[(size_t)j * (size_t)width + (size_t)c] = sum / (double)(last - first + 1);
        }
        if (pos) pos[j] = pos_base + last;
    }
    return k;
}

/*
 * Attention of Tq query tokens of one sequence over [nuggets ; local tokens].
 *
 *   Q        [Tq, H, dh]     query i sits at position q_pos0 + i
 *   cK, cV   [>= clen, H, dh] nugget cache rows, row j at position cpos[j]
 *   lK, lV   [>= llen, H, dh] uncompressed local rows, row j at lpos0 + j
 *   O        [Tq, H, dh] fp64 out;  lse [Tq, H] fp64 out (may be NULL)
 *
 * A key is visible to a query iff key position <= query position.  Per head:
 * logit_j = scale * <q, k_j>;  p = softmax over the visible keys;
 * o = sum_j p_j v_j.  No visible key: o = 0, lse = -inf.
 */
void oracle_attend(const void *Q, int dtype, int Tq, int q_pos0, int H, int dh, double scale,
                   const void *cK, const void *cV, const int32_t *cpos, int clen,
                   const void *lK, const void *lV, int llen, int lpos0,
                   double *O, double *lse) {
    int unit;
#pragma omp parallel for schedule(dynamic, 1)
    for (unit = 0; unit < Tq * H; ++unit) {
        int qi = unit / H, h = unit % H;
        int p_q = q_pos0 + qi;
        int nmax = clen + llen;
        double *logit = (double *)malloc(sizeof(double) * (size_t)(nmax > 0 ? nmax : 1));
        /* (source, row) of each visible key: source 0 = nugget cache, 1 = local */
        int *src = (int *)malloc(sizeof(int) * (size_t)(nmax > 0 ? nmax : 1));
        int *row = (int *)malloc(sizeof(int) * (size_t)(nmax > 0 ? nmax : 1));
        int nvis = 0;
        for (int j = 0; j < clen; ++j)
            if (cpos[j] <= p_q) { src[nvis] = 0; row[nvis] = j; ++nvis; }
        for (int j = 0; j < llen; ++j)
            if (lpos0 + j <= p_q) { src[nvis] = 1; row[nvis] = j; ++nvis; }

        size_t qbase = ((size_t)qi * (size_t)H + (size_t)h) * (size_t)dh;
        double *o = O + qbase;
        for (int c = 0; c < dh; ++c) o[c] = 0.0;
        if (nvis == 0) {
            if (lse) lse[(size_t)qi * (size_t)H + (size_t)h] = -INFINITY;
            free(logit); free(src); free(row);
            continue;
        }
        double mx = -INFINITY;
        for (int v = 0; v < nvis; ++v) {
            const void *Kb = src[v] == 0 ? cK : lK;
            size_t kbase = ((size_t)row[v] * (size_t)H + (size_t)h) * (size_t)dh;
            double dot = 0.0;
            for (int c = 0; c < dh; ++c)
                dot += load_elem(Q, dtype, qbase + (size_t)c) * load_elem(Kb, dtype, kbase + (size_t)c);
            logit[v] = dot * scale;
            if (logit[v] > mx) mx = logit[v];
        }
        double denom = 0.0;
        for (int v = 0; v < nvis; ++v) {
            logit[v] = exp(logit[v] - mx);
            denom += logit[v];
        }
        for (int v = 0; v < nvis; ++v) {
            const void *Vb = src[v] == 0 ? cV : lV;
            size_t vbase = ((size_t)row[v] * (size_t)H + (size_t)h) * (size_t)dh;
            double p = logit[v] / denom;
            for (int c = 0; c < dh; ++c) o[c] += p * load_elem(Vb, dtype, vbase + (size_t)c);
        }
        if (lse) lse[(size_t)qi * (size_t)H + (size_t)h] = mx + log(denom);
        free(logit); free(src); free(row);
    }
}

/* Number of OpenMP threads the parallel loops above will use. */
#ifdef _OPENMP
#include <omp.h>
int oracle_threads(void) { return omp_get_max_threads(); }
void oracle_set_threads(int t) { if (t > 0) omp_set_num_threads(t); }
#else
int oracle_threads(void) { return 1; }
void oracle_set_threads(int t) { (void)t; }
#endif
