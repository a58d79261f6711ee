/*
 * PrefixKV CPU oracle -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, single-threaded restatement of what the PrefixKV hot path
 * computes, written from the paper's definitions.  It exists so that the CUDA
 * library can be checked element by element; it shares no code, header, table
 * or helper with that library, and nothing in the product may call it.
 *
 * Floating-point work is done in fp64 (inputs arrive as fp32 values, which
 * hold bf16 exactly); the two places where an fp32 value decides an integer
 * (the sort key and the fixed-point weight) use the fp32 score itself.
 *
 * Notation follows the paper: L layers, H heads, N prompt tokens, D head dim,
 * I_l^n importance, s_l^j sorted indices, P_l^o cumulative priority, p the
 * information-retention ratio, R_l retained ratio (here the integer R_l * N).
 *
 * Pins (tests/test_oracle_*.py): harmonic-number closed form and softmax
 * column sums via a library softmax for the score; a library log-sum-exp and
 * the closed form log(m) for zero queries for the normaliser; library stable sort for the
 * order; exact rational arithmetic for the cumulative weights; brute-force
 * enumeration of every breakpoint of p and a hand-worked example for the
 * search; library dense attention for decode; a hand example, one-hot keys
 * and a library normalised matrix product for cache merging.  Unpinned: nothing in this file
 * (iteration counts and model quality reported by the paper are not
 * reproducible without its data and are not claimed).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum {
    ORC_OK = 0,
    ORC_BAD_SCORE = 1,        /* NaN, inf or negative importance          */
    ORC_RANGE = 2,            /* fixed-point total does not fit in 2^53   */
    ORC_BUDGET_TOO_SMALL = 3, /* budget < L: one row per layer is minimal */
    ORC_BAD_LENGTH = 4        /* given length outside [1, N]              */
};

/* ------------------------------------------------------------------------
 * Importance score, Sec. 3.2: a_l^{i,m,n} is the causal softmax over keys
 * j <= m of scale * (q^{i,m} . k^{i,j}); I_l^n averages over heads i the sum
 * over queries m of a_l^{i,m,n}.  (The printed formula has no scale; scale = 1
 * reproduces it.  The max subtraction leaves the quotient unchanged.)
 *
 * q, k: [H][N][D] fp32, one layer of one sample.  out_f32[N] is I rounded once
 * to fp32; out_f64[N] (may be NULL) is the unrounded value.
 * ---------------------------------------------------------------------- */
void orc_score_layer(const float *q, const float *k, int H, int N, int D,
                     double scale, float *out_f32, double *out_f64)
{
    double *col = (double *)calloc((size_t)N, sizeof(double));
    double *s = (double *)malloc((size_t)N * sizeof(double));
    for (int i = 0; i < H; ++i) {
        const float *qh = q + (size_t)i * N * D;
        const float *kh = k + (size_t)i * N * D;
        for (int m = 0; m < N; ++m) {
            double mx = -INFINITY;
            for (int j = 0; j <= m; ++j) {
                double dot = 0.0;
                for (int d = 0; d < D; ++d)
                    dot += (double)qh[(size_t)m * D + d] * (double)kh[(size_t)j * D + d];
                s[j] = scale * dot;
                if (s[j] > mx) mx = s[j];
            }
            double z = 0.0;
            for (int j = 0; j <= m; ++j) z += exp(s[j] - mx);
            for (int j = 0; j <= m; ++j) col[j] += exp(s[j] - mx) / z;
        }
    }
    for (int n = 0; n < N; ++n) {
        double v = col[n] / (double)H;
        if (out_f64) out_f64[n] = v;
        out_f32[n] = (float)v;
    }
    free(s);
    free(col);
}

/* ------------------------------------------------------------------------
 * Normaliser of the same softmax, Sec. 3.2: for every head i and query m the
 * natural logarithm of sum over keys j <= m of exp(scale * (q^{i,m} . k^{i,j})),
 * i.e. the denominator of a_l^{i,m,n} in the log domain.  A prefill attention
 * kernel usually keeps exactly this value per query; the library accepts it in
 * place of recomputing it.  q, k: [H][N][D]; out: [H][N] fp64.
 * ---------------------------------------------------------------------- */
void orc_lse_layer(const float *q, const float *k, int H, int N, int D, double scale,
                   double *out)
{
    double *s = (double *)malloc((size_t)N * sizeof(double));
    for (int i = 0; i < H; ++i) {
        const float *qh = q + (size_t)i * N * D;
        const float *kh = k + (size_t)i * N * D;
        for (int m = 0; m < N; ++m) {
            double mx = -INFINITY;
            for (int j = 0; j <= m; ++j) {
                double dot = 0.0;
                for (int d = 0; d < D; ++d)
                    dot += (double)qh[(size_t)m * D + d] * (double)kh[(size_t)j * D + d];
                s[j] = scale * dot;
                if (s[j] > mx) mx = s[j];
            }
            double z = 0.0;
            for (int j = 0; j <= m; ++j) z += exp(s[j] - mx);
            out[(size_t)i * N + m] = mx + log(z);
        }
    }
    free(s);
}

/* ------------------------------------------------------------------------
 * Priority sequence, Sec. 3.2: indices sorted by importance, descending.
 * Ties are broken by position ascending (the paper is silent; this makes the
 * order unique).  -0.0 and +0.0 compare equal, as IEEE says.  Insertion sort:
 * slow, stable, obviously right.
 * ---------------------------------------------------------------------- */
static int precedes(const float *I, int32_t a, int32_t b)
{
    if (I[a] > I[b]) return 1;
    if (I[a] < I[b]) return 0;
    return a < b;
}

void orc_sort_desc(const float *I, int N, int32_t *order)
{
    for (int n = 0; n < N; ++n) {
        int32_t cur = n;
        int j = n;
        while (j > 0 && precedes(I, cur, order[j - 1])) {
            order[j] = order[j - 1];
            --j;
        }
        order[j] = cur;
    }
}

/* ------------------------------------------------------------------------
 * Cumulative priority, Sec. 3.2: P_l^o = sum_{j <= oN} of the normalised
 * importance of s_l^j.  The normaliser is never divided out: P >= p is tested
 * as cum >= p * total.  Sums are kept in 2^-32 fixed point so that they do not
 * depend on summation order: w = round-half-even(I * 2^32) (the product is
 * exact in fp64), cum[j] = w_0 + ... + w_j in uint64.
 * Returns ORC_BAD_SCORE / ORC_RANGE when the inputs break the preconditions.
 * ---------------------------------------------------------------------- */
int orc_cumulative(const float *I, const int32_t *order, int N, uint64_t *cum)
{
    uint64_t run = 0;
    for (int j = 0; j < N; ++j) {
        float v = I[order[j]];
        if (!(v >= 0.0f) || isinf(v)) return ORC_BAD_SCORE;
        double scaled = ldexp((double)v, 32);
        if (scaled >= 9007199254740992.0) return ORC_RANGE;
        uint64_t w = (uint64_t)llrint(scaled); /* default rounding: half-even */
        run += w;
        if (run >= (1ull << 53)) return ORC_RANGE;
        cum[j] = run;
    }
    return ORC_OK;
}

/* ------------------------------------------------------------------------
 * Retained length of one layer for a given p, Sec. 3.3:
 * R_l = min{ o | P_l^o >= p }, returned as the row count R_l * N in [1, N].
 * p >= 1 keeps everything by definition; otherwise the threshold is
 * theta = ceil(p * total) and the answer is the first 1-based j with
 * cum[j] >= theta.
 * ---------------------------------------------------------------------- */
int32_t orc_length_for_p(const uint64_t *cum, int N, double p)
{
    if (p >= 1.0) return N;
    double total = (double)cum[N - 1];
    volatile double prod = p * total; /* one rounded multiply, no contraction */
    uint64_t theta = (uint64_t)ceil(prod);
    int32_t below = 0;
    for (int j = 0; j < N; ++j)
        if (cum[j] < theta) ++below;
    int32_t n = 1 + below;
    if (n > N) n = N;
    return n;
}

static int64_t total_length(const uint64_t *cum, int L, int N, double p, int32_t *len)
{
    int64_t S = 0;
    for (int l = 0; l < L; ++l) {
        len[l] = orc_length_for_p(cum + (size_t)l * N, N, p);
        S += len[l];
    }
    return S;
}

/* ------------------------------------------------------------------------
 * Binary search for p, Algorithm 1 and Eq. 1, with the budget as an integer
 * number of rows summed over layers (r * L * N).  delta = S(p) - budget.
 * delta == 0 returns p; delta < 0 raises p1; otherwise lowers p2.  The printed
 * loop condition never becomes false, so the search also stops when the
 * interval is no wider than tol, after max_iters evaluations, or when fp64
 * cannot split the interval further; it then returns the lower end p1, whose
 * configuration never exceeds the budget.
 *
 * Sec. 3.3 also lets the search end as soon as delta is within a small
 * threshold (Tab. "robustness-delta": the threshold is a fraction of sum R_l,
 * here a number of rows), after which the configuration is scaled to the
 * budget.  The threshold is given per side: a midpoint is accepted when
 *   -slack_under <= delta <= slack_over.
 * slack_over = 0 never accepts a configuration above the budget; with
 * slack_under = slack_over the test is the printed |delta| <= threshold, and
 * the accepted configuration may exceed the budget until it is rescaled
 * (orc_apportion).
 *
 * cum: [L][N].  Outputs: len[L], *p_out, *iters_out (evaluations of S at a
 * midpoint).  Returns ORC_BUDGET_TOO_SMALL if budget < L.
 * ---------------------------------------------------------------------- */
int orc_search(const uint64_t *cum, int L, int N, int64_t budget, double tol,
               int32_t max_iters, int64_t slack_under, int64_t slack_over, int32_t *len,
               double *p_out, int32_t *iters_out)
{
    *iters_out = 0;
    if (budget < (int64_t)L) {
        *p_out = 0.0;
        for (int l = 0; l < L; ++l) len[l] = 1;
        return ORC_BUDGET_TOO_SMALL;
    }
    if ((int64_t)L * (int64_t)N <= budget) {
        total_length(cum, L, N, 1.0, len);
        *p_out = 1.0;
        return ORC_OK;
    }
    double p1 = 0.0, p2 = 1.0;
    int32_t iters = 0;
    for (;;) {
        double p = (p1 + p2) / 2.0;
        if (p == p1 || p == p2 || iters == max_iters || p2 - p1 <= tol) break;
        int64_t S = total_length(cum, L, N, p, len);
        ++iters;
        int64_t delta = S - budget;
        if (delta >= -slack_under && delta <= slack_over) {
            *p_out = p;
            *iters_out = iters;
            return ORC_OK;
        }
        if (delta < 0) p1 = p; else p2 = p;
    }
    total_length(cum, L, N, p1, len);
    *p_out = p1;
    *iters_out = iters;
    return ORC_OK;
}

/* ------------------------------------------------------------------------
 * Lengths given from outside (offline configuration, Sec. 3.3 last paragraph,
 * or the uniform R_j = r of Sec. 3.2): validate only.
 * ---------------------------------------------------------------------- */
int orc_check_lengths(const int32_t *len_in, int L, int N)
{
    for (int l = 0; l < L; ++l)
        if (len_in[l] < 1 || len_in[l] > N) return ORC_BAD_LENGTH;
    return ORC_OK;
}

/* ------------------------------------------------------------------------
 * Compression after prefilling, Sec. 3.1 / Fig. 2(a): keep the first `len`
 * entries of the priority sequence, the same set for every head.  kept[] lists
 * the retained positions in ascending position; rows are copied in that order.
 * src: [H][N][D]; dst: [len][H][D].
 * ---------------------------------------------------------------------- */
void orc_retained_positions(const int32_t *order, int N, int32_t len, int32_t *kept)
{
    unsigned char *flag = (unsigned char *)calloc((size_t)N, 1);
    for (int j = 0; j < len; ++j) flag[order[j]] = 1;
    int32_t w = 0;
    for (int n = 0; n < N; ++n)
        if (flag[n]) kept[w++] = n;
    free(flag);
}

void orc_gather_rows(const float *src, int H, int N, int D, const int32_t *kept,
                     int32_t len, float *dst)
{
    for (int r = 0; r < len; ++r)
        for (int h = 0; h < H; ++h)
            memcpy(dst + ((size_t)r * H + h) * D,
                   src + ((size_t)h * N + kept[r]) * D, (size_t)D * sizeof(float));
}

/* ------------------------------------------------------------------------
 * Cache merging, Sec. 4.3 ("Eviction or merging", Tab. "merge"): instead of
 * being dropped, every pruned vector is merged into one retained vector.  With
 * Omega_r the retained positions (kept[], ascending) and Omega_p the others,
 * each pruned key k^m is matched to the retained key with the largest metric
 *   Position:  c^{mn} = -|m - n|
 *   Feature:   c^{mn} = (k^m . k^n) / (|k^m| |k^n|)     (0 when a norm is 0)
 * T^n collects the pruned positions matched to n, and the retained vector is
 * replaced by the plain average of itself and the vectors in T^n.  The
 * operation is done per head and is the same for keys and values.
 * Readings (the paper is silent): the match is taken on the keys and applied to
 * the values as well; among equal metrics the retained vector at the lower
 * position wins.
 *
 * orc_merge_match: k [H][N][D]; match[H][N] receives, for every position, the
 * index r into kept[] it belongs to (its own index for a retained position).
 * gap[H][N] (may be NULL) receives best minus second-best metric of a pruned
 * position (+inf when only one candidate), so that a test can tell a real
 * decision from a near tie.  mode: 1 = Position, 2 = Feature.
 * ---------------------------------------------------------------------- */
void orc_merge_match(const float *k, int H, int N, int D, const int32_t *kept, int32_t len,
                     int mode, int32_t *match, double *gap)
{
    int32_t *slot = (int32_t *)malloc((size_t)N * sizeof(int32_t));
    for (int n = 0; n < N; ++n) slot[n] = -1;
    for (int r = 0; r < len; ++r) slot[kept[r]] = r;
    for (int h = 0; h < H; ++h) {
        const float *kh = k + (size_t)h * N * D;
        for (int m = 0; m < N; ++m) {
            int32_t *out = match + (size_t)h * N + m;
            if (slot[m] >= 0) {
                *out = slot[m];
                if (gap) gap[(size_t)h * N + m] = INFINITY;
                continue;
            }
            double best = -INFINITY, second = -INFINITY;
            int32_t arg = -1;
            double nm = 0.0;
            for (int d = 0; d < D; ++d) nm += (double)kh[(size_t)m * D + d] * (double)kh[(size_t)m * D + d];
            for (int r = 0; r < len; ++r) {
                const int n = kept[r];
                double c;
                if (mode == 1) {
                    c = -fabs((double)m - (double)n);
                } else {
                    double dot = 0.0, nn = 0.0;
                    for (int d = 0; d < D; ++d) {
                        dot += (double)kh[(size_t)m * D + d] * (double)kh[(size_t)n * D + d];
                        nn += (double)kh[(size_t)n * D + d] * (double)kh[(size_t)n * D + d];
                    }
                    c = (nm > 0.0 && nn > 0.0) ? dot / (sqrt(nm) * sqrt(nn)) : 0.0;
                }
                if (c > best) { /* strict: an equal metric later in kept[] (a higher position) loses */
                    second = best;
                    best = c;
                    arg = r;
                } else if (c > second) {
                    second = c;
                }
            }
            *out = arg;
            if (gap) gap[(size_t)h * N + m] = best - second;
        }
    }
    free(slot);
}

/* The merged cache rows for a given assignment: dst[r][h][:] = average of src[h][kept[r]][:] and
 * of every src[h][m][:] with match[h][m] == r, m not retained.  src [H][N][D]; dst [len][H][D]. */
void orc_merge_rows(const float *src, int H, int N, int D, const int32_t *kept, int32_t len,
                    const int32_t *match, double *dst)
{
    int32_t *count = (int32_t *)malloc((size_t)len * sizeof(int32_t));
    for (int h = 0; h < H; ++h) {
        for (int r = 0; r < len; ++r) {
            count[r] = 0;
            for (int d = 0; d < D; ++d) dst[((size_t)r * H + h) * D + d] = 0.0;
        }
        for (int m = 0; m < N; ++m) {
            const int32_t r = match[(size_t)h * N + m];
            count[r] += 1; /* the retained vector itself is listed under its own index */
            for (int d = 0; d < D; ++d)
                dst[((size_t)r * H + h) * D + d] += (double)src[((size_t)h * N + m) * D + d];
        }
        for (int r = 0; r < len; ++r)
            for (int d = 0; d < D; ++d) dst[((size_t)r * H + h) * D + d] /= (double)count[r];
    }
    free(count);
}

/* ------------------------------------------------------------------------
 * Decode attention, Sec. 3.1: the newest token's query attends to every cached
 * row (its own key/value row has already been appended).
 * kc, vc: [rows][H][D]; q: [H][D]; out: [H][D] in fp64.
 * ---------------------------------------------------------------------- */
void orc_decode_attn(const float *q, const float *kc, const float *vc, int rows,
                     int H, int D, double scale, double *out)
{
    double *s = (double *)malloc((size_t)rows * sizeof(double));
    for (int h = 0; h < H; ++h) {
        double mx = -INFINITY;
        for (int r = 0; r < rows; ++r) {
            double dot = 0.0;
            for (int d = 0; d < D; ++d)
                dot += (double)q[(size_t)h * D + d] * (double)kc[((size_t)r * H + h) * D + d];
            s[r] = scale * dot;
            if (s[r] > mx) mx = s[r];
        }
        double z = 0.0;
        for (int r = 0; r < rows; ++r) z += exp(s[r] - mx);
        for (int d = 0; d < D; ++d) {
            double acc = 0.0;
            for (int r = 0; r < rows; ++r)
                acc += (exp(s[r] - mx) / z) * (double)vc[((size_t)r * H + h) * D + d];
            out[(size_t)h * D + d] = acc;
        }
    }
    free(s);
}

/* ------------------------------------------------------------------------
 * Lorenz curve / Gini coefficient of a layer's priority sequence, Sec. 3.2
 * (Fig. 3): area between the equality line and the curve, doubled, with the
 * curve drawn over the ascending importance order (trapezoids).
 * ---------------------------------------------------------------------- */
double orc_gini(const float *I, const int32_t *order, int N)
{
    double total = 0.0;
    for (int n = 0; n < N; ++n) total += (double)I[n];
    if (!(total > 0.0)) return 0.0;
    double area = 0.0, run = 0.0;
    for (int j = N - 1; j >= 0; --j) { /* ascending = reverse of the priority order */
        double prev = run;
        run += (double)I[order[j]] / total;
        area += (prev + run) / (2.0 * N);
    }
    return 1.0 - 2.0 * area;
}

/* ------------------------------------------------------------------------
 * Meeting the budget exactly after the search (Sec. 3.3 says the configuration
 * found is scaled to the target budget and prints no formula) and deriving one
 * configuration from several samples (Sec. 3.3, last paragraph; the
 * aggregation is not specified either).  Reading used for both, an integer
 * apportionment:
 *   every layer keeps its one mandatory row; the other E = budget - L rows are
 *   split in proportion to weight[l]: layer l first gets floor(weight[l] * E / W)
 *   rows (W = sum of weights), at most N - 1; what is then left over is dealt
 *   out one row at a time to the layers that still have room, in the order of
 *   their division remainders (largest first, ties to the lower layer), going
 *   round as often as needed.
 *   rescale:  weight[l] = len[l] - 1 of the searched configuration
 *   estimate: weight[l] = sum over samples of (len[b][l] - 1)
 * Properties: the result sums to min(budget, L * N) exactly; a configuration
 * that already sums to the budget is returned unchanged; a configuration below
 * the budget only grows; one above it (a search ended by the two-sided
 * threshold) only shrinks, never below one row.  All arithmetic is integer.
 * ---------------------------------------------------------------------- */
typedef struct {
    int64_t rem;
    int layer;
} orc_rem_t;

static int by_remainder(const void *a, const void *b)
{
    const orc_rem_t *x = (const orc_rem_t *)a, *y = (const orc_rem_t *)b;
    if (x->rem != y->rem) return x->rem > y->rem ? -1 : 1;
    return x->layer < y->layer ? -1 : (x->layer > y->layer ? 1 : 0);
}

int orc_apportion(const int64_t *weight, int L, int64_t budget, int N, int32_t *len_out)
{
    if (budget < (int64_t)L) return ORC_BUDGET_TOO_SMALL;
    int64_t W = 0;
    for (int l = 0; l < L; ++l) {
        if (weight[l] < 0) return ORC_BAD_LENGTH;
        W += weight[l];
    }
    const int64_t E = budget - L, room = (int64_t)N - 1;
    orc_rem_t *queue = (orc_rem_t *)malloc((size_t)L * sizeof(orc_rem_t));
    int64_t left = E;
    for (int l = 0; l < L; ++l) {
        /* all weights zero: every layer counts the same */
        const int64_t w = W == 0 ? 1 : weight[l], sum = W == 0 ? L : W;
        /* w * E < 2^63 for every supported size (w <= 2^30 rows, E <= 2^24 rows) */
        int64_t share = (w * E) / sum;
        if (share > room) share = room;
        len_out[l] = (int32_t)(1 + share);
        left -= share;
        queue[l].rem = (w * E) % sum;
        queue[l].layer = l;
    }
    qsort(queue, (size_t)L, sizeof(orc_rem_t), by_remainder);
    /* one row at a time, round after round, to whoever still has room */
    while (left > 0) {
        int64_t before = left;
        for (int i = 0; i < L && left > 0; ++i) {
            int l = queue[i].layer;
            if (len_out[l] < N) {
                len_out[l] += 1;
                left -= 1;
            }
        }
        if (left == before) break; /* every layer already keeps all N rows */
    }
    free(queue);
    return ORC_OK;
}

/* ------------------------------------------------------------------------
 * Keeping the configuration while decoding (Sec. 3.1: during generation the
 * vectors at a fixed distance behind the newest token are pruned so that the
 * layer-wise configuration is kept; Fig. 2a: the cache keeps the compression
 * proportions found after prefilling).  The distance and the exact rule are left to the
 * cited work; reading used here, per layer:
 *   R_l = len0 / N is the layer's proportion.  When generated token g arrives
 *   (g = 0, 1, ...) the layer may hold floor(len0 * (N + g + 1) / N) rows.  If
 *   adding the token would exceed that, the token generated d steps earlier
 *   (g - d) is dropped -- if it is still cached -- and the new row takes its
 *   slot; otherwise the new row is appended.  Prompt rows are never dropped.
 * ring[d + 1] holds the row index of each of the last d + 1 generated tokens
 * (-1 once dropped), indexed by token % (d + 1).  n = rows cached now.
 * Outputs: *dst = row the new token is written to, *evict = 1 if it replaced
 * token g - d; returns the row count afterwards.  d = 0 never drops anything.
 * ---------------------------------------------------------------------- */
int32_t orc_decode_slot(int32_t len0, int32_t N, int32_t g, int32_t n, int32_t d, int32_t *ring,
                        int32_t *dst, int32_t *evict)
{
    *evict = 0;
    *dst = n;
    if (d > 0) {
        int64_t target = ((int64_t)len0 * ((int64_t)N + g + 1)) / N;
        if ((int64_t)n + 1 > target && g >= d && ring[(g - d) % (d + 1)] >= 0) {
            *evict = 1;
            *dst = ring[(g - d) % (d + 1)];
            ring[(g - d) % (d + 1)] = -1;
        }
        ring[g % (d + 1)] = *dst;
    }
    return *evict ? n : n + 1;
}
