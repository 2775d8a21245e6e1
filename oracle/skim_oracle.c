/*
 * skim_oracle.c -- plain CPU oracle for the SKIM row-clustering path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement of
 * what the path computes.  It shares no code with the CUDA implementation and must
 * never be used by it: only the test-suite, the smoke check and the benchmark's
 * CPU-baseline leg may build, load or call it.
 *
 * What it follows (SKIM, arXiv 2412.04180):
 *   - weighted 1-D K-means of one weight row with per-element importance, objective
 *     sum_j g_ij (w_ij - wq_ij)^2                       -- Section 3.2 (sensitivity,
 *     diagonal form) and Section 4.1 (S-diag for K-means); Algorithm 3, error
 *     pre-recording loop and final clustering loop.
 *   - greedy bit allocation                               -- Section 4.2, Algorithm 1.
 *   - scaling vector  Wq = Quant(W * alpha^-1) * alpha    -- Section 4.3, Algorithm 2.
 *   - packing rows grouped by bit-width                   -- Section 4.2, last paragraph.
 *   - unpacking: dequantised weights and the matrix-vector product from the packed form
 *                                                         -- Section 4 overview, Sections 4.2, 4.3.
 *   - the L-full error  (w - wq) X X^T (w - wq)^T  of a row -- Section 3.4; Section 4.2; Algorithm 3.
 *
 * Readings where the paper is silent (kept identical on the CUDA side):
 *   - init: centroid j of k = sorted_row[ floor((2j+1) m / (2k)) ] (index quantiles).
 *   - exactly `iters` (assign, update) pairs, then one more assign against the final
 *     centroids; err and labels use that last assignment.
 *   - assign: nearest centroid by a plain scan j = 0..k-1.  A tie between two different
 *     centroid values (an element exactly at their midpoint) goes to the lower value; a tie
 *     between equal-valued centroids goes to the copy on the element's side (the highest
 *     copy for an element above that value, else the lowest).  With ascending centroids
 *     this is the 1-D quantiser rule  label = #{ j : (c_j + c_{j+1})/2 < x }  and it keeps
 *     the centroids ascending through every update.
 *   - update: c_j = sum g x / sum g over the members; a cluster whose weight sum is
 *     not > 0 keeps its centroid.
 *   - if the row has D <= k distinct values: centroids are those values ascending, padded
 *     with the largest; err = 0; no iterations.
 *   - the error recorded in the table is the K-means objective itself (diagonal form).
 *   - between iterations the centroids are held as IEEE binary32 (the precision of the
 *     library's centroid output); all sums are binary64.  `round_fp32 = 0` keeps them
 *     binary64 instead (used by the textbook pins).
 *   - a scaled row is clustered on x~ = float(w) * r_j with r_j = 1.0f / s_j, the product
 *     taken in binary32, so that both sides cluster bit-identical numbers.
 *
 * Parity pins: every function here is pinned by tests that do not call the CUDA path
 * (closed forms, brute force, exact DP, library K-means, finite differences).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define SKIM_ORACLE_MAX_K 256

/* ------------------------------------------------------------------ number formats */

/* IEEE binary16 bit pattern -> float, exact. */
static float half_bits_to_float(uint16_t h)
{
    uint32_t sign = (uint32_t)(h >> 15) & 1u;
    uint32_t exp = (uint32_t)(h >> 10) & 0x1fu;
    uint32_t man = (uint32_t)h & 0x3ffu;
    float v;
    if (exp == 0) {
        v = ldexpf((float)man, -24);                 /* subnormal or zero */
    } else if (exp == 31) {
        v = man ? NAN : INFINITY;
    } else {
        v = ldexpf((float)(man | 0x400u), (int)exp - 25);
    }
    return sign ? -v : v;
}

/* float -> IEEE binary16 bit pattern, round to nearest even. */
static uint16_t float_to_half_bits(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    uint32_t sign = (u >> 16) & 0x8000u;
    uint32_t mag = u & 0x7fffffffu;
    if (mag >= 0x7f800000u) {                        /* inf or nan */
        return (uint16_t)(sign | 0x7c00u | (mag > 0x7f800000u ? 0x200u : 0u));
    }
    double a = fabs((double)f);
    if (a >= 65520.0) return (uint16_t)(sign | 0x7c00u);   /* rounds to inf */
    if (a < ldexp(1.0, -14)) {
        /* subnormal half: multiples of 2^-24 */
        double q = nearbyint(a * ldexp(1.0, 24));   /* default mode: ties to even */
        return (uint16_t)(sign | (uint32_t)q);      /* q == 1024 lands on the smallest normal */
    }
    int e;
    double fr = frexp(a, &e);                        /* a = fr * 2^e, fr in [0.5, 1) */
    double q = nearbyint(fr * 2048.0);               /* 11 significant bits */
    if (q == 2048.0) { q = 1024.0; e += 1; }
    uint32_t he = (uint32_t)(e - 1 + 15);
    return (uint16_t)(sign | (he << 10) | ((uint32_t)q - 1024u));
}

uint16_t skim_oracle_float_to_half(float f) { return float_to_half_bits(f); }
float skim_oracle_half_to_float(uint16_t h) { return half_bits_to_float(h); }

/* The value that is clustered for element (., j): the fp16 weight, times r_j = 1.0f/s_j in
 * binary32 when a scale vector is given (Section 4.3: W * alpha^-1). */
static double clustered_value(uint16_t w, const float *s, int64_t j)
{
    float x = half_bits_to_float(w);
    if (s) {
        volatile float r = 1.0f / s[j];
        volatile float p = x * r;
        x = p;
    }
    if (x == 0.0f) x = 0.0f;                          /* -0 and +0 are one value */
    return (double)x;
}

static int cmp_double(const void *a, const void *b)
{
    double x = *(const double *)a, y = *(const double *)b;
    return (x > y) - (x < y);
}

/* ------------------------------------------------------------------ one row, one k */

/* Nearest centroid, plain scan over ascending centroids.  Equal distances: keep the earlier
 * centroid unless the later one lies below x (then the two are equal-valued copies below x,
 * or x sits past both), see the tie rule in the header. */
static int nearest_centroid(double x, const double *c, int k)
{
    int best = 0;
    double bd = fabs(x - c[0]);
    for (int j = 1; j < k; ++j) {
        double d = fabs(x - c[j]);
        if (d < bd || (d == bd && c[j] < x)) { bd = d; best = j; }
    }
    return best;
}

static double objective(const double *x, const double *g, int64_t m, const double *c, const int32_t *label)
{
    double e = 0.0;
    for (int64_t j = 0; j < m; ++j) {
        double d = x[j] - c[label[j]];
        e += g[j] * d * d;
    }
    return e;
}

/*
 * Weighted 1-D K-means of one row (Algorithm 3, the Kmeans(W_i, weights=G_i, 2^b) call,
 * objective of Section 3.2's diagonal form).
 *   x, g      [m]   values to cluster and their importance (g >= 0)
 *   c         [k]   out: centroids, ascending
 *   label     [m]   out: cluster index of every element (final assignment)
 *   err             out: sum g (x - c[label])^2 for the final assignment
 *   trace           out, optional [2*iters+1]: objective after every assign and every update
 *   n_distinct      out, optional: number of distinct values, capped at k+1
 * Returns 0, or -1 on bad arguments / allocation failure.
 */
int skim_oracle_kmeans_row(const double *x, const double *g, int64_t m, int k, int iters,
                           int round_fp32, double *c, int32_t *label, double *err,
                           double *trace, int *n_distinct)
{
    if (m <= 0 || k <= 0 || k > SKIM_ORACLE_MAX_K || iters < 0) return -1;
    double *sorted = (double *)malloc((size_t)m * sizeof(double));
    if (!sorted) return -1;
    memcpy(sorted, x, (size_t)m * sizeof(double));
    qsort(sorted, (size_t)m, sizeof(double), cmp_double);

    /* distinct values (up to k+1 of them) */
    double distinct[SKIM_ORACLE_MAX_K + 1];
    int D = 0;
    for (int64_t j = 0; j < m && D <= k; ++j) {
        if (j == 0 || sorted[j] != sorted[j - 1]) distinct[D++] = sorted[j];
    }
    if (n_distinct) *n_distinct = D;

    if (D <= k) {
        /* every value gets its own centroid: zero error, no iterations */
        for (int j = 0; j < k; ++j) c[j] = distinct[j < D ? j : D - 1];
        for (int64_t j = 0; j < m; ++j) label[j] = nearest_centroid(x[j], c, k);
        *err = 0.0;
        if (trace) for (int t = 0; t < 2 * iters + 1; ++t) trace[t] = 0.0;
        free(sorted);
        return 0;
    }

    /* index-quantile init */
    for (int j = 0; j < k; ++j) {
        int64_t idx = ((int64_t)(2 * j + 1) * m) / (int64_t)(2 * k);
        c[j] = sorted[idx];
    }
    free(sorted);

    for (int it = 0; it < iters; ++it) {
        double sg[SKIM_ORACLE_MAX_K], sgx[SKIM_ORACLE_MAX_K];
        for (int j = 0; j < k; ++j) { sg[j] = 0.0; sgx[j] = 0.0; }
        /* assign */
        for (int64_t j = 0; j < m; ++j) {
            int l = nearest_centroid(x[j], c, k);
            label[j] = l;
            sg[l] += g[j];
            sgx[l] += g[j] * x[j];
        }
        if (trace) trace[2 * it] = objective(x, g, m, c, label);
        /* update */
        for (int j = 0; j < k; ++j) {
            if (sg[j] > 0.0) {
                double cj = sgx[j] / sg[j];
                c[j] = round_fp32 ? (double)(float)cj : cj;
            }
        }
        if (trace) trace[2 * it + 1] = objective(x, g, m, c, label);
    }
    /* final assignment against the final centroids */
    for (int64_t j = 0; j < m; ++j) label[j] = nearest_centroid(x[j], c, k);
    *err = objective(x, g, m, c, label);
    if (trace) trace[2 * iters] = *err;
    return 0;
}

/* ------------------------------------------------------------------ all rows, all bit-widths */

static int check_bit_set(const int *bit_set, int n_bits)
{
    if (!bit_set || n_bits <= 0) return -1;
    for (int b = 0; b < n_bits; ++b) {
        if (bit_set[b] < 1 || bit_set[b] > 8) return -1;
        if (b && bit_set[b] != bit_set[b - 1] + 1) return -1;
    }
    return 0;
}

/*
 * Error pre-recording (Algorithm 3, the double loop over rows and candidate bit-widths) and,
 * with `row_bits`, the final clustering at the allocated width (Algorithm 3, second row loop).
 *   W          fp16 bit patterns, row-major, leading dimension ld
 *   importance float, same layout
 *   s          optional scale vector [cols] (NULL = none)
 *   row_bits   optional [rows]: cluster row i only at bit-width row_bits[i]; other slots untouched
 *   centroids  out [rows][sum_b 2^b] double, bit-width blocks in bit_set order
 *   codes      out, optional [n_bits][rows][cols] uint8 labels
 *   err        out [rows][n_bits] double
 *   trace      out, optional [rows][n_bits][2*iters+1]
 */
int skim_oracle_cluster_rows(const uint16_t *W, const float *importance, int64_t rows, int64_t cols,
                             int64_t ld, const float *s, const uint8_t *row_bits,
                             const int *bit_set, int n_bits, int iters, int round_fp32,
                             double *centroids, uint8_t *codes, double *err, double *trace)
{
    if (!W || !importance || rows < 0 || cols <= 0 || ld < cols || iters < 0) return -1;
    if (check_bit_set(bit_set, n_bits)) return -1;
    int sumk = 0;
    for (int b = 0; b < n_bits; ++b) sumk += 1 << bit_set[b];
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < rows; ++i) {
        double *x = (double *)malloc((size_t)cols * sizeof(double));
        double *g = (double *)malloc((size_t)cols * sizeof(double));
        int32_t *label = (int32_t *)malloc((size_t)cols * sizeof(int32_t));
        if (!x || !g || !label) {
            failed = 1;
        } else {
            for (int64_t j = 0; j < cols; ++j) {
                x[j] = clustered_value(W[i * ld + j], s, j);
                g[j] = (double)importance[i * ld + j];
            }
            int off = 0;
            for (int b = 0; b < n_bits; ++b) {
                int k = 1 << bit_set[b];
                if (!row_bits || row_bits[i] == bit_set[b]) {
                    double e = 0.0;
                    double *tr = trace ? trace + ((size_t)i * n_bits + b) * (size_t)(2 * iters + 1) : NULL;
                    if (skim_oracle_kmeans_row(x, g, cols, k, iters, round_fp32,
                                               centroids + (size_t)i * sumk + off, label, &e, tr, NULL))
                        failed = 1;
                    err[(size_t)i * n_bits + b] = e;
                    if (codes) {
                        uint8_t *dst = codes + ((size_t)b * rows + i) * (size_t)cols;
                        for (int64_t j = 0; j < cols; ++j) dst[j] = (uint8_t)label[j];
                    }
                }
                off += k;
            }
        }
        free(x); free(g); free(label);
    }
    return failed ? -1 : 0;
}

/* ------------------------------------------------------------------ greedy bit allocation */

/*
 * Algorithm 1 (Section 4.2).  All rows start at b_min; the row whose next bit removes the
 * most error (E[i,b_i] - E[i,b_i+1], lowest row index on ties) is raised by one bit, until
 * the total reaches T = floor(rows * budget + 1e-6).  Gains are differences of the float
 * table entries taken in binary64.
 *   err   [rows][n_bits] float, column b is bit-width b_min + b
 *   bits  out [rows]
 *   total out: T
 * Returns 0, -1 on bad arguments, -2 if the budget is outside [b_min, b_max].
 */
int skim_oracle_allocate_bits(const float *err, int64_t rows, int n_bits, int b_min, double budget,
                              uint8_t *bits, int64_t *total)
{
    if (!err || !bits || rows <= 0 || n_bits <= 0 || b_min < 1) return -1;
    int b_max = b_min + n_bits - 1;
    int64_t T = (int64_t)floor((double)rows * budget + 1e-6);
    int64_t K = T - rows * (int64_t)b_min;
    if (K < 0 || K > rows * (int64_t)(b_max - b_min)) return -2;
    for (int64_t i = 0; i < rows; ++i) bits[i] = (uint8_t)b_min;
    for (int64_t step = 0; step < K; ++step) {
        int64_t best = -1;
        double best_gain = 0.0;
        for (int64_t i = 0; i < rows; ++i) {
            if (bits[i] >= b_max) continue;
            int b = bits[i] - b_min;
            double gain = (double)err[i * n_bits + b] - (double)err[i * n_bits + b + 1];
            if (best < 0 || gain > best_gain) { best = i; best_gain = gain; }
        }
        bits[best] += 1;
    }
    if (total) *total = T;
    return 0;
}

/*
 * Algorithm 1 with its stopping rule taken literally: bits are handed out "until sum_i b_i >= n * bit",
 * so a non-integer n * bit is rounded UP (the total may exceed the budget by less than one bit), where
 * skim_oracle_allocate_bits rounds down to honour the "<=" of Section 4.2's constraint.
 */
int skim_oracle_allocate_bits_until(const float *err, int64_t rows, int n_bits, int b_min, double budget,
                                    uint8_t *bits, int64_t *total)
{
    if (!err || !bits || rows <= 0 || n_bits <= 0 || b_min < 1) return -1;
    int b_max = b_min + n_bits - 1;
    if (!(budget >= (double)b_min && budget <= (double)b_max)) return -2;
    double want = (double)rows * budget - 1e-6;
    int64_t sum = rows * (int64_t)b_min;
    for (int64_t i = 0; i < rows; ++i) bits[i] = (uint8_t)b_min;
    while ((double)sum < want) {
        int64_t best = -1;
        double best_gain = 0.0;
        for (int64_t i = 0; i < rows; ++i) {
            if (bits[i] >= b_max) continue;
            int b = bits[i] - b_min;
            double gain = (double)err[i * n_bits + b] - (double)err[i * n_bits + b + 1];
            if (best < 0 || gain > best_gain) { best = i; best_gain = gain; }
        }
        if (best < 0) break;
        bits[best] += 1;
        sum += 1;
    }
    if (total) *total = sum;
    return 0;
}

/*
 * Allocation started from the floor of the budget (appendix with the results on other model
 * families: mixed precision is switched off at integer budgets, and at non-integer ones the
 * allocation is initialised with the budget rounded down).  Every row starts at floor(budget);
 * Algorithm 1's loop then hands out the remaining T - rows * floor(budget) bits exactly as above.
 */
int skim_oracle_allocate_bits_floor(const float *err, int64_t rows, int n_bits, int b_min, double budget,
                                    uint8_t *bits, int64_t *total)
{
    if (!err || !bits || rows <= 0 || n_bits <= 0 || b_min < 1) return -1;
    int b_max = b_min + n_bits - 1;
    if (!(budget >= (double)b_min && budget <= (double)b_max)) return -2;
    int64_t T = (int64_t)floor((double)rows * budget + 1e-6);
    int start = (int)floor(budget + 1e-9);
    if (start > b_max) start = b_max;
    int64_t K = T - rows * (int64_t)start;
    if (K < 0 || K > rows * (int64_t)(b_max - start)) return -2;
    for (int64_t i = 0; i < rows; ++i) bits[i] = (uint8_t)start;
    for (int64_t step = 0; step < K; ++step) {
        int64_t best = -1;
        double best_gain = 0.0;
        for (int64_t i = 0; i < rows; ++i) {
            if (bits[i] >= b_max) continue;
            int b = bits[i] - b_min;
            double gain = (double)err[i * n_bits + b] - (double)err[i * n_bits + b + 1];
            if (best < 0 || gain > best_gain) { best = i; best_gain = gain; }
        }
        bits[best] += 1;
    }
    if (total) *total = T;
    return 0;
}

/*
 * The exact solution of the allocation problem of Section 4.2 (minimise sum_i Err(w_i, b_i) subject
 * to the bit budget), by the dynamic programme the paper mentions and sets aside for its quadratic
 * cost: the yardstick for Algorithm 1.  The total is fixed to the same T = floor(rows * budget + 1e-6)
 * the greedy reaches.  With s = (bits handed out so far beyond b_min per row),
 *   f_0(0) = 0,   f_i(s) = min_u f_{i-1}(s - u) + E[i-1][u],   u = 0 .. n_bits-1 (smallest u on ties),
 * and the answer is f_rows(T - rows * b_min), with the widths recovered by walking the choices back.
 *   bits out [rows];  cost out (may be NULL): the minimum, summed in row order in binary64.
 */
int skim_oracle_allocate_optimal(const float *err, int64_t rows, int n_bits, int b_min, double budget,
                                 uint8_t *bits, int64_t *total, double *cost)
{
    if (!err || !bits || rows <= 0 || n_bits <= 0 || b_min < 1) return -1;
    int b_max = b_min + n_bits - 1;
    int64_t T = (int64_t)floor((double)rows * budget + 1e-6);
    int64_t K = T - rows * (int64_t)b_min;
    if (K < 0 || K > rows * (int64_t)(b_max - b_min)) return -2;
    double *prev = (double *)malloc((size_t)(K + 1) * sizeof(double));
    double *cur = (double *)malloc((size_t)(K + 1) * sizeof(double));
    uint8_t *choice = (uint8_t *)malloc((size_t)rows * (size_t)(K + 1));
    if (!prev || !cur || !choice) { free(prev); free(cur); free(choice); return -3; }
    for (int64_t s = 0; s <= K; ++s) prev[s] = INFINITY;
    prev[0] = 0.0;
    for (int64_t i = 0; i < rows; ++i) {
        for (int64_t s = 0; s <= K; ++s) {
            double best = INFINITY;
            int bu = 0;
            for (int u = 0; u < n_bits && u <= s; ++u) {
                double v = prev[s - u] + (double)err[i * n_bits + u];
                if (v < best) { best = v; bu = u; }
            }
            cur[s] = best;
            choice[(size_t)i * (size_t)(K + 1) + (size_t)s] = (uint8_t)bu;
        }
        double *t = prev; prev = cur; cur = t;
    }
    if (cost) *cost = prev[K];
    int64_t s = K;
    for (int64_t i = rows - 1; i >= 0; --i) {
        int u = choice[(size_t)i * (size_t)(K + 1) + (size_t)s];
        bits[i] = (uint8_t)(b_min + u);
        s -= u;
    }
    free(prev); free(cur); free(choice);
    if (total) *total = T;
    return s == 0 ? 0 : -4;
}

/* ------------------------------------------------------------------ emission */

/* Words in one packed row of `cols` codes of `b` bits: ceil(cols*b/32), rounded up to 4 words. */
int64_t skim_oracle_row_stride_words(int64_t cols, int b)
{
    int64_t w = (cols * (int64_t)b + 31) / 32;
    return (w + 3) / 4 * 4;
}

/*
 * Final codebook and code emission (Algorithm 3: labels and centroids at the allocated width;
 * Section 4.2: rows of equal width are gathered and packed together).
 *   bits        [rows] allocated width of every row
 *   centroids   [rows][sum_b 2^b] float, as produced by the clustering (only the block of the
 *               row's own width is read)
 *   packed      out: for width b (ascending) the rows of that width in ascending row index,
 *               each a little-endian bitstream (element j in bits [j*b, (j+1)*b)) stored as
 *               32-bit words with stride skim_oracle_row_stride_words(cols, b); zero padded
 *   row_order   out [rows]: source row of every packed row
 *   group_start out [n_bits+1]: first packed-row index of every width group
 *   group_word  out [n_bits+1]: word offset of every width group inside `packed`
 *   lut         out [rows][2^b_max] fp16 bit patterns, entries beyond 2^b_i repeat the last
 *   codes       out, optional [rows][cols] unpacked labels
 */
int skim_oracle_emit(const uint16_t *W, int64_t rows, int64_t cols, int64_t ld, const float *s,
                     const uint8_t *bits, const float *centroids, const int *bit_set, int n_bits,
                     uint32_t *packed, int32_t *row_order, int64_t *group_start, int64_t *group_word,
                     uint16_t *lut, uint8_t *codes)
{
    if (!W || !bits || !centroids || rows <= 0 || cols <= 0 || ld < cols) return -1;
    if (check_bit_set(bit_set, n_bits)) return -1;
    int sumk = 0, kmax = 1 << bit_set[n_bits - 1];
    for (int b = 0; b < n_bits; ++b) sumk += 1 << bit_set[b];

    /* group rows by width, ascending width then ascending row */
    int64_t pos = 0, word = 0;
    for (int b = 0; b < n_bits; ++b) {
        group_start[b] = pos;
        group_word[b] = word;
        int64_t cnt = 0;
        for (int64_t i = 0; i < rows; ++i) {
            if (bits[i] == bit_set[b]) { row_order[pos + cnt] = (int32_t)i; ++cnt; }
        }
        pos += cnt;
        word += cnt * skim_oracle_row_stride_words(cols, bit_set[b]);
    }
    group_start[n_bits] = pos;
    group_word[n_bits] = word;
    if (pos != rows) return -3;                       /* some row has a width outside bit_set */
    memset(packed, 0, (size_t)word * sizeof(uint32_t));

    for (int b = 0; b < n_bits; ++b) {
        int width = bit_set[b], k = 1 << width, off = 0;
        for (int u = 0; u < b; ++u) off += 1 << bit_set[u];
        int64_t stride = skim_oracle_row_stride_words(cols, width);
        for (int64_t p = group_start[b]; p < group_start[b + 1]; ++p) {
            int64_t i = row_order[p];
            double c[SKIM_ORACLE_MAX_K];
            for (int j = 0; j < k; ++j) c[j] = (double)centroids[(size_t)i * sumk + off + j];
            uint32_t *dst = packed + group_word[b] + (p - group_start[b]) * stride;
            for (int64_t j = 0; j < cols; ++j) {
                double x = clustered_value(W[i * ld + j], s, j);
                uint32_t code = (uint32_t)nearest_centroid(x, c, k);
                if (codes) codes[(size_t)i * cols + j] = (uint8_t)code;
                int64_t bit = j * width;
                for (int t = 0; t < width; ++t) {
                    if ((code >> t) & 1u) dst[(bit + t) / 32] |= 1u << ((bit + t) % 32);
                }
            }
            for (int j = 0; j < kmax; ++j) {
                float cv = centroids[(size_t)i * sumk + off + (j < k ? j : k - 1)];
                lut[(size_t)i * kmax + j] = float_to_half_bits(cv);
            }
        }
    }
    return 0;
}

/* ------------------------------------------------------------------ unpacking: dequantised weights */

/* Code of element j in a packed row of `width`-bit codes (little-endian bit stream). */
static uint32_t packed_code(const uint32_t *row_words, int64_t j, int width)
{
    uint32_t code = 0;
    int64_t bit = j * width;
    for (int t = 0; t < width; ++t) code |= ((row_words[(bit + t) / 32] >> ((bit + t) % 32)) & 1u) << t;
    return code;
}

/*
 * Dequantised weights from the packed form (Section 4 overview: the weights are recovered
 * from labels, centroids and the scaling vector; Section 4.3: Wq = Quant(W * alpha^-1) * alpha;
 * Section 4.2, last paragraph: rows are unpacked group by group).
 *   Wq[i][j] = binary16( float(lut[i][code_ij]) * s_j )   product in binary32, then one more
 *   round-to-nearest-even to binary16; with no scale (s == NULL) Wq is the codebook entry itself.
 * out: [rows][cols] binary16 bit patterns, in source-row order.
 */
int skim_oracle_dequantize(const uint32_t *packed, const int32_t *row_order, const int64_t *group_start,
                           const int64_t *group_word, const uint16_t *lut, const float *s, int64_t rows,
                           int64_t cols, const int *bit_set, int n_bits, uint16_t *out)
{
    if (!packed || !row_order || !group_start || !group_word || !lut || !out || rows <= 0 || cols <= 0) return -1;
    if (check_bit_set(bit_set, n_bits)) return -1;
    int kmax = 1 << bit_set[n_bits - 1];
    for (int b = 0; b < n_bits; ++b) {
        int width = bit_set[b];
        int64_t stride = skim_oracle_row_stride_words(cols, width);
        for (int64_t p = group_start[b]; p < group_start[b + 1]; ++p) {
            int64_t i = row_order[p];
            const uint32_t *src = packed + group_word[b] + (p - group_start[b]) * stride;
            for (int64_t j = 0; j < cols; ++j) {
                uint16_t entry = lut[(size_t)i * kmax + packed_code(src, j, width)];
                if (s) {
                    volatile float prod = half_bits_to_float(entry) * s[j];   /* binary32 product */
                    out[(size_t)i * cols + j] = float_to_half_bits(prod);
                } else {
                    out[(size_t)i * cols + j] = entry;
                }
            }
        }
    }
    return 0;
}

/*
 * Matrix-vector product with the quantised matrix taken straight from its packed form (the
 * inference-side consumer of the packing of Section 4.2):
 *   y_i = sum_j float(lut[i][code_ij]) * z_j,   z_j = float(x_j) * s_j in binary32 (z = x when
 *   s == NULL), the sum in binary64.  abs_sum (may be NULL) receives sum_j |term|, the scale of
 *   the rounding error of a lower-precision accumulation.
 *   x: [cols] binary16 bit patterns;  y, abs_sum: [rows] double, source-row order.
 */
int skim_oracle_matvec(const uint32_t *packed, const int32_t *row_order, const int64_t *group_start,
                       const int64_t *group_word, const uint16_t *lut, const float *s, const uint16_t *x,
                       int64_t rows, int64_t cols, const int *bit_set, int n_bits, double *y, double *abs_sum)
{
    if (!packed || !row_order || !group_start || !group_word || !lut || !x || !y || rows <= 0 || cols <= 0) return -1;
    if (check_bit_set(bit_set, n_bits)) return -1;
    int kmax = 1 << bit_set[n_bits - 1];
    for (int b = 0; b < n_bits; ++b) {
        int width = bit_set[b];
        int64_t stride = skim_oracle_row_stride_words(cols, width);
        for (int64_t p = group_start[b]; p < group_start[b + 1]; ++p) {
            int64_t i = row_order[p];
            const uint32_t *src = packed + group_word[b] + (p - group_start[b]) * stride;
            double acc = 0.0, mag = 0.0;
            for (int64_t j = 0; j < cols; ++j) {
                volatile float z = s ? half_bits_to_float(x[j]) * s[j] : half_bits_to_float(x[j]);
                double term = (double)half_bits_to_float(lut[(size_t)i * kmax + packed_code(src, j, width)]) * (double)z;
                acc += term;
                mag += fabs(term);
            }
            y[i] = acc;
            if (abs_sum) abs_sum[i] = mag;
        }
    }
    return 0;
}

/* ------------------------------------------------------------------ scaling-vector update */

/*
 * Loss and gradient of the scaling vector with the labels held fixed (Algorithm 2, inner
 * repeat: c = calc_centroids(W * alpha^-1, L); Wq = replace(c, L) * alpha; loss = Err(W, Wq)),
 * with the diagonal error  loss = sum_ij g_ij (W_ij - alpha_j c_{i,l_ij})^2  and importance-
 * weighted centroids  c_ik = sum_{j in k} g_ij W_ij / alpha_j  /  sum_{j in k} g_ij.
 *   labels [rows][cols] uint8,  alpha [cols] double,  grad out [cols] (may be NULL)
 */
int skim_oracle_scale_loss_grad(const uint16_t *W, const float *importance, int64_t rows, int64_t cols,
                                int64_t ld, const uint8_t *labels, const double *alpha,
                                double *loss_out, double *grad)
{
    if (!W || !importance || !labels || !alpha || rows <= 0 || cols <= 0 || ld < cols) return -1;
    double loss = 0.0;
    if (grad) for (int64_t j = 0; j < cols; ++j) grad[j] = 0.0;
    for (int64_t i = 0; i < rows; ++i) {
        double G[SKIM_ORACLE_MAX_K], S[SKIM_ORACLE_MAX_K], c[SKIM_ORACLE_MAX_K], R[SKIM_ORACLE_MAX_K];
        for (int k = 0; k < SKIM_ORACLE_MAX_K; ++k) { G[k] = 0.0; S[k] = 0.0; c[k] = 0.0; R[k] = 0.0; }
        for (int64_t j = 0; j < cols; ++j) {
            double w = (double)half_bits_to_float(W[i * ld + j]);
            double g = (double)importance[i * ld + j];
            int l = labels[i * cols + j];
            G[l] += g;
            S[l] += g * w / alpha[j];
        }
        for (int k = 0; k < SKIM_ORACLE_MAX_K; ++k) if (G[k] > 0.0) c[k] = S[k] / G[k];
        for (int64_t j = 0; j < cols; ++j) {
            double w = (double)half_bits_to_float(W[i * ld + j]);
            double g = (double)importance[i * ld + j];
            int l = labels[i * cols + j];
            double r = w - alpha[j] * c[l];
            loss += g * r * r;
            R[l] += g * r * alpha[j];
        }
        if (grad) {
            for (int64_t j = 0; j < cols; ++j) {
                double w = (double)half_bits_to_float(W[i * ld + j]);
                double g = (double)importance[i * ld + j];
                int l = labels[i * cols + j];
                double r = w - alpha[j] * c[l];
                double d = -2.0 * g * r * c[l];
                if (G[l] > 0.0) d += 2.0 * R[l] * g * w / (alpha[j] * alpha[j] * G[l]);
                grad[j] += d;
            }
        }
    }
    *loss_out = loss;
    return 0;
}

/*
 * `steps` Adam updates of alpha with the labels fixed (Section 5.1: Adam, learning rate lr0,
 * multiplied by `decay` every `decay_every` steps; default betas 0.9 / 0.999, eps 1e-8).
 *   alpha      in/out [cols]
 *   loss_trace out, optional [steps]: loss at the alpha each step started from
 */
int skim_oracle_scale_update(const uint16_t *W, const float *importance, int64_t rows, int64_t cols,
                             int64_t ld, const uint8_t *labels, double *alpha, int steps, double lr0,
                             double decay, int decay_every, double beta1, double beta2, double eps,
                             double *loss_trace)
{
    if (steps < 0 || decay_every <= 0) return -1;
    double *m1 = (double *)calloc((size_t)cols, sizeof(double));
    double *m2 = (double *)calloc((size_t)cols, sizeof(double));
    double *grad = (double *)malloc((size_t)cols * sizeof(double));
    if (!m1 || !m2 || !grad) { free(m1); free(m2); free(grad); return -1; }
    int rc = 0;
    for (int t = 0; t < steps && !rc; ++t) {
        double loss;
        rc = skim_oracle_scale_loss_grad(W, importance, rows, cols, ld, labels, alpha, &loss, grad);
        if (loss_trace) loss_trace[t] = loss;
        double lr = lr0 * pow(decay, (double)(t / decay_every));
        double bc1 = 1.0 - pow(beta1, (double)(t + 1));
        double bc2 = 1.0 - pow(beta2, (double)(t + 1));
        for (int64_t j = 0; j < cols; ++j) {
            m1[j] = beta1 * m1[j] + (1.0 - beta1) * grad[j];
            m2[j] = beta2 * m2[j] + (1.0 - beta2) * grad[j] * grad[j];
            double mh = m1[j] / bc1, vh = m2[j] / bc2;
            alpha[j] -= lr * mh / (sqrt(vh) + eps);
        }
    }
    free(m1); free(m2); free(grad);
    return rc;
}

/* ------------------------------------------------------------------ exact 1-D weighted K-means */

typedef struct { double x, g; } oracle_pair;

static int cmp_pair(const void *a, const void *b)
{
    double x = ((const oracle_pair *)a)->x, y = ((const oracle_pair *)b)->x;
    return (x > y) - (x < y);
}

/*
 * The optimum of the clustering objective of Section 3.2 (diagonal form), sum_j g_j (x_j - c_{l_j})^2, over ALL
 * assignments to k centroids, for one row: in one dimension the optimal clusters are intervals of the sorted
 * row, so the textbook dynamic programme over split points finds it,
 *     F_1(i) = cost(0, i),   F_j(i) = min_{j-1 <= t < i} F_{j-1}(t) + cost(t, i),
 *     cost(t, i) = sum g x^2 - (sum g x)^2 / sum g  over the sorted elements t .. i-1 (0 without weight),
 * every t tried (no monotonicity assumed), smallest t on ties.  This is the yardstick for the Lloyd
 * iterations of Algorithm 3, which only reach a local optimum.
 *   ks [nk] ascending cluster counts; c out: concatenated blocks of ks[u] centroids (weighted means of the
 *   intervals, ascending; an interval without weight takes the mean of its first and last value);
 *   err out [nk]: the optimum.  A row with D <= k distinct values gets them as centroids, padded with the
 *   largest, and err = 0, as in skim_oracle_kmeans_row.
 */
int skim_oracle_kmeans_exact_row(const double *x, const double *g, int64_t m, const int *ks, int nk, double *c, double *err)
{
    if (!x || !g || !ks || !c || !err || m <= 0 || nk <= 0) return -1;
    int kmax = ks[nk - 1];
    if (kmax > SKIM_ORACLE_MAX_K) return -1;
    oracle_pair *v = (oracle_pair *)malloc((size_t)m * sizeof(oracle_pair));
    double *p0 = (double *)malloc((size_t)(m + 1) * 3 * sizeof(double));
    if (!v || !p0) { free(v); free(p0); return -1; }
    double *p1 = p0 + (m + 1), *p2 = p1 + (m + 1);
    for (int64_t j = 0; j < m; ++j) { v[j].x = (x[j] == 0.0) ? 0.0 : x[j]; v[j].g = g[j]; }
    qsort(v, (size_t)m, sizeof(oracle_pair), cmp_pair);
    p0[0] = p1[0] = p2[0] = 0.0;
    int64_t distinct = 1;
    for (int64_t j = 0; j < m; ++j) {
        p0[j + 1] = p0[j] + v[j].g;
        p1[j + 1] = p1[j] + v[j].g * v[j].x;
        p2[j + 1] = p2[j] + v[j].g * v[j].x * v[j].x;
        if (j && v[j].x != v[j - 1].x) ++distinct;
    }
    int64_t limit = (int64_t)kmax < m ? (int64_t)kmax : m;      /* layers that can have non-empty intervals */
    double *F = (double *)malloc((size_t)(limit + 1) * (size_t)(m + 1) * sizeof(double));
    int32_t *T = (int32_t *)malloc((size_t)(limit + 1) * (size_t)(m + 1) * sizeof(int32_t));
    if (!F || !T) { free(v); free(p0); free(F); free(T); return -1; }
#define COST(t, i) ((p0[i] - p0[t]) > 0.0 ? (p2[i] - p2[t]) - (p1[i] - p1[t]) * (p1[i] - p1[t]) / (p0[i] - p0[t]) : 0.0)
    for (int64_t i = 1; i <= m; ++i) { F[1 * (m + 1) + i] = COST(0, i); T[1 * (m + 1) + i] = 0; }
    for (int64_t j = 2; j <= limit; ++j) {
        for (int64_t i = j; i <= m; ++i) {
            double best = 0.0;
            int64_t bt = -1;
            for (int64_t t = j - 1; t < i; ++t) {
                double val = F[(j - 1) * (m + 1) + t] + COST(t, i);
                if (bt < 0 || val < best) { best = val; bt = t; }
            }
            F[j * (m + 1) + i] = best;
            T[j * (m + 1) + i] = (int32_t)bt;
        }
    }
#undef COST
    int off = 0;
    for (int u = 0; u < nk; ++u) {
        int k = ks[u];
        if (distinct <= (int64_t)k) {
            int q = 0;
            for (int64_t j = 0; j < m; ++j)
                if (j == 0 || v[j].x != v[j - 1].x) c[off + q++] = v[j].x;
            for (; q < k; ++q) c[off + q] = v[m - 1].x;
            err[u] = 0.0;
        } else {
            int64_t i = m;
            for (int j = k; j >= 1; --j) {
                int64_t t = (j == 1) ? 0 : T[(int64_t)j * (m + 1) + i];
                double s0 = p0[i] - p0[t];
                c[off + j - 1] = s0 > 0.0 ? (p1[i] - p1[t]) / s0 : 0.5 * (v[t].x + v[i - 1].x);
                i = t;
            }
            double e = F[(int64_t)k * (m + 1) + m];
            err[u] = e > 0.0 ? e : 0.0;
        }
        off += k;
    }
    free(v); free(p0); free(F); free(T);
    return 0;
}

/* Exact clustering of every row of a matrix at every width of bit_set (the counterpart of
 * skim_oracle_cluster_rows with the Lloyd iterations replaced by the optimum). */
int skim_oracle_cluster_rows_exact(const uint16_t *W, const float *importance, int64_t rows, int64_t cols, int64_t ld,
                                   const float *s, const int *bit_set, int n_bits, double *centroids, double *err)
{
    if (!W || !importance || !centroids || !err || rows <= 0 || cols <= 0 || ld < cols) return -1;
    if (check_bit_set(bit_set, n_bits)) return -1;
    int ks[8], sumk = 0;
    for (int b = 0; b < n_bits; ++b) { ks[b] = 1 << bit_set[b]; sumk += ks[b]; }
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < rows; ++i) {
        double *x = (double *)malloc((size_t)cols * 2 * sizeof(double));
        if (!x) { failed = 1; continue; }
        double *g = x + cols;
        for (int64_t j = 0; j < cols; ++j) {
            x[j] = clustered_value(W[i * ld + j], s, j);
            g[j] = (double)importance[i * ld + j];
        }
        if (skim_oracle_kmeans_exact_row(x, g, cols, ks, n_bits, centroids + (size_t)i * sumk, err + (size_t)i * n_bits)) failed = 1;
        free(x);
    }
    return failed ? -4 : 0;
}

/* ------------------------------------------------------------------ L-full error (Section 3.4) */

/*
 * Residual of a row against its quantised form, the operand of the L-full error (Section 3.4: the error of
 * row i is (w_i - wq_i) X X^T (w_i - wq_i)^T; Section 4 overview and Section 4.3: wq = replace(c, l) * alpha).
 *   label   the 1-D quantiser rule on the clustered value (as in skim_oracle_emit)
 *   wq      the binary32 product  c[label] * alpha_j   (alpha == NULL: c[label] itself)
 *   d       binary16( (float(w) - wq) * 2^exp2 ), the difference taken in binary32, the power-of-two scaling
 *           exact, then one rounding to nearest even.  The scaling keeps small residuals out of the
 *           binary16 subnormal range; the error routine divides it out again.
 * row_bits == NULL: every row uses the centroid block of `width`; else row i uses width row_bits[i].
 * D out [rows][ldd] binary16 bit patterns.
 */
int skim_oracle_residual(const uint16_t *W, int64_t rows, int64_t cols, int64_t ld, const float *s,
                         const uint8_t *row_bits, int width, const float *centroids, const int *bit_set,
                         int n_bits, int exp2, uint16_t *D, int64_t ldd)
{
    if (!W || !centroids || !D || rows <= 0 || cols <= 0 || ld < cols || ldd < cols) return -1;
    if (check_bit_set(bit_set, n_bits)) return -1;
    int sumk = 0;
    for (int b = 0; b < n_bits; ++b) sumk += 1 << bit_set[b];
    for (int64_t i = 0; i < rows; ++i) {
        int wd = row_bits ? (int)row_bits[i] : width, off = 0, found = 0;
        for (int b = 0; b < n_bits; ++b) {
            if (bit_set[b] == wd) { found = 1; break; }
            off += 1 << bit_set[b];
        }
        if (!found) return -3;
        int k = 1 << wd;
        double c[SKIM_ORACLE_MAX_K];
        for (int j = 0; j < k; ++j) c[j] = (double)centroids[(size_t)i * sumk + off + j];
        for (int64_t j = 0; j < cols; ++j) {
            double x = clustered_value(W[i * ld + j], s, j);
            int label = nearest_centroid(x, c, k);
            float cq = centroids[(size_t)i * sumk + off + label];
            float q = s ? cq * s[j] : cq;
            float r = half_bits_to_float(W[i * ld + j]) - q;
            D[i * ldd + j] = float_to_half_bits(ldexpf(r, exp2));
        }
    }
    return 0;
}

/*
 * L-full error of every row (Section 3.4, the form the paper names L-full; Section 4.2: "Err refers to the
 * L-full form"; Algorithm 3, the line that fills the error table):  err_i = d_i H d_i^T  with H = X X^T,
 * written out as the double sum over j and k in binary64.  D holds the scaled residuals of
 * skim_oracle_residual (binary16), H [cols][ldh] binary16; the result is divided by 4^exp2.
 * mag (optional) receives sum_jk |d_j H_jk d_k| / 4^exp2, the scale of the rounding error of any
 * reduced-precision evaluation.
 */
int skim_oracle_err_lfull(const uint16_t *D, int64_t rows, int64_t cols, int64_t ldd, const uint16_t *H,
                          int64_t ldh, int exp2, double *err, double *mag)
{
    if (!D || !H || !err || rows <= 0 || cols <= 0 || ldd < cols || ldh < cols) return -1;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < rows; ++i) {
        double *d = (double *)malloc((size_t)cols * sizeof(double));
        if (!d) { failed = 1; continue; }
        for (int64_t j = 0; j < cols; ++j) d[j] = (double)half_bits_to_float(D[i * ldd + j]);
        double acc = 0.0, absacc = 0.0;
        for (int64_t j = 0; j < cols; ++j) {
            for (int64_t k = 0; k < cols; ++k) {
                double t = d[j] * (double)half_bits_to_float(H[j * ldh + k]) * d[k];
                acc += t;
                absacc += fabs(t);
            }
        }
        err[i] = ldexp(acc, -2 * exp2);
        if (mag) mag[i] = ldexp(absacc, -2 * exp2);
        free(d);
    }
    return failed ? -4 : 0;
}

/*
 * Loss and gradient of the scaling vector in the L-full form (Section 4.3: "the loss calculation adopts the L-full
 * form"; Algorithm 2, inner repeat; Section 3.4 for the form itself), labels fixed:
 *     c_ik  = sum_{j in k} g_ij W_ij / alpha_j  /  sum_{j in k} g_ij     (importance-weighted, as in the diagonal version)
 *     d_ij  = W_ij - alpha_j c_{i,l_ij}
 *     loss  = sum_i d_i H d_i^T,   H = X X^T (binary16, symmetric)
 * With Y = D H the derivative with respect to d_ij is 2 Y_ij, so, both through the explicit alpha_j and through the
 * re-fitted centroids,
 *     d loss / d alpha_j = sum_i [ -2 Y_ij c_{i,l_ij} + 2 R_{i,l_ij} g_ij W_ij / (alpha_j^2 G_{i,l_ij}) ],
 *     R_ik = sum_{j in k} Y_ij alpha_j,   G_ik = sum_{j in k} g_ij.
 * round_d != 0: the residual enters the contraction as the library's operand does, binary16(float(d) * 2^exp2) / 2^exp2
 * (the gradient treats that rounding as the identity); round_d == 0: exact d (used by the finite-difference pin).
 *   grad out [cols], may be NULL.
 */
int skim_oracle_scale_loss_grad_lfull(const uint16_t *W, const float *importance, int64_t rows, int64_t cols,
                                      int64_t ld, const uint8_t *labels, const double *alpha, const uint16_t *H,
                                      int64_t ldh, int exp2, int round_d, double *loss_out, double *grad)
{
    if (!W || !importance || !labels || !alpha || !H || rows <= 0 || cols <= 0 || ld < cols || ldh < cols) return -1;
    double *Hd = (double *)malloc((size_t)cols * (size_t)cols * sizeof(double));
    double *rowbuf = (double *)malloc((size_t)cols * 2 * sizeof(double));
    if (!Hd || !rowbuf) { free(Hd); free(rowbuf); return -1; }
    for (int64_t j = 0; j < cols; ++j)
        for (int64_t k = 0; k < cols; ++k) Hd[j * cols + k] = (double)half_bits_to_float(H[j * ldh + k]);
    double *d = rowbuf, *y = rowbuf + cols;
    double loss = 0.0;
    if (grad) for (int64_t j = 0; j < cols; ++j) grad[j] = 0.0;
    for (int64_t i = 0; i < rows; ++i) {
        double G[SKIM_ORACLE_MAX_K], S[SKIM_ORACLE_MAX_K], c[SKIM_ORACLE_MAX_K], R[SKIM_ORACLE_MAX_K];
        for (int k = 0; k < SKIM_ORACLE_MAX_K; ++k) { G[k] = 0.0; S[k] = 0.0; c[k] = 0.0; R[k] = 0.0; }
        for (int64_t j = 0; j < cols; ++j) {
            double w = (double)half_bits_to_float(W[i * ld + j]);
            double g = (double)importance[i * ld + j];
            int l = labels[i * cols + j];
            G[l] += g;
            S[l] += g * w / alpha[j];
        }
        for (int k = 0; k < SKIM_ORACLE_MAX_K; ++k) if (G[k] > 0.0) c[k] = S[k] / G[k];
        for (int64_t j = 0; j < cols; ++j) {
            double w = (double)half_bits_to_float(W[i * ld + j]);
            double r = w - alpha[j] * c[labels[i * cols + j]];
            if (round_d) r = ldexp((double)half_bits_to_float(float_to_half_bits(ldexpf((float)r, exp2))), -exp2);
            d[j] = r;
        }
        for (int64_t k = 0; k < cols; ++k) {
            double acc = 0.0;
            for (int64_t j = 0; j < cols; ++j) acc += d[j] * Hd[j * cols + k];
            y[k] = acc;
        }
        for (int64_t j = 0; j < cols; ++j) {
            loss += y[j] * d[j];
            R[labels[i * cols + j]] += y[j] * alpha[j];
        }
        if (grad) {
            for (int64_t j = 0; j < cols; ++j) {
                double w = (double)half_bits_to_float(W[i * ld + j]);
                double g = (double)importance[i * ld + j];
                int l = labels[i * cols + j];
                double t = -2.0 * y[j] * c[l];
                if (G[l] > 0.0) t += 2.0 * R[l] * g * w / (alpha[j] * alpha[j] * G[l]);
                grad[j] += t;
            }
        }
    }
    free(Hd); free(rowbuf);
    *loss_out = loss;
    return 0;
}

/* `steps` Adam updates of alpha on the L-full loss (schedule and constants as in skim_oracle_scale_update). */
int skim_oracle_scale_update_lfull(const uint16_t *W, const float *importance, int64_t rows, int64_t cols, int64_t ld,
                                   const uint8_t *labels, const uint16_t *H, int64_t ldh, int exp2, int round_d,
                                   double *alpha, int steps, double lr0, double decay, int decay_every, double beta1,
                                   double beta2, double eps, double *loss_trace)
{
    if (steps < 0 || decay_every <= 0) return -1;
    double *m1 = (double *)calloc((size_t)cols, sizeof(double));
    double *m2 = (double *)calloc((size_t)cols, sizeof(double));
    double *grad = (double *)malloc((size_t)cols * sizeof(double));
    if (!m1 || !m2 || !grad) { free(m1); free(m2); free(grad); return -1; }
    int rc = 0;
    for (int t = 0; t < steps && !rc; ++t) {
        double loss;
        rc = skim_oracle_scale_loss_grad_lfull(W, importance, rows, cols, ld, labels, alpha, H, ldh, exp2, round_d, &loss, grad);
        if (loss_trace) loss_trace[t] = loss;
        double lr = lr0 * pow(decay, (double)(t / decay_every));
        double bc1 = 1.0 - pow(beta1, (double)(t + 1));
        double bc2 = 1.0 - pow(beta2, (double)(t + 1));
        for (int64_t j = 0; j < cols; ++j) {
            m1[j] = beta1 * m1[j] + (1.0 - beta1) * grad[j];
            m2[j] = beta2 * m2[j] + (1.0 - beta2) * grad[j] * grad[j];
            double mh = m1[j] / bc1, vh = m2[j] / bc2;
            alpha[j] -= lr * mh / (sqrt(vh) + eps);
        }
    }
    free(m1); free(m2); free(grad);
    return rc;
}

int skim_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
