/*
 * Plain fp64 CPU oracle for Gradient Agreement Filtering (arxiv 2412.18052).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement
 * of what the method computes, written from the paper; the tests and the CPU
 * baseline leg of the benchmark call it, the product library never does.  It
 * shares no code, header, table or helper with the CUDA path.
 *
 * Every loop is a single sequential pass in double precision, in the order the
 * paper states the steps (Algorithm 1; Eq. 4 for the cosine distance; Eq. 5 for
 * the final division).  No blocking, no vectorisation tricks, no reordering.
 *
 * Conventions that the paper leaves open (each listed again in the design
 * notes of the repository):
 *   - zero-norm rule: if either vector of a pair has squared norm 0, cos := 0,
 *     so the distance is 1.                               [parity unpinned]
 *   - cos is clamped to [-1, 1] so the distance stays in the range [0, 2] the
 *     paper states in its introduction.
 *   - a NaN distance is rejected (the comparison d <= tau is false).
 *                                                          [parity unpinned]
 *   - the update/skip block of Algorithm 1 is read as sitting after the inner
 *     loop: one g/c per macrobatch (Section 3.1, Eq. 5).   [parity unpinned]
 *
 * Element types: dtype 0 = IEEE binary32, dtype 1 = bfloat16 given as 16-bit
 * patterns.  Both widen to double exactly.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };

/* Exact widening of element d of a buffer to double. */
static double elem(const void *buf, int64_t d, int dtype)
{
    if (dtype == ORACLE_F32) {
        return (double)((const float *)buf)[d];
    } else {
        /* bfloat16 is the upper half of a binary32 */
        uint32_t bits = ((uint32_t)((const uint16_t *)buf)[d]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
}

/* Eq. 4 on three already-computed sums: 1 - p / (sqrt(na) sqrt(nb)). */
static double distance_from_sums(double p, double na, double nb)
{
    double cosv;
    if (na == 0.0 || nb == 0.0) {
        cosv = 0.0;                       /* zero-norm rule */
    } else {
        cosv = p / (sqrt(na) * sqrt(nb));
        if (cosv > 1.0) cosv = 1.0;       /* keep D_c inside [0, 2] */
        if (cosv < -1.0) cosv = -1.0;
    }
    return 1.0 - cosv;
}

/*
 * Cosine distance between two buffers (Eq. 4).
 * stats, if not NULL, receives {x.y, |x|^2, |y|^2}.
 */
int gaf_oracle_cosdist(const void *x, const void *y, int64_t D, int dtype,
                       double *dist_out, double *stats)
{
    double p = 0.0, nx = 0.0, ny = 0.0;
    for (int64_t d = 0; d < D; ++d) {
        double a = elem(x, d, dtype);
        double b = elem(y, d, dtype);
        p += a * b;
        nx += a * a;
        ny += b * b;
    }
    *dist_out = distance_from_sums(p, nx, ny);
    if (stats) { stats[0] = p; stats[1] = nx; stats[2] = ny; }
    return 0;
}

/*
 * Algorithm 1, inner part (one macrobatch): seed, test each remaining
 * micro-gradient against the running SUM of accepted ones, add it if its
 * cosine distance is <= tau, count, and finally divide by the count (Eq. 5).
 *
 *   grads   K pointers to D elements each
 *   order   permutation of 0..K-1, order[0] is the seed s; NULL = identity
 *   forced  NULL, or K entries indexed by step t (entry 0 unused):
 *           -1 = decide by the test, 0 = force reject, 1 = force accept
 *   g       D doubles: running sum during the call, g/c on return
 *   mask    K bytes by ORIGINAL index; mask[s] = 1
 *   dist    K doubles by original index; dist[s] = 0
 *   stats   NULL or 3*K doubles by original index: {g_i.g, |g|^2, |g_i|^2}
 *           as seen by the test of g_i (zeros for the seed)
 */
int gaf_oracle_filter_accumulate(const void *const *grads, int K, int64_t D,
                                 int dtype, double tau, const int32_t *order,
                                 const int8_t *forced, double *g,
                                 uint8_t *mask, double *dist, int32_t *count,
                                 double *stats)
{
    if (K < 1) return 1;
    int s = order ? order[0] : 0;

    /* g <- g_s ; c <- 1 */
    for (int64_t d = 0; d < D; ++d) g[d] = elem(grads[s], d, dtype);
    int32_t c = 1;
    mask[s] = 1;
    dist[s] = 0.0;
    if (stats) { stats[3 * s] = stats[3 * s + 1] = stats[3 * s + 2] = 0.0; }

    /* for i in [1, k], i != s */
    for (int t = 1; t < K; ++t) {
        int i = order ? order[t] : t;
        const void *gi = grads[i];

        double p = 0.0, ng = 0.0, ni = 0.0;
        for (int64_t d = 0; d < D; ++d) {
            double v = elem(gi, d, dtype);
            p += v * g[d];
            ng += g[d] * g[d];
            ni += v * v;
        }
        double dc = distance_from_sums(p, ng, ni);
        dist[i] = dc;
        if (stats) { stats[3 * i] = p; stats[3 * i + 1] = ng; stats[3 * i + 2] = ni; }

        int accept = (dc <= tau);          /* false for NaN */
        if (forced && forced[t] >= 0) accept = forced[t];

        if (accept) {
            for (int64_t d = 0; d < D; ++d) g[d] += elem(gi, d, dtype);
            c += 1;
            mask[i] = 1;
        } else {
            mask[i] = 0;
        }
    }

    /* g_GAF = g / c */
    for (int64_t d = 0; d < D; ++d) g[d] = g[d] / (double)c;
    *count = c;
    return 0;
}

/*
 * Order-indifferent variant sketched at the end of Section 3.1: every micro-gradient
 * in turn acts as the initial one and the others follow "around the ring", i.e. for
 * seed s the processing order is s, s+1, ..., K-1, 0, ..., s-1; Algorithm 1 runs on
 * each of the K orders and the result with the largest agreement is kept.
 * Reading taken where the paper leaves it open: agreement = the accepted count c;
 * ties go to the smallest s.                                 [parity unpinned]
 *   g, mask, dist, count   as in gaf_oracle_filter_accumulate, for the winning seed
 *   seed_out               the winning seed
 *   counts_out             NULL or K entries: c obtained with each seed
 *   work                   D doubles of scratch
 */
int gaf_oracle_filter_any_seed(const void *const *grads, int K, int64_t D, int dtype,
                               double tau, double *g, uint8_t *mask, double *dist,
                               int32_t *count, int32_t *seed_out, int32_t *counts_out,
                               double *work)
{
    if (K < 1 || K > 4096) return 1;
    int32_t order[4096];
    uint8_t m[4096];
    double dd[4096];
    int best_seed = -1;
    int32_t best_count = 0;
    for (int s = 0; s < K; ++s) {
        for (int t = 0; t < K; ++t) order[t] = (s + t) % K;
        int32_t c = 0;
        gaf_oracle_filter_accumulate(grads, K, D, dtype, tau, order, NULL, work, m, dd, &c, NULL);
        if (counts_out) counts_out[s] = c;
        if (c > best_count) { best_count = c; best_seed = s; }
    }
    for (int t = 0; t < K; ++t) order[t] = (best_seed + t) % K;
    gaf_oracle_filter_accumulate(grads, K, D, dtype, tau, order, NULL, g, mask, dist, count, NULL);
    *seed_out = best_seed;
    return 0;
}

/*
 * Bucketed variant (Section 5 notes that inside a ring all-reduce the cosine distance
 * would have to be applied "to buckets at a time"): the D parameters are cut into S
 * consecutive buckets, bucket b = elements [offsets[b], offsets[b+1]), and Algorithm 1
 * followed by Eq. 5 runs on every bucket independently -- its own running sum, its own
 * decisions, its own count.                                     [parity unpinned]
 *   offsets  S+1 ascending element offsets, offsets[0] = 0, offsets[S] = D
 *   g        D doubles: per-bucket g/c on return
 *   mask     S*K bytes, row b = bucket b, by original index
 *   dist     S*K doubles;  count  S entries
 */
int gaf_oracle_filter_bucketed(const void *const *grads, int K, int64_t D, int dtype,
                               double tau, const int32_t *order, int S,
                               const int64_t *offsets, double *g, uint8_t *mask,
                               double *dist, int32_t *count)
{
    if (K < 1 || K > 4096 || S < 1 || offsets[0] != 0 || offsets[S] != D) return 1;
    size_t esize = dtype == ORACLE_F32 ? 4 : 2;
    const void *sub[4096];
    for (int b = 0; b < S; ++b) {
        int64_t lo = offsets[b], hi = offsets[b + 1];
        if (hi < lo) return 1;
        for (int i = 0; i < K; ++i) sub[i] = (const char *)grads[i] + (size_t)lo * esize;
        int rc = gaf_oracle_filter_accumulate(sub, K, hi - lo, dtype, tau, order, NULL, g + lo,
                                              mask + (size_t)b * K, dist + (size_t)b * K,
                                              count + b, NULL);
        if (rc) return rc;
    }
    return 0;
}

/*
 * Pairwise cosine distances between K micro-gradients (the quantity the
 * paper's cosine-distance figures plot).  gram and dist are K*K row-major.
 * Diagonal: 0 when the norm is non-zero; rows/columns of a zero-norm vector
 * are all 1, diagonal included (zero-norm rule).
 */
int gaf_oracle_pairwise(const void *const *grads, int K, int64_t D, int dtype,
                        double *gram, double *dist)
{
    for (int i = 0; i < K; ++i) {
        for (int j = i; j < K; ++j) {
            double p = 0.0;
            for (int64_t d = 0; d < D; ++d)
                p += elem(grads[i], d, dtype) * elem(grads[j], d, dtype);
            gram[i * K + j] = p;
            gram[j * K + i] = p;
        }
    }
    for (int i = 0; i < K; ++i) {
        for (int j = 0; j < K; ++j) {
            double dc;
            if (i == j && gram[i * K + i] > 0.0) dc = 0.0;
            else dc = distance_from_sums(gram[i * K + j], gram[i * K + i], gram[j * K + j]);
            dist[i * K + j] = dc;
        }
    }
    return 0;
}

/* Plain average of Eq. 2, (1/k) sum_i g_i -- the aggregation GAF replaces. */
int gaf_oracle_plain_average(const void *const *grads, int K, int64_t D,
                             int dtype, double *out)
{
    for (int64_t d = 0; d < D; ++d) {
        double sum = 0.0;
        for (int i = 0; i < K; ++i) sum += elem(grads[i], d, dtype);
        out[d] = sum / (double)K;
    }
    return 0;
}
