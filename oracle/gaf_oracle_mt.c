/*
 * The fp64 CPU oracle of Algorithm 1 + Eq. 5 split over several host threads.
 *
 * TEST INFRASTRUCTURE ONLY, like gaf_oracle.c: this file exists so that the
 * benchmark can report a CPU baseline on ALL host cores beside the
 * single-thread one.  It is the same statement of the method -- the same plain
 * loops in double precision, in the paper's order -- with every pass over the D
 * parameters cut into consecutive chunks, one chunk per thread, and the three
 * sums of a test combined in chunk order (a fixed order, so results do not
 * depend on thread timing).  Nothing else is changed: no blocking, no
 * vectorisation tricks, no fusion of steps.  Element widening and Eq. 4 are the
 * single-thread file's own functions (included below), so there is one
 * definition of each.  tests/ pins it against the single-thread routine.
 */
#include <pthread.h>
#include <stdlib.h>

#include "gaf_oracle.c"

enum { PASS_SEED, PASS_SUMS, PASS_ADD, PASS_DIVIDE };

typedef struct {
    int pass;
    const void *src;            /* the gradient this pass reads (seed or g_i) */
    int dtype;
    double *g;                  /* running sum */
    int64_t lo, hi;             /* this thread's chunk of the D parameters */
    double divisor;             /* PASS_DIVIDE */
    double p, ng, ni;           /* PASS_SUMS: this chunk's partial sums */
} chunk_job;

static void *run_chunk(void *arg)
{
    chunk_job *j = (chunk_job *)arg;
    double *g = j->g;
    switch (j->pass) {
    case PASS_SEED:             /* g <- g_s */
        for (int64_t d = j->lo; d < j->hi; ++d) g[d] = elem(j->src, d, j->dtype);
        break;
    case PASS_SUMS: {           /* g_i.g, |g|^2, |g_i|^2 over the chunk */
        double p = 0.0, ng = 0.0, ni = 0.0;
        for (int64_t d = j->lo; d < j->hi; ++d) {
            double v = elem(j->src, d, j->dtype);
            p += v * g[d];
            ng += g[d] * g[d];
            ni += v * v;
        }
        j->p = p; j->ng = ng; j->ni = ni;
        break;
    }
    case PASS_ADD:              /* g <- g + g_i */
        for (int64_t d = j->lo; d < j->hi; ++d) g[d] += elem(j->src, d, j->dtype);
        break;
    case PASS_DIVIDE:           /* g <- g / c */
        for (int64_t d = j->lo; d < j->hi; ++d) g[d] = g[d] / j->divisor;
        break;
    }
    return NULL;
}

/* One pass over all chunks: one thread per chunk, joined before returning. */
static int run_pass(chunk_job *jobs, pthread_t *threads, int n, int pass, const void *src, double divisor)
{
    for (int c = 0; c < n; ++c) {
        jobs[c].pass = pass; jobs[c].src = src; jobs[c].divisor = divisor;
        if (pthread_create(&threads[c], NULL, run_chunk, &jobs[c]) != 0) {
            for (int k = 0; k < c; ++k) pthread_join(threads[k], NULL);
            return 1;
        }
    }
    for (int c = 0; c < n; ++c) pthread_join(threads[c], NULL);
    return 0;
}

/*
 * Algorithm 1 (one macrobatch) + Eq. 5 on `n_threads` threads.  Arguments as
 * gaf_oracle_filter_accumulate (without forced decisions and statistics).
 */
int gaf_oracle_filter_accumulate_mt(const void *const *grads, int K, int64_t D,
                                    int dtype, double tau, const int32_t *order,
                                    double *g, uint8_t *mask, double *dist,
                                    int32_t *count, int n_threads)
{
    if (K < 1 || n_threads < 1 || n_threads > 4096) return 1;
    chunk_job *jobs = (chunk_job *)calloc((size_t)n_threads, sizeof *jobs);
    pthread_t *threads = (pthread_t *)calloc((size_t)n_threads, sizeof *threads);
    if (!jobs || !threads) { free(jobs); free(threads); return 1; }
    for (int c = 0; c < n_threads; ++c) {
        jobs[c].dtype = dtype; jobs[c].g = g;
        jobs[c].lo = D / n_threads * c + (c < D % n_threads ? c : D % n_threads);
        jobs[c].hi = jobs[c].lo + D / n_threads + (c < D % n_threads ? 1 : 0);
    }
    int rc = 0;
    int s = order ? order[0] : 0;
    rc |= run_pass(jobs, threads, n_threads, PASS_SEED, grads[s], 0.0);
    int32_t cnt = 1;
    mask[s] = 1;
    dist[s] = 0.0;
    for (int t = 1; t < K && !rc; ++t) {
        int i = order ? order[t] : t;
        rc |= run_pass(jobs, threads, n_threads, PASS_SUMS, grads[i], 0.0);
        double p = 0.0, ng = 0.0, ni = 0.0;
        for (int c = 0; c < n_threads; ++c) { p += jobs[c].p; ng += jobs[c].ng; ni += jobs[c].ni; }
        double dc = distance_from_sums(p, ng, ni);
        dist[i] = dc;
        if (dc <= tau) {
            rc |= run_pass(jobs, threads, n_threads, PASS_ADD, grads[i], 0.0);
            cnt += 1;
            mask[i] = 1;
        } else {
            mask[i] = 0;
        }
    }
    if (!rc) rc |= run_pass(jobs, threads, n_threads, PASS_DIVIDE, NULL, (double)cnt);
    *count = cnt;
    free(jobs);
    free(threads);
    return rc;
}
