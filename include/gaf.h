/*
 * gaf.h -- C ABI of the Gradient Agreement Filtering hot path for NVIDIA B200
 * (sm_100a).  Method: "Gradient Agreement Filtering", arxiv 2412.18052.
 *
 * Given K flattened micro-gradients of D parameters and a cosine-distance
 * threshold tau, the library computes the cosine distance of Eq. 4 between the
 * running sum of accepted micro-gradients and each incoming one, accepts or
 * rejects it as Algorithm 1 states (D_c <= tau), and returns the filtered
 * macro-gradient g/c of Eq. 5, the accept mask and the count c.  A K x K
 * pairwise cosine-distance matrix (the quantity the paper's cosine-distance
 * figures track) is provided for analysis.
 *
 * General conventions
 *   - "device" pointers are CUDA global-memory addresses on the current device,
 *     "host" pointers are ordinary process memory.
 *   - The caller owns every buffer, including the workspace.  The library
 *     allocates no device memory and keeps no state between calls other than
 *     what lives in the caller's workspace.
 *   - Every call is asynchronous on `cuda_stream` (a cudaStream_t passed as
 *     void*; NULL = the legacy default stream) and never synchronises, except
 *     gaf_read_status and the *_host convenience call, which say so.  Some
 *     kernels are launched with programmatic stream serialisation and signal
 *     early that the launch behind them may be placed: an ordinary launch
 *     behind a call is ordered after it as usual; a launch that the caller
 *     itself makes programmatic must, as always with such launches, wait for
 *     its predecessor (griddepcontrol.wait / cudaGridDependencySynchronize)
 *     before it reads the call's outputs.
 *   - Gradient buffers are read-only.  Every device pointer must be 16-byte
 *     aligned (else GAF_ERR_ALIGN).  D need not be a multiple of anything; with
 *     D == 0 the element buffers may be NULL.
 *   - dtype: GAF_F32 = IEEE binary32, GAF_BF16 = bfloat16.  Arithmetic on
 *     elements is binary32: products of at most 64 pairs are summed in binary32
 *     before they are widened (on the tensor-core paths that bfloat16 gradients
 *     take from 7 gradients on: binary32 accumulators over at most 512 products);
 *     the Gram sums of up to 4 binary32 gradients are taken in binary64
 *     throughout, where every product is exact.  Sums are carried in binary64
 *     from the thread level up and reduced in a fixed order, so results are
 *     bitwise reproducible on the same GPU model.  The scalar arithmetic of
 *     Eq. 4 and the comparison with tau are binary64.
 *   - Conventions where the paper is silent: a pair with a zero-norm member has
 *     cos := 0 (distance 1); cos is clamped to [-1, 1]; a NaN distance is
 *     rejected.  Either event sets a bit in the status word (see
 *     gaf_read_status) and is otherwise not an error.
 *   - Return value: GAF_OK or an error code; on an error detected on the host
 *     nothing was launched.
 */
#ifndef GAF_H_
#define GAF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GAF_MAX_K 64            /* largest number of micro-gradients per call */
#define GAF_MAX_BUCKETS 256     /* largest number of buckets of the bucketed variant */

enum { GAF_F32 = 0, GAF_BF16 = 1 };

enum {
    GAF_OK = 0,
    GAF_ERR_ARG = 1,            /* NULL pointer, K or D out of range, bad dtype/order/schedule */
    GAF_ERR_ALIGN = 2,          /* a device pointer is not 16-byte aligned */
    GAF_ERR_ALIAS = 3,          /* macro_out overlaps an input gradient */
    GAF_ERR_WORKSPACE = 4,      /* workspace missing, misaligned or too small */
    GAF_ERR_CUDA = 5,           /* a CUDA runtime call failed (launch, copy) */
    GAF_ERR_RESERVED = 6,       /* not used */
    GAF_ERR_UNSUPPORTED = 7,    /* the requested schedule cannot run for this call (K too large for it, or the
                                   device is still busy with a one-launch call on another stream) */
    GAF_ERR_TOO_LARGE = 8       /* size beyond the fixed limit of gaf_cosdist_static */
};

/* How gaf_filter_accumulate walks the K-1 sequential decisions of Algorithm 1.
 * All schedules produce the same mask and a bit-identical macro-gradient (the
 * accepted gradients are always added in processing order in binary32); they
 * differ in launch structure and in how many bytes cross HBM. */
enum {
    GAF_SCHED_AUTO = 0,         /* the library picks: Gram-first where a one-pass Gram kernel
                                   pays off (K <= 32; bfloat16: K <= 64), else stepwise.
                                   For K <= 8 the one-launch form is taken for K = 2, for binary32
                                   inputs of at most 512 MB in all, and for bfloat16 inputs except 7
                                   or 8 gradients of more than 1 GB in all (tensor-core Gram then);
                                   if the device refuses that launch, two launches. */
    GAF_SCHED_STEPWISE = 1,     /* streaming: one launch per step; each launch adds the
                                   gradient accepted at step t to the running sum and, in
                                   the same pass, takes the three dot products of the
                                   updated sum with the candidate of step t+1; decisions
                                   stay on the device */
    GAF_SCHED_GRAM = 2,         /* Gram-first: every gradient is read once to build the
                                   K x K Gram matrix, the K-1 decisions are taken on it (dot
                                   products are bilinear), then the accepted gradients are
                                   read once more to write g/c.  The distances agree with
                                   the stepwise schedule to rounding.  Two launches. */
    GAF_SCHED_GRAM_FUSED = 3    /* Gram-first as ONE launch (K <= 8) of a grid sized to what the device
                                   holds at once: the same two passes, every CTA taking the decisions
                                   itself from the partial sums all CTAs left in the workspace, so that
                                   part of what the first pass read (shared memory, L2) need not cross
                                   HBM again.  Identical outputs to GAF_SCHED_GRAM.  GAF_ERR_UNSUPPORTED
                                   for K > 8.  Such a call needs the whole device for its CTAs to meet:
                                   calls on one stream are ordered and fine; a second one on ANOTHER
                                   stream while the first stream still has work pending returns
                                   GAF_ERR_UNSUPPORTED (GAF_SCHED_AUTO takes two launches then), and so
                                   does a call on a stream that is being captured into a graph (what
                                   runs beside the node is decided at replay).  The one
                                   wait on other CTAs is bounded: GAF_STATUS_TIMEOUT if it ever runs out
                                   (only when something else, another process say, keeps part of the
                                   device busy for seconds).
                                   With K = 2 (the setting of the paper's experiments, Section 4) the
                                   result is either the mean of both gradients or the seed alone, and
                                   the first pass writes one of the two while it reads: the one the
                                   latest two such calls on the same workspace both ended with (a word
                                   in the workspace; a fresh workspace guesses "both"; no guess while
                                   the latest two differ).  A call whose decision matches the guess
                                   moves (2 b + 4) D bytes and has no second pass; one that does not
                                   rewrites the output.  The values never depend on the guess.
                                   GAF_SCHED_AUTO takes this form for K = 2 at every length. */
};

/* Bits of the device status word. */
enum {
    GAF_STATUS_ZERO_NORM = 1,   /* some tested pair had a zero norm (distance set to 1) */
    GAF_STATUS_NONFINITE = 2,   /* some sum was NaN or Inf */
    GAF_STATUS_TIMEOUT = 4,     /* a bounded wait inside a kernel (tensor-core Gram pipeline,
                                   one-launch Gram-first schedule) ran out; the outputs of that
                                   call are not valid */
    GAF_STATUS_ILL_CONDITIONED = 8  /* after some accept the running sum g of the c accepted gradients
                                   had c * sum_i |g_i|^2 > 167 |g|^2: the accepted gradients nearly
                                   cancel (only possible with tau > 1, when a gradient that points
                                   against the sum is accepted).  |g|^2 is then a small difference of
                                   large binary32-rounded terms and neither the 1e-5 on the distances
                                   of Eq. 4 nor the 1e-6 on the binary32 macro-gradient is guaranteed
                                   from that step on.  The outputs are still what the arithmetic
                                   gave; not an error. */
};

/* Human-readable name of a return code.  Host only; never NULL. */
const char *gaf_error_string(int code);

/*
 * Size in bytes of the workspace a call with these K, D, dtype needs (the
 * maximum over the three operations).  Host only, touches no GPU.
 * Errors: GAF_ERR_ARG for K outside [1, GAF_MAX_K], D < 0, bad dtype or NULL.
 */
int gaf_workspace_bytes(int K, int64_t D, int dtype, size_t *bytes_out);

/*
 * Prepare a workspace: clears its control block (asynchronous memset on the
 * stream).  Needed once after allocation; every call leaves the workspace ready
 * for the next one.  A workspace serves one call at a time: calls that share a
 * workspace must be ordered on one stream.
 *   workspace        device, 256-byte aligned, >= gaf_workspace_bytes(...)
 */
int gaf_workspace_init(void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Cosine distance of Eq. 4 between two buffers:
 *     D_c(x, y) = 1 - x.y / (|x| |y|).
 *   x, y        device, D elements of `dtype` each
 *   dist_out    device, 1 float
 *   stats_out   device, 3 doubles {x.y, |x|^2, |y|^2}; may be NULL
 */
int gaf_cosdist(const void *x, const void *y, int64_t D, int dtype,
                float *dist_out, double *stats_out,
                void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Algorithm 1 for one macrobatch followed by Eq. 5 (Section 3.1):
 *     g <- g_{order[0]};  c <- 1
 *     for t = 1 .. K-1, i = order[t]:
 *         if D_c(g_i, g) <= tau:  g <- g + g_i;  c <- c + 1
 *     macro_out <- g / c
 * The test is against the running SUM g; the division happens once, at the end.
 * The update/skip rule of the paper (skip the optimiser step when c == 1) is
 * the caller's: read count_out.
 *
 *   grads       HOST array of K device pointers, D elements of `dtype` each
 *   K           1 .. GAF_MAX_K (K == 1 returns the seed, c = 1)
 *   D           >= 0
 *   tau         threshold; tau >= 2 accepts everything (plain mean of Eq. 2),
 *               tau < 0 rejects everything
 *   order       HOST, permutation of 0..K-1, order[0] = seed s; NULL = identity
 *               (the paper samples s at random: do that on the host)
 *   macro_out   device, D floats (binary32 also for bf16 inputs); doubles as
 *               the running sum during the call; must not overlap any input
 *   mask_out    device, K bytes, by ORIGINAL index i: 1 accepted, 0 rejected;
 *               mask[s] = 1
 *   dist_out    device, K floats, by original index: D_c(g_i, g) at the moment
 *               g_i was tested; dist[s] = 0; may be NULL
 *   count_out   device, 1 int32: c
 *   schedule    one of GAF_SCHED_*
 */
int gaf_filter_accumulate(const void *const *grads, int K, int64_t D, int dtype,
                          double tau, const int32_t *order,
                          float *macro_out, uint8_t *mask_out, float *dist_out,
                          int32_t *count_out,
                          void *workspace, size_t workspace_bytes,
                          int schedule, void *cuda_stream);

/*
 * The same call `repeats` times back to back on the stream, cycling through `n_sets` sets of
 * inputs (call r reads set r mod n_sets): exactly what a host loop in C around
 * gaf_filter_accumulate does, for callers -- benchmarks above all -- driven from an interpreted
 * language whose own per-call cost would otherwise be measured instead of the library's.  Every
 * repetition overwrites the same outputs; gaf_last_launch_count() reports the launches of all
 * repetitions together.
 *   grads       HOST array of n_sets * K device pointers, set after set
 *   repeats     >= 0;  n_sets >= 1;  everything else as in gaf_filter_accumulate
 */
int gaf_filter_accumulate_repeat(int repeats, int n_sets, const void *const *grads, int K, int64_t D,
                                 int dtype, double tau, const int32_t *order,
                                 float *macro_out, uint8_t *mask_out, float *dist_out,
                                 int32_t *count_out,
                                 void *workspace, size_t workspace_bytes,
                                 int schedule, void *cuda_stream);

/*
 * Order-indifferent variant, as sketched at the end of Section 3.1: Algorithm 1 is
 * order dependent (a first gradient orthogonal to all others wastes the whole
 * macrobatch), so every micro-gradient in turn acts as the initial one, the
 * others following in ring order s, s+1, ..., K-1, 0, ..., s-1, and the result
 * with the largest agreement is kept.  Where the paper leaves it open: agreement
 * is the accepted count c; ties go to the smallest s.  All K walks run on one
 * K x K Gram matrix (dot products are bilinear), so the cost is that of
 * gaf_filter_accumulate with GAF_SCHED_GRAM: every gradient read once, the
 * accepted ones once more.
 *   mask_out, dist_out, count_out, macro_out   as in gaf_filter_accumulate, for
 *               the winning seed (dist[seed] = 0); the accepted gradients are added
 *               in the winning ring order
 *   seed_out    device, 1 int32: the winning seed
 */
int gaf_filter_accumulate_any_seed(const void *const *grads, int K, int64_t D, int dtype,
                                   double tau,
                                   float *macro_out, uint8_t *mask_out, float *dist_out,
                                   int32_t *count_out, int32_t *seed_out,
                                   void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Bucketed variant.  Section 5 notes that inside a ring all-reduce the cosine distance
 * would be applied "to buckets at a time": here the D parameters are cut into S
 * consecutive buckets (the tensors of a network, the buckets of an all-reduce) and
 * Algorithm 1 + Eq. 5 run on every bucket independently -- its own running sum,
 * decisions and count.  Gram-first: one pass builds a K x K Gram matrix per bucket,
 * the decisions are walked per bucket, one pass writes every bucket's g/c.
 *   K           1 .. 8
 *   S, offsets  1 <= S <= GAF_MAX_BUCKETS; HOST array of S+1 ascending element offsets,
 *               offsets[0] = 0, offsets[S] = D; every offset but the last must be a
 *               multiple of 8 elements (else GAF_ERR_ALIGN); empty buckets are legal
 *   macro_out   device, D floats: bucket b holds its g/c
 *   mask_out    device, S*K bytes, row b = bucket b, by original index
 *   dist_out    device, S*K floats or NULL;  count_out  device, S int32
 */
int gaf_filter_accumulate_bucketed(const void *const *grads, int K, int64_t D, int dtype,
                                   double tau, const int32_t *order,
                                   int S, const int64_t *offsets,
                                   float *macro_out, uint8_t *mask_out, float *dist_out,
                                   int32_t *count_out,
                                   void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Streaming form of Algorithm 1, for micro-gradients that arrive one at a time (as
 * they do around a ring, Section 1 / Section 3.1): the loop body of Algorithm 1 per
 * call.  The state lives in `workspace` (one stream of calls per workspace) and in
 * the caller's running-sum buffer `acc` (D floats, 16-byte aligned).
 *   gaf_stream_begin   g <- seed; c <- 1
 *   gaf_stream_push    gradient number t (t = 1, 2, ... in arrival order, t < GAF_MAX_K):
 *                      D_c(g_t, g) by Eq. 4; if <= tau: g <- g + g_t, c <- c + 1.
 *                      `g` may be reused as soon as the call's work on the stream is done.
 *   gaf_stream_end     acc <- g / c (Eq. 5); mask_out[K], dist_out[K] (may be NULL) in
 *                      ARRIVAL order (entry 0 = seed: 1 and 0), count_out = c
 * Same arithmetic as gaf_filter_accumulate with GAF_SCHED_STEPWISE: the result is
 * bit-identical to that call on the same gradients in arrival order.
 */
int gaf_stream_begin(const void *seed, int64_t D, int dtype, float *acc,
                     void *workspace, size_t workspace_bytes, void *cuda_stream);
int gaf_stream_push(const void *g, int t, int64_t D, int dtype, double tau, float *acc,
                    void *workspace, size_t workspace_bytes, void *cuda_stream);
int gaf_stream_end(int K, int64_t D, float *acc, uint8_t *mask_out, float *dist_out,
                   int32_t *count_out,
                   void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * The same operation for gradients that live in HOST memory (pinned memory
 * makes the copies asynchronous and fast).  Copies each gradient to the device
 * staging area, runs gaf_filter_accumulate, copies the results back and
 * SYNCHRONISES the stream before returning.
 *   grads_host      HOST array of K host pointers, D elements each
 *   macro_out_host  host, D floats;  mask_out_host host, K bytes;
 *   dist_out_host   host, K floats or NULL;  count_out_host host, 1 int32
 *   staging         device, 256-byte aligned scratch for inputs and outputs,
 *                   >= gaf_host_staging_bytes(K, D, dtype)
 */
int gaf_host_staging_bytes(int K, int64_t D, int dtype, size_t *bytes_out);
int gaf_filter_accumulate_host(const void *const *grads_host, int K, int64_t D, int dtype,
                               double tau, const int32_t *order,
                               float *macro_out_host, uint8_t *mask_out_host,
                               float *dist_out_host, int32_t *count_out_host,
                               void *staging, size_t staging_bytes,
                               void *workspace, size_t workspace_bytes,
                               int schedule, void *cuda_stream);

/*
 * Pairwise cosine distances between K micro-gradients (Eq. 4 for every pair;
 * what the paper's cosine-distance-over-training figures plot):
 *     G = X X^T,  dist[i][j] = 1 - G_ij / (sqrt(G_ii) sqrt(G_jj)).
 *   grads       HOST array of K device pointers
 *   dist_out    device, K*K floats row-major; symmetric; diagonal 0 (1 for a
 *               zero-norm gradient, whose whole row and column are 1)
 *   gram_out    device, K*K doubles row-major (the Gram matrix); may be NULL
 * bfloat16 with 17 to 42 gradients runs fastest when the gradients are rows of one matrix (see
 * gaf_last_gram_loader); any other placement is accepted.
 */
int gaf_pairwise_cosdist(const void *const *grads, int K, int64_t D, int dtype,
                         float *dist_out, double *gram_out,
                         void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Read the device status word of the most recent call that used `workspace`.
 * SYNCHRONISES the stream.  *status_out receives GAF_STATUS_* bits.
 */
int gaf_read_status(const void *workspace, void *cuda_stream, int *status_out);

/*
 * gaf_cosdist for callers that cannot allocate device memory.  (The paper has no
 * counterpart of this entry point: it exists for integration reasons only.)
 *
 * Every other call here needs a workspace that the caller allocated.  Some
 * callers cannot provide one: code that runs inside another framework's memory
 * pool with allocation disabled, a plug-in called at a point where cudaMalloc
 * would stall the whole device, a host program that is not allowed to touch the
 * allocator after start-up.  This variant computes the same D_c(x, y) of Eq. 4
 * with the same kernel, but keeps its scratch memory (one ticket, one status
 * word, 512 per-CTA partial triples: 12,544 bytes) in a fixed array inside the
 * library's device image.  It calls no cudaMalloc / cudaFree and no allocating
 * library routine.
 *
 *   x, y        device, D elements of `dtype`, 16-byte aligned
 *   D           0 .. GAF_STATIC_MAX_D; larger D returns GAF_ERR_TOO_LARGE
 *               ("size beyond the fixed limit ...") and launches nothing
 *   dist_out    device, 1 float;  stats_out  device, 3 doubles or NULL
 *
 * Things to know:
 *   - Every GPU on which the library is loaded holds the array until the
 *     process exits.
 *   - The first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress, with that device current) and remembers it.  Make
 *     that first call outside any stream capture.
 *   - All calls share the one array, which keeps the previous call's contents;
 *     each call clears the words that must start at zero (an asynchronous
 *     16-word memset on the stream ahead of the kernel).  Two calls that can
 *     overlap on the GPU (different streams without ordering, or two host
 *     threads on one device) race on it: order them.
 *   - The status word is not readable through gaf_read_status (that call takes a
 *     workspace); the zero-norm convention still applies (distance 1).
 *   - Asynchronous on `cuda_stream`, like gaf_cosdist.
 */
#define GAF_STATIC_MAX_D ((int64_t)1 << 31)
int gaf_cosdist_static(const void *x, const void *y, int64_t D, int dtype,
                       float *dist_out, double *stats_out, void *cuda_stream);

/* Number of kernel launches the most recent gaf_* call of this thread issued
 * (host-side counter, for benchmarks; gaf_cosdist_static counts too). */
int gaf_last_launch_count(void);

/* The GAF_SCHED_* value the most recent gaf_filter_accumulate call of this thread ran with
 * (what GAF_SCHED_AUTO resolved to).  Host-side, for benchmarks and tests. */
int gaf_last_schedule(void);

/* How the tensor-memory Gram kernel (bfloat16, 17 to 64 gradients) of this thread's most recent call fetched
 * its tiles: 0 the call did not use that kernel, 1 16-byte asynchronous copies, 2 tensor copies (TMA) --
 * taken when the gradients are rows of one matrix: grads[i] = grads[0] + i * stride with a positive stride
 * that is a multiple of 128 bytes (the layout an all-gather of flattened, padded micro-gradients leaves),
 * 64 <= D < 2^31, at most 42 gradients (beyond that the 16-byte copies measured faster).  The tensor
 * copies are 3 to 10 % faster up to 32 gradients and 20 to 27 % with 33 to 42; both give the same Gram matrix
 * up to the rounding order inside one MMA.
 * Host-side, for tests. */
int gaf_last_gram_loader(void);

/*
 * Test hook for the bounded waits inside the kernels (failure detection without a faulted GPU).
 * Two kernels wait on something another part of the same launch produces: the one-launch
 * Gram-first schedule (its CTAs poll one word for the decisions) and the tensor-core Gram
 * pipeline (mbarrier waits between loaders, MMA issuer and epilogue).  Every such wait gives up
 * after a fixed number of attempts -- seconds in normal use, never reached -- raises
 * GAF_STATUS_TIMEOUT and lets the kernel return in an orderly way (copies in flight are awaited,
 * tensor memory is freed).  This call lets a test see that path run, for the following launches of
 * the calling thread:
 *   wait_limit   attempts before a wait gives up; 0 restores the built-in limits
 *   withhold     non-zero: the awaited signal is never given (the deciding CTA does not publish the
 *                decision word; the first tile's barrier expects one arrival more than will come),
 *                so that every wait runs out.  Nothing traps and nothing waits without a limit.
 * The outputs of a call made with `withhold` set are not valid; the workspace stays usable: the next
 * ordinary call on it is correct.  Always returns GAF_OK.  Off by default; not for production use.
 */
int gaf_test_set_wait_fault(unsigned int wait_limit, int withhold);

#ifdef __cplusplus
}
#endif
#endif /* GAF_H_ */
