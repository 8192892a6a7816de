// Gram-first schedule of Algorithm 1.
//
// The test of step t needs <g_i, g>, |g|^2 and |g_i|^2 where g is the sum of the
// gradients accepted so far.  Dot products are bilinear, so all of them follow from
// the K x K Gram matrix G_ij = <g_i, g_j> of the raw micro-gradients:
//     <g_i, sum_A g_j> = sum_{j in A} G_ji,     |sum_A g_j|^2 = sum_{j,l in A} G_jl.
// The schedule therefore reads every gradient ONCE to build G (binary64 sums), walks
// the K-1 sequential decisions of Algorithm 1 on K^2 scalars in a single thread, and
// then reads only the accepted gradients once more to write g/c (Eq. 5):
// ((K + c) b + 4) D bytes instead of one pass over the running sum per step, and no
// grid-wide serialisation per step.  The accepted gradients are added in processing
// order in binary32, so the macro-gradient is bit-identical to the streaming
// schedules'; the distances differ from theirs only by rounding (the running sum is
// never rounded to binary32 here).
#pragma once

#include "gaf_device.cuh"

namespace gaf {

constexpr int kGsThreads = 512;
constexpr int kGsMaxK = 8;                  // gradients the one-pass register-tiled Gram handles
constexpr int kGsMaxCtas = 296;
constexpr int kGsPartialStride = 320;       // per-CTA partials are stored [pair][CTA]: the totalling loads coalesce
constexpr int kGsFlushEvery = 16;           // iterations between binary64 flushes
constexpr int kMsThreads = 512;
constexpr int kMsLongRun = 8;                // chunks per run of the masked-mean pass on long vectors
constexpr int kReplayMaxK = 8;               // the table form of the walk: 2^(K-1) - 1 cases

struct ReplayArgs {
    int K;
    double tau;
    int idx[GAF_MAX_K];                     // original index of the gradient processed at step t
    uint8_t *mask_out;
    float *dist_out;                        // may be null
    int32_t *count_out;
    Control *ctl;
};

// Algorithm 1 on the Gram matrix (indexed by processing step): one thread.
// gram is K x K row-major in binary64.  With `publish` the decisions, distances and count go
// to the outputs and the control block; the accept bits (bit t = step t) are returned either way.
__device__ __forceinline__ unsigned long long replay_on_gram(const ReplayArgs &r, const volatile double *gram,
                                                             bool publish) {
    const int K = r.K;
    Control *c = r.ctl;
    int status = 0, count = 1;
    unsigned long long bits = 1ull;         // step 0 is the seed
    double na = gram[0];                    // |g|^2 of the running sum
    double norm_sq = gram[0];               // sum of |g_i|^2 over the accepted gradients
    if (publish) {
        c->decision[0] = 1;
        r.mask_out[r.idx[0]] = 1;
        if (r.dist_out) r.dist_out[r.idx[0]] = 0.0f;
    }
    for (int t = 1; t < K; ++t) {
        double p = 0.0;                     // <g_t, running sum>
        for (int u = 0; u < t; ++u)
            if ((bits >> u) & 1ull) p += gram[(size_t)u * K + t];
        const double ng = gram[(size_t)t * K + t];
        const double d = cosine_distance(p, na, ng, &status);
        const int accept = (d <= r.tau) ? 1 : 0;
        if (publish) {
            c->decision[t] = accept;
            c->sums[t][0] = p; c->sums[t][1] = na; c->sums[t][2] = ng;
            r.mask_out[r.idx[t]] = (uint8_t)accept;
            if (r.dist_out) r.dist_out[r.idx[t]] = (float)d;
        }
        if (accept) {
            bits |= 1ull << t;
            na = na + 2.0 * p + ng;         // |g + g_t|^2
            norm_sq += ng;
            ++count;
            status |= ill_conditioned(count, norm_sq, na);
        }
    }
    if (publish) {
        c->accept_bits = bits;
        c->ring_seed = -1;
        c->count = count;
        // (OR, not store: an earlier kernel of the operation may have raised a bit; the first kernel cleared the word)
        if (status) atomicOr(&c->status, status);
        *r.count_out = count;
    }
    return bits;
}

// The same walk for K <= 8 with its latency taken out of the serial part.  Step t's test depends on
// the earlier decisions only through WHICH gradients were accepted, so one thread per (step t,
// accept pattern of steps 1..t-1) evaluates Eq. 4 for that case -- 2^(K-1) - 1 threads, all at once --
// and thread 0 then only follows the decisions through the table.  Every case repeats the sums of
// the sequential walk in the same order, so the results are the same to the last bit.
// All threads of the block call (blockDim.x >= 128).  `early(bits)` is called by thread 0 as soon as
// the accept bits are known, before the outputs are written.  With `publish` false nothing is written
// to global memory (the one-launch schedule runs the walk in every CTA and lets one of them publish).
struct ReplayTable {
    double d[127], p[127], na[127];
    unsigned char accept[127], status[127];
};
struct NoEarlyBits {
    __device__ __forceinline__ void operator()(unsigned long long) const {}
};
template <int KT, typename Early = NoEarlyBits>
__device__ __forceinline__ void replay_on_gram_parallel(const ReplayArgs &r, const double *gram, ReplayTable &tb,
                                                        Early early = Early(), bool publish = true) {
    constexpr int K = KT;
    const int tid = threadIdx.x;
    constexpr int cases = (1 << (K - 1)) - 1;
    if (tid < cases) {
        const int t = 32 - __clz(tid + 1);                      // tid + 1 in [2^(t-1), 2^t)
        const unsigned int m = (unsigned int)(tid + 1) - (1u << (t - 1));
        // step v accepted in this case (bits of m at and above t-1 are zero)
        auto in = [&](int v) { return v == 0 || ((m >> (v - 1)) & 1u); };
        // Branch-free (neighbouring lanes hold different cases): a gradient that is not in the case
        // contributes an added 0.0, which leaves a binary64 sum unchanged, and its update of |g|^2
        // is computed and dropped.
        double na = gram[0], norm_sq = gram[0];
        int cnt = 1;
#pragma unroll
        for (int u = 1; u < K - 1; ++u) {
            double pu = 0.0;
#pragma unroll
            for (int v = 0; v < u; ++v) pu += in(v) ? gram[v * K + u] : 0.0;
            const double grown = na + 2.0 * pu + gram[u * K + u];
            na = in(u) ? grown : na;
            norm_sq += in(u) ? gram[u * K + u] : 0.0;
            cnt += in(u) ? 1 : 0;
        }
        double p = 0.0;
#pragma unroll
        for (int v = 0; v < K - 1; ++v) p += (v < t && in(v)) ? gram[v * K + t] : 0.0;
        int status = 0;
        const double ng = gram[t * K + t];
        const double d = cosine_distance(p, na, ng, &status);
        const int accept = (d <= r.tau) ? 1 : 0;
        // the sum this case would leave behind, if it accepts
        status |= accept ? ill_conditioned(cnt + 1, norm_sq + ng, na + 2.0 * p + ng) : 0;
        tb.d[tid] = d; tb.p[tid] = p; tb.na[tid] = na;
        tb.accept[tid] = (unsigned char)accept;
        tb.status[tid] = (unsigned char)status;
    }
    __syncthreads();
    if (tid == 0) {
        unsigned int m = 0;
        int node[kReplayMaxK];
        for (int t = 1; t < K; ++t) {
            node[t] = (1 << (t - 1)) - 1 + (int)m;
            if (tb.accept[node[t]]) m |= 1u << (t - 1);
        }
        const unsigned long long bits = 1ull | ((unsigned long long)m << 1);
        early(bits);
        if (!publish) return;
        Control *c = r.ctl;
        int status = 0, count = 1;
        c->decision[0] = 1;
        r.mask_out[r.idx[0]] = 1;
        if (r.dist_out) r.dist_out[r.idx[0]] = 0.0f;
        for (int t = 1; t < K; ++t) {
            const int i = node[t], accept = tb.accept[i];
            c->decision[t] = accept;
            c->sums[t][0] = tb.p[i]; c->sums[t][1] = tb.na[i]; c->sums[t][2] = gram[t * K + t];
            r.mask_out[r.idx[t]] = (uint8_t)accept;
            if (r.dist_out) r.dist_out[r.idx[t]] = (float)tb.d[i];
            status |= tb.status[i];
            count += accept;
        }
        c->accept_bits = bits;
        c->ring_seed = -1;
        c->count = count;
        if (status) atomicOr(&c->status, status);
        *r.count_out = count;
        __threadfence();
    }
}

// Order-indifferent variant (end of Section 3.1): Algorithm 1 from every seed s with the
// others following in ring order s, s+1, ..., K-1, 0, ..., s-1; the seed with the largest
// accepted count wins, ties to the smallest s.  Threads 0..K-1 of the calling block each walk
// one seed on the Gram matrix (by ORIGINAL index); thread 0 then publishes the winner.
// `scratch` holds K ints + K unsigned long longs in shared memory.  All threads must call.
struct RingArgs {
    int K;
    double tau;
    uint8_t *mask_out;
    float *dist_out;                        // may be null
    int32_t *count_out;
    int32_t *seed_out;
    Control *ctl;
};

__device__ __forceinline__ void ring_walk_one_seed(const RingArgs &r, const volatile double *gram, int s,
                                                   int &count_out, unsigned long long &bits_out, int &status_out,
                                                   float *dist_by_index) {
    const int K = r.K;
    unsigned long long bits = 1ull << s;    // bit i set = gradient i (original index) accepted
    int count = 1, status = 0;
    double na = gram[(size_t)s * K + s], norm_sq = na;
    if (dist_by_index) dist_by_index[s] = 0.0f;
    for (int t = 1; t < K; ++t) {
        const int i = (s + t) % K;
        double p = 0.0;
        for (int u = 0; u < t; ++u) {       // accepted gradients in processing order
            const int j = (s + u) % K;
            if ((bits >> j) & 1ull) p += gram[(size_t)j * K + i];
        }
        const double ng = gram[(size_t)i * K + i];
        const double d = cosine_distance(p, na, ng, &status);
        if (dist_by_index) dist_by_index[i] = (float)d;
        if (d <= r.tau) {
            bits |= 1ull << i;
            na = na + 2.0 * p + ng;
            norm_sq += ng;
            ++count;
            status |= ill_conditioned(count, norm_sq, na);
        }
    }
    count_out = count; bits_out = bits; status_out = status;
}

// `early`, when given, is called by thread 0 with (winning seed, its accept bits) as soon as they are
// known, before the outputs are written.
struct NoEarlyNotice {
    __device__ __forceinline__ void operator()(int, unsigned long long) const {}
};
template <typename Early = NoEarlyNotice>
__device__ __forceinline__ void ring_replay_on_gram(const RingArgs &r, const volatile double *gram,
                                                    int *sh_count, unsigned long long *sh_bits,
                                                    Early early = Early()) {
    const int K = r.K;
    if ((int)threadIdx.x < K) {
        int c, st;
        unsigned long long b;
        ring_walk_one_seed(r, gram, threadIdx.x, c, b, st, nullptr);
        sh_count[threadIdx.x] = c;
        sh_bits[threadIdx.x] = b;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int best = 0;
        for (int s = 1; s < K; ++s)
            if (sh_count[s] > sh_count[best]) best = s;
        early(best, sh_bits[best]);
        // walk the winner once more to write its distances and status
        int c, st;
        unsigned long long b;
        ring_walk_one_seed(r, gram, best, c, b, st, r.dist_out);
        for (int i = 0; i < K; ++i) r.mask_out[i] = (uint8_t)((b >> i) & 1ull);
        Control *ctl = r.ctl;
        ctl->accept_bits = b;
        ctl->ring_seed = best;
        ctl->count = c;
        if (st) atomicOr(&ctl->status, st);
        *r.count_out = c;
        *r.seed_out = best;
        __threadfence();
    }
}

// The any-seed walks in table form (K <= 8), as replay_on_gram_parallel does for one order: one thread
// per (seed, step t, accept pattern of the seed's steps 1..t-1) evaluates Eq. 4 on the Gram matrix by
// ORIGINAL index (step v of seed s is gradient (s + v) mod K), one thread per seed then follows its
// decisions through the table, and thread 0 picks the largest count (ties to the smallest seed) and
// publishes.  Same sums in the same order as ring_walk_one_seed: identical outputs.
// All threads of the block call; `early(seed, bits)` as in ring_replay_on_gram; `publish` as in
// replay_on_gram_parallel.
template <int KT>
struct RingTable {
    static constexpr int kCases = (1 << (KT - 1)) - 1;          // per seed
    float d[KT * kCases + 1];
    unsigned char accept[KT * kCases + 1], status[KT * kCases + 1];
    int count[KT];
    unsigned int steps[KT];                                     // bit t-1 = step t of this seed accepted
};
template <int KT, typename Early = NoEarlyNotice>
__device__ __forceinline__ void ring_replay_parallel(const RingArgs &r, const double *gram, RingTable<KT> &tb,
                                                     Early early = Early(), bool publish = true) {
    constexpr int K = KT, C = RingTable<KT>::kCases;
    for (int idx = threadIdx.x; idx < K * C; idx += blockDim.x) {
        const int s = idx / C, cs = idx - s * C;
        const int t = 32 - __clz(cs + 1);
        const unsigned int m = (unsigned int)(cs + 1) - (1u << (t - 1));
        auto in = [&](int v) { return v == 0 || ((m >> (v - 1)) & 1u); };
        auto gi = [&](int v) { const int i = s + v; return i >= K ? i - K : i; };      // gradient of step v
        double na = gram[s * K + s], norm_sq = na;
        int cnt = 1;
#pragma unroll
        for (int u = 1; u < K - 1; ++u) {
            double pu = 0.0;
#pragma unroll
            for (int v = 0; v < u; ++v) pu += in(v) ? gram[gi(v) * K + gi(u)] : 0.0;
            const double guu = gram[gi(u) * K + gi(u)];
            const double grown = na + 2.0 * pu + guu;
            na = in(u) ? grown : na;
            norm_sq += in(u) ? guu : 0.0;
            cnt += in(u) ? 1 : 0;
        }
        double p = 0.0;
#pragma unroll
        for (int v = 0; v < K - 1; ++v) p += (v < t && in(v)) ? gram[gi(v) * K + gi(t)] : 0.0;
        int status = 0;
        const double ng = gram[gi(t) * K + gi(t)];
        const double d = cosine_distance(p, na, ng, &status);
        const int accept = (d <= r.tau) ? 1 : 0;
        status |= accept ? ill_conditioned(cnt + 1, norm_sq + ng, na + 2.0 * p + ng) : 0;
        tb.d[idx] = (float)d;
        tb.accept[idx] = (unsigned char)accept;
        tb.status[idx] = (unsigned char)status;
    }
    __syncthreads();
    if ((int)threadIdx.x < K) {
        const int s = threadIdx.x;
        unsigned int m = 0;
        int count = 1;
        for (int t = 1; t < K; ++t) {
            const int node = s * C + (1 << (t - 1)) - 1 + (int)m;
            if (tb.accept[node]) { m |= 1u << (t - 1); ++count; }
        }
        tb.count[s] = count;
        tb.steps[s] = m;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int best = 0;
        for (int s = 1; s < K; ++s)
            if (tb.count[s] > tb.count[best]) best = s;
        const unsigned int steps = tb.steps[best];
        unsigned long long bits = 1ull << best;                 // by original index
        for (int t = 1; t < K; ++t)
            if ((steps >> (t - 1)) & 1u) bits |= 1ull << ((best + t) % K);
        early(best, bits);
        if (!publish) return;
        int status = 0;
        unsigned int m = 0;
        if (r.dist_out) r.dist_out[best] = 0.0f;
        for (int t = 1; t < K; ++t) {
            const int node = best * C + (1 << (t - 1)) - 1 + (int)m;
            if (r.dist_out) r.dist_out[(best + t) % K] = tb.d[node];
            status |= tb.status[node];
            if (tb.accept[node]) m |= 1u << (t - 1);
        }
        for (int i = 0; i < K; ++i) r.mask_out[i] = (uint8_t)((bits >> i) & 1ull);
        Control *ctl = r.ctl;
        ctl->accept_bits = bits;
        ctl->ring_seed = best;
        ctl->count = tb.count[best];
        if (status) atomicOr(&ctl->status, status);
        *r.count_out = tb.count[best];
        *r.seed_out = best;
        __threadfence();
    }
}

// ------------------------------------------------ one-pass Gram for K <= 8 ----

struct GramSmallArgs {
    const void *g[kGsMaxK];                 // processing order
    int64_t D;
    int64_t keep_from;                      // elements from here on are loaded "keep in L2"
    double *partials;                       // [pair][kGsPartialStride]
    double *gram;                           // [K][K]
    ReplayArgs replay;                      // used when pair_dist_out is null and ring.K == 0
    float *pair_dist_out;                   // pairwise mode: K x K distances instead of the walk
    double *pair_gram_out;                  // pairwise mode: optional copy of the Gram matrix
    RingArgs ring;                          // any-seed mode when ring.K > 0 (rows are in original order)
    int mma_run;                            // gram_mma_kernel: trips per run of a CTA (even, >= 2)
};

// 16-byte read-only load with an explicit L2 eviction policy.
__device__ __forceinline__ uint4 ld16_policy(const void *p, uint64_t policy) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p), "l"(policy));
    return r;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}

template <typename T> struct GsVec;         // one 16-byte load per gradient and iteration
template <> struct GsVec<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ void load(const float *base, int64_t e, uint64_t policy, float (&v)[4]) {
        uint4 r = ld16_policy(base + e, policy);
        v[0] = __uint_as_float(r.x); v[1] = __uint_as_float(r.y);
        v[2] = __uint_as_float(r.z); v[3] = __uint_as_float(r.w);
    }
};
template <> struct GsVec<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ void load(const __nv_bfloat16 *base, int64_t e, uint64_t policy,
                                                float (&v)[8]) {
        uint4 r = ld16_policy(base + e, policy);
        unsigned int w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            v[2 * k] = bf16_bits_to_float(w[k] & 0xFFFFu);
            v[2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u);
        }
    }
};

// Fixed-order totals of the per-CTA partial sums ([pair][CTA] layout), by the whole calling block:
// one warp per pair (several pairs per warp when there are more pairs than warps, all loads issued
// before the first add: this is the serial tail of the call), lane-strided sums, then a shuffle tree.
// Fills the symmetric K x K matrix in shared memory and, when `gram_out` is given, in global memory.
template <int KT>
__device__ __forceinline__ void total_gram_partials(const double *part, int n_ctas, double *sgram, double *gram_out) {
    constexpr int NP = KT * (KT + 1) / 2;
    constexpr int kWarps = kGsThreads / 32;
    constexpr int PW = (NP + kWarps - 1) / kWarps;             // pairs per warp
    constexpr int kRounds = (kGsMaxCtas + 31) / 32;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    double v[PW][kRounds];
#pragma unroll
    for (int w = 0; w < PW; ++w) {
        const int p = warp + w * kWarps;
#pragma unroll
        for (int k = 0; k < kRounds; ++k) {
            const int i = lane + 32 * k;
            v[w][k] = (p < NP && i < n_ctas) ? __ldcg(part + (size_t)p * kGsPartialStride + i) : 0.0;
        }
    }
#pragma unroll
    for (int w = 0; w < PW; ++w) {
        const int p = warp + w * kWarps;
        double s = 0.0;
#pragma unroll
        for (int k = 0; k < kRounds; ++k) s += v[w][k];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) s += shfl_down_f64(s, d);
        if (lane == 0 && p < NP) {
            int r = 0, rem = p;                                 // decode p -> (r, c), r <= c
            while (rem >= KT - r) { rem -= KT - r; ++r; }
            const int c = r + rem;
            sgram[r * KT + c] = s;
            sgram[c * KT + r] = s;
            if (gram_out) {
                gram_out[r * KT + c] = s;
                gram_out[c * KT + r] = s;
            }
        }
    }
}

// Accumulator of the register-tiled Gram kernels (K <= 8).
// binary32 inputs, up to 4 gradients: binary64.  A product of two binary32 values is exact in binary64, so
// the Gram sums are exact up to binary64 rounding and need no periodic flush; binary64 FMAs (half the
// binary32 rate on this GPU) keep up with HBM here (measured: the same pass time, and a shorter call because
// the flushes are gone).  With 5 to 8 gradients there are up to 1.4 binary64 operations per byte read and
// the long passes, which run under the power cap, lost 8 %: binary32 chains there.
// bfloat16 inputs: binary32 chains (a product of two bfloat16 values is exact in binary32; there are twice
// as many products per byte), widened to binary64 every kGsFlushEvery rounds like the binary32 chains above.
template <typename T, int KT> struct GsAcc {
    using type = float;
    static constexpr bool kPeriodicFlush = true;
};
template <> struct GsAcc<float, 1> { using type = double; static constexpr bool kPeriodicFlush = false; };
template <> struct GsAcc<float, 2> { using type = double; static constexpr bool kPeriodicFlush = false; };
template <> struct GsAcc<float, 3> { using type = double; static constexpr bool kPeriodicFlush = false; };
template <> struct GsAcc<float, 4> { using type = double; static constexpr bool kPeriodicFlush = false; };
__device__ __forceinline__ float gs_fma(float a, float b, float s) { return fmaf(a, b, s); }
__device__ __forceinline__ double gs_fma(float a, float b, double s) { return fma((double)a, (double)b, s); }

// What every one-pass Gram kernel for K <= 8 does once its warps have left their sums in
// sacc[warp][pair] (upper triangle, row-major pair index): per-CTA partial sums in a fixed order,
// last-CTA election, fixed-order totals, then the walk of Algorithm 1 (or the any-seed walks, or the
// pairwise distances).  All threads of the block call.
template <int KT>
__device__ __forceinline__ void gram_small_tail(const GramSmallArgs &a, double (*sacc)[KT * (KT + 1) / 2]) {
    constexpr int NP = KT * (KT + 1) / 2;
    __shared__ bool is_last;
    // the streaming part of this CTA is over: a kernel launched as a programmatic dependent
    // (the masked-mean pass) may start occupying SMs; it still waits for this whole grid
    // before it reads anything
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    __syncthreads();
    if (threadIdx.x < NP) {
        // the 16 warps' sums in four short chains (a fixed order, so still reproducible)
        double s4[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            s4[c] = sacc[4 * c][threadIdx.x];
#pragma unroll
            for (int w = 1; w < 4; ++w) s4[c] += sacc[4 * c + w][threadIdx.x];
        }
        a.partials[(size_t)threadIdx.x * kGsPartialStride + blockIdx.x] = (s4[0] + s4[1]) + (s4[2] + s4[3]);
    }
    __syncthreads();
    if (threadIdx.x == 0) is_last = take_last_ticket(&a.replay.ctl->ticket, gridDim.x);
    __syncthreads();
    if (!is_last) return;

    // last CTA: fixed-order totals (one warp per pair; all of a lane's loads are issued together,
    // this is the serial tail of the call), then the scalar walk out of shared memory
    __shared__ double sgram[KT * KT];
    total_gram_partials<KT>(a.partials, gridDim.x, sgram, a.gram);
    __syncthreads();
    if (a.ring.K > 0) {
        __shared__ RingTable<KT> ring_table;
        ring_replay_parallel<KT>(a.ring, sgram, ring_table);
        return;
    }
    if (a.pair_dist_out == nullptr) {
        __shared__ ReplayTable table;
        replay_on_gram_parallel<KT>(a.replay, sgram, table);
        return;
    }
    // pairwise mode: Eq. 4 for every pair
    if (threadIdx.x < KT * KT) {
        const int i = threadIdx.x / KT, j = threadIdx.x % KT;
        const double gii = sgram[i * KT + i], gjj = sgram[j * KT + j], gij = sgram[threadIdx.x];
        int status = 0;
        const double d = (i == j && gii > 0.0) ? 0.0 : cosine_distance(gij, gii, gjj, &status);
        a.pair_dist_out[threadIdx.x] = (float)d;
        if (a.pair_gram_out) a.pair_gram_out[threadIdx.x] = gij;
        if (status) atomicOr(&a.replay.ctl->status, status);
    }
}

template <typename T, int KT>
__global__ void __launch_bounds__(kGsThreads, (KT <= 4 ? 2 : 1)) gram_small_kernel(const __grid_constant__ GramSmallArgs a) {
    constexpr int NP = KT * (KT + 1) / 2;   // upper triangle
    constexpr int N = GsVec<T>::N;
    __shared__ double sacc[kGsThreads / 32][NP];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (blockIdx.x == 0 && threadIdx.x == 0) a.replay.ctl->status = 0;      // first kernel of the operation
    for (int p = lane; p < NP; p += 32) sacc[warp][p] = 0.0;
    __syncwarp();

    const T *row[KT];
#pragma unroll
    for (int r = 0; r < KT; ++r) row[r] = static_cast<const T *>(a.g[r]);

    using Acc = typename GsAcc<T, KT>::type;
    Acc acc[NP];
#pragma unroll
    for (int p = 0; p < NP; ++p) acc[p] = Acc(0);

    auto flush = [&]() {
#pragma unroll
        for (int p = 0; p < NP; ++p) {
            Acc v = acc[p];
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) v += __shfl_down_sync(0xFFFFFFFFu, v, d);
            if (lane == 0) sacc[warp][p] += (double)v;
            acc[p] = Acc(0);
        }
    };

    // The masked-mean pass that follows walks the vectors from their end: the tail of
    // this pass is loaded "evict last" so that it is still in L2 then; the head, which
    // cannot survive anyway, is loaded "evict first".
    const uint64_t pol_first = l2_policy_evict_first(), pol_last = l2_policy_evict_last();
    const int64_t n_vec = a.D / N;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    int since_flush = 0;
    // The trip count is the same for all lanes of a warp (the bound is tested on the warp's first
    // vector): the flush below shuffles across the whole warp, so the lanes must reach it together.
    const int64_t warp_first = (int64_t)blockIdx.x * blockDim.x + (threadIdx.x & ~31);
    for (int64_t qw = warp_first; qw < n_vec; qw += stride) {
        const int64_t q = qw + lane;
        if (q < n_vec) {
            float x[KT][N];
            const uint64_t pol = (q * N >= a.keep_from) ? pol_last : pol_first;
#pragma unroll
            for (int r = 0; r < KT; ++r) GsVec<T>::load(row[r], q * N, pol, x[r]);
            int p = 0;
#pragma unroll
            for (int r = 0; r < KT; ++r)
#pragma unroll
                for (int c = r; c < KT; ++c, ++p) {
                    Acc s = acc[p];
#pragma unroll
                    for (int k = 0; k < N; ++k) s = gs_fma(x[r][k], x[c][k], s);
                    acc[p] = s;
                }
        }
        if (GsAcc<T, KT>::kPeriodicFlush && ++since_flush == kGsFlushEvery) { flush(); since_flush = 0; }
    }
    // ragged tail (D mod N elements), first CTA
    const int64_t tail0 = n_vec * N;
    if (blockIdx.x == 0 && tail0 + threadIdx.x < a.D) {
        const int64_t e = tail0 + threadIdx.x;
        float x[KT];
#pragma unroll
        for (int r = 0; r < KT; ++r) x[r] = load1<T>(row[r], e);
        int p = 0;
#pragma unroll
        for (int r = 0; r < KT; ++r)
#pragma unroll
            for (int c = r; c < KT; ++c, ++p) acc[p] = gs_fma(x[r], x[c], acc[p]);
    }
    flush();
    gram_small_tail<KT>(a, sacc);
}

// Scalar walk as its own launch (Gram matrix produced by the tiled pairwise kernels).
// `perm` maps processing step -> row of `gram_by_index` (K x K by original index).
__global__ void gram_replay_kernel(ReplayArgs r, const double *gram_by_index, double *gram_by_step) {
    const int K = r.K;
    for (int i = threadIdx.x; i < K * K; i += blockDim.x) {
        const int t = i / K, u = i % K;
        gram_by_step[i] = gram_by_index[(size_t)r.idx[t] * K + r.idx[u]];
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) { replay_on_gram(r, gram_by_step, true); __threadfence(); }
}

// Any-seed walk as its own launch (Gram matrix by original index from the tiled or
// tensor-core kernels).  One block of at least K threads.
__global__ void gram_ring_replay_kernel(RingArgs r, const double *gram_by_index) {
    __shared__ int ring_count[GAF_MAX_K];
    __shared__ unsigned long long ring_bits[GAF_MAX_K];
    ring_replay_on_gram(r, gram_by_index, ring_count, ring_bits);
}

// ------------------------------------------------------- masked mean (Eq. 5) --

// Eight consecutive elements as loaded (streaming, evict-first), widened on use.
template <typename T> struct RawOct;
template <> struct RawOct<float> {
    float4 a, b;
    static __device__ __forceinline__ RawOct load(const float *base, int64_t e) {
        const float4 *p = reinterpret_cast<const float4 *>(base + e);
        return {__ldcs(p), __ldcs(p + 1)};
    }
    __device__ __forceinline__ void widen(float (&v)[8]) const {
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    }
};
template <> struct RawOct<__nv_bfloat16> {
    uint4 r;
    static __device__ __forceinline__ RawOct load(const __nv_bfloat16 *base, int64_t e) {
        return {__ldcs(reinterpret_cast<const uint4 *>(base + e))};
    }
    __device__ __forceinline__ void widen(float (&v)[8]) const {
        const unsigned int w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            v[2 * k] = bf16_bits_to_float(w[k] & 0xFFFFu);
            v[2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u);
        }
    }
};

struct MaskedMeanArgs {
    const void *g[GAF_MAX_K];               // processing order; original order in any-seed mode, where
                                            // the order starts at the winning seed and wraps around
    int K;
    int64_t D;
    float *out;
    const Control *ctl;
    int run;                                // chunks (of one CTA's 512 groups of 8 elements) a CTA takes in a row
};

// out = (((g_0 + g_a) + g_b) + ...) / c over the accepted steps a < b < ..., binary32,
// in processing order: the same association as the streaming schedule.  The vector is
// walked from its END: the Gram pass that ran just before walked it from the start, so
// its last-read lines are the ones still in L2.  A CTA takes `run` consecutive chunks, then
// jumps ahead by the whole grid's share: with run = U the grid works on one compact window of
// every vector at any moment (short vectors: every CTA has work); on long vectors longer runs
// keep an SM inside the same pages for several trips, which the address translation needs
// (12 GB through this pass: 5.5 TB/s with run = U, measured, against the 6.5 TB/s it reaches
// on shorter vectors).
template <typename T>
__global__ void __launch_bounds__(kMsThreads, 2) masked_mean_kernel(const __grid_constant__ MaskedMeanArgs a) {
    __shared__ const T *list[GAF_MAX_K];
    __shared__ int n_list;
    __shared__ float cdiv_s;
    // when launched as a programmatic dependent of the Gram pass: wait until that grid has
    // completed and its writes (the accept bits) are visible; otherwise a no-op
    asm volatile("griddepcontrol.wait;" ::: "memory");
    unsigned long long bits = 0;
    int seed = -1;
    if (threadIdx.x == 0) {
        bits = __ldcg(&a.ctl->accept_bits);                      // (two independent L2 loads)
        seed = __ldcg(&a.ctl->ring_seed);
    }
    if (threadIdx.x == 0) {
        const int start = seed < 0 ? 0 : seed;
        int n = 0;
        for (int t = 0; t < a.K; ++t) {
            const int i = (start + t) % a.K;
            if ((bits >> i) & 1ull) list[n++] = static_cast<const T *>(a.g[i]);
        }
        n_list = n;
        cdiv_s = (float)n;
    }
    __syncthreads();
    const int n = n_list;
    const float cdiv = cdiv_s;
    const int64_t n_oct = a.D / kOct;
    // U groups of 8 elements per thread and round (two for 2-byte inputs, so that as many bytes
    // are in flight as with 4-byte inputs); loads stay packed until they are added
    constexpr int U = sizeof(T) == 2 ? 2 : 1;
    constexpr int kChunk = 3;                       // further gradients fetched together
    const int64_t n_chunks = (n_oct + kMsThreads - 1) / kMsThreads;
    const int64_t run = a.run;
    for (int64_t base = (int64_t)blockIdx.x * run; base < n_chunks; base += (int64_t)gridDim.x * run)
    for (int64_t rr = 0; rr < run && base + rr < n_chunks; rr += U) {
        int64_t e[U];
        bool ok[U];
        RawOct<T> first[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t o = (base + rr + u) * kMsThreads + threadIdx.x;
            ok[u] = rr + u < run && o < n_oct;
            e[u] = (n_oct - 1 - (ok[u] ? o : 0)) * kOct;
            if (ok[u]) first[u] = RawOct<T>::load(list[0], e[u]);
        }
        float v[U][8];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (ok[u]) first[u].widen(v[u]);
        for (int i = 1; i < n; i += kChunk) {
            RawOct<T> w[U][kChunk];
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int j = 0; j < kChunk; ++j)
                    if (ok[u] && i + j < n) w[u][j] = RawOct<T>::load(list[i + j], e[u]);
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int j = 0; j < kChunk; ++j)
                    if (ok[u] && i + j < n) {
                        float x[8];
                        w[u][j].widen(x);
#pragma unroll
                        for (int k = 0; k < 8; ++k) v[u][k] += x[k];
                    }
        }
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (ok[u]) {
#pragma unroll
                for (int k = 0; k < 8; ++k) v[u][k] = v[u][k] / cdiv;
                store8(a.out, e[u], v[u], true);
            }
    }
    const int64_t tail0 = n_oct * kOct;
    if (blockIdx.x == 0 && tail0 + threadIdx.x < a.D) {
        const int64_t e = tail0 + threadIdx.x;
        float v = load1<T>(list[0], e);
        for (int i = 1; i < n; ++i) v += load1<T>(list[i], e);
        a.out[e] = v / cdiv;
    }
}

}  // namespace gaf
