// Bucketed variant: the parameter vector is cut into S consecutive buckets (for example the
// tensors of a network, or the buckets of a ring all-reduce) and Algorithm 1 + Eq. 5 run on every
// bucket independently.  Gram-first, as for the whole vector: one pass builds a K x K Gram matrix
// PER BUCKET, a small kernel walks Algorithm 1 per bucket, one pass writes every bucket's g/c.
//
// Work split: every CTA owns one contiguous range of the D elements (equal shares), and inside
// it handles the part of every bucket that intersects the range.  A (CTA c, bucket b) intersection
// writes its partial Gram sums to slot c + b, which is unique because both indices only grow along
// the vector.  The per-bucket totals are taken over the CTAs in ascending order (fixed order).
#pragma once

#include "gaf_device.cuh"
#include "gaf_gramfilter.cuh"

namespace gaf {

constexpr int kBkThreads = 512;
constexpr int kBkMaxBuckets = GAF_MAX_BUCKETS;
constexpr int kBkMaxCtas = 296;

struct BucketTable {
    int S;
    int64_t off[kBkMaxBuckets + 1];         // element offsets, off[0] = 0, off[S] = D
};

// Largest b with off[b] <= e (e < D).
__device__ __forceinline__ int bucket_of(const BucketTable &bt, int64_t e) {
    int lo = 0, hi = bt.S;                  // off[lo] <= e < off[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (bt.off[mid] <= e) lo = mid; else hi = mid;
    }
    return lo;
}

// Element range of CTA c out of G: equal shares in units of 8 elements; the last CTA also takes
// the D mod 8 leftover.
__device__ __forceinline__ void cta_range(int64_t D, int c, int G, int64_t &lo, int64_t &hi) {
    const int64_t n_oct = D / kOct;
    lo = (n_oct * c / G) * kOct;
    hi = (c == G - 1) ? D : (n_oct * (c + 1) / G) * kOct;
}

struct BucketGramArgs {
    const void *g[kGsMaxK];                 // processing order
    int64_t D;
    int64_t keep_elems;                     // the last so many elements of every CTA's range are loaded "keep in L2"
    double *partials;                       // [slot][64], slot = cta + bucket
    Control *ctl;
};

template <typename T, int KT>
__global__ void __launch_bounds__(kBkThreads, (KT <= 4 ? 2 : 1))
bucket_gram_kernel(const __grid_constant__ BucketGramArgs a, const __grid_constant__ BucketTable bt) {
    constexpr int NP = KT * (KT + 1) / 2;
    constexpr int N = GsVec<T>::N;
    __shared__ double sacc[kBkThreads / 32][NP];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const T *row[KT];
#pragma unroll
    for (int r = 0; r < KT; ++r) row[r] = static_cast<const T *>(a.g[r]);
    // the mean pass walks every CTA's range from its end: the end of the range is asked to stay in L2
    const uint64_t pol_first = l2_policy_evict_first(), pol_last = l2_policy_evict_last();
    if (blockIdx.x == 0 && threadIdx.x == 0) a.ctl->status = 0;     // first kernel of the operation

    int64_t lo, hi;
    cta_range(a.D, blockIdx.x, gridDim.x, lo, hi);
    if (lo >= hi) return;
    int b = bucket_of(bt, lo);
    while (true) {
        const int64_t s0 = lo > bt.off[b] ? lo : bt.off[b];
        const int64_t s1 = hi < bt.off[b + 1] ? hi : bt.off[b + 1];
        if (s1 > s0) {
            for (int p = lane; p < NP; p += 32) sacc[warp][p] = 0.0;
            __syncwarp();
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
            // s0 is a multiple of 8 elements (bucket offsets and CTA ranges are), so vector loads are aligned
            const int64_t n_vec = (s1 - s0) / N;
            int since_flush = 0;
            // warp-uniform trip count: the flush shuffles across the whole warp
            for (int64_t qw = threadIdx.x & ~31; qw < n_vec; qw += kBkThreads) {
                const int64_t q = qw + lane;
                if (q < n_vec) {
                    float x[KT][N];
                    const uint64_t pol = (s0 + q * N >= hi - a.keep_elems) ? pol_last : pol_first;
#pragma unroll
                    for (int r = 0; r < KT; ++r) GsVec<T>::load(row[r], s0 + q * N, pol, x[r]);
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
            const int64_t t0 = s0 + n_vec * N;          // fewer than N leftover elements
            if (t0 + threadIdx.x < s1) {
                float x[KT];
#pragma unroll
                for (int r = 0; r < KT; ++r) x[r] = load1<T>(row[r], t0 + threadIdx.x);
                int p = 0;
#pragma unroll
                for (int r = 0; r < KT; ++r)
#pragma unroll
                    for (int c = r; c < KT; ++c, ++p) acc[p] = gs_fma(x[r], x[c], acc[p]);
            }
            flush();
            __syncthreads();
            if (threadIdx.x < NP) {
                double s = 0.0;
                for (int w = 0; w < kBkThreads / 32; ++w) s += sacc[w][threadIdx.x];
                a.partials[(size_t)(blockIdx.x + b) * 64 + threadIdx.x] = s;
            }
            __syncthreads();
        }
        if (bt.off[b + 1] >= hi || b + 1 >= bt.S) break;
        ++b;
    }
    // the per-bucket walk is launched as a programmatic dependent: its blocks may be placed now
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

struct BucketWalkArgs {
    int K;
    int64_t D;
    int ctas;                               // grid of the Gram pass
    double tau;
    const double *partials;
    uint8_t *mask_out;                      // [S][K], by original index
    float *dist_out;                        // [S][K] or null
    int32_t *count_out;                     // [S]
    unsigned long long *bits;               // [S], bit t = step t accepted (workspace)
    int idx[kGsMaxK];                       // original index of step t
    Control *ctl;
};

// One CTA per bucket (64 pairs x 16 chains of threads): totals over the intersecting CTAs in
// ascending order, then the walk.
constexpr int kWalkChains = 16;
__global__ void __launch_bounds__(64 * kWalkChains)
bucket_walk_kernel(const __grid_constant__ BucketWalkArgs a, const __grid_constant__ BucketTable bt) {
    __shared__ double sgram[kGsMaxK * kGsMaxK];
    __shared__ double part[kWalkChains][64];
    const int b = blockIdx.x, K = a.K, NP = K * (K + 1) / 2;
    const int64_t b0 = bt.off[b], b1 = bt.off[b + 1];
    // CTAs of the Gram pass whose range meets [b0, b1)
    int c_first = 0, c_last = -1;
    if (b1 > b0) {
        int lo = 0, hi = a.ctas - 1;            // first CTA with range end > b0
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            int64_t l, h;
            cta_range(a.D, mid, a.ctas, l, h);
            if (h > b0) hi = mid; else lo = mid + 1;
        }
        c_first = lo;
        lo = c_first; hi = a.ctas - 1;          // last CTA with range start < b1
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            int64_t l, h;
            cta_range(a.D, mid, a.ctas, l, h);
            if (l < b1) lo = mid; else hi = mid - 1;
        }
        c_last = lo;
    }
    const int p = threadIdx.x & 63, chain = threadIdx.x >> 6;
    // programmatic dependent of the Gram pass: wait for that grid and its partial sums; the mean pass
    // behind this kernel may be placed at once (it waits for this grid in turn)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    {
        const int n = c_last - c_first + 1;
        const int per = (n + kWalkChains - 1) / kWalkChains;
        const int c0 = c_first + chain * per, c1 = min(c_last + 1, c0 + per);
        double s = 0.0;
        if (p < NP) {
            for (int c = c0; c < c1; ++c) {
                int64_t l, h;
                cta_range(a.D, c, a.ctas, l, h);
                const int64_t s0 = l > b0 ? l : b0, s1 = h < b1 ? h : b1;
                if (s1 > s0) s += __ldcg(a.partials + (size_t)(c + b) * 64 + p);
            }
        }
        part[chain][p] = s;
    }
    __syncthreads();
    if ((int)threadIdx.x < NP) {
        double s = 0.0;
#pragma unroll
        for (int c = 0; c < kWalkChains; ++c) s += part[c][threadIdx.x];
        int r = 0, rem = threadIdx.x;
        while (rem >= K - r) { rem -= K - r; ++r; }
        const int cc = r + rem;
        sgram[r * K + cc] = s;
        sgram[cc * K + r] = s;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int status = 0, count = 1;
        unsigned long long bits = 1ull;
        double na = sgram[0], norm_sq = sgram[0];
        uint8_t *mask = a.mask_out + (size_t)b * K;
        float *dist = a.dist_out ? a.dist_out + (size_t)b * K : nullptr;
        mask[a.idx[0]] = 1;
        if (dist) dist[a.idx[0]] = 0.0f;
        for (int t = 1; t < K; ++t) {
            double p = 0.0;
            for (int u = 0; u < t; ++u)
                if ((bits >> u) & 1ull) p += sgram[u * K + t];
            const double ng = sgram[t * K + t];
            const double d = cosine_distance(p, na, ng, &status);
            const int accept = (d <= a.tau) ? 1 : 0;
            mask[a.idx[t]] = (uint8_t)accept;
            if (dist) dist[a.idx[t]] = (float)d;
            if (accept) {
                bits |= 1ull << t; na = na + 2.0 * p + ng; norm_sq += ng; ++count;
                status |= ill_conditioned(count, norm_sq, na);
            }
        }
        a.bits[b] = bits;
        a.count_out[b] = count;
        if (status) atomicOr(&a.ctl->status, status);
    }
}

struct BucketMeanArgs {
    const void *g[kGsMaxK];                 // processing order
    int K;
    int64_t D;
    float *out;
    const unsigned long long *bits;         // [S]
};

template <typename T>
__global__ void __launch_bounds__(kBkThreads, 2)
bucket_mean_kernel(const __grid_constant__ BucketMeanArgs a, const __grid_constant__ BucketTable bt) {
    __shared__ const T *list[kGsMaxK];
    __shared__ int n_list;
    int64_t lo, hi;
    cta_range(a.D, blockIdx.x, gridDim.x, lo, hi);
    // programmatic dependent of the per-bucket walk: wait for its accept bits
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (lo >= hi) return;
    // the range is walked from its END (buckets last to first, each from its end): the Gram pass
    // walked it from the start, so its last-read lines are the ones still in L2
    int b = bucket_of(bt, hi - 1);
    while (true) {
        const int64_t s0 = lo > bt.off[b] ? lo : bt.off[b];
        const int64_t s1 = hi < bt.off[b + 1] ? hi : bt.off[b + 1];
        if (s1 > s0) {
            __syncthreads();
            if (threadIdx.x == 0) {
                const unsigned long long bits = __ldcg(a.bits + b);
                int n = 0;
                for (int t = 0; t < a.K; ++t)
                    if ((bits >> t) & 1ull) list[n++] = static_cast<const T *>(a.g[t]);
                n_list = n;
            }
            __syncthreads();
            const int n = n_list;
            const float cdiv = (float)n;
            const int64_t n_oct = (s1 - s0) / kOct;
            for (int64_t o = threadIdx.x; o < n_oct; o += kBkThreads) {
                const int64_t e = s0 + (n_oct - 1 - o) * kOct;
                float v[8];
                RawOct<T>::load(list[0], e).widen(v);
                for (int i = 1; i < n; i += 3) {
                    RawOct<T> w[3];
#pragma unroll
                    for (int j = 0; j < 3; ++j)
                        if (i + j < n) w[j] = RawOct<T>::load(list[i + j], e);
#pragma unroll
                    for (int j = 0; j < 3; ++j)
                        if (i + j < n) {
                            float x[8];
                            w[j].widen(x);
#pragma unroll
                            for (int k = 0; k < 8; ++k) v[k] += x[k];
                        }
                }
#pragma unroll
                for (int k = 0; k < 8; ++k) v[k] = v[k] / cdiv;
                store8(a.out, e, v, true);
            }
            const int64_t t0 = s0 + n_oct * kOct;
            if (t0 + threadIdx.x < s1) {
                const int64_t e = t0 + threadIdx.x;
                float v = load1<T>(list[0], e);
                for (int i = 1; i < n; ++i) v += load1<T>(list[i], e);
                a.out[e] = v / cdiv;
            }
        }
        if (bt.off[b] <= lo || b == 0) break;
        --b;
    }
}

}  // namespace gaf
