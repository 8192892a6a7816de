// Gram-first schedule of Algorithm 1 as ONE launch (K <= 8).
//
// The two-launch form (gaf_gramfilter.cuh) reads every gradient once for the Gram
// matrix and the accepted ones a second time for g/c (Eq. 5).  When the whole call
// lasts tens of microseconds, what the second pass has to fetch again is a large part
// of the cost.  Here one grid whose CTAs are all resident at once does both passes, so
// that part of what the first pass read is still ON CHIP when the second pass starts:
//   pass 1   every thread walks its vectors (grid-stride), accumulating the Gram
//            partial sums exactly as gram_small_kernel does, and parks the raw loads
//            of its FIRST R rounds in shared memory (the last rounds are the ones L2
//            still holds afterwards: shared memory and L2 then keep different data);
//   decide   every CTA stores its partial sums and adds itself to an arrival counter;
//            when the counter is full every CTA totals the partials in the same fixed
//            order and walks Algorithm 1 (Eq. 4 in binary64) on the Gram matrix ITSELF --
//            all CTAs get the same bits, nobody waits for a published result (one trip
//            through L2 less than electing a CTA to decide); CTA 0 writes the outputs;
//   pass 2   the same thread visits the same vectors: the rounds that were not parked
//            from the last one down (the end of the vectors was loaded "keep in L2"),
//            then the parked rounds straight from shared memory, adding the accepted
//            gradients in processing order in binary32 and dividing by c.
// Same sums, same order of additions as the two-launch form: identical outputs.
//
// The grid is sized by the host to what the device holds at once.  The kernel is launched with
// programmatic stream serialisation: it waits for whatever precedes it on the stream before it
// touches memory, and lets the launch behind it be placed as soon as its own decisions are taken
// (that launch waits in turn), which hides most of the launch latency of back-to-back calls.
// The one wait on other CTAs is bounded and ends in GAF_STATUS_TIMEOUT.
#pragma once

#include <type_traits>

#include "gaf_device.cuh"
#include "gaf_gramfilter.cuh"

namespace gaf {

constexpr unsigned int kFusedSpinLimit = 1u << 23;   // polls of an L2 round trip plus a 20 ns sleep each: seconds
constexpr unsigned int kFusedCallUnit = 4096;        // what one call adds to the arrival counter in all
constexpr int kFusedCallShift = 12;

struct GramFusedArgs {
    const void *g[kGsMaxK];                 // processing order (original order in any-seed mode)
    int64_t D;
    int64_t keep_from;                      // elements from here on are loaded "keep in L2"
    int park_rounds;                        // R: rounds per thread parked in shared memory
    double *partials;                       // [pair][kGsPartialStride]
    double *gram;                           // [K][K]
    float *out;                             // D floats
    ReplayArgs replay;                      // used when ring.K == 0
    RingArgs ring;                          // any-seed mode when ring.K > 0
    unsigned int spin_limit;                // polls a waiting CTA makes before it gives up
    int test_withhold;                      // test hook, normally 0: the waiting CTAs are never shown the full
                                            // counter, so that every wait runs out
};

__device__ __forceinline__ unsigned int ld_relaxed_u32(const unsigned int *p) {
    unsigned int v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int *p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Adds to a counter, ordered after everything this CTA wrote before (its threads' stores reach this
// thread through the barrier in front of the call).
__device__ __forceinline__ void red_release_add_u32(unsigned int *p, unsigned int v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

template <typename T> struct FusedVec;      // one 16-byte vector of a gradient, widened
template <> struct FusedVec<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ void widen(const uint4 &r, float (&v)[4]) {
        v[0] = __uint_as_float(r.x); v[1] = __uint_as_float(r.y);
        v[2] = __uint_as_float(r.z); v[3] = __uint_as_float(r.w);
    }
};
template <> struct FusedVec<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ void widen(const uint4 &r, float (&v)[8]) {
        const unsigned int w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            v[2 * k] = bf16_bits_to_float(w[k] & 0xFFFFu);
            v[2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u);
        }
    }
};

template <int N>
__device__ __forceinline__ void store_vec_streaming(float *dst, const float (&v)[N]) {
#pragma unroll
    for (int h = 0; h < N / 4; ++h)
        __stcs(reinterpret_cast<float4 *>(dst) + h, make_float4(v[4 * h], v[4 * h + 1], v[4 * h + 2], v[4 * h + 3]));
}

// Rounds of the second pass a thread keeps in flight, by the number of gradients it has to fetch per
// round (8 loads of 16 bytes per thread at most, 2 rounds at least up to 4 gradients).
template <int NN> struct FusedInFlight { static constexpr int U = NN <= 1 ? 8 : (NN == 2 ? 4 : (NN <= 4 ? 2 : 1)); };

template <typename T, int KT>
__global__ void __launch_bounds__(kGsThreads, (KT <= 4 ? 2 : 1))
gram_fused_kernel(const __grid_constant__ GramFusedArgs a) {
    constexpr int NP = KT * (KT + 1) / 2;
    constexpr int N = FusedVec<T>::N;
    // With two gradients (the paper's own experiments: Section 4) the output can only be the mean of both or the
    // seed alone, so the first pass writes one of the two while it forms the sums -- the one the latest two calls on
    // this workspace both ended with (decisions of consecutive training steps go together; no guess while they
    // differ) -- and the second pass runs only when this call decides otherwise: 12 bytes per fp32 element instead
    // of 20 (16 for the seed alone) when the guess holds, 24 when it does not, the usual 20 / 16 without a guess.
    // The guess changes which stores happen, never their values.
    constexpr bool kSpeculative = KT == 2;
    extern __shared__ uint4 parked[];       // [round][gradient][thread]
    __shared__ double sacc[kGsThreads / 32][NP];
    __shared__ double sgram[KT * KT];
    __shared__ const T *list[kGsMaxK];      // accepted gradients in the order they are added
    __shared__ int list_row[kGsMaxK];       // ... and their row in `parked`
    __shared__ int n_list;                  // c, or -1 when the wait ran out
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    Control *ctl = a.replay.ctl;

    // Launched with programmatic stream serialisation, this grid may be placed while the launch before
    // it on the stream is still winding down: nothing that launch (or the producer of the gradients)
    // wrote may be touched before it has completed.  A no-op after an ordinary predecessor.
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // call generation before this CTA has arrived: it cannot change until every CTA has, this one included
    unsigned int gen0 = 0;
    if (tid == 0) {
        gen0 = ld_relaxed_u32(&ctl->fused_arrivals) >> kFusedCallShift;
        if (blockIdx.x == 0) ctl->status = 0;
    }
    for (int p = lane; p < NP; p += 32) sacc[warp][p] = 0.0;
    __syncwarp();
    // (read before this CTA arrives, hence before any CTA can have decided and written the next guess)
    // 0 / 1: the latest two such calls both kept both gradients / the seed alone: write that now;
    // 2 / 3: they differed (the latest kept both / the seed alone): no guess, two passes as with more gradients
    const unsigned int hint = kSpeculative ? ld_relaxed_u32(&ctl->pair_hint) : 2u;
    const bool guessing = hint < 2u, guess_seed_alone = (hint & 1u) != 0;

    const T *row[KT];
#pragma unroll
    for (int r = 0; r < KT; ++r) row[r] = static_cast<const T *>(a.g[r]);

    const uint64_t pol_first = l2_policy_evict_first(), pol_last = l2_policy_evict_last();
    const int64_t n_vec = a.D / N;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    // rounds of this warp (the same for all its lanes: the flush shuffles across the warp)
    const int64_t warp_first = (int64_t)blockIdx.x * blockDim.x + (tid & ~31);
    const int64_t rounds = warp_first < n_vec ? (n_vec - warp_first + stride - 1) / stride : 0;
    const int64_t parked_rounds = rounds < a.park_rounds ? rounds : a.park_rounds;   // the FIRST ones
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

    const int64_t tail0 = n_vec * N;
    // ---- pass 1: Gram partial sums; the first rounds stay in shared memory ----
    // (with two gradients a thread would have only two 16-byte loads in flight: it fetches two rounds at a time;
    // the rounds are still consumed in order, so the sums are the same)
    constexpr int U1 = KT <= 2 ? 2 : 1;
    int since_flush = 0;
    for (int64_t j0 = 0; j0 < rounds; j0 += U1) {
        int64_t q[U1];
        bool ok[U1];
        uint4 raw[U1][KT];
#pragma unroll
        for (int u = 0; u < U1; ++u) {
            q[u] = warp_first + (j0 + u) * stride + lane;
            ok[u] = j0 + u < rounds && q[u] < n_vec;
            if (ok[u]) {
                const uint64_t pol = (q[u] * N >= a.keep_from) ? pol_last : pol_first;
#pragma unroll
                for (int r = 0; r < KT; ++r) raw[u][r] = ld16_policy(row[r] + q[u] * N, pol);
            }
        }
#pragma unroll
        for (int u = 0; u < U1; ++u) {
            const int64_t j = j0 + u;
            if (j >= rounds) break;
            if (ok[u]) {
                if (j < parked_rounds) {
                    uint4 *slot = parked + (size_t)j * KT * kGsThreads + tid;
#pragma unroll
                    for (int r = 0; r < KT; ++r) slot[r * kGsThreads] = raw[u][r];
                }
                float x[KT][N];
#pragma unroll
                for (int r = 0; r < KT; ++r) FusedVec<T>::widen(raw[u][r], x[r]);
                if (kSpeculative && guessing) {
                    // two gradients: the guessed result is written now
                    float v[N];
#pragma unroll
                    for (int k = 0; k < N; ++k) v[k] = guess_seed_alone ? x[0][k] : (x[0][k] + x[1][k]) / 2.0f;
                    store_vec_streaming<N>(a.out + q[u] * N, v);
                }
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
    }
    // ragged tail (D mod N elements), first CTA
    if (blockIdx.x == 0 && tail0 + tid < a.D) {
        const int64_t e = tail0 + tid;
        float x[KT];
#pragma unroll
        for (int r = 0; r < KT; ++r) x[r] = load1<T>(row[r], e);
        if (kSpeculative && guessing) a.out[e] = guess_seed_alone ? x[0] : (x[0] + x[1]) / 2.0f;
        int p = 0;
#pragma unroll
        for (int r = 0; r < KT; ++r)
#pragma unroll
            for (int c = r; c < KT; ++c, ++p) acc[p] = gs_fma(x[r], x[c], acc[p]);
    }
    flush();
    __syncthreads();
    if (tid < NP) {
        // the 16 warps' sums in four short chains (a fixed order, so still reproducible)
        double s4[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            s4[c] = sacc[4 * c][tid];
#pragma unroll
            for (int w = 1; w < 4; ++w) s4[c] += sacc[4 * c + w][tid];
        }
        a.partials[(size_t)tid * kGsPartialStride + blockIdx.x] = (s4[0] + s4[1]) + (s4[2] + s4[3]);
    }
    __syncthreads();

    // ---- decide: arrive, wait until every CTA has, then total the partials and walk Algorithm 1 here ----
    if (tid == 0) {
        red_release_add_u32(&ctl->fused_arrivals, blockIdx.x == 0 ? kFusedCallUnit - (gridDim.x - 1) : 1u);
        unsigned int polls = 0;
        bool ok = true;
        // (the acquire orders the loads of the partials below, through the barrier, after every CTA's stores)
        while ((ld_acquire_u32(&ctl->fused_arrivals) >> kFusedCallShift) == gen0 || a.test_withhold) {
            __nanosleep(20);
            if (++polls > a.spin_limit) { ok = false; break; }
        }
        n_list = ok ? 0 : -1;
        if (!ok) atomicOr(&ctl->status, GAF_STATUS_TIMEOUT);
    }
    __syncthreads();
    if (n_list < 0) return;                 // every CTA has arrived all the same: the counter is whole again
    const bool publisher = blockIdx.x == 0;
    total_gram_partials<KT>(a.partials, gridDim.x, sgram, publisher ? a.gram : nullptr);
    __syncthreads();
    {
        // every CTA takes the same sums in the same order, hence the same decisions; one of them writes them out
        auto take = [&](int seed, unsigned long long bits) {
            const int start = seed < 0 ? 0 : seed;
            int n = 0;
            for (int t = 0; t < KT; ++t) {
                const int i = (start + t) % KT;
                if ((bits >> i) & 1ull) { list[n] = static_cast<const T *>(a.g[i]); list_row[n] = i; ++n; }
            }
            n_list = n;
        };
        if (a.ring.K > 0) {
            __shared__ RingTable<KT> ring_table;
            ring_replay_parallel<KT>(a.ring, sgram, ring_table, take, publisher);
        } else {
            __shared__ ReplayTable table;
            replay_on_gram_parallel<KT>(a.replay, sgram, table, [&](unsigned long long bits) { take(-1, bits); }, publisher);
        }
    }
    __syncthreads();
    const int n = n_list;
    const float cdiv = (float)n;
    // the launch behind this one on the stream may be placed from here on (it waits for this grid itself)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // two gradients: when the first pass guessed right, it has written the result already (the same additions and
    // the same division as below).  Otherwise every thread overwrites, below, exactly what it wrote then.
    if constexpr (kSpeculative) {
        const bool seed_alone = n == 1 && list_row[0] == 0;     // (the order-indifferent variant may keep row 1 alone)
        const unsigned int outcome = n == 1 ? 1u : 0u;
        if (publisher && tid == 0) ctl->pair_hint = outcome == (hint & 1u) ? outcome : (2u | outcome);
        if (guessing && (guess_seed_alone ? seed_alone : n == 2)) return;
    }

    // ---- pass 2a: the rounds that were not parked, last first (what pass 1 read last is what L2 still
    //      holds), several rounds in flight per thread; specialised on the number of accepted gradients ----
    auto pass2a = [&](auto nn_tag) {
        constexpr int NN = decltype(nn_tag)::value;
        constexpr int U = FusedInFlight<NN>::U;
        for (int64_t j0 = rounds - 1; j0 >= parked_rounds; j0 -= U) {
            int64_t q[U];
            bool ok[U];
            uint4 w[U][NN];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int64_t ju = j0 - u;
                q[u] = warp_first + ju * stride + lane;
                ok[u] = ju >= parked_rounds && q[u] < n_vec;
#pragma unroll
                for (int i = 0; i < NN; ++i)
                    if (ok[u]) w[u][i] = ld16_policy(list[i] + q[u] * N, pol_first);
            }
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (ok[u]) {
                    float v[N];
                    FusedVec<T>::widen(w[u][0], v);
#pragma unroll
                    for (int i = 1; i < NN; ++i) {
                        float x[N];
                        FusedVec<T>::widen(w[u][i], x);
#pragma unroll
                        for (int k = 0; k < N; ++k) v[k] += x[k];
                    }
#pragma unroll
                    for (int k = 0; k < N; ++k) v[k] = v[k] / cdiv;
                    store_vec_streaming<N>(a.out + q[u] * N, v);
                }
        }
    };
    switch (n) {
        case 1: pass2a(std::integral_constant<int, 1>()); break;
        case 2: if constexpr (KT >= 2) pass2a(std::integral_constant<int, 2>()); break;
        case 3: if constexpr (KT >= 3) pass2a(std::integral_constant<int, 3>()); break;
        case 4: if constexpr (KT >= 4) pass2a(std::integral_constant<int, 4>()); break;
        case 5: if constexpr (KT >= 5) pass2a(std::integral_constant<int, 5>()); break;
        case 6: if constexpr (KT >= 6) pass2a(std::integral_constant<int, 6>()); break;
        case 7: if constexpr (KT >= 7) pass2a(std::integral_constant<int, 7>()); break;
        default: if constexpr (KT >= 8) pass2a(std::integral_constant<int, 8>()); break;
    }
    // ---- pass 2b: the parked rounds, from shared memory ----
    for (int64_t j = 0; j < parked_rounds; ++j) {
        const int64_t q = warp_first + j * stride + lane;
        if (q < n_vec) {
            const uint4 *slot = parked + (size_t)j * KT * kGsThreads + tid;
            float v[N];
            FusedVec<T>::widen(slot[list_row[0] * kGsThreads], v);
            for (int i = 1; i < n; ++i) {
                float x[N];
                FusedVec<T>::widen(slot[list_row[i] * kGsThreads], x);
#pragma unroll
                for (int k = 0; k < N; ++k) v[k] += x[k];
            }
#pragma unroll
            for (int k = 0; k < N; ++k) v[k] = v[k] / cdiv;
            store_vec_streaming<N>(a.out + q * N, v);
        }
    }
    if (blockIdx.x == 0 && tail0 + tid < a.D) {
        const int64_t e = tail0 + tid;
        float v = load1<T>(list[0], e);
        for (int i = 1; i < n; ++i) v += load1<T>(list[i], e);
        a.out[e] = v / cdiv;
    }
}

}  // namespace gaf
