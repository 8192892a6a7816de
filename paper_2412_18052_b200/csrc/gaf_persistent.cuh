// Persistent schedule of Algorithm 1: ONE cooperative launch, one CTA per SM, for
// all K passes over the gradients.
//
//   * Every CTA owns a fixed, contiguous slice of the D parameters for the whole
//     call, so the slice of the running sum it re-reads in pass s is the one it
//     wrote in pass s-1 (no cross-CTA data hazards, and it tends to stay in L2).
//   * A producer thread streams tiles of the three operands (running sum, the
//     candidate of the next step, the gradient accepted at this step) from global
//     to shared memory with bulk asynchronous copies that signal mbarriers;
//     eight consumer warps do the arithmetic out of shared memory.
//   * The K-1 accept decisions are grid-wide serialisation points: every CTA
//     publishes its three partial sums, arrives at a counter in global memory,
//     and once all have arrived every CTA totals the partials in the same fixed
//     order and evaluates Eq. 4 and the test D_c <= tau itself (identical
//     arithmetic, identical answer).  The producer keeps prefetching the
//     decision-independent operands of the next pass across that wait; only the
//     loads of the just-decided gradient wait for the decision.
//   * Every wait is bounded; when one runs out the CTA sets GAF_STATUS_TIMEOUT,
//     drains its copies in flight and leaves.
#pragma once

#include "gaf_device.cuh"

namespace gaf {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kPersistThreads = kConsumerThreads + 32;     // + one producer warp
constexpr int kTile = 4096;                                 // elements per operand tile
constexpr int kMaxStages = 8;
constexpr unsigned int kDefaultSpinLimit = 1u << 24;        // polls (>= ~40 ns each)

struct PersistArgs {
    const void *g[GAF_MAX_K];       // gradients in processing order (g[0] = seed)
    int idx[GAF_MAX_K];             // their original indices
    int K;
    int64_t D;
    double tau;
    float *acc;                     // running sum == macro_out
    uint8_t *mask_out;
    float *dist_out;                // may be null
    int32_t *count_out;
    Control *ctl;
    double *partials;               // [2][gridDim.x][3]
    int stages;
    unsigned int spin_limit;
};

// ------------------------------------------------------------- PTX helpers --

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_test(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bulk asynchronous copy global -> this CTA's shared memory; completion is counted
// in bytes on `bar`.  Source, destination and size are multiples of 16 bytes.
__device__ __forceinline__ void bulk_load(void *dst_smem, const void *src_gmem, uint32_t bytes,
                                          uint64_t *bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1], %2, [%3], %4;" ::"r"(smem_u32(dst_smem)),
        "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t policy_evict_normal() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
    return p;
}
// Orders this thread's earlier generic-proxy accesses before later asynchronous-proxy
// accesses (the bulk copies that will re-read what was just stored).
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ void consumer_bar() {
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory");
}
__device__ __forceinline__ unsigned int ld_acquire(const unsigned int *p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Four consecutive elements out of a shared-memory tile, widened to binary32.
template <typename T>
__device__ __forceinline__ void lds4(const unsigned char *tile, int q, float (&v)[4]);
template <>
__device__ __forceinline__ void lds4<float>(const unsigned char *tile, int q, float (&v)[4]) {
    float4 a = reinterpret_cast<const float4 *>(tile)[q];
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
}
template <>
__device__ __forceinline__ void lds4<__nv_bfloat16>(const unsigned char *tile, int q, float (&v)[4]) {
    uint2 r = reinterpret_cast<const uint2 *>(tile)[q];
    v[0] = bf16_bits_to_float(r.x & 0xFFFFu); v[1] = __uint_as_float(r.x & 0xFFFF0000u);
    v[2] = bf16_bits_to_float(r.y & 0xFFFFu); v[3] = __uint_as_float(r.y & 0xFFFF0000u);
}
__device__ __forceinline__ float dot4(const float (&a)[4], const float (&b)[4]) {
    return fmaf(a[1], b[1], a[0] * b[0]) + fmaf(a[3], b[3], a[2] * b[2]);
}

// Shared-memory bookkeeping next to the operand stages.
struct PersistShared {
    uint64_t full[kMaxStages];      // producer -> consumers: operands of this stage landed
    uint64_t empty[kMaxStages];     // consumers -> producer: stage may be overwritten
    double scratch[3 * kConsumerWarps];
    int decision[GAF_MAX_K];        // by pass
    volatile int decided;           // passes 0..decided have a decision
    volatile int abort;            // set by whoever runs out of patience
    int quit;                      // abort as sampled once per pass (uniform for all consumers)
    int count;
};

enum PassKind { kPassFirst = 0, kPassMid = 1, kPassLast = 2 };

// Arithmetic of one tile.  `stage` holds [running sum or seed | next candidate | current gradient].
template <typename T, int KIND>
__device__ __forceinline__ void consume_tile(const unsigned char *stage, int cnt, float *acc_tile,
                                             bool accept, float cdiv, Sums3 &s, int ctid) {
    const unsigned char *a0 = stage;
    const unsigned char *a1 = stage + kTile * 4;
    const unsigned char *b = a1 + kTile * sizeof(T);
    const int nq = cnt >> 2;
#pragma unroll 4
    for (int q = ctid; q < nq; q += kConsumerThreads) {
        float v[4], gn[4];
        if (KIND == kPassFirst) lds4<T>(a0, q, v);
        else lds4<float>(a0, q, v);
        if (KIND != kPassLast) lds4<T>(a1, q, gn);
        if (KIND != kPassFirst && accept) {
            float gc[4];
            lds4<T>(b, q, gc);
#pragma unroll
            for (int k = 0; k < 4; ++k) v[k] += gc[k];
        }
        float4 *dst = reinterpret_cast<float4 *>(acc_tile) + q;
        if (KIND == kPassLast) {
            __stcs(dst, make_float4(v[0] / cdiv, v[1] / cdiv, v[2] / cdiv, v[3] / cdiv));
        } else if (KIND == kPassFirst || accept) {
            *dst = make_float4(v[0], v[1], v[2], v[3]);
        }
        if (KIND != kPassLast) {
            s.p += (double)dot4(v, gn);
            s.na += (double)dot4(v, v);
            s.ng += (double)dot4(gn, gn);
        }
    }
}

// The D mod 8 trailing elements, handled with plain loads by the last CTA.
template <typename T>
__device__ __forceinline__ void consume_ragged(const PersistArgs &a, int pass, bool accept,
                                               float cdiv, Sums3 &s, int ctid) {
    const int64_t e = (a.D / kOct) * kOct + ctid;
    if (e >= a.D) return;
    const bool first = pass == 0, last = pass == a.K - 1;
    float v = first ? load1<T>(static_cast<const T *>(a.g[0]), e) : a.acc[e];
    if (!first && accept) v += load1<T>(static_cast<const T *>(a.g[pass]), e);
    if (last) a.acc[e] = v / cdiv;
    else if (first || accept) a.acc[e] = v;
    if (!last) {
        float gn = load1<T>(static_cast<const T *>(a.g[pass + 1]), e);
        s.p += (double)(v * gn);
        s.na += (double)(v * v);
        s.ng += (double)(gn * gn);
    }
}

template <typename T>
__global__ void __launch_bounds__(kPersistThreads, 1) persistent_kernel(PersistArgs a) {
    extern __shared__ __align__(128) unsigned char stage_mem[];
    __shared__ PersistShared sh;

    constexpr uint32_t kStageBytes = kTile * 4 + 2 * kTile * sizeof(T);
    const int NS = a.stages;
    const int G = gridDim.x, cta = blockIdx.x;
    const int K = a.K;

    // this CTA's slice, in units of 8 elements so every bulk copy is 16-byte aligned
    const int64_t n_oct = a.D / kOct;
    const int64_t lo = (n_oct * cta / G) * kOct;
    const int64_t hi = (n_oct * (cta + 1) / G) * kOct;
    const int my_n = (int)((hi - lo + kTile - 1) / kTile);
    const long long total = (long long)K * my_n;

    if (threadIdx.x == 0) {
        for (int i = 0; i < NS; ++i) {
            mbar_init(&sh.full[i], 2);                  // producer arrives twice per use
            mbar_init(&sh.empty[i], kConsumerWarps);
        }
        sh.decided = 0;
        sh.abort = 0;
        sh.quit = 0;
        sh.count = 1;
        sh.decision[0] = 1;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
        if (cta == 0) {
            a.ctl->status = 0;
            a.ctl->count = 1;
            a.ctl->decision[0] = 1;
            a.mask_out[a.idx[0]] = 1;
            if (a.dist_out) a.dist_out[a.idx[0]] = 0.0f;
        }
    }
    __syncthreads();

    if (threadIdx.x >= kConsumerThreads) {
        // ------------------------------------------------------ producer -----
        if (threadIdx.x != kConsumerThreads) return;
        const uint64_t pol_stream = policy_evict_first();
        const uint64_t pol_acc = policy_evict_normal();
        long long a_iss = 0, b_iss = 0, freed = 0;
        unsigned int idle = 0;
        bool timed_out = false;
        while (b_iss < total) {
            bool progressed = false;
            if (freed < a_iss) {
                const int st = (int)(freed % NS);
                if (mbar_test(&sh.empty[st], (uint32_t)((freed / NS) & 1))) { ++freed; progressed = true; }
            }
            // operands that do not depend on the pending decision
            if (a_iss < total && a_iss - freed < NS && (a_iss < my_n || a_iss - my_n < freed)) {
                const int pass = (int)(a_iss / my_n), k = (int)(a_iss % my_n);
                const int st = (int)(a_iss % NS);
                const int64_t e0 = lo + (int64_t)k * kTile;
                const uint32_t cnt = (uint32_t)min((int64_t)kTile, hi - e0);
                unsigned char *stage = stage_mem + (size_t)st * kStageBytes;
                const uint32_t gbytes = cnt * (uint32_t)sizeof(T);
                if (pass == 0) {
                    mbar_arrive_expect_tx(&sh.full[st], 2 * gbytes);
                    bulk_load(stage, static_cast<const T *>(a.g[0]) + e0, gbytes, &sh.full[st], pol_stream);
                    bulk_load(stage + kTile * 4, static_cast<const T *>(a.g[1]) + e0, gbytes, &sh.full[st],
                              pol_stream);
                } else {
                    const bool has_next = pass < K - 1;
                    mbar_arrive_expect_tx(&sh.full[st], cnt * 4 + (has_next ? gbytes : 0));
                    bulk_load(stage, a.acc + e0, cnt * 4, &sh.full[st], pol_acc);
                    if (has_next)
                        bulk_load(stage + kTile * 4, static_cast<const T *>(a.g[pass + 1]) + e0, gbytes,
                                  &sh.full[st], pol_stream);
                }
                ++a_iss;
                progressed = true;
            }
            // the gradient decided at this pass: loaded only if it was accepted
            if (b_iss < a_iss) {
                const int pass = (int)(b_iss / my_n);
                if (pass == 0 || sh.decided >= pass) {
                    const int st = (int)(b_iss % NS);
                    if (pass > 0 && sh.decision[pass]) {
                        const int k = (int)(b_iss % my_n);
                        const int64_t e0 = lo + (int64_t)k * kTile;
                        const uint32_t cnt = (uint32_t)min((int64_t)kTile, hi - e0);
                        const uint32_t gbytes = cnt * (uint32_t)sizeof(T);
                        unsigned char *stage = stage_mem + (size_t)st * kStageBytes;
                        mbar_arrive_expect_tx(&sh.full[st], gbytes);
                        bulk_load(stage + kTile * 4 + kTile * sizeof(T),
                                  static_cast<const T *>(a.g[pass]) + e0, gbytes, &sh.full[st], pol_stream);
                    } else {
                        mbar_arrive(&sh.full[st]);
                    }
                    ++b_iss;
                    progressed = true;
                }
            }
            if (progressed) { idle = 0; continue; }
            if (sh.abort || ++idle > a.spin_limit) { timed_out = true; break; }
            __nanosleep(40);
        }
        if (timed_out) {
            sh.abort = 1;
            atomicOr(&a.ctl->status, GAF_STATUS_TIMEOUT);
            // let every stage with copies in flight complete, then wait for them (bounded)
            for (long long n = b_iss; n < a_iss; ++n) mbar_arrive(&sh.full[(int)(n % NS)]);
            for (long long n = freed; n < a_iss; ++n) {
                const int st = (int)(n % NS);
                for (unsigned int spin = 0; spin < a.spin_limit; ++spin) {
                    if (mbar_test(&sh.full[st], (uint32_t)((n / NS) & 1))) break;
                    __nanosleep(40);
                }
            }
        }
        return;
    }

    // ---------------------------------------------------------- consumers ----
    const int ctid = threadIdx.x, warp = ctid >> 5, lane = ctid & 31;
    bool accept = true;
    int count = 1;
    long long n = 0;                                    // running (pass, tile) sequence number
    for (int pass = 0; pass < K; ++pass) {
        const bool last = pass == K - 1;
        const float cdiv = (float)count;
        Sums3 s = {0.0, 0.0, 0.0};
        for (int k = 0; k < my_n; ++k, ++n) {
            const int st = (int)(n % NS);
            const uint32_t parity = (uint32_t)((n / NS) & 1);
            bool ok = true;
            unsigned int spin = 0;
            while (!mbar_test(&sh.full[st], parity)) {
                if (sh.abort || ++spin > a.spin_limit) { ok = false; break; }
                if (spin > 64) __nanosleep(40);
            }
            if (!ok) {
                if (!sh.abort) { sh.abort = 1; atomicOr(&a.ctl->status, GAF_STATUS_TIMEOUT); }
                break;
            }
            const int64_t e0 = lo + (int64_t)k * kTile;
            const int cnt = (int)min((int64_t)kTile, hi - e0);
            const unsigned char *stage = stage_mem + (size_t)st * kStageBytes;
            if (pass == 0) consume_tile<T, kPassFirst>(stage, cnt, a.acc + e0, accept, cdiv, s, ctid);
            else if (!last) consume_tile<T, kPassMid>(stage, cnt, a.acc + e0, accept, cdiv, s, ctid);
            else consume_tile<T, kPassLast>(stage, cnt, a.acc + e0, accept, cdiv, s, ctid);
            // stores to the running sum are re-read by bulk copies in the next pass
            if (!last && (pass == 0 || accept)) fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.empty[st]);
        }
        if (cta == G - 1) consume_ragged<T>(a, pass, accept, cdiv, s, ctid);
        if (last) break;

        // ---- decision of pass+1: publish partials, grid barrier, total, Eq. 4 ----
        s = warp_reduce(s);
        if (lane == 0) {
            sh.scratch[3 * warp] = s.p; sh.scratch[3 * warp + 1] = s.na; sh.scratch[3 * warp + 2] = s.ng;
        }
        consumer_bar();
        double *part = a.partials + (size_t)(pass & 1) * G * 3;
        if (warp == 0) {
            if (lane == 0) {
                Sums3 r = {0.0, 0.0, 0.0};
                for (int w = 0; w < kConsumerWarps; ++w) {
                    r.p += sh.scratch[3 * w]; r.na += sh.scratch[3 * w + 1]; r.ng += sh.scratch[3 * w + 2];
                }
                part[3 * cta] = r.p; part[3 * cta + 1] = r.na; part[3 * cta + 2] = r.ng;
                if (!sh.abort) {
                    __threadfence();
                    atomicAdd(&a.ctl->barrier, 1u);
                    const unsigned int want = (unsigned int)(pass + 1) * (unsigned int)G;
                    unsigned int spin = 0;
                    while (ld_acquire(&a.ctl->barrier) < want) {
                        if (++spin > a.spin_limit) {
                            sh.abort = 1;
                            atomicOr(&a.ctl->status, GAF_STATUS_TIMEOUT);
                            break;
                        }
                        __nanosleep(32);
                    }
                    __threadfence();
                }
            }
            __syncwarp();
            if (lane == 0) sh.quit = sh.abort;
            __syncwarp();
            if (!sh.quit) {
                Sums3 tot = warp_sum_partials(part, G);
                if (lane == 0) {
                    int status = 0;
                    const double d = cosine_distance(tot.p, tot.na, tot.ng, &status);
                    const int acc_it = (d <= a.tau) ? 1 : 0;
                    sh.count += acc_it;
                    sh.decision[pass + 1] = acc_it;
                    __threadfence_block();
                    sh.decided = pass + 1;
                    if (cta == 0) {
                        Control *c = a.ctl;
                        c->decision[pass + 1] = acc_it;
                        c->sums[pass + 1][0] = tot.p; c->sums[pass + 1][1] = tot.na; c->sums[pass + 1][2] = tot.ng;
                        c->count = sh.count;
                        if (status) atomicOr(&c->status, status);
                        a.mask_out[a.idx[pass + 1]] = (uint8_t)acc_it;
                        if (a.dist_out) a.dist_out[a.idx[pass + 1]] = (float)d;
                    }
                }
            }
        }
        consumer_bar();
        if (sh.quit) return;
        accept = sh.decision[pass + 1] != 0;
        count = sh.count;
    }
    if (sh.abort) return;

    // leave the workspace ready for the next call
    if (ctid == 0) {
        if (cta == 0) *a.count_out = count;
        const unsigned int old = atomicInc(&a.ctl->exit_ticket, (unsigned int)G - 1);
        if (old == (unsigned int)G - 1) {
            a.ctl->barrier = 0;
            __threadfence();
        }
    }
}

// ------------------------------------------------------------- host side ----

inline size_t persistent_stage_bytes(int dtype) {
    return size_t(kTile) * 4 + 2 * size_t(kTile) * (dtype == GAF_F32 ? 4 : 2);
}

inline bool persistent_supported(int coop, int smem_optin) {
    return coop != 0 && size_t(smem_optin) >= 2 * persistent_stage_bytes(GAF_F32);
}

template <typename T>
int launch_persistent(const void *const *g, int K, int64_t D, double tau, const int32_t *ord,
                      float *macro_out, uint8_t *mask_out, float *dist_out, int32_t *count_out,
                      Control *ctl, double *partials, int sms, cudaStream_t st) {
    PersistArgs a{};
    for (int t = 0; t < K; ++t) { a.g[t] = g[ord[t]]; a.idx[t] = ord[t]; }
    a.K = K; a.D = D; a.tau = tau; a.acc = macro_out; a.mask_out = mask_out; a.dist_out = dist_out;
    a.count_out = count_out; a.ctl = ctl; a.partials = partials;
    a.spin_limit = kDefaultSpinLimit;

    int dev = 0, smem_optin = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GAF_ERR_CUDA;
    if (cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
        return GAF_ERR_CUDA;
    const size_t stage = size_t(kTile) * 4 + 2 * size_t(kTile) * sizeof(T);
    const size_t reserve = 2048;    // static shared memory of the kernel
    int stages = int((size_t(smem_optin) - reserve) / stage);
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) return GAF_ERR_UNSUPPORTED;
    a.stages = stages;
    const size_t dyn = stages * stage;
    if (cudaFuncSetAttribute(persistent_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) !=
        cudaSuccess)
        return GAF_ERR_CUDA;
    // one CTA per SM, never more CTAs than there are 8-element groups
    int grid = sms;
    if (grid > kMaxCtas / 2) grid = kMaxCtas / 2;
    const int64_t n_oct = D / kOct;
    if (n_oct < grid) grid = n_oct > 0 ? int(n_oct) : 1;
    void *params[] = {&a};
    cudaError_t err = cudaLaunchCooperativeKernel((const void *)persistent_kernel<T>, dim3(grid),
                                                  dim3(kPersistThreads), params, dyn, st);
    if (err != cudaSuccess) { cudaGetLastError(); return GAF_ERR_CUDA; }
    return GAF_OK;
}

}  // namespace gaf
