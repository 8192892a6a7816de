// Resident schedule of Algorithm 1: ONE cooperative launch for all K passes, one
// CTA per SM, with the running sum g kept ON CHIP between passes.
//
//   * Every CTA owns a fixed contiguous slice of the D parameters and every thread
//     a fixed set of 4-element groups of it, for the whole call.  The thread's part
//     of the running sum lives in up to three tiers: registers (the first kRegQuads
//     groups; none by default), shared memory (as many as fit), and -- only when the
//     slice is too large -- the output buffer in global memory, always touched by the
//     same thread, so that program order alone keeps it coherent.  For D up to about
//     8.4 M (148 SMs) the running sum never travels: a pass reads the candidate of the
//     next step (and the gradient accepted at this step, usually still in L2), and
//     the only global write of the call is g/c at the end.
//   * Loads are plain 128-bit coalesced loads, issued in batches ahead of the
//     arithmetic; element arithmetic is binary32, sums are binary64 per thread and
//     reduced in a fixed order (bitwise reproducible).
//   * The K-1 accept decisions are grid-wide serialisation points: every CTA
//     publishes its three partial sums, arrives at a counter in global memory, waits
//     (bounded) for all arrivals, totals the partials in the same fixed order and
//     evaluates Eq. 4 and the test D_c <= tau itself.
//   * When the bounded wait runs out the CTA sets GAF_STATUS_TIMEOUT and leaves.
#pragma once

#include "gaf_device.cuh"

namespace gaf {

#ifndef GAF_RES_THREADS
#define GAF_RES_THREADS 512
#endif
#ifndef GAF_RES_REGQ
#define GAF_RES_REGQ 0
#endif
#ifndef GAF_RES_BATCH
#define GAF_RES_BATCH 4
#endif
#ifndef GAF_RES_SPILL_BATCH
#define GAF_RES_SPILL_BATCH 2
#endif
constexpr int kResThreads = GAF_RES_THREADS;
constexpr int kRegQuads = GAF_RES_REGQ;           // 4-element groups of g held in registers per thread
constexpr int kBatch = GAF_RES_BATCH;             // groups whose loads are issued together
constexpr int kSpillBatch = GAF_RES_SPILL_BATCH;  // same, for the groups that live in global memory
constexpr unsigned int kResSpinLimit = 1u << 24;
static_assert(kRegQuads % kBatch == 0, "register tier is processed in whole batches");

struct ResArgs {
    const void *g[GAF_MAX_K];       // gradients in processing order (g[0] = seed)
    int idx[GAF_MAX_K];             // their original indices
    int K;
    int64_t D;
    double tau;
    float *acc;                     // macro_out; also the global tier of the running sum
    uint8_t *mask_out;
    float *dist_out;                // may be null
    int32_t *count_out;
    Control *ctl;
    double *partials;               // [2][gridDim.x][3]
    int smem_slots;                 // shared-memory groups per thread
    unsigned int spin_limit;
};

enum ResPass { kResFirst = 0, kResMid = 1, kResLast = 2 };

__device__ __forceinline__ unsigned int res_ld_acquire(const unsigned int *p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ float res_dot4(const float (&a)[4], const float (&b)[4]) {
    return fmaf(a[1], b[1], a[0] * b[0]) + fmaf(a[3], b[3], a[2] * b[2]);
}

// Four consecutive elements from global memory, widened to binary32.  KEEP = the
// data is likely to be read again in the next pass (leave it in L2); otherwise
// it is a streaming, evict-first load.
template <typename T, bool KEEP>
__device__ __forceinline__ void ldg4(const T *__restrict__ base, int64_t e, float (&v)[4]);
template <>
__device__ __forceinline__ void ldg4<float, true>(const float *__restrict__ base, int64_t e, float (&v)[4]) {
    float4 a = __ldg(reinterpret_cast<const float4 *>(base + e));
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
}
template <>
__device__ __forceinline__ void ldg4<float, false>(const float *__restrict__ base, int64_t e, float (&v)[4]) {
    float4 a = __ldcs(reinterpret_cast<const float4 *>(base + e));
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
}
__device__ __forceinline__ void unpack_bf16x4(uint2 r, float (&v)[4]) {
    v[0] = bf16_bits_to_float(r.x & 0xFFFFu); v[1] = __uint_as_float(r.x & 0xFFFF0000u);
    v[2] = bf16_bits_to_float(r.y & 0xFFFFu); v[3] = __uint_as_float(r.y & 0xFFFF0000u);
}
template <>
__device__ __forceinline__ void ldg4<__nv_bfloat16, true>(const __nv_bfloat16 *__restrict__ base, int64_t e,
                                                          float (&v)[4]) {
    unpack_bf16x4(__ldg(reinterpret_cast<const uint2 *>(base + e)), v);
}
template <>
__device__ __forceinline__ void ldg4<__nv_bfloat16, false>(const __nv_bfloat16 *__restrict__ base, int64_t e,
                                                           float (&v)[4]) {
    unpack_bf16x4(__ldcs(reinterpret_cast<const uint2 *>(base + e)), v);
}

// Arithmetic of one 4-element group in one pass.  `v` enters as the group's part of
// the running sum (the seed in the first pass) and leaves as what is stored back.
template <int PASS>
__device__ __forceinline__ void combine(float (&v)[4], const float (&gc)[4], const float (&gn)[4],
                                        bool accept, float cdiv, Sums3 &s) {
    if (PASS != kResFirst && accept) {
#pragma unroll
        for (int k = 0; k < 4; ++k) v[k] += gc[k];
    }
    if (PASS != kResLast) {
        s.p += (double)res_dot4(v, gn);
        s.na += (double)res_dot4(v, v);
        s.ng += (double)res_dot4(gn, gn);
    } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) v[k] = v[k] / cdiv;
    }
}

struct ResSlice {
    int64_t lo;                     // first element of the CTA's slice
    int nq;                         // 4-element groups in the slice
    int j_smem_end;                 // per-thread group index where the shared-memory tier ends
    int j_end;                      // per-thread group count (ceil)
};

// One pass over the thread's groups.  gc = gradient decided at this pass (added if
// accepted), gn = candidate of the next step.
template <typename T, int PASS>
__device__ __forceinline__ void run_pass(const ResArgs &a, const ResSlice &sl, float4 (&racc)[kRegQuads > 0 ? kRegQuads : 1],
                                         float4 *sacc, const T *__restrict__ gc_base,
                                         const T *__restrict__ gn_base, bool accept, float cdiv, Sums3 &s) {
    const int t = threadIdx.x;
    const bool need_gc = (PASS == kResFirst) || accept;       // first pass: "gc" is the seed itself
    float *__restrict__ out = a.acc;

    // ---- tier 1: registers (static indices: fully unrolled) ----
#pragma unroll
    for (int jb = 0; jb < kRegQuads; jb += kBatch) {
        float gc[kBatch][4], gn[kBatch][4];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int q = t + (jb + u) * kResThreads;
            if (q < sl.nq) {
                const int64_t e = sl.lo + (int64_t)q * 4;
                if (need_gc) ldg4<T, false>(gc_base, e, gc[u]);
                if (PASS != kResLast) ldg4<T, true>(gn_base, e, gn[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int q = t + (jb + u) * kResThreads;
            if (q < sl.nq) {
                float v[4];
                if (PASS == kResFirst) { v[0] = gc[u][0]; v[1] = gc[u][1]; v[2] = gc[u][2]; v[3] = gc[u][3]; }
                else { v[0] = racc[jb + u].x; v[1] = racc[jb + u].y; v[2] = racc[jb + u].z; v[3] = racc[jb + u].w; }
                combine<PASS>(v, gc[u], gn[u], accept, cdiv, s);
                if (PASS == kResLast) __stcs(reinterpret_cast<float4 *>(out + sl.lo) + q, make_float4(v[0], v[1], v[2], v[3]));
                else racc[jb + u] = make_float4(v[0], v[1], v[2], v[3]);
            }
        }
    }
    // ---- tier 2: shared memory (thread-private slots, conflict-free 16-byte accesses) ----
#pragma unroll 1
    for (int jb = kRegQuads; jb < sl.j_smem_end; jb += kBatch) {
        float gc[kBatch][4], gn[kBatch][4];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int j = jb + u, q = t + j * kResThreads;
            if (j < sl.j_smem_end && q < sl.nq) {
                const int64_t e = sl.lo + (int64_t)q * 4;
                if (need_gc) ldg4<T, false>(gc_base, e, gc[u]);
                if (PASS != kResLast) ldg4<T, true>(gn_base, e, gn[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int j = jb + u, q = t + j * kResThreads;
            if (j < sl.j_smem_end && q < sl.nq) {
                float4 *slot = sacc + (size_t)(j - kRegQuads) * kResThreads + t;
                float v[4];
                if (PASS == kResFirst) { v[0] = gc[u][0]; v[1] = gc[u][1]; v[2] = gc[u][2]; v[3] = gc[u][3]; }
                else { const float4 r = *slot; v[0] = r.x; v[1] = r.y; v[2] = r.z; v[3] = r.w; }
                combine<PASS>(v, gc[u], gn[u], accept, cdiv, s);
                const float4 r = make_float4(v[0], v[1], v[2], v[3]);
                if (PASS == kResLast) __stcs(reinterpret_cast<float4 *>(out + sl.lo) + q, r);
                else if (PASS == kResFirst || accept) *slot = r;
            }
        }
    }
    // ---- tier 3: what does not fit on chip lives in the output buffer, always touched by
    //      the same thread (program order keeps it coherent) ----
#pragma unroll 1
    for (int jb = sl.j_smem_end; jb < sl.j_end; jb += kSpillBatch) {
        float gc[kSpillBatch][4], gn[kSpillBatch][4], v[kSpillBatch][4];
#pragma unroll
        for (int u = 0; u < kSpillBatch; ++u) {
            const int j = jb + u, q = t + j * kResThreads;
            if (j < sl.j_end && q < sl.nq) {
                const int64_t e = sl.lo + (int64_t)q * 4;
                if (need_gc) ldg4<T, false>(gc_base, e, gc[u]);
                if (PASS != kResLast) ldg4<T, true>(gn_base, e, gn[u]);
                if (PASS != kResFirst) {
                    const float4 r = *reinterpret_cast<const float4 *>(out + e);
                    v[u][0] = r.x; v[u][1] = r.y; v[u][2] = r.z; v[u][3] = r.w;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kSpillBatch; ++u) {
            const int j = jb + u, q = t + j * kResThreads;
            if (j < sl.j_end && q < sl.nq) {
                if (PASS == kResFirst) {
                    v[u][0] = gc[u][0]; v[u][1] = gc[u][1]; v[u][2] = gc[u][2]; v[u][3] = gc[u][3];
                }
                combine<PASS>(v[u], gc[u], gn[u], accept, cdiv, s);
                const float4 r = make_float4(v[u][0], v[u][1], v[u][2], v[u][3]);
                float4 *gdst = reinterpret_cast<float4 *>(out + sl.lo) + q;
                if (PASS == kResLast) __stcs(gdst, r);
                else if (PASS == kResFirst || accept) *gdst = r;
            }
        }
    }
}

// The D mod 8 trailing elements: plain scalar accesses by the last CTA (global tier).
template <typename T>
__device__ __forceinline__ void run_ragged(const ResArgs &a, int pass, bool accept, float cdiv, Sums3 &s) {
    const int64_t e = (a.D / kOct) * kOct + threadIdx.x;
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

// Grid-wide decision of step pass+1: publish this CTA's sums, wait (bounded) for all
// CTAs, total in fixed order, evaluate Eq. 4 and the test.  Returns false on timeout.
struct DecideArgs {                 // what the decision needs, passed by value: taking the address
    Control *ctl;                   // of the kernel's parameter block would force a per-thread
    double *partials;               // copy of it into local memory
    double tau;
    uint8_t *mask_out;
    float *dist_out;
    unsigned int spin_limit;
    int idx_next;                   // original index of the gradient being decided
};

__device__ __noinline__ bool decide(DecideArgs a, int pass, Sums3 s, double *scratch, int count,
                                    int &sh_decision, int &sh_count, int &sh_abort) {
    const int G = gridDim.x, cta = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    Sums3 blk = block_reduce(s, scratch);
    double *part = a.partials + (size_t)(pass & 1) * G * 3;
    if (warp == 0) {
        if (lane == 0) {
            part[3 * cta] = blk.p; part[3 * cta + 1] = blk.na; part[3 * cta + 2] = blk.ng;
            __threadfence();
            atomicAdd(&a.ctl->barrier, 1u);
            const unsigned int want = (unsigned int)(pass + 1) * (unsigned int)G;
            unsigned int spin = 0;
            while (res_ld_acquire(&a.ctl->barrier) < want) {
                if (++spin > a.spin_limit) {
                    sh_abort = 1;
                    atomicOr(&a.ctl->status, GAF_STATUS_TIMEOUT);
                    break;
                }
                __nanosleep(20);
            }
            __threadfence();
        }
        __syncwarp();
        Sums3 tot = warp_sum_partials(part, G);
        if (lane == 0) {
            int status = 0;
            const double d = cosine_distance(tot.p, tot.na, tot.ng, &status);
            const int acc_it = (d <= a.tau) ? 1 : 0;
            sh_decision = acc_it;
            sh_count = count + acc_it;
            if (cta == 0 && !sh_abort) {
                Control *c = a.ctl;
                c->decision[pass + 1] = acc_it;
                c->sums[pass + 1][0] = tot.p; c->sums[pass + 1][1] = tot.na; c->sums[pass + 1][2] = tot.ng;
                c->count = count + acc_it;
                if (status) atomicOr(&c->status, status);
                a.mask_out[a.idx_next] = (uint8_t)acc_it;
                if (a.dist_out) a.dist_out[a.idx_next] = (float)d;
            }
        }
    }
    __syncthreads();
    return sh_abort == 0;               // written by one thread before the barrier: uniform
}

template <typename T>
__global__ void __launch_bounds__(kResThreads, 1) resident_kernel(ResArgs a) {
    extern __shared__ __align__(16) unsigned char res_smem[];
    __shared__ double scratch[3 * (kResThreads / 32)];
    __shared__ int sh_decision, sh_count, sh_abort;

    float4 *sacc = reinterpret_cast<float4 *>(res_smem);
    const int G = gridDim.x, cta = blockIdx.x, K = a.K;

    ResSlice sl;
    {
        const int64_t n_oct = a.D / kOct;
        sl.lo = (n_oct * cta / G) * kOct;
        const int64_t hi = (n_oct * (cta + 1) / G) * kOct;
        sl.nq = (int)((hi - sl.lo) >> 2);
        sl.j_end = (sl.nq + kResThreads - 1) / kResThreads;
        sl.j_smem_end = min(sl.j_end, kRegQuads + a.smem_slots);
    }
    if (threadIdx.x == 0) {
        sh_abort = 0;
        if (cta == 0) {
            a.ctl->status = 0;
            a.ctl->count = 1;
            a.ctl->decision[0] = 1;
            a.mask_out[a.idx[0]] = 1;
            if (a.dist_out) a.dist_out[a.idx[0]] = 0.0f;
        }
    }
    float4 racc[kRegQuads > 0 ? kRegQuads : 1];
    bool accept = true;
    int count = 1;
    {
        Sums3 s = {0.0, 0.0, 0.0};
        const T *gc = static_cast<const T *>(a.g[0]);
        const T *gn = static_cast<const T *>(a.g[1]);
        run_pass<T, kResFirst>(a, sl, racc, sacc, gc, gn, true, 1.0f, s);
        if (cta == G - 1) run_ragged<T>(a, 0, true, 1.0f, s);
        if (!decide(DecideArgs{a.ctl, a.partials, a.tau, a.mask_out, a.dist_out, a.spin_limit, a.idx[1]}, 0, s,
                    scratch, count, sh_decision, sh_count, sh_abort))
            return;
        accept = sh_decision != 0;
        count = sh_count;
        __syncthreads();
    }
    for (int pass = 1; pass < K - 1; ++pass) {
        Sums3 s = {0.0, 0.0, 0.0};
        const T *gc = static_cast<const T *>(a.g[pass]);
        const T *gn = static_cast<const T *>(a.g[pass + 1]);
        run_pass<T, kResMid>(a, sl, racc, sacc, gc, gn, accept, 1.0f, s);
        if (cta == G - 1) run_ragged<T>(a, pass, accept, 1.0f, s);
        if (!decide(DecideArgs{a.ctl, a.partials, a.tau, a.mask_out, a.dist_out, a.spin_limit, a.idx[pass + 1]},
                    pass, s, scratch, count, sh_decision, sh_count, sh_abort))
            return;
        accept = sh_decision != 0;
        count = sh_count;
        __syncthreads();
    }
    {
        Sums3 s = {0.0, 0.0, 0.0};
        const T *gc = static_cast<const T *>(a.g[K - 1]);
        run_pass<T, kResLast>(a, sl, racc, sacc, gc, gc, accept, (float)count, s);
        if (cta == G - 1) run_ragged<T>(a, K - 1, accept, (float)count, s);
    }

    // leave the workspace ready for the next call
    if (threadIdx.x == 0) {
        if (cta == 0) *a.count_out = count;
        const unsigned int old = atomicInc(&a.ctl->exit_ticket, (unsigned int)G - 1);
        if (old == (unsigned int)G - 1) {
            a.ctl->barrier = 0;
            __threadfence();
        }
    }
}

// ------------------------------------------------------------- host side ----

// Elements of running sum that stay on chip with `sms` CTAs and `smem_optin` bytes
// of opt-in shared memory per CTA.
inline int resident_smem_slots(int smem_optin) {
    const int reserve = 2048;                       // static shared memory of the kernel
    int slots = (smem_optin - reserve) / (16 * kResThreads);
    return slots < 0 ? 0 : slots;
}
inline int64_t resident_capacity(int sms, int smem_optin) {
    return int64_t(sms) * (kRegQuads + resident_smem_slots(smem_optin)) * kResThreads * 4;
}

template <typename T>
int launch_resident(const void *const *g, int K, int64_t D, double tau, const int32_t *ord,
                    float *macro_out, uint8_t *mask_out, float *dist_out, int32_t *count_out,
                    Control *ctl, double *partials, int sms, int smem_optin, cudaStream_t st) {
    ResArgs a{};
    for (int t = 0; t < K; ++t) { a.g[t] = g[ord[t]]; a.idx[t] = ord[t]; }
    a.K = K; a.D = D; a.tau = tau; a.acc = macro_out; a.mask_out = mask_out; a.dist_out = dist_out;
    a.count_out = count_out; a.ctl = ctl; a.partials = partials;
    a.spin_limit = kResSpinLimit;
    a.smem_slots = resident_smem_slots(smem_optin);
    const size_t dyn = size_t(a.smem_slots) * 16 * kResThreads;
    if (cudaFuncSetAttribute(resident_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) !=
        cudaSuccess)
        return GAF_ERR_CUDA;
    int grid = sms;
    if (grid > kMaxCtas / 2) grid = kMaxCtas / 2;
    const int64_t n_oct = D / kOct;
    if (n_oct < grid) grid = n_oct > 0 ? int(n_oct) : 1;
    void *params[] = {&a};
    cudaError_t err = cudaLaunchCooperativeKernel((const void *)resident_kernel<T>, dim3(grid),
                                                  dim3(kResThreads), params, dyn, st);
    if (err != cudaSuccess) { cudaGetLastError(); return GAF_ERR_CUDA; }
    return GAF_OK;
}

}  // namespace gaf
