// Device-side building blocks shared by the GAF kernels: element loads, the
// fixed-order reductions, the workspace control block and the scalar decision
// of Algorithm 1 (Eq. 4 evaluated in binary64).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/gaf.h"

namespace gaf {

constexpr int kMaxCtas = 2048;          // most CTAs any kernel here launches
constexpr int kOct = 8;                 // elements handled per inner step

// Control block at the start of the caller's workspace.
struct Control {
    unsigned int ticket;                // last-block election, wraps to 0 by itself
    unsigned int pair_hint;             // one-launch schedule with two gradients: what the latest two calls kept (0 both, 1 the seed alone, 2 | latest: they differed)
    unsigned int reserved1;
    int status;                         // GAF_STATUS_* bits of the latest call
    int count;                          // running c of Algorithm 1
    int ring_seed;                      // any-seed variant: the winning seed, else -1
    unsigned long long accept_bits;     // Gram-first schedule: bit t set = step t accepted
    int decision[GAF_MAX_K];            // by step t: 1 accept, 0 reject
    double sums[GAF_MAX_K][3];          // by step t: {g_i.g, |g|^2, |g_i|^2}
    float stream_dist[GAF_MAX_K];       // streaming form: distance of arrival t
    uint8_t stream_mask[GAF_MAX_K];     // streaming form: decision of arrival t
    double norm_sq_sum;                 // stepwise and streaming forms: sum of |g_i|^2 over the accepted gradients
    // One-launch Gram-first schedule: the arrival counter its CTAs add to and poll, alone in its cache
    // line.  Every call adds 4096 in all (one per CTA, the first CTA makes up the difference), so bits
    // 12..31 count calls and bits 0..11 the CTAs of the running call that have arrived.
    alignas(128) unsigned int fused_arrivals;
    unsigned int fused_pad[31];
};
constexpr size_t kControlBytes = 4096;  // sizeof(Control) rounded up
static_assert(sizeof(Control) <= kControlBytes, "control block");
// After the control block: double partials[kMaxCtas][3], then operation-specific space.
constexpr size_t kPartialsOffset = kControlBytes;
constexpr size_t kPartialsBytes = size_t(kMaxCtas) * 3 * sizeof(double);
constexpr size_t kExtraOffset = kPartialsOffset + kPartialsBytes;

// ------------------------------------------------------------- election ----

// Takes a ticket that elects the last CTA of a grid of `ctas`; returns true in the CTA that took the
// last one.  One atomic with release and acquire semantics at GPU scope: what this CTA wrote before
// (and, through a barrier, what its other threads wrote) is visible to whoever sees the ticket, and
// the last CTA's later loads (again through a barrier for its other threads) see every other CTA's
// writes -- no separate fences.  The counter wraps to 0 after the last ticket, so a workspace is
// initialised once and reused.
__device__ __forceinline__ bool take_last_ticket(unsigned int *ticket, unsigned int ctas) {
    unsigned int old;
    asm volatile("atom.acq_rel.gpu.global.inc.u32 %0, [%1], %2;" : "=r"(old) : "l"(ticket), "r"(ctas - 1) : "memory");
    return old == ctas - 1;
}

// ---------------------------------------------------------------- loads -----

__device__ __forceinline__ float bf16_bits_to_float(unsigned int hi16) {
    return __uint_as_float(hi16 << 16);
}

// Eight consecutive elements starting at element index e (multiple of 8), widened
// to binary32.  Streaming (evict-first) loads: every gradient element is used once
// per pass.
template <typename T>
__device__ __forceinline__ void load8_stream(const T *base, int64_t e, float (&v)[8]);

template <>
__device__ __forceinline__ void load8_stream<float>(const float *base, int64_t e, float (&v)[8]) {
    const float4 *p = reinterpret_cast<const float4 *>(base + e);
    float4 a = __ldcs(p), b = __ldcs(p + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

template <>
__device__ __forceinline__ void load8_stream<__nv_bfloat16>(const __nv_bfloat16 *base, int64_t e,
                                                            float (&v)[8]) {
    uint4 r = __ldcs(reinterpret_cast<const uint4 *>(base + e));
    unsigned int w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        v[2 * k] = bf16_bits_to_float(w[k] & 0xFFFFu);
        v[2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u);
    }
}

template <typename T>
__device__ __forceinline__ float load1(const T *base, int64_t e);
template <>
__device__ __forceinline__ float load1<float>(const float *base, int64_t e) { return base[e]; }
template <>
__device__ __forceinline__ float load1<__nv_bfloat16>(const __nv_bfloat16 *base, int64_t e) {
    return bf16_bits_to_float(reinterpret_cast<const unsigned short *>(base)[e]);
}

__device__ __forceinline__ void load8_acc(const float *acc, int64_t e, float (&v)[8]) {
    const float4 *p = reinterpret_cast<const float4 *>(acc + e);
    float4 a = p[0], b = p[1];
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

__device__ __forceinline__ void store8(float *dst, int64_t e, const float (&v)[8], bool streaming) {
    float4 a = make_float4(v[0], v[1], v[2], v[3]);
    float4 b = make_float4(v[4], v[5], v[6], v[7]);
    float4 *p = reinterpret_cast<float4 *>(dst + e);
    if (streaming) { __stcs(p, a); __stcs(p + 1, b); }
    else { p[0] = a; p[1] = b; }
}

// Binary32 sum of eight products, as a fixed balanced tree (short chains: the
// rounding error of each leaf stays at the 1e-7 level and is averaged out by the
// binary64 accumulation above it).
__device__ __forceinline__ float dot8(const float (&a)[8], const float (&b)[8]) {
    float s0 = fmaf(a[1], b[1], a[0] * b[0]);
    float s1 = fmaf(a[3], b[3], a[2] * b[2]);
    float s2 = fmaf(a[5], b[5], a[4] * b[4]);
    float s3 = fmaf(a[7], b[7], a[6] * b[6]);
    return (s0 + s1) + (s2 + s3);
}

// ------------------------------------------------------------ reductions ----

struct Sums3 {
    double p, na, ng;                   // <acc, g>, |acc|^2, |g|^2
};

__device__ __forceinline__ double shfl_down_f64(double v, int delta) {
    return __shfl_down_sync(0xFFFFFFFFu, v, delta);
}

__device__ __forceinline__ Sums3 warp_reduce(Sums3 s) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        s.p += shfl_down_f64(s.p, d);
        s.na += shfl_down_f64(s.na, d);
        s.ng += shfl_down_f64(s.ng, d);
    }
    return s;                           // lane 0 holds the warp's sums
}

// Sum over the block in a fixed order; the result is valid in thread 0 only.
// `scratch` must hold 3 * (blockDim.x / 32) doubles.
__device__ __forceinline__ Sums3 block_reduce(Sums3 s, double *scratch) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    s = warp_reduce(s);
    if (lane == 0) {
        scratch[3 * warp] = s.p; scratch[3 * warp + 1] = s.na; scratch[3 * warp + 2] = s.ng;
    }
    __syncthreads();
    Sums3 r = {0.0, 0.0, 0.0};
    if (threadIdx.x == 0) {
        for (int w = 0; w < nwarps; ++w) {
            r.p += scratch[3 * w]; r.na += scratch[3 * w + 1]; r.ng += scratch[3 * w + 2];
        }
    }
    __syncthreads();
    return r;
}

// One warp sums `n` per-CTA partial triples in a fixed order (lane-strided, then
// a shuffle tree).  Every lane must call; lane 0 returns the total.  The partials
// were published with a fence before the ticket that elected this CTA, so plain
// L2 loads (which the compiler may issue together) see them.
__device__ __forceinline__ Sums3 warp_sum_partials(const double *partials, int n) {
    const int lane = threadIdx.x & 31;
    Sums3 s = {0.0, 0.0, 0.0};
    // batches of 10 entries per lane (320 CTAs) whose loads are all issued before the first add:
    // this runs on the serial tail of a launch, one L2 round trip per batch
    for (int base = 0; base < n; base += 320) {
        double a[10], b[10], c[10];
#pragma unroll
        for (int k = 0; k < 10; ++k) {
            const int i = base + lane + 32 * k;
            const bool ok = i < n;
            a[k] = ok ? __ldcg(partials + 3 * i) : 0.0;
            b[k] = ok ? __ldcg(partials + 3 * i + 1) : 0.0;
            c[k] = ok ? __ldcg(partials + 3 * i + 2) : 0.0;
        }
#pragma unroll
        for (int k = 0; k < 10; ++k) { s.p += a[k]; s.na += b[k]; s.ng += c[k]; }
    }
    return warp_reduce(s);
}

// --------------------------------------------------------------- decision ---

// Eq. 4 on the three sums, in binary64:  D_c = 1 - p / (sqrt(na) sqrt(ng)),
// with the zero-norm and clamping conventions of the header.  Returns the
// distance and ORs status bits into *status.
__device__ __forceinline__ double cosine_distance(double p, double na, double ng, int *status) {
    double cosv;
    if (na == 0.0 || ng == 0.0) {
        cosv = 0.0;
        *status |= GAF_STATUS_ZERO_NORM;
    } else {
        cosv = p / (sqrt(na) * sqrt(ng));
        cosv = cosv > 1.0 ? 1.0 : cosv;
        cosv = cosv < -1.0 ? -1.0 : cosv;
    }
    if (!(isfinite(p) && isfinite(na) && isfinite(ng))) *status |= GAF_STATUS_NONFINITE;
    return 1.0 - cosv;
}

// Conditioning of a running sum g of c accepted gradients.  Every schedule forms |g|^2 (and g itself)
// from binary32-rounded quantities, so its relative error is about 6e-8 kappa with
//     kappa = c * sum_i |g_i|^2 / |g|^2   (>= (sum_i |g_i|)^2 / |g|^2 >= 1),
// which is at most c while no accepted gradient points against the sum (tau <= 1), and grows without
// bound when accepted gradients nearly cancel (possible only with tau > 1).  Beyond kIllKappa the
// distance tolerance of 1e-5 (6e-8 kappa > 1e-5) and the 1e-6 of the binary32 macro-gradient are no
// longer guaranteed: the call says so with GAF_STATUS_ILL_CONDITIONED.  `norm_sq_sum` = sum_i |g_i|^2
// and `na` = |g|^2, both for the sum AFTER an accept.
constexpr double kIllKappa = 167.0;
__device__ __forceinline__ int ill_conditioned(int c, double norm_sq_sum, double na) {
    return ((double)c * norm_sq_sum > kIllKappa * na) ? GAF_STATUS_ILL_CONDITIONED : 0;
}

}  // namespace gaf
