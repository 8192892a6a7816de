// Stepwise schedule of Algorithm 1: one launch per step, the accept decision of
// step t taken on the device by the last CTA to finish and read by the launch
// of step t+1.  Each launch fuses "add the gradient accepted at step t" with
// "three dot products against the candidate of step t+1", so the running sum is
// read once per step.  Also the two-buffer cosine distance of Eq. 4.
#pragma once

#include "gaf_device.cuh"

namespace gaf {

constexpr int kStepThreads = 512;

struct StepArgs {
    const void *g_seed;     // FIRST: the seed gradient (source of the running sum)
    const void *g_cur;      // MID/LAST: candidate of this step (added if accepted)
    const void *g_next;     // FIRST/MID: candidate of the next step (dot products)
    float *acc;             // running sum g == macro_out
    int64_t D;
    Control *ctl;
    double *partials;
    double tau;
    int t;                  // step whose decision this launch consumes (0 for FIRST)
    int i_next;             // original index of g_next
    uint8_t *mask_out;
    float *dist_out;        // may be null
    int32_t *count_out;
    int seed_index;         // original index of the seed
    int K;
};

enum StepMode { kFirst = 0, kMid = 1, kLast = 2, kOnly = 3 };

// Last-CTA finaliser: total the partials in fixed order, evaluate Eq. 4 and the
// test D_c <= tau, publish the decision of step t+1.
__device__ __forceinline__ void finalize_step(const StepArgs &a, Sums3 mine, int step_next) {
    __shared__ bool is_last;
    if (threadIdx.x == 0) {
        a.partials[3 * blockIdx.x] = mine.p;
        a.partials[3 * blockIdx.x + 1] = mine.na;
        a.partials[3 * blockIdx.x + 2] = mine.ng;
        is_last = take_last_ticket(&a.ctl->ticket, gridDim.x);
    }
    __syncthreads();
    if (!is_last || threadIdx.x >= 32) return;
    Sums3 tot = warp_sum_partials(a.partials, gridDim.x);
    if (threadIdx.x == 0) {
        int status = 0;
        double d = cosine_distance(tot.p, tot.na, tot.ng, &status);
        int accept = (d <= a.tau) ? 1 : 0;
        Control *c = a.ctl;
        c->decision[step_next] = accept;
        c->sums[step_next][0] = tot.p; c->sums[step_next][1] = tot.na; c->sums[step_next][2] = tot.ng;
        c->count += accept;
        if (step_next == 1) c->norm_sq_sum = tot.na;        // the running sum is still the seed alone
        if (accept) {
            // conditioning of the sum this accept leaves behind: |g + g_i|^2 from the three sums
            // (c->count and c->norm_sq_sum are touched by the deciding thread of each launch only)
            c->norm_sq_sum += tot.ng;
            status |= ill_conditioned(c->count, c->norm_sq_sum, tot.na + 2.0 * tot.p + tot.ng);
        }
        if (status) atomicOr(&c->status, status);
        a.mask_out[a.i_next] = (uint8_t)accept;
        if (a.dist_out) a.dist_out[a.i_next] = (float)d;
        __threadfence();
    }
}

template <typename T, int MODE>
__global__ void __launch_bounds__(kStepThreads, 2) step_kernel(StepArgs a) {
    __shared__ double scratch[3 * (kStepThreads / 32)];
    const T *g_seed = static_cast<const T *>(a.g_seed);
    const T *g_cur = static_cast<const T *>(a.g_cur);
    const T *g_next = static_cast<const T *>(a.g_next);
    float *acc = a.acc;

    int accept = 0, count = 1;
    if (MODE == kMid || MODE == kLast) {
        // launched as a programmatic dependent of the previous step's launch: its blocks are placed
        // while that grid winds down, and wait here until it has completed and its decision is visible
        asm volatile("griddepcontrol.wait;" ::: "memory");
        accept = *reinterpret_cast<volatile int *>(&a.ctl->decision[a.t]);
        count = *reinterpret_cast<volatile int *>(&a.ctl->count);
    }
    if ((MODE == kFirst || MODE == kOnly) && blockIdx.x == 0 && threadIdx.x == 0) {
        // fresh call: c = 1, mask[s] = 1, dist[s] = 0, status cleared
        a.ctl->count = 1;
        a.ctl->status = 0;
        a.ctl->decision[0] = 1;
        a.mask_out[a.seed_index] = 1;
        if (a.dist_out) a.dist_out[a.seed_index] = 0.0f;
        if (MODE == kOnly) *a.count_out = 1;
    }
    const float inv_note = (float)count;   // Eq. 5 divides by c (true division below)

    Sums3 s = {0.0, 0.0, 0.0};
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    const int64_t n_oct = a.D / kOct;

    for (int64_t o = tid; o < n_oct; o += nthreads) {
        const int64_t e = o * kOct;
        float v[8], gc[8], gn[8];
        if (MODE == kFirst || MODE == kOnly) load8_stream<T>(g_seed, e, v);
        else load8_acc(acc, e, v);
        if (MODE == kFirst || MODE == kMid) load8_stream<T>(g_next, e, gn);
        if ((MODE == kMid || MODE == kLast) && accept) {
            load8_stream<T>(g_cur, e, gc);
#pragma unroll
            for (int k = 0; k < 8; ++k) v[k] += gc[k];
        }
        if (MODE == kLast) {
#pragma unroll
            for (int k = 0; k < 8; ++k) v[k] = v[k] / inv_note;
            store8(acc, e, v, true);
        } else if (MODE == kFirst || MODE == kOnly || accept) {
            store8(acc, e, v, MODE == kOnly);
        }
        if (MODE == kFirst || MODE == kMid) {
            s.p += (double)dot8(v, gn);
            s.na += (double)dot8(v, v);
            s.ng += (double)dot8(gn, gn);
        }
    }
    // ragged tail: D mod 8 elements, one per thread of the first CTA
    const int64_t tail0 = n_oct * kOct;
    if (blockIdx.x == 0 && tail0 + threadIdx.x < a.D) {
        const int64_t e = tail0 + threadIdx.x;
        float v = (MODE == kFirst || MODE == kOnly) ? load1<T>(g_seed, e) : acc[e];
        if ((MODE == kMid || MODE == kLast) && accept) v += load1<T>(g_cur, e);
        if (MODE == kLast) acc[e] = v / inv_note;
        else if (MODE == kFirst || MODE == kOnly || accept) acc[e] = v;
        if (MODE == kFirst || MODE == kMid) {
            float gn = load1<T>(g_next, e);
            s.p += (double)(v * gn);
            s.na += (double)(v * v);
            s.ng += (double)(gn * gn);
        }
    }

    if (MODE == kFirst || MODE == kMid) {
        // the streaming part of this CTA is over: the next step's launch may start placing blocks
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        Sums3 blk = block_reduce(s, scratch);
        finalize_step(a, blk, a.t + 1);
    } else if (MODE == kLast) {
        if (blockIdx.x == 0 && threadIdx.x == 0) *a.count_out = count;
    }
}

// ------------------------------------------------------- Eq. 4, two buffers --

struct CosArgs {
    const void *x, *y;
    int64_t D;
    Control *ctl;
    double *partials;
    float *dist_out;
    double *stats_out;      // may be null
};

template <typename T>
__global__ void __launch_bounds__(kStepThreads, 2) cosdist_kernel(CosArgs a) {
    __shared__ double scratch[3 * (kStepThreads / 32)];
    __shared__ bool is_last;
    const T *x = static_cast<const T *>(a.x);
    const T *y = static_cast<const T *>(a.y);
    // launched with programmatic stream serialisation by gaf_cosdist: nothing the launch before it on the stream
    // wrote is touched before that launch has completed (a no-op after an ordinary predecessor or launch)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (blockIdx.x == 0 && threadIdx.x == 0) a.ctl->status = 0;

    Sums3 s = {0.0, 0.0, 0.0};
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    const int64_t n_oct = a.D / kOct;
    for (int64_t o = tid; o < n_oct; o += nthreads) {
        float xv[8], yv[8];
        load8_stream<T>(x, o * kOct, xv);
        load8_stream<T>(y, o * kOct, yv);
        s.p += (double)dot8(xv, yv);
        s.na += (double)dot8(xv, xv);
        s.ng += (double)dot8(yv, yv);
    }
    const int64_t tail0 = n_oct * kOct;
    if (blockIdx.x == 0 && tail0 + threadIdx.x < a.D) {
        float xv = load1<T>(x, tail0 + threadIdx.x), yv = load1<T>(y, tail0 + threadIdx.x);
        s.p += (double)(xv * yv);
        s.na += (double)(xv * xv);
        s.ng += (double)(yv * yv);
    }
    // the streaming part of this CTA is over: the launch behind this one may be placed (it waits for this grid)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    Sums3 blk = block_reduce(s, scratch);
    if (threadIdx.x == 0) {
        a.partials[3 * blockIdx.x] = blk.p;
        a.partials[3 * blockIdx.x + 1] = blk.na;
        a.partials[3 * blockIdx.x + 2] = blk.ng;
        is_last = take_last_ticket(&a.ctl->ticket, gridDim.x);
    }
    __syncthreads();
    if (!is_last || threadIdx.x >= 32) return;
    Sums3 tot = warp_sum_partials(a.partials, gridDim.x);
    if (threadIdx.x == 0) {
        int status = 0;
        double d = cosine_distance(tot.p, tot.na, tot.ng, &status);
        *a.dist_out = (float)d;
        if (a.stats_out) { a.stats_out[0] = tot.p; a.stats_out[1] = tot.na; a.stats_out[2] = tot.ng; }
        if (status) atomicOr(&a.ctl->status, status);
    }
}

}  // namespace gaf
