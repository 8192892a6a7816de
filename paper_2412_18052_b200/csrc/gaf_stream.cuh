// Streaming form of Algorithm 1 for micro-gradients that arrive one at a time (as they
// do around a ring): begin(seed), push(g_1), push(g_2), ..., end().  Each push is Algorithm
// 1's loop body for one gradient: the three dot products against the running sum, Eq. 4,
// the test D_c <= tau on the device, and -- in a second launch that returns at once when
// the gradient was rejected -- g <- g + g_i.  The state (running count, decisions,
// distances) lives in the caller's workspace; the running sum is the caller's buffer.
// The arithmetic per element is that of the stepwise schedule, so the result is
// bit-identical to gaf_filter_accumulate on the same gradients in arrival order.
#pragma once

#include "gaf_device.cuh"

namespace gaf {

constexpr int kStreamThreads = 512;

struct StreamArgs {
    const void *g;          // the arriving gradient
    float *acc;             // running sum
    int64_t D;
    Control *ctl;
    double *partials;
    double tau;
    int t;                  // arrival index, 1 .. GAF_MAX_K-1 (0 is the seed)
};

// Three dot products of (running sum, g); the last CTA decides step t.
template <typename T>
__global__ void __launch_bounds__(kStreamThreads, 2) stream_test_kernel(StreamArgs a) {
    __shared__ double scratch[3 * (kStreamThreads / 32)];
    __shared__ bool is_last;
    const T *g = static_cast<const T *>(a.g);
    Sums3 s = {0.0, 0.0, 0.0};
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    const int64_t n_oct = a.D / kOct;
    for (int64_t o = tid; o < n_oct; o += nthreads) {
        float v[8], x[8];
        load8_acc(a.acc, o * kOct, v);
        load8_stream<T>(g, o * kOct, x);
        s.p += (double)dot8(v, x);
        s.na += (double)dot8(v, v);
        s.ng += (double)dot8(x, x);
    }
    const int64_t tail0 = n_oct * kOct;
    if (blockIdx.x == 0 && tail0 + threadIdx.x < a.D) {
        const float v = a.acc[tail0 + threadIdx.x], x = load1<T>(g, tail0 + threadIdx.x);
        s.p += (double)(v * x);
        s.na += (double)(v * v);
        s.ng += (double)(x * x);
    }
    // the streaming part of this CTA is over: the add launch may start placing blocks
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
        const double d = cosine_distance(tot.p, tot.na, tot.ng, &status);
        const int accept = (d <= a.tau) ? 1 : 0;
        Control *c = a.ctl;
        c->decision[a.t] = accept;
        c->sums[a.t][0] = tot.p; c->sums[a.t][1] = tot.na; c->sums[a.t][2] = tot.ng;
        c->stream_mask[a.t] = (uint8_t)accept;
        c->stream_dist[a.t] = (float)d;
        c->count += accept;
        if (a.t == 1) c->norm_sq_sum = tot.na;              // the running sum is still the seed alone
        if (accept) {
            c->norm_sq_sum += tot.ng;
            status |= ill_conditioned(c->count, c->norm_sq_sum, tot.na + 2.0 * tot.p + tot.ng);
        }
        if (status) atomicOr(&c->status, status);
        __threadfence();
    }
}

// g <- g + g_i if step t was accepted.
template <typename T>
__global__ void __launch_bounds__(kStreamThreads, 2) stream_add_kernel(StreamArgs a) {
    // launched as a programmatic dependent of the test: placed while that grid winds down, it waits
    // here until the test has completed and its decision is visible
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (*reinterpret_cast<volatile int *>(&a.ctl->decision[a.t]) == 0) return;
    const T *g = static_cast<const T *>(a.g);
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    const int64_t n_oct = a.D / kOct;
    for (int64_t o = tid; o < n_oct; o += nthreads) {
        float v[8], x[8];
        load8_acc(a.acc, o * kOct, v);
        load8_stream<T>(g, o * kOct, x);
#pragma unroll
        for (int k = 0; k < 8; ++k) v[k] += x[k];
        store8(a.acc, o * kOct, v, false);
    }
    const int64_t tail0 = n_oct * kOct;
    if (blockIdx.x == 0 && tail0 + threadIdx.x < a.D)
        a.acc[tail0 + threadIdx.x] += load1<T>(g, tail0 + threadIdx.x);
}

struct StreamEndArgs {
    float *acc;             // in: running sum; out: g / c (Eq. 5)
    int64_t D;
    int K;                  // gradients seen, seed included
    const Control *ctl;
    uint8_t *mask_out;      // K bytes, arrival order
    float *dist_out;        // K floats or null
    int32_t *count_out;
};

__global__ void __launch_bounds__(kStreamThreads, 2) stream_end_kernel(StreamEndArgs a) {
    const int count = *reinterpret_cast<const volatile int *>(&a.ctl->count);
    const float cdiv = (float)count;
    if (blockIdx.x == 0) {
        for (int t = threadIdx.x; t < a.K; t += blockDim.x) {
            a.mask_out[t] = t == 0 ? (uint8_t)1 : a.ctl->stream_mask[t];
            if (a.dist_out) a.dist_out[t] = t == 0 ? 0.0f : a.ctl->stream_dist[t];
        }
        if (threadIdx.x == 0) *a.count_out = count;
    }
    if (count == 1) return;                 // g / 1: nothing to do
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    const int64_t n_oct = a.D / kOct;
    for (int64_t o = tid; o < n_oct; o += nthreads) {
        float v[8];
        load8_acc(a.acc, o * kOct, v);
#pragma unroll
        for (int k = 0; k < 8; ++k) v[k] = v[k] / cdiv;
        store8(a.acc, o * kOct, v, true);
    }
    const int64_t tail0 = n_oct * kOct;
    if (blockIdx.x == 0 && tail0 + threadIdx.x < a.D) a.acc[tail0 + threadIdx.x] /= cdiv;
}

}  // namespace gaf
