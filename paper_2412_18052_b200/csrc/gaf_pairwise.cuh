// Pairwise cosine-distance matrix (Eq. 4 for every pair of K micro-gradients):
// Gram matrix G = X X^T over D, then dist_ij = 1 - G_ij / (sqrt(G_ii) sqrt(G_jj)).
//
// CUDA-core version: the K x K matrix is cut into 8 x 8 tiles of pairs; a CTA owns
// one tile (upper triangle only) and one slice of D, and every thread keeps the 64
// partial dot products of its tile in registers.  Binary32 accumulation runs over
// short chunks and is flushed into binary64 shared-memory accumulators; per-CTA
// partials are summed in a fixed order by a second kernel, whose last CTA derives
// the distances.
#pragma once

#include "gaf_device.cuh"

namespace gaf {

constexpr int kGramTile = 8;
constexpr int kGramThreads = 256;
constexpr int kGramFlushEvery = 64;     // inner iterations between binary64 flushes
constexpr int kGramMaxSlices = 296;     // most D-slices (CTAs along x)

struct GramArgs {
    const void *g[GAF_MAX_K];
    int K;
    int64_t D;
    int tiles;              // ceil(K / 8)
    double *partials;       // [tile_pair][slice][64]
    double *gram;           // [K][K]
    float *dist_out;        // [K][K]
    double *gram_out;       // [K][K] or null
    Control *ctl;
    int slices;
};

template <typename T>
__device__ __forceinline__ void load4(const T *base, int64_t e, float (&v)[4]);
template <>
__device__ __forceinline__ void load4<float>(const float *base, int64_t e, float (&v)[4]) {
    float4 a = __ldcs(reinterpret_cast<const float4 *>(base + e));
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
}
template <>
__device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16 *base, int64_t e, float (&v)[4]) {
    uint2 r = __ldcs(reinterpret_cast<const uint2 *>(base + e));
    v[0] = bf16_bits_to_float(r.x & 0xFFFFu); v[1] = __uint_as_float(r.x & 0xFFFF0000u);
    v[2] = bf16_bits_to_float(r.y & 0xFFFFu); v[3] = __uint_as_float(r.y & 0xFFFF0000u);
}

// Decode the linear upper-triangle tile index into (ti, tj), ti <= tj.
__device__ __forceinline__ void tile_pair(int idx, int tiles, int &ti, int &tj) {
    ti = 0;
    while (idx >= tiles - ti) { idx -= tiles - ti; ++ti; }
    tj = ti + idx;
}

template <typename T>
__global__ void __launch_bounds__(kGramThreads) gram_tile_kernel(GramArgs a) {
    __shared__ double sacc[kGramThreads / 32][kGramTile * kGramTile];
    int ti, tj;
    tile_pair(blockIdx.y, a.tiles, ti, tj);
    const bool diag = (ti == tj);
    const T *ri[kGramTile], *rj[kGramTile];
#pragma unroll
    for (int r = 0; r < kGramTile; ++r) {
        // rows past K alias the last valid row; their products are never read back
        int i = min(ti * kGramTile + r, a.K - 1), j = min(tj * kGramTile + r, a.K - 1);
        ri[r] = static_cast<const T *>(a.g[i]);
        rj[r] = static_cast<const T *>(a.g[j]);
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) a.ctl->status = 0;   // first kernel of the operation
    for (int p = lane; p < kGramTile * kGramTile; p += 32) sacc[warp][p] = 0.0;
    __syncwarp();

    float acc[kGramTile][kGramTile];
#pragma unroll
    for (int r = 0; r < kGramTile; ++r)
#pragma unroll
        for (int c = 0; c < kGramTile; ++c) acc[r][c] = 0.0f;

    auto flush = [&]() {
#pragma unroll
        for (int r = 0; r < kGramTile; ++r)
#pragma unroll
            for (int c = 0; c < kGramTile; ++c) {
                float v = acc[r][c];
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) v += __shfl_down_sync(0xFFFFFFFFu, v, d);
                if (lane == 0) sacc[warp][r * kGramTile + c] += (double)v;
                acc[r][c] = 0.0f;
            }
    };

    const int64_t n_quad = a.D / 4;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    int since_flush = 0;
    // warp-uniform trip count: the flush shuffles across the whole warp
    const int64_t warp_first = (int64_t)blockIdx.x * blockDim.x + (threadIdx.x & ~31);
    for (int64_t qw = warp_first; qw < n_quad; qw += stride) {
        const int64_t q = qw + lane;
        if (q < n_quad) {
            float xi[kGramTile][4], xj[kGramTile][4];
#pragma unroll
            for (int r = 0; r < kGramTile; ++r) load4<T>(ri[r], q * 4, xi[r]);
            if (!diag) {
#pragma unroll
                for (int r = 0; r < kGramTile; ++r) load4<T>(rj[r], q * 4, xj[r]);
            }
#pragma unroll
            for (int r = 0; r < kGramTile; ++r)
#pragma unroll
                for (int c = 0; c < kGramTile; ++c) {
                    if (diag && c < r) continue;
                    const float *y = diag ? xi[c] : xj[c];
                    float s = acc[r][c];
                    s = fmaf(xi[r][0], y[0], s); s = fmaf(xi[r][1], y[1], s);
                    s = fmaf(xi[r][2], y[2], s); s = fmaf(xi[r][3], y[3], s);
                    acc[r][c] = s;
                }
        }
        if (++since_flush == kGramFlushEvery) { flush(); since_flush = 0; }
    }
    // ragged tail (D mod 4 elements): lanes 0..2 of warp 0 in slice 0
    const int64_t tail0 = n_quad * 4;
    if (blockIdx.x == 0 && tail0 + threadIdx.x < a.D) {
        const int64_t e = tail0 + threadIdx.x;
        float xi[kGramTile], xj[kGramTile];
#pragma unroll
        for (int r = 0; r < kGramTile; ++r) { xi[r] = load1<T>(ri[r], e); xj[r] = load1<T>(rj[r], e); }
#pragma unroll
        for (int r = 0; r < kGramTile; ++r)
#pragma unroll
            for (int c = 0; c < kGramTile; ++c) acc[r][c] = fmaf(xi[r], xj[c], acc[r][c]);
    }
    flush();
    __syncthreads();
    if (threadIdx.x < kGramTile * kGramTile) {
        double s = 0.0;
        for (int w = 0; w < kGramThreads / 32; ++w) s += sacc[w][threadIdx.x];
        a.partials[((size_t)blockIdx.y * gridDim.x + blockIdx.x) * 64 + threadIdx.x] = s;
    }
}

// One CTA per tile pair: sums the slices in a fixed order, writes both triangles of
// the Gram matrix; the last CTA to finish turns the Gram matrix into distances.
constexpr int kFinishParts = 16;        // each entry's slices are summed in 16 independent chains
__global__ void __launch_bounds__(64 * kFinishParts) gram_finish_kernel(GramArgs a) {
    __shared__ double part[kFinishParts][64];
    __shared__ bool is_last;
    int ti, tj;
    tile_pair(blockIdx.x, a.tiles, ti, tj);
    const int p = threadIdx.x & 63, chain = threadIdx.x >> 6;
    // launched as a programmatic dependent of the Gram kernel: wait until that grid has completed
    // and its partial sums are visible (a no-op in an ordinary launch)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    {
        const int per = (a.slices + kFinishParts - 1) / kFinishParts;
        const int lo = chain * per, hi = min(a.slices, lo + per);
        double s = 0.0;
        const double *src = a.partials + (size_t)blockIdx.x * a.slices * 64 + p;
#pragma unroll 4
        for (int sl = lo; sl < hi; ++sl) s += __ldcg(src + (size_t)sl * 64);
        part[chain][p] = s;
    }
    __syncthreads();
    if (threadIdx.x < 64) {
        double s = 0.0;
#pragma unroll
        for (int c = 0; c < kFinishParts; ++c) s += part[c][p];
        int r = p / kGramTile, c = p % kGramTile;
        int i = ti * kGramTile + r, j = tj * kGramTile + c;
        if (i < a.K && j < a.K && i <= j) {
            a.gram[(size_t)i * a.K + j] = s;
            a.gram[(size_t)j * a.K + i] = s;
        }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned int old = atomicInc(&a.ctl->ticket, gridDim.x - 1);
        is_last = (old == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    const volatile double *G = a.gram;
    int status = 0;
    for (int idx = threadIdx.x; idx < a.K * a.K; idx += blockDim.x) {
        int i = idx / a.K, j = idx % a.K;
        double gii = G[(size_t)i * a.K + i], gjj = G[(size_t)j * a.K + j], gij = G[idx];
        double d;
        if (i == j && gii > 0.0) d = 0.0;
        else d = cosine_distance(gij, gii, gjj, &status);
        a.dist_out[idx] = (float)d;
        if (a.gram_out) a.gram_out[idx] = gij;
    }
    if (status) atomicOr(&a.ctl->status, status);
}

}  // namespace gaf
