// Pairwise cosine-distance matrix (Eq. 4 for every pair of K micro-gradients):
// Gram matrix G = X X^T over D, then dist_ij = 1 - G_ij / (sqrt(G_ii) sqrt(G_jj)).
//
// What the Gram kernels for more than 8 gradients share (gaf_gram_panel.cuh on CUDA cores,
// gaf_gram_tc.cuh on tensor cores): the K x K matrix cut into 8 x 8 tiles of pairs, per-CTA
// binary64 partial sums in a [tile pair][slice][64] layout, and the finishing kernel that totals
// the slices in a fixed order and whose last CTA derives the distances.
#pragma once

#include "gaf_device.cuh"

namespace gaf {

constexpr int kGramTile = 8;
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

// Decode the linear upper-triangle tile index into (ti, tj), ti <= tj.
__device__ __forceinline__ void tile_pair(int idx, int tiles, int &ti, int &tj) {
    ti = 0;
    while (idx >= tiles - ti) { idx -= tiles - ti; ++ti; }
    tj = ti + idx;
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
    // a dependent of this launch may be placed now (it waits for this grid before it touches global memory)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
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
    __syncthreads();
    if (threadIdx.x == 0) is_last = take_last_ticket(&a.ctl->ticket, gridDim.x);
    __syncthreads();
    if (!is_last) return;
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
