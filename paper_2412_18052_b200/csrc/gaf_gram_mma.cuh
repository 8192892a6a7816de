// One-pass Gram matrix of up to 8 bfloat16 micro-gradients on the warp-level tensor-core path
// (mma.sync m16n8k16, bf16 x bf16 -> binary32).
//
// Why: with bfloat16 inputs the register-tiled CUDA-core kernel needs 36 multiply-adds plus the
// widening of every element per 16 bytes read and runs the binary32 pipes close to half busy;
// the 128 x 128 tcgen05 tile of gaf_gram_tc.cuh, built for 9..64 gradients, keeps only its
// diagonal 8 x 8 blocks with 8 gradients (1/16 of its work).  Both cost power, and under the
// power cap clock, on vectors long enough to matter.  One m16n8k16 MMA per 16 elements does the
// whole 8 x 8 block with half of its rows used, and its operands come straight from the 16-byte
// global loads: no shared-memory staging, no widening.
//
// Mapping.  G = X X^T with A[i][k] = X[i][d_k] (16 x 16, rows 8..15 zero) and B[k][j] = X[j][d_k]
// (16 x 8).  In the m16n8k16 fragment layout lane (g, t) = (lane / 4, lane % 4) supplies row g of A at
// columns {2t, 2t+1} and {2t+8, 2t+9}, and column g of B at the same k -- the same two registers.  The
// order of k inside one MMA does not matter as long as A and B agree, so lane (g, t) simply loads
// 16 bytes (8 elements) of gradient g at element offset 8 t of the warp's 32-element chunk and feeds
// them as two MMAs.  Lane (g, t) ends up with G[g][2t], G[g][2t+1]: the 32 lanes hold the whole 8 x 8
// matrix.  With fewer than 8 gradients the lanes of the absent rows load nothing and feed zeros.
//
// Sums: binary32 inside the tensor core over chains of at most kMmaChain MMAs (256 products), widened
// to binary64 registers after each chain; fixed-order sums from there on, like gram_small_kernel, whose
// tail (per-CTA partials, last-CTA totals, walk of Algorithm 1) this kernel shares.
#pragma once

#include "gaf_device.cuh"
#include "gaf_gramfilter.cuh"

namespace gaf {

constexpr int kMmaThreads = 512;        // as gram_small_kernel: the tail's fixed-order sums assume 16 warps
constexpr int kMmaChain = 16;           // MMAs accumulated in binary32 before widening (4 warp tiles)
constexpr int kMmaTileElems = 64;       // elements of every gradient one warp consumes per step (2 loads per lane)
constexpr int kMmaLongRun = 8;          // trips per run on long vectors (even); short vectors use 2

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], unsigned int a_lo, unsigned int a_hi) {
    // rows 8..15 of A are zero; B uses the same registers as A's rows 0..7
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%4, %6}, "
                 "{%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a_lo), "r"(0u), "r"(a_hi), "r"(0u));
}

template <int KT>
__global__ void __launch_bounds__(kMmaThreads, 2) gram_mma_kernel(const __grid_constant__ GramSmallArgs a) {
    static_assert(kMmaThreads == kGsThreads, "the shared tail sums 16 warps");
    constexpr int NP = KT * (KT + 1) / 2;
    __shared__ double sacc[kMmaThreads / 32][NP];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    if (blockIdx.x == 0 && threadIdx.x == 0) a.replay.ctl->status = 0;      // first kernel of the operation

    const bool have = g < KT;
    const unsigned short *rowp = static_cast<const unsigned short *>(a.g[have ? g : 0]);
    const uint64_t pol_first = l2_policy_evict_first(), pol_last = l2_policy_evict_last();
    const int64_t n_tiles = a.D / kMmaTileElems;
    float c[4] = {0.f, 0.f, 0.f, 0.f};
    double d0 = 0.0, d1 = 0.0;          // G[g][2t], G[g][2t+1]
    int chain = 0;
    // Tiles are dealt in runs: a CTA takes `run` consecutive trips' worth of tiles (run x 16 tiles, contiguous in
    // every gradient), then jumps ahead by the whole grid's share.  With run = 2 the grid reads one compact window
    // of every gradient at any moment, which is what short vectors want (every CTA has work).  On long vectors that
    // window moves on by a 2 MB page of every gradient per trip, each SM needs 8 fresh address translations per
    // trip, and the pass fell from 6.5 TB/s at 1.6 GB of inputs to 5.2 TB/s at 16 GB; with runs of 8 trips an SM
    // stays inside its pages four times longer and 16 GB stream at 6.6 TB/s.
    constexpr int kWarps = kMmaThreads / 32;
    const int run = a.mma_run;
    const int64_t cta_run_tiles = (int64_t)run * kWarps;                 // tiles of one run of one CTA
    const int64_t grid_run_tiles = cta_run_tiles * gridDim.x;            // tiles of one run of the whole grid
    for (int64_t base = (int64_t)blockIdx.x * cta_run_tiles; base < n_tiles; base += grid_run_tiles) {
        // two tiles per trip, all four loads issued before the first MMA (trip counts are the same for a warp's lanes)
        for (int rr = 0; rr < run; rr += 2) {
            const int64_t tile = base + (int64_t)rr * kWarps + warp, tile2 = tile + kWarps;
            if (tile >= n_tiles) break;
            const int64_t e0 = tile * kMmaTileElems + t * 8, e1 = tile2 * kMmaTileElems + t * 8;
            const bool second = tile2 < n_tiles;
            uint4 r[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) r[k] = make_uint4(0u, 0u, 0u, 0u);
            if (have) {
                const uint64_t p0 = (e0 >= a.keep_from) ? pol_last : pol_first;
                r[0] = ld16_policy(rowp + e0, p0);
                r[1] = ld16_policy(rowp + e0 + 32, p0);
                if (second) {
                    const uint64_t p1 = (e1 >= a.keep_from) ? pol_last : pol_first;
                    r[2] = ld16_policy(rowp + e1, p1);
                    r[3] = ld16_policy(rowp + e1 + 32, p1);
                }
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                mma_bf16_16816(c, r[k].x, r[k].y);
                mma_bf16_16816(c, r[k].z, r[k].w);
            }
            chain += 8;
            if (chain >= kMmaChain) {
                d0 += (double)c[0]; d1 += (double)c[1];
                c[0] = c[1] = c[2] = c[3] = 0.f;
                chain = 0;
            }
        }
    }
    d0 += (double)c[0]; d1 += (double)c[1];
    // the 8 x 8 matrix of this warp -> upper-triangle slots of sacc (row-major pair index)
    for (int p = lane; p < NP; p += 32) sacc[warp][p] = 0.0;
    __syncwarp();
    {
        const int i = g;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int j = 2 * t + h;
            if (i <= j && j < KT) sacc[warp][i * KT - i * (i - 1) / 2 + (j - i)] = h ? d1 : d0;
        }
    }
    // ragged end (D mod 64 elements), first CTA: one thread per pair, plain binary64 products
    const int64_t tail0 = n_tiles * kMmaTileElems;
    __syncthreads();
    if (blockIdx.x == 0 && (int)threadIdx.x < NP && tail0 < a.D) {
        int i = 0, rem = threadIdx.x;
        while (rem >= KT - i) { rem -= KT - i; ++i; }
        const int j = i + rem;
        const __nv_bfloat16 *xi = static_cast<const __nv_bfloat16 *>(a.g[i]), *xj = static_cast<const __nv_bfloat16 *>(a.g[j]);
        double s = 0.0;
        for (int64_t e = tail0; e < a.D; ++e) s += (double)load1<__nv_bfloat16>(xi, e) * (double)load1<__nv_bfloat16>(xj, e);
        sacc[0][threadIdx.x] += s;
    }
    gram_small_tail<KT>(a, sacc);
}

// ------------------------------------------------------------------------------------------------
// The same idea for 9..16 bfloat16 gradients: two blocks of 8 rows.  Lane (g, t) loads 8 elements of
// gradient g and of gradient g + 8 -- two loads of 16 bytes per 32-element chunk -- and those registers
// are at once the A fragment of the 16-row block (rows g and g + 8) and the B fragments of the two
// 8-column blocks.  Two 16 x 8 tiles cover the upper triangle: 4 MMAs per 32 elements, three quarters of
// whose work is kept, against one eighth for the 128 x 128 tcgen05 tile with 16 gradients.  No
// shared-memory staging, no barriers in the streaming loop.  Measured at D = 11.2 M: 54 / 58 / 64 us with
// 9 / 12 / 16 gradients against 64 / 69 / 74 us on the tcgen05 kernel.  The form with 3 and 4 row blocks
// (up to 32 gradients, 12 MMAs per 32 elements) was built and measured as well: 210 us against 145 us at 32
// gradients -- the warp-level MMA rate of this GPU (about 150 TFLOP/s here) is what 32 gradients need at
// HBM speed, so from 17 gradients on the tcgen05 tile stays.
// Per-CTA partial sums go out in the [tile pair][slice][64] layout of the tiled Gram kernels
// (gaf_pairwise.cuh), so gram_finish_kernel totals them.

struct GramWideArgs {
    const void *g[16];
    int K;
    int64_t D;
    int64_t keep_from;
    double *partials;           // [tile pair][slice][64]
    Control *ctl;
    int run;                    // tiles per warp a CTA takes in a row (even)
};

constexpr int kWideThreads = 512;
constexpr int kWideMaxK = 16;

__device__ __forceinline__ void mma_bf16_16816_full(float (&c)[4], unsigned int a0, unsigned int a1, unsigned int a2,
                                                    unsigned int a3, unsigned int b0, unsigned int b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                 "{%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__global__ void __launch_bounds__(kWideThreads, 2) gram_mma_wide_kernel(const __grid_constant__ GramWideArgs a) {
    constexpr int NB = 2;                           // blocks of 8 rows
    constexpr int NT = 2;                           // 16 x 8 tiles: columns 0..7 and 8..15
    extern __shared__ double wide_red[];            // [warp][tile][lane][4] at the end
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    if (blockIdx.x == 0 && threadIdx.x == 0) a.ctl->status = 0;            // first kernel of the operation

    const unsigned short *rowp[NB];
    bool have[NB];
#pragma unroll
    for (int m = 0; m < NB; ++m) {
        have[m] = g + 8 * m < a.K;
        rowp[m] = static_cast<const unsigned short *>(a.g[have[m] ? g + 8 * m : 0]);
    }
    const uint64_t pol_first = l2_policy_evict_first(), pol_last = l2_policy_evict_last();
    const int64_t n_tiles = a.D / kMmaTileElems;
    float c[NT][4];
    double d[NT][4];
#pragma unroll
    for (int i = 0; i < NT; ++i)
#pragma unroll
        for (int k = 0; k < 4; ++k) { c[i][k] = 0.f; d[i][k] = 0.0; }
    int chain = 0;
    constexpr int kWarps = kWideThreads / 32;
    const int run = a.run;
    const int64_t cta_run_tiles = (int64_t)run * kWarps, grid_run_tiles = cta_run_tiles * gridDim.x;
    for (int64_t base = (int64_t)blockIdx.x * cta_run_tiles; base < n_tiles; base += grid_run_tiles) {
        for (int rr = 0; rr < run; ++rr) {
            const int64_t tile = base + (int64_t)rr * kWarps + warp;
            if (tile >= n_tiles) break;
            // one tile of 64 elements: two chunks of 32, all 2 NB loads issued before the first MMA
            const int64_t e0 = tile * kMmaTileElems + t * 8;
            const uint64_t pol = (e0 >= a.keep_from) ? pol_last : pol_first;
            uint4 r[2][NB];
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int m = 0; m < NB; ++m)
                    r[h][m] = have[m] ? ld16_policy(rowp[m] + e0 + 32 * h, pol) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    unsigned int lo[NB], hi[NB];
#pragma unroll
                    for (int m = 0; m < NB; ++m) {
                        lo[m] = half ? r[h][m].z : r[h][m].x;
                        hi[m] = half ? r[h][m].w : r[h][m].y;
                    }
#pragma unroll
                    for (int cb = 0; cb < NB; ++cb)
                        mma_bf16_16816_full(c[cb], lo[0], lo[1], hi[0], hi[1], lo[cb], hi[cb]);
                }
            chain += 4;
            if (chain >= kMmaChain) {
#pragma unroll
                for (int i = 0; i < NT; ++i)
#pragma unroll
                    for (int k = 0; k < 4; ++k) { d[i][k] += (double)c[i][k]; c[i][k] = 0.f; }
                chain = 0;
            }
        }
    }
    // the streaming part of this CTA is over: the finishing kernel may be placed (it waits for this grid)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
#pragma unroll
    for (int i = 0; i < NT; ++i)
#pragma unroll
        for (int k = 0; k < 4; ++k) wide_red[((size_t)(warp * NT + i) * 32 + lane) * 4 + k] = d[i][k] + (double)c[i][k];
    __syncthreads();
    const int tiles8 = NB;                           // 8 x 8 blocks per side
    for (int e = threadIdx.x; e < NT * 128; e += kWideThreads) {
        // the 16 warps in a fixed order
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) s += wide_red[(size_t)w * NT * 128 + e];
        const int cb = e >> 7, ln = (e >> 2) & 31, k = e & 3;
        const int bi = k >> 1, bj = cb;                                   // 8 x 8 block, row and column inside it:
        const int row = ln >> 2, col = 2 * (ln & 3) + (k & 1);
        if (bi > bj || bi >= tiles8) continue;                            // below the diagonal: not wanted
        int tp = 0;
        for (int q = 0; q < bi; ++q) tp += tiles8 - q;
        tp += bj - bi;
        a.partials[((size_t)tp * gridDim.x + blockIdx.x) * 64 + row * 8 + col] = s;
    }
    // ragged end (D mod 64 elements), first CTA: plain binary64 products, added to its own slots
    const int64_t tail0 = n_tiles * kMmaTileElems;
    if (blockIdx.x == 0 && tail0 < a.D) {
        __syncthreads();
        for (int p = threadIdx.x; p < a.K * a.K; p += kWideThreads) {
            const int i = p / a.K, j = p % a.K;
            if (i > j) continue;
            const __nv_bfloat16 *xi = static_cast<const __nv_bfloat16 *>(a.g[i]), *xj = static_cast<const __nv_bfloat16 *>(a.g[j]);
            double s = 0.0;
            for (int64_t e = tail0; e < a.D; ++e) s += (double)load1<__nv_bfloat16>(xi, e) * (double)load1<__nv_bfloat16>(xj, e);
            const int bi = i >> 3, bj = j >> 3;
            int tp = 0;
            for (int q = 0; q < bi; ++q) tp += tiles8 - q;
            tp += bj - bi;
            a.partials[((size_t)tp * gridDim.x + blockIdx.x) * 64 + (i & 7) * 8 + (j & 7)] += s;
        }
    }
}

}  // namespace gaf
