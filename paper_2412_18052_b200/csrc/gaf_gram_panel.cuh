// Gram matrix G = X X^T for any number of gradients up to GAF_MAX_K and both input types, on
// CUDA cores, reading every gradient ONCE from HBM (the general path: binary32 with more than 8
// gradients; fewer go to the one-pass register-tiled kernel, bfloat16 with 9 to 64 to the tensor
// cores).
//
// The K x K matrix is cut into 8 x 8 tiles of pairs (upper triangle: P = T(T+1)/2 tile pairs for
// T = ceil(K/8)).  One CTA per SM streams panels of the D axis -- all K rows x one chunk of
// consecutive elements, at most 32 KB -- through a ring of five shared-memory stages filled by
// 16-byte cp.async copies (four panels, up to 128 KB, in flight per SM).  Every warp owns ONE tile
// pair for the whole kernel; with few tile pairs several warps share a pair and split each panel's
// steps between them.  Per step a lane reads two consecutive elements of the 8 + 8 rows of its pair
// out of shared memory (conflict-free) and updates the 64 partial dot products of the tile, kept in
// registers (36 on a diagonal tile).  With more than 12 tile pairs (K > 32) the pairs are split
// over gridDim.y groups of CTAs, each of which streams the whole panel.
// Binary32 accumulation runs over 64 products per accumulator, then the warp's sums go to
// binary64 in shared memory; at the end the warps of a pair are added in a fixed order and the
// tile's 64 binary64 partials are written in the [tile pair][slice][64] layout that
// gram_finish_kernel totals in a fixed order.
// Shared-memory reads bound this kernel (8 x 8 tiles give 4 multiply-adds per word read), not
// the FMA pipes.
#pragma once

#include "gaf_device.cuh"
#include "gaf_pairwise.cuh"

namespace gaf {

constexpr int kPanelStages = 5;
constexpr int kPanelMaxWarps = 12;          // warps per CTA (384 threads leave each 168 registers)
constexpr int kPanelFlushEvery = 32;        // steps of two products per accumulator between binary64 flushes

struct GramPanelArgs {
    const void *g[GAF_MAX_K];
    int K;
    int64_t D;
    int tiles;              // T = ceil(K / 8)
    int pairs;              // T (T + 1) / 2
    int pairs_per_cta;      // gridDim.y = ceil(pairs / pairs_per_cta)
    double *partials;       // [tile pair][slice][64]
    Control *ctl;
};

__device__ __forceinline__ void panel_cp_async16(void *dst_smem, const void *src, unsigned int src_bytes) {
    // copies the first src_bytes (0..16) bytes and zero-fills the rest of the 16
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((unsigned int)__cvta_generic_to_shared(dst_smem)),
                 "l"(src), "r"(src_bytes)
                 : "memory");
}
__device__ __forceinline__ void panel_cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void panel_cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <typename T> struct PanelLane;     // two consecutive elements of one row, as a lane reads them
template <> struct PanelLane<float> {
    static constexpr int kBytes = 8;
    static __device__ __forceinline__ void load(const unsigned char *p, float (&v)[2]) {
        const float2 x = *reinterpret_cast<const float2 *>(p);
        v[0] = x.x; v[1] = x.y;
    }
};
template <> struct PanelLane<__nv_bfloat16> {
    static constexpr int kBytes = 4;
    static __device__ __forceinline__ void load(const unsigned char *p, float (&v)[2]) {
        const unsigned int w = *reinterpret_cast<const unsigned int *>(p);
        v[0] = bf16_bits_to_float(w & 0xFFFFu); v[1] = __uint_as_float(w & 0xFFFF0000u);
    }
};

// SHIFT: bytes of one gradient in one panel = 16 << SHIFT; WPP: warps that share a tile pair.  Both
// are compile-time so that shared-memory addresses are immediates and a warp's steps unroll.
template <typename T, int SHIFT, int WPP>
__global__ void __launch_bounds__(kPanelMaxWarps * 32, 1) gram_panel_kernel(const __grid_constant__ GramPanelArgs a) {
    extern __shared__ uint4 panel_smem[];                       // [stage][8 T rows][row_bytes]
    __shared__ double wsum[kPanelMaxWarps][64];
    __shared__ const unsigned char *rowp[GAF_MAX_K];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nthreads = blockDim.x;
    constexpr int RB = 16 << SHIFT;
    const int rows_padded = a.tiles * 8;
    const size_t stage_bytes = (size_t)rows_padded * RB;
    unsigned char *smem = reinterpret_cast<unsigned char *>(panel_smem);

    if (blockIdx.x == 0 && blockIdx.y == 0 && tid == 0) a.ctl->status = 0;          // first kernel of the operation
    for (int i = tid; i < a.K; i += nthreads) rowp[i] = static_cast<const unsigned char *>(a.g[i]);
    for (int p = lane; p < 64; p += 32) wsum[warp][p] = 0.0;
    // rows of absent gradients (K not a multiple of 8) stay zero in every stage
    {
        const int absent_from = a.K * (RB / 16), per_stage = rows_padded * (RB / 16);
        for (int s = 0; s < kPanelStages; ++s)
            for (int i = absent_from + tid; i < per_stage; i += nthreads)
                panel_smem[(size_t)s * per_stage + i] = make_uint4(0, 0, 0, 0);
    }
    __syncthreads();

    // this warp's tile pair, and which of the pair's warps it is
    constexpr int wpp = WPP;
    const int pair_local = warp / wpp, sub = warp - pair_local * wpp;
    const int pair = blockIdx.y * a.pairs_per_cta + pair_local;
    const bool active = pair_local < a.pairs_per_cta && pair < a.pairs;
    int ti = 0, tj = 0;
    if (active) tile_pair(pair, a.tiles, ti, tj);
    const bool diag = ti == tj;

    float acc[8][8];
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[r][c] = 0.0f;
    // Warp-wide sums of the 64 accumulators by recursive halving: in the round with distance d a lane
    // keeps the half of its values chosen by its bit d, adding its partner's copy of that half, so
    // 62 shuffles (not 320) leave every lane with two complete sums, which it adds to the warp's
    // binary64 totals.  A fixed tree: results do not depend on timing.
    auto flush = [&]() {
        float v[64];
#pragma unroll
        for (int r = 0; r < 8; ++r)
#pragma unroll
            for (int c = 0; c < 8; ++c) { v[r * 8 + c] = acc[r][c]; acc[r][c] = 0.0f; }
#pragma unroll
        for (int d = 16, n = 32; d >= 1; d >>= 1, n >>= 1) {
            const bool upper = (lane & d) != 0;
#pragma unroll
            for (int i = 0; i < n; ++i) {
                const float send = upper ? v[i] : v[i + n];
                const float keep = upper ? v[i + n] : v[i];
                v[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, d);
            }
        }
        // lane bits 4..0 chose halves of 64, 32, 16, 8, 4: this lane holds entries idx and idx + 1
        const int idx = ((lane >> 4) & 1) * 32 + ((lane >> 3) & 1) * 16 + ((lane >> 2) & 1) * 8 +
                        ((lane >> 1) & 1) * 4 + (lane & 1) * 2;
        wsum[warp][idx] += (double)v[0];
        wsum[warp][idx + 1] += (double)v[1];
    };

    // panels are dealt round-robin to the CTAs of a group: at any moment the grid reads one
    // compact window of every gradient
    const int64_t chunk_elems = RB / (int)sizeof(T);
    const int64_t n_chunks = (a.D + chunk_elems - 1) / chunk_elems;
    const int64_t G = gridDim.x;
    const int n_mine = blockIdx.x < n_chunks ? (int)((n_chunks - blockIdx.x + G - 1) / G) : 0;
    constexpr int pieces_per_row = RB / 16;
    const int pieces = a.K * pieces_per_row;
    const int64_t total_bytes = a.D * (int64_t)sizeof(T);

    // Every panel has the same shape: which 16-byte pieces this thread copies, from where (relative to
    // the panel's first byte in the row) and to where (relative to the stage) is worked out once.
    constexpr int kMaxMine = 8;                         // pieces of one panel per thread (<= 2048 / 256)
    const unsigned char *src_rel[kMaxMine];
    int dst_rel[kMaxMine];
#pragma unroll
    for (int k = 0; k < kMaxMine; ++k) {
        const int p = tid + k * nthreads;
        src_rel[k] = nullptr;
        dst_rel[k] = 0;
        if (p < pieces) {
            const int row = p >> SHIFT, col = p & (pieces_per_row - 1);
            src_rel[k] = rowp[row] + col * 16;
            dst_rel[k] = row * RB + col * 16;
        }
    }
    auto issue = [&](int it) {
        if (it < n_mine) {
            unsigned char *stage = smem + (size_t)(it % kPanelStages) * stage_bytes;
            const int64_t byte0 = (blockIdx.x + (int64_t)it * G) * RB;             // offset of the panel in every row
            if (byte0 + RB <= total_bytes) {
#pragma unroll
                for (int k = 0; k < kMaxMine; ++k)
                    if (src_rel[k] != nullptr) panel_cp_async16(stage + dst_rel[k], src_rel[k] + byte0, 16u);
            } else {
                // ragged end of the vectors: copy what exists, zero-fill the rest of each piece
#pragma unroll
                for (int k = 0; k < kMaxMine; ++k)
                    if (src_rel[k] != nullptr) {
                        const int64_t left = total_bytes - byte0 - (dst_rel[k] & (RB - 1));
                        const unsigned int n = left >= 16 ? 16u : (left > 0 ? (unsigned int)left : 0u);
                        // (a piece wholly past the end reads nothing: any valid address will do)
                        panel_cp_async16(stage + dst_rel[k], n ? src_rel[k] + byte0 : src_rel[k] - (dst_rel[k] & (RB - 1)), n);
                    }
            }
        }
        panel_cp_async_commit();                                                    // (an empty group keeps the count in step)
    };

    constexpr int LB = PanelLane<T>::kBytes;
    constexpr int steps = RB / (32 * LB);
    static_assert(steps % WPP == 0, "a panel's steps divide evenly between the warps of a pair");
    int since_flush = 0;
    for (int it = 0; it < kPanelStages - 1; ++it) issue(it);
    for (int it = 0; it < n_mine; ++it) {
        panel_cp_async_wait<kPanelStages - 2>();        // this thread's copies of panel `it` have landed
        __syncthreads();                                // ... everybody's have, and panel it-1 is no longer read
        issue(it + kPanelStages - 1);                   // refills the stage of panel it-1
        if (active) {
            const unsigned char *stage = smem + (size_t)(it % kPanelStages) * stage_bytes;
            const unsigned char *bi = stage + (size_t)(ti * 8) * RB + lane * LB;
            const unsigned char *bj = stage + (size_t)(tj * 8) * RB + lane * LB;
#pragma unroll
            for (int s0 = 0; s0 < steps; s0 += wpp) {
                const int s = s0 + sub;
                float xi[8][2];
#pragma unroll
                for (int r = 0; r < 8; ++r) PanelLane<T>::load(bi + (size_t)r * RB + s * (32 * LB), xi[r]);
                if (diag) {
#pragma unroll
                    for (int r = 0; r < 8; ++r)
#pragma unroll
                        for (int c = r; c < 8; ++c)
                            acc[r][c] = fmaf(xi[r][1], xi[c][1], fmaf(xi[r][0], xi[c][0], acc[r][c]));
                } else {
                    float xj[8][2];
#pragma unroll
                    for (int r = 0; r < 8; ++r) PanelLane<T>::load(bj + (size_t)r * RB + s * (32 * LB), xj[r]);
#pragma unroll
                    for (int r = 0; r < 8; ++r)
#pragma unroll
                        for (int c = 0; c < 8; ++c)
                            acc[r][c] = fmaf(xi[r][1], xj[c][1], fmaf(xi[r][0], xj[c][0], acc[r][c]));
                }
                if (++since_flush == kPanelFlushEvery) { flush(); since_flush = 0; }
            }
        }
    }
    panel_cp_async_wait<0>();
    // the streaming part of this CTA is over: the finishing kernel may start placing its blocks
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (active) flush();
    __syncthreads();
    if (active && sub == 0) {
        // the pair's warps in a fixed order
        double v0 = 0.0, v1 = 0.0;
        for (int k = 0; k < wpp; ++k) { v0 += wsum[warp + k][lane]; v1 += wsum[warp + k][lane + 32]; }
        double *dst = a.partials + ((size_t)pair * gridDim.x + blockIdx.x) * 64;
        dst[lane] = v0;
        dst[lane + 32] = v1;
    }
}

}  // namespace gaf
