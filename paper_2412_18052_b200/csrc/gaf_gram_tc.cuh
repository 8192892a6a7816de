// Tensor-core Gram matrix for bfloat16 micro-gradients (K <= 64): G = X X^T with the
// D parameters as the contraction axis, on the 5th-generation tensor cores
// (tcgen05.mma, accumulators in tensor memory).
//
// Why tensor cores here: with K = 32 the Gram matrix needs 528 multiply-adds per
// 64 bytes read, about 107 TFLOP/s at HBM speed -- more than the binary32 pipes
// deliver, and a fraction of what the tensor pipes do.
//
// Shape of one MMA: the K gradients are too few to fill the 128 rows of a tile, so R =
// 128 / Kp different 64-element chunks of the D axis are stacked in the rows (Kp = K
// rounded up to 8, 16, 32 or 64).  The same shared-memory tile serves as both operands (A = B,
// both K-major, 128-byte swizzle), so D = A A^T is 128 x 128; the entries whose row and column
// hold the same chunk are R partial Gram matrices, the others mix different chunks and are
// ignored.  Two row orders, one per way of filling the tiles:
//   chunk-major     row c Kp + i = chunk c of gradient i: the partial Gram matrices are the R
//                   diagonal Kp x Kp blocks (16-byte-copy loaders);
//   gradient-major  row i R + c: R consecutive chunks of a gradient sit in consecutive rows, which
//                   is what one tensor copy of a {64 elements, R chunks, Kp gradients} box writes
//                   and lets it fetch R x 128 contiguous bytes per gradient; the partial Gram
//                   matrix of chunk c is then the entries (i R + c, j R + c), picked out of all
//                   128 columns by the epilogue.
//
// Pipeline per CTA (one CTA per SM; tiles of the D axis are dealt round-robin to the CTAs):
//   loaders    a ring of kTcStages tiles of 64 KB in swizzled shared memory, filled in one of two ways.
//              TMA form (the gradients are rows of one matrix: equal distances, multiples of 128
//              bytes, between their addresses): one thread of warp 4 issues one tensor copy
//              (cp.async.bulk.tensor) per 16 KB block, completing on the tile's mbarrier by byte
//              count; chunks past the end and gradients past K arrive as zeros, and the one block
//              that holds a ragged last chunk is fetched row by row through a second, element-
//              granular map.  Measured at 32 gradients: 0.120 ms against 0.134 ms with the 16-byte
//              copies at D = 11.2 M (6.0 TB/s), 1.27 against 1.41 ms at D = 124 M; a box of one chunk of
//              every gradient (128 contiguous bytes per gradient) ran at 3.7 TB/s only.
//              Otherwise warps 4-11 issue 16-byte cp.async copies, each thread's batch arriving on
//              the mbarrier by itself;
//   MMA warp   one thread issues the MMAs (16 per tile, K = 16 each) into one of two
//              128-column accumulator buffers in tensor memory and commits to mbarriers;
//   warps 0-3  epilogue: every kTcDrain tiles read the finished buffer with tcgen05.ld and
//              add it to binary64 registers (short binary32 accumulation chains only).
// A tile is kTcSub swizzle blocks (kTcSub x 64 elements per row): the issuing thread pays
// one barrier handshake per tile, which at one block per tile cost more than the MMAs.  Measured
// at 32 gradients, D = 11.2 M, in a long loop of calls: six tiles of two blocks 139-149 us, three tiles of
// four blocks 125-134 us (fewer, larger handshakes; 64 gradients: 289 -> 252 us).
// At the end the R chunk blocks are summed in a fixed order and the CTA writes its partial
// Gram matrix in the [tile pair][slice][64] layout of the CUDA-core version, so the same
// finishing kernel totals the slices.  Every wait is bounded.
#pragma once

#include <type_traits>

#include <cuda.h>        // CUtensorMap (the type only: the encoder is fetched from the driver at run time)

#include "gaf_device.cuh"

namespace gaf {

#ifndef GAF_TC_LOADER_WARPS
#define GAF_TC_LOADER_WARPS 8
#endif
#ifndef GAF_TC_STAGES
#define GAF_TC_STAGES 3
#endif
#ifndef GAF_TC_SUB
#define GAF_TC_SUB 4
#endif
constexpr int kTcLoaderWarps = GAF_TC_LOADER_WARPS;
constexpr int kTcLoaders = kTcLoaderWarps * 32;
constexpr int kTcStages = GAF_TC_STAGES;
constexpr int kTcSub = GAF_TC_SUB;              // 128-row x 128-byte swizzle blocks per tile (one handshake per tile)
constexpr int kTcBlockBytes = 128 * 128;        // one such block: 128 rows x 128 bytes
constexpr int kTcStageBytes = kTcSub * kTcBlockBytes;
constexpr int kTcDrain = 8 / kTcSub;            // tiles accumulated in tensor memory between drains (32 MMAs)
constexpr int kTcMaxK = 64;
constexpr int kTcTmemCols = 256;                // two accumulator buffers of 128 columns
constexpr unsigned int kTcSpinLimit = 1u << 19;       // attempts of up to ~2 us each
constexpr int kStatusTimeoutBit = 4;            // GAF_STATUS_TIMEOUT

struct GramTcArgs {
    const void *g[kTcMaxK];
    int K;                  // gradients
    int Kp;                 // 8, 16, 32 or 64
    int R;                  // tensor-copy form: chunks of D stacked in the 128 rows, floor(128 / K) (2..7)
    int box_k;              // tensor-copy form: gradients a box covers (K, or Kp when that stacks as many chunks)
    int64_t D;
    double *partials;       // [tile pair][slice][64]
    int tiles;              // ceil(K / 8)
    Control *ctl;
    unsigned int spin_limit;    // attempts (of up to ~2 us each) a wait makes before it gives up
    int test_extra_arrival;     // test hook, normally 0: the first tile's barrier expects one arrival more
                                // than will ever come, so that every wait of the pipeline runs out
};

// ----------------------------------------------------------------- PTX --------

__device__ __forceinline__ uint32_t tc_smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void tc_mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(tc_smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void tc_mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(tc_smem_u32(bar)) : "memory");
}
// One attempt at waiting for the phase with the given parity: the hardware suspends the
// thread until the phase completes or about `hint_ns` nanoseconds have passed, whichever is
// first, and wakes it at once on completion (unlike a sleep-and-poll loop, whose sleep
// granularity would be paid on every tile).
__device__ __forceinline__ bool tc_mbar_try(uint64_t *bar, uint32_t parity, uint32_t hint_ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(tc_smem_u32(bar)), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok != 0;
}
// Bounded wait: false when the limit ran out or another thread already gave up.
__device__ __forceinline__ bool tc_mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag,
                                             unsigned int limit) {
    for (unsigned int spin = 0; spin < limit; ++spin) {
        if (tc_mbar_try(bar, parity, 2000u)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
// The same for a whole warp: one lane polls (32 lanes polling one mbarrier are 32 serialised
// shared-memory operations per round), the others learn the outcome through the shuffle,
// which also orders their later accesses after the polling lane's acquire.
__device__ __forceinline__ bool tc_mbar_wait_warp(uint64_t *bar, uint32_t parity, volatile int *abort_flag,
                                                  unsigned int limit) {
    int ok = 1;
    if ((threadIdx.x & 31) == 0) ok = tc_mbar_wait(bar, parity, abort_flag, limit) ? 1 : 0;
    return __shfl_sync(0xFFFFFFFFu, ok, 0) != 0;
}
__device__ __forceinline__ void tc_cp_async16(uint32_t dst_smem, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_smem), "l"(src) : "memory");
}
// The same, reading only the first `src_bytes` (0..16) bytes and zero-filling the rest.
__device__ __forceinline__ void tc_cp_async16_zfill(uint32_t dst_smem, const void *src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst_smem), "l"(src), "r"(src_bytes) : "memory");
}
// Asynchronous arrival (counted among the barrier's expected arrivals) once all earlier
// cp.async copies of this thread have completed.
__device__ __forceinline__ void tc_cp_async_arrive(uint64_t *bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(tc_smem_u32(bar)) : "memory");
}
// One arrival that also announces `bytes` of asynchronous copies to come (the phase completes when both the
// arrivals and the bytes are in).
__device__ __forceinline__ void tc_mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(tc_smem_u32(bar)), "r"(bytes) : "memory");
}
// Tensor copy of one box of a two-dimensional tensor map into (swizzled) shared memory; x is the element
// coordinate along D (a multiple of 64 here, so the copy starts on a 128-byte boundary), y the first row.
__device__ __forceinline__ void tc_tma_load_2d(uint32_t dst_smem, const CUtensorMap *map, int32_t x, int32_t y,
                                               uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst_smem), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(tc_smem_u32(bar))
        : "memory");
}
// The same for a box of a three-dimensional map ({element, chunk, gradient}; x = 0 here).
__device__ __forceinline__ void tc_tma_load_3d(uint32_t dst_smem, const CUtensorMap *map, int32_t x, int32_t y, int32_t z,
                                               uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst_smem), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(tc_smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void tc_cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory operand descriptor: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);       // start address, 16-byte units
    d |= (uint64_t)1 << 16;                              // leading byte offset (unused with swizzle)
    d |= (uint64_t)(1024 >> 4) << 32;                    // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                              // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                              // 128-byte swizzle
    return d;
}
// Instruction descriptor: bf16 x bf16 -> f32, both operands K-major, M = 128, N = 128.
constexpr uint32_t kTcInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(kTcInstrDesc), "r"(accumulate)
        : "memory");
}
// All MMAs issued so far by this thread arrive on the barrier once they have completed.
__device__ __forceinline__ void tc_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(tc_smem_u32(bar))
                 : "memory");
}
// 32 lanes x 32 columns of 32-bit accumulators: thread = lane (row), registers = columns.
__device__ __forceinline__ void tc_tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

struct GramTcShared {
    uint64_t full[kTcStages];       // loaders -> MMA: tile landed
    uint64_t empty[kTcStages];      // MMA -> loaders: tile consumed
    uint64_t acc_full[2];           // MMA -> epilogue: accumulator buffer complete
    uint64_t acc_empty[2];          // epilogue -> MMA: accumulator buffer read out
    uint64_t drained;               // MMA thread, after a wait gave up: the MMAs it had issued are complete
    uint32_t tmem_base;
    volatile int abort_flag;
};

// WIDE: Kp = 64.  A row's diagonal block is then 64 columns wide, twice what one epilogue thread can
// carry in binary64 registers, so a second set of four epilogue warps (after the MMA warp; a warp reads
// the tensor-memory lanes 32 (warp mod 4) .. + 31) takes the upper 32 columns of each block.
//
// TMA: the tiles are filled by tensor copies, gradient-major rows (Kp is 32 or 64 then): `tmap` has the
// dimensions {64, D / 64, K} of bfloat16 and the box {64, R, K}, `tmap_row` the dimensions {D, K} and the box
// {64, 1}; both with the 128-byte swizzle and zero fill outside.  Otherwise neither map is touched.
// Threads of a launch: four epilogue warps, the loader warps (one with tensor copies), the MMA warp, and four
// more epilogue warps for 33..64 gradients.
__host__ __device__ constexpr int tc_mma_warp(bool tma) { return 4 + (tma ? 1 : kTcLoaderWarps); }
__host__ __device__ constexpr int tc_threads(bool wide, bool tma) { return (tc_mma_warp(tma) + 1) * 32 + (wide ? 128 : 0); }

// GM: gradient-major rows (always with tensor copies; with 16-byte copies up to 42 gradients, where they stack more
// chunks than the padded chunk-major order).
template <bool WIDE, bool TMA, bool GM>
__global__ void __launch_bounds__(tc_threads(WIDE, TMA), 1)
gram_tc_kernel(const __grid_constant__ GramTcArgs a, const __grid_constant__ CUtensorMap tmap,
               const __grid_constant__ CUtensorMap tmap_row) {
    constexpr int kThreads = tc_threads(WIDE, TMA);
    constexpr int kMmaWarp = tc_mma_warp(TMA);
    extern __shared__ unsigned char tc_dyn_smem[];
    __shared__ GramTcShared sh;

    // tiles must start on a 1024-byte boundary (swizzle atom)
    unsigned char *tiles = reinterpret_cast<unsigned char *>(
        (reinterpret_cast<uintptr_t>(tc_dyn_smem) + 1023) & ~uintptr_t(1023));
    const uint32_t tiles_u32 = tc_smem_u32(tiles);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Chunks of D stacked in the rows.  The 16-byte-copy form pads the gradients to Kp, so that a chunk's partial
    // Gram matrix is a diagonal block; the tensor-copy form needs no such padding (its epilogue picks single
    // columns) and stacks as many chunks as fit: 7 with 17 or 18 gradients, 3 with 33 to 42.
    static_assert(GM || !TMA, "tensor copies write gradient-major rows");
    const int K = a.K, Kp = a.Kp, R = GM ? a.R : 128 / Kp;
    const int rows_filled = TMA ? a.box_k * R : K * R;     // gradient-major: rows that the copies write
    const int64_t unit = (int64_t)R * 64 * kTcSub;       // elements of D per tile and gradient
    // the last tile may be partial: its missing elements are zero-filled by the copies
    const int64_t n_units = (a.D + unit - 1) / unit;
    // tiles are dealt round-robin to the CTAs, so that at any moment the whole grid reads one
    // compact window of every gradient (DRAM row locality), not 148 far-apart places
    const int64_t G = gridDim.x;
    const int n_tiles = (int)((n_units - blockIdx.x + G - 1) / G);
    const int n_blocks = (n_tiles + kTcDrain - 1) / kTcDrain;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kTcStages; ++s) {
            // every loader thread arrives (TMA form: the issuing thread, plus the tile's bytes)
            tc_mbar_init(&sh.full[s], (TMA ? 1 : kTcLoaders) + ((s == 0 && a.test_extra_arrival) ? 1 : 0));
            tc_mbar_init(&sh.empty[s], 1);               // one commit
        }
        for (int b = 0; b < 2; ++b) {
            tc_mbar_init(&sh.acc_full[b], 1);
            tc_mbar_init(&sh.acc_empty[b], WIDE ? 256 : 128);    // every epilogue thread arrives
        }
        tc_mbar_init(&sh.drained, 1);
        sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // rows that no copy ever writes stay zero for the whole kernel: those of absent gradients (K < Kp), or, with
    // tensor copies, the rows past the K R that a box fills
    if (GM ? rows_filled < 128 : K < Kp) {
        for (int idx = threadIdx.x; idx < kTcStages * kTcSub * 128 * 8; idx += kThreads) {
            const int row = (idx >> 3) & 127;
            if (GM ? row >= rows_filled : (row % Kp) >= K) reinterpret_cast<uint4 *>(tiles)[idx] = make_uint4(0, 0, 0, 0);
        }
        tc_fence_async_smem();
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc_smem_u32(&sh.tmem_base)),
                     "r"(kTcTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = sh.tmem_base;
    // Everything above touched only this CTA's shared and tensor memory.  The kernel is launched as a programmatic
    // dependent of its predecessor on the stream: wait for that grid (its results, and its last reads of the
    // workspace) before the first access to global memory.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (blockIdx.x == 0 && threadIdx.x == 0) a.ctl->status = 0;      // first kernel of the operation

    // epilogue warps: which 32 rows (tensor-memory lanes) and which 32 columns of them this warp reads --
    // the columns that hold the rows' diagonal block(s): the 32 on the diagonal, or one half of the 64
    // (gradient-major rows: the first of all 128 columns, or of the half that holds this warp set's 32 gradients)
    const int epi_q = warp & 3;
    const int epi_col0 = GM ? ((WIDE && warp > kMmaWarp) ? 64 : 0)
                             : (WIDE ? (epi_q >> 1) * 64 + (warp > kMmaWarp ? 32 : 0) : epi_q * 32);
    double gsum[32];                                     // epilogue: this row's 32 loaded columns
#pragma unroll
    for (int j = 0; j < 32; ++j) gsum[j] = 0.0;

    if (TMA && warp >= 4 && warp < kMmaWarp) {
        // ------------------------------------------------------ loader (tensor copies) ----
        // (one warp; lane 0 does the handshakes and the block copies, all lanes share the row copies)
        {
            const int64_t full_chunks = a.D / 64;            // what the chunk-granular map covers
            const bool ragged = (a.D % 64) != 0;
            int issued = 0;
            for (int it = 0; it < n_tiles; ++it) {
                const int s = it % kTcStages;
                if (it >= kTcStages &&
                    !tc_mbar_wait_warp(&sh.empty[s], (uint32_t)((it / kTcStages - 1) & 1), &sh.abort_flag, a.spin_limit))
                    break;
                const int64_t elem0 = (blockIdx.x + it * G) * unit;   // first element of the tile, per gradient
                const uint32_t tile = tiles_u32 + (uint32_t)s * kTcStageBytes;
                if (lane == 0) tc_mbar_arrive_expect_tx(&sh.full[s], (uint32_t)(kTcSub * a.box_k * R * 128));
                __syncwarp();
                for (int b = 0; b < kTcSub; ++b) {
                    // block b: chunks chunk0 .. chunk0 + R - 1 of every gradient, row i R + c
                    const int64_t chunk0 = elem0 / 64 + (int64_t)b * R;
                    const uint32_t block = tile + (uint32_t)b * kTcBlockBytes;
                    if (!(ragged && chunk0 <= full_chunks && full_chunks < chunk0 + R)) {
                        if (lane == 0) tc_tma_load_3d(block, &tmap, 0, (int32_t)chunk0, 0, &sh.full[s]);
                    } else {
                        // the one block of the whole vector that holds the partial last chunk: row by row through
                        // the element-granular map, which fills what lies past D with zeros; the lanes issue
                        // up to four rows each (one thread issuing all of them took 5 us)
                        for (int row = lane; row < a.box_k * R; row += 32)
                            tc_tma_load_2d(block + (uint32_t)row * 128u, &tmap_row,
                                           (int32_t)((chunk0 + row % R) * 64), row / R, &sh.full[s]);
                    }
                }
                issued = it + 1;
            }
            // The last copies must have landed before the CTA leaves its shared memory to the next one, also when
            // a wait gave up somewhere and nobody consumes them (bounded like every wait; ignores the abort flag).
            if (lane == 0)
                for (int it = issued > kTcStages ? issued - kTcStages : 0; it < issued; ++it)
                    for (unsigned int spin = 0; spin < a.spin_limit; ++spin)
                        if (tc_mbar_try(&sh.full[it % kTcStages], (uint32_t)((it / kTcStages) & 1), 2000u)) break;
        }
        __syncwarp();
    } else if (warp >= 4 && warp < kMmaWarp) {
        // ------------------------------------------------------ loaders (16-byte copies) ----
        const int tl = threadIdx.x - 128;                // 0..kTcLoaders-1
        const int run = kTcSub * R * 8;                  // 16-byte pieces of one gradient in a tile (contiguous)
        const int pieces = K * run;                      // 16-byte pieces per tile
        // Every tile has the same shape: work out once which pieces this thread copies, from
        // where (relative to the tile's first element) and to which swizzled position.
        constexpr int kMaxMine = kTcStageBytes / 16 / kTcLoaders;
        const unsigned char *src_base[kMaxMine];
        uint32_t dst_off[kMaxMine];
        int rel_elem[kMaxMine];                          // element offset of the piece inside the tile
#pragma unroll
        for (int k = 0; k < kMaxMine; ++k) {
            const int p = tl + k * kTcLoaders;
            src_base[k] = nullptr;
            dst_off[k] = 0;
            rel_elem[k] = 0;
            if (p < pieces) {
                const int i = p / run, rem = p % run;
                const int q = rem >> 3, j = rem & 7;     // 64-element chunk within the run, piece within it
                const int blk = q / R, c = q % R;        // which swizzle block, which row group
                const int row = GM ? i * R + c : c * Kp + i;
                rel_elem[k] = q * 64 + j * 8;
                src_base[k] = static_cast<const unsigned char *>(a.g[i]) + (int64_t)rel_elem[k] * 2;
                dst_off[k] = (uint32_t)(blk * kTcBlockBytes + row * 128 + ((j ^ (row & 7)) << 4));
            }
        }
        for (int it = 0; it < n_tiles; ++it) {
            const int s = it % kTcStages;
            if (it >= kTcStages &&
                !tc_mbar_wait_warp(&sh.empty[s], (uint32_t)((it / kTcStages - 1) & 1), &sh.abort_flag, a.spin_limit))
                break;
            const int64_t elem0 = (blockIdx.x + it * G) * unit;       // first element of the tile, per gradient
            const int64_t byte0 = elem0 * 2;
            const uint32_t tile = tiles_u32 + (uint32_t)s * kTcStageBytes;
            if (elem0 + unit <= a.D) {
#pragma unroll
                for (int k = 0; k < kMaxMine; ++k)
                    if (src_base[k] != nullptr) tc_cp_async16(tile + dst_off[k], src_base[k] + byte0);
            } else {
                // ragged end of the vectors: copy what exists, zero-fill the rest of each piece
#pragma unroll
                for (int k = 0; k < kMaxMine; ++k)
                    if (src_base[k] != nullptr) {
                        const int64_t left = (a.D - elem0 - rel_elem[k]) * 2;         // bytes that exist from here on
                        const uint32_t n = left >= 16 ? 16u : (left > 0 ? (uint32_t)left : 0u);
                        // (a piece that lies wholly past the end reads nothing: point it at the buffer's start)
                        tc_cp_async16_zfill(tile + dst_off[k], n ? src_base[k] + byte0 : src_base[k] - (int64_t)rel_elem[k] * 2, n);
                    }
            }
            // arrives on the tile's barrier when this thread's copies above have landed
            tc_cp_async_arrive(&sh.full[s]);
        }
        tc_cp_async_wait_all();
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------ MMA issuer -----
        if (lane == 0) {
            for (int it = 0; it < n_tiles; ++it) {
                const int s = it % kTcStages;
                const int blk = it / kTcDrain, buf = blk & 1;
                const bool first_of_block = (it % kTcDrain) == 0;
                if (first_of_block && blk >= 2) {
                    // the epilogue must have read this buffer's previous contents
                    if (!tc_mbar_wait(&sh.acc_empty[buf], (uint32_t)((blk / 2 - 1) & 1), &sh.abort_flag, a.spin_limit)) break;
                }
                if (!tc_mbar_wait(&sh.full[s], (uint32_t)((it / kTcStages) & 1), &sh.abort_flag, a.spin_limit)) break;
                // a tile written by cp.async (generic proxy) is read by the MMA through the asynchronous
                // proxy: order the two before the first MMA of the tile (tensor copies are of that proxy already)
                if (!TMA) tc_fence_async_smem();
                tc_fence_after_sync();
#pragma unroll
                for (int b = 0; b < kTcSub; ++b) {
                    const uint64_t desc = tc_smem_desc(tiles_u32 + (uint32_t)s * kTcStageBytes + b * kTcBlockBytes);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        // 16 elements = 32 bytes further along K inside the swizzle atom
                        const uint64_t dk = desc + (uint64_t)(k * 2);
                        tc_mma(tmem_base + (uint32_t)buf * 128, dk, dk, (first_of_block && b == 0 && k == 0) ? 0u : 1u);
                    }
                }
                tc_commit(&sh.empty[s]);
                if ((it % kTcDrain) == kTcDrain - 1 || it == n_tiles - 1) tc_commit(&sh.acc_full[buf]);
            }
            // Tensor memory must not be freed under MMAs still in flight (a wait that gave up, here or in
            // another warp, skips the handshakes that normally guarantee it): one more commit arrives when
            // everything issued so far has completed.  Bounded like every wait; it ignores the abort flag.
            tc_commit(&sh.drained);
            for (unsigned int spin = 0; spin < a.spin_limit; ++spin)
                if (tc_mbar_try(&sh.drained, 0u, 2000u)) break;
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------ epilogue -------
        if constexpr (!GM) {
            for (int blk = 0; blk < n_blocks; ++blk) {
                const int buf = blk & 1;
                // (warp-uniform outcome: the load below needs the whole warp)
                if (!tc_mbar_wait_warp(&sh.acc_full[buf], (uint32_t)((blk / 2) & 1), &sh.abort_flag, a.spin_limit)) break;
                tc_fence_after_sync();
                uint32_t r[32];
                tc_tmem_ld32(tmem_base + ((uint32_t)(epi_q * 32) << 16) + (uint32_t)(buf * 128 + epi_col0), r);
                tc_fence_before_sync();
                tc_mbar_arrive(&sh.acc_empty[buf]);
#pragma unroll
                for (int j = 0; j < 32; ++j) gsum[j] += (double)__uint_as_float(r[j]);
            }
        } else {
            // Gradient-major rows: this row holds chunk c of its gradient, its Gram entries are the columns j R + c.
            // All 128 columns are read, 32 at a time, and every row keeps, per gradient j, the column of its own
            // chunk (one select per column; j and the column's chunk are compile-time), then adds those.  RR = R,
            // J0 = the first of the 32 gradients this warp set keeps.
            const int c = (epi_q * 32 + lane) % R;
            auto drain_all = [&](auto rr_tag, auto j0_tag, auto nj_tag) {
                // NJ: how many gradients, from J0 on, this warp set keeps (what is never indexed costs no register)
                constexpr int RR = decltype(rr_tag)::value, J0 = decltype(j0_tag)::value, NJ = decltype(nj_tag)::value;
                for (int blk = 0; blk < n_blocks; ++blk) {
                    const int buf = blk & 1;
                    if (!tc_mbar_wait_warp(&sh.acc_full[buf], (uint32_t)((blk / 2) & 1), &sh.abort_flag, a.spin_limit)) break;
                    tc_fence_after_sync();
                    const uint32_t taddr = tmem_base + ((uint32_t)(epi_q * 32) << 16) + (uint32_t)(buf * 128);
                    uint32_t sel[NJ];                        // the column of this row's chunk, per gradient
#pragma unroll
                    for (int j = 0; j < NJ; ++j) sel[j] = 0u;
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        // (a batch none of whose columns belongs to this warp set's gradients is not read)
                        if ((32 * t + 31) / RR < J0 || (32 * t) / RR >= J0 + NJ) continue;
                        uint32_t r[32];
                        tc_tmem_ld32(taddr + (uint32_t)(32 * t), r);
#pragma unroll
                        for (int n = 0; n < 32; ++n) {
                            const int col = 32 * t + n;
                            const int j = col / RR, cc = col % RR;
                            if (j >= J0 && j < J0 + NJ) sel[j - J0] = (cc == c) ? r[n] : sel[j - J0];
                        }
                    }
                    tc_fence_before_sync();
                    tc_mbar_arrive(&sh.acc_empty[buf]);
#pragma unroll
                    for (int j = 0; j < NJ; ++j) gsum[j] += (double)__uint_as_float(sel[j]);
                }
            };
            // (two chunks: up to 64 gradients, 32 per warp set; three: up to 42, 21 per set; four and more: one set)
            using std::integral_constant;
            typedef integral_constant<int, 0> I0;
            const bool upper = WIDE && warp > kMmaWarp;
            if constexpr (WIDE) {
                if (R == 2) {
                    if (!upper) drain_all(integral_constant<int, 2>(), I0(), integral_constant<int, 32>());
                    else drain_all(integral_constant<int, 2>(), integral_constant<int, 32>(), integral_constant<int, 32>());
                } else {
                    if (!upper) drain_all(integral_constant<int, 3>(), I0(), integral_constant<int, 21>());
                    else drain_all(integral_constant<int, 3>(), integral_constant<int, 21>(), integral_constant<int, 21>());
                }
            } else {
                switch (R) {
                    case 4: drain_all(integral_constant<int, 4>(), I0(), integral_constant<int, 32>()); break;
                    case 5: drain_all(integral_constant<int, 5>(), I0(), integral_constant<int, 25>()); break;
                    case 6: drain_all(integral_constant<int, 6>(), I0(), integral_constant<int, 21>()); break;
                    default: drain_all(integral_constant<int, 7>(), I0(), integral_constant<int, 18>()); break;
                }
            }
        }
    }

    // ---------------------------------------------- reduce the R chunk blocks ----
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTcTmemCols) : "memory");
    }
    if (sh.abort_flag) {
        if (threadIdx.x == 0) atomicOr(&a.ctl->status, kStatusTimeoutBit);
        return;
    }
    // the streaming part of this CTA is over: the finishing kernel, launched as a programmatic
    // dependent, may be placed now; it still waits for this whole grid before it reads the partials
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // the tile ring is idle now: reuse it as red[c][i][j] (R * Kp * Kp doubles, at most 96 KB)
    double *red = reinterpret_cast<double *>(tiles);
    if (warp < 4 || warp > kMmaWarp) {
        const int row = epi_q * 32 + lane;               // row of the 128 x 128 result
        if constexpr (GM) {
            const int i = row / R, c = row % R;
            // (the same split of the gradients between the warp sets as in the drain)
            const int per_set = WIDE ? (R == 2 ? 32 : 21) : 32;
            const int j0 = (WIDE && warp > kMmaWarp) ? per_set : 0;
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (j < per_set && j0 + j < Kp) red[((size_t)c * Kp + i) * Kp + j0 + j] = gsum[j];
        } else {
            const int c = row / Kp, i = row % Kp;
            const int off = c * Kp - epi_col0;           // where this chunk's block starts in the loaded columns
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const int jj = j - off;
                if (jj >= 0 && jj < Kp) red[((size_t)c * Kp + i) * Kp + jj] = gsum[j];
            }
        }
    }
    __syncthreads();
    const int slices = gridDim.x;
    for (int e = threadIdx.x; e < Kp * Kp; e += kThreads) {
        const int i = e / Kp, j = e % Kp;
        if (i > j || j >= K) continue;
        double s = 0.0;
        for (int c = 0; c < R; ++c) s += red[((size_t)c * Kp + i) * Kp + j];
        const int ti = i >> 3, tj = j >> 3;
        int tp = 0;
        for (int r = 0; r < ti; ++r) tp += a.tiles - r;
        tp += tj - ti;
        a.partials[((size_t)tp * slices + blockIdx.x) * 64 + (i & 7) * 8 + (j & 7)] = s;
    }
}

}  // namespace gaf
