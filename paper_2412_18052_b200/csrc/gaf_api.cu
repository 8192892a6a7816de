// Host side of the C ABI declared in include/gaf.h: argument checks, workspace
// carve-up and kernel launches.  No device memory is allocated here.
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>
#include <cstring>
#include <mutex>
#include <type_traits>

#include "../../include/gaf.h"
#include "gaf_bucketed.cuh"
#include "gaf_device.cuh"
#include "gaf_fused.cuh"
#include "gaf_gram_mma.cuh"
#include "gaf_gram_panel.cuh"
#include "gaf_gram_tc.cuh"
#include "gaf_gramfilter.cuh"
#include "gaf_host.h"
#include "gaf_pairwise.cuh"
#include "gaf_stepwise.cuh"
#include "gaf_stream.cuh"

namespace {

using namespace gaf;

thread_local int g_launches = 0;
thread_local int g_schedule = 0;       // what the latest gaf_filter_accumulate resolved AUTO to

// Test hook (gaf_test_set_wait_fault): poll limit and withheld signal for the next launches of this thread.
thread_local unsigned int g_test_wait_limit = 0;       // 0: the kernels' own limits
thread_local int g_test_withhold = 0;
thread_local int g_gram_loader = 0;    // tensor-memory Gram kernel of the latest call: 0 not used, 1 16-byte copies, 2 tensor copies

constexpr int kMaxDevices = 64;

struct DeviceInfo {
    int dev = 0;
    int sms = 0;
    int l2_bytes = 0;
    int smem_per_sm = 0;                // shared memory of one SM
    int smem_per_cta_max = 0;           // opt-in limit of one CTA
};

// What is worked out once per device and kept for the life of the process: the device's attributes and, per
// kernel instantiation, its launch plan (occupancy, shared-memory attributes, grid).  A call then costs
// argument checks and the launch itself: at a million elements the driver queries were a third of the call.
// Device memory is not involved; the tables are guarded by one mutex on their slow path only.
std::mutex g_plan_mutex;

// Runs `make(slot)` once per (table slot, device); afterwards the slot is read without the lock.
template <typename Plan, typename Make>
int plan_once(Plan &slot, std::atomic<int> &ready, Make &&make) {
    if (ready.load(std::memory_order_acquire)) return GAF_OK;
    std::lock_guard<std::mutex> lock(g_plan_mutex);
    if (ready.load(std::memory_order_relaxed)) return GAF_OK;
    if (int rc = make(slot)) return rc;             // nothing is remembered about a failure
    ready.store(1, std::memory_order_release);
    return GAF_OK;
}

struct DeviceSlot { DeviceInfo info; std::atomic<int> ready{0}; };
DeviceSlot g_devices[kMaxDevices];

// Attributes of the current device.
bool device_info(DeviceInfo *out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return false;
    DeviceSlot &slot = g_devices[dev];
    const int rc = plan_once(slot.info, slot.ready, [dev](DeviceInfo &d) {
        d.dev = dev;
        if (cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return GAF_ERR_CUDA;
        if (cudaDeviceGetAttribute(&d.l2_bytes, cudaDevAttrL2CacheSize, dev) != cudaSuccess) return GAF_ERR_CUDA;
        if (cudaDeviceGetAttribute(&d.smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev) != cudaSuccess)
            return GAF_ERR_CUDA;
        if (cudaDeviceGetAttribute(&d.smem_per_cta_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
            return GAF_ERR_CUDA;
        return d.sms > 0 ? GAF_OK : GAF_ERR_CUDA;
    });
    if (rc != GAF_OK) return false;
    *out = slot.info;
    return true;
}

// One slot per device for a kernel instantiation: `static PerDevice<Plan> table;` inside a function template
// gives every instantiation its own table.
template <typename Plan>
struct PerDevice {
    Plan plan[kMaxDevices];
    std::atomic<int> ready[kMaxDevices];
    PerDevice() { for (auto &r : ready) r.store(0, std::memory_order_relaxed); }
};
struct DynSmemPlan { int dyn = 0; };    // "the dynamic shared memory limit of this kernel has been raised"
struct OccPlan { int occ = 1; };
struct FusedPlan { int occ = 0, park = 0, dyn = 0; };

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t elem_bytes(int dtype) { return dtype == GAF_F32 ? 4 : 2; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Launch `kernel` as a programmatic dependent of the launch before it on the stream: its blocks may be
// placed while that grid winds down; the kernel itself waits (griddepcontrol.wait) for that grid.
template <typename... KArgs, typename... Args>
cudaError_t launch_dependent_smem(void (*kernel)(KArgs...), int grid, int threads, size_t dyn_smem, cudaStream_t st,
                                  const Args &...args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(threads); cfg.dynamicSmemBytes = dyn_smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}
template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), int grid, int threads, cudaStream_t st, const Args &...args) {
    return launch_dependent_smem(kernel, grid, threads, 0, st, args...);
}

// macro_out (D floats) must not overlap any input gradient.
bool overlaps_inputs(const float *macro_out, const void *const *grads, int K, int64_t D, int dtype) {
    const uintptr_t o0 = reinterpret_cast<uintptr_t>(macro_out), o1 = o0 + size_t(D) * 4;
    for (int i = 0; i < K; ++i) {
        const uintptr_t g0 = reinterpret_cast<uintptr_t>(grads[i]);
        const uintptr_t g1 = g0 + size_t(D) * elem_bytes(dtype);
        if (o0 < g1 && g0 < o1) return true;
    }
    return false;
}

// `order` (NULL = identity) must be a permutation of 0..K-1; copies it to `ord`.
bool read_order(const int32_t *order, int K, int32_t *ord) {
    bool seen[GAF_MAX_K] = {false};
    for (int t = 0; t < K; ++t) {
        const int32_t i = order ? order[t] : t;
        if (i < 0 || i >= K || seen[i]) return false;
        seen[i] = true;
        ord[t] = i;
    }
    return true;
}

// CTAs for a streaming kernel of `threads` threads that handles 8 elements per
// thread and iteration: two per SM, fewer when D is small.
int stream_grid(int64_t D, int threads, int sms) {
    int64_t need = (D / kOct + threads - 1) / threads;
    int64_t cap = int64_t(sms) * 2;
    if (cap > kMaxCtas) cap = kMaxCtas;
    if (need < 1) need = 1;
    return int(need < cap ? need : cap);
}

// Which Gram kernel.  The 128-row tcgen05 tile pays off from 9 bfloat16 gradients on.  Up to 8 the one-pass
// kernels for few gradients are faster at every length: with exactly 8, where the 128 x 128 product keeps 1/16 of
// its work, the warp-level MMA kernel streams 16 GB of inputs at 6.6 TB/s against 5.2 TB/s (measured).
constexpr int kPanelAutoMaxK = 32;
bool use_tensor_gram(int K, int64_t D, int dtype) {
    (void)D;
    return dtype == GAF_BF16 && K > kGsMaxK && K <= kTcMaxK;
}
bool use_small_gram(int K, int64_t D, int dtype) {
    return K >= 2 && K <= kGsMaxK && !use_tensor_gram(K, D, dtype);
}

// Layout after the per-CTA triples: Gram partials [tile pair][slice][64] doubles, the
// Gram matrix by original index, the Gram matrix by processing step, a K x K float
// scratch for distances nobody asked for.
size_t gram_partials_bytes(int K) {
    const int tiles = (K + kGramTile - 1) / kGramTile;
    const size_t pairs = size_t(tiles) * (tiles + 1) / 2;
    return pairs * kGramMaxSlices * 64 * sizeof(double);
}
size_t gram_matrix_bytes(int K) { return round_up(size_t(K) * K * sizeof(double), 256); }
// Bucketed variant: partial slots [ctas + buckets][64] doubles and one bit mask per bucket.
size_t bucketed_extra_bytes() {
    return size_t(kBkMaxCtas + kBkMaxBuckets) * 64 * sizeof(double) + size_t(kBkMaxBuckets) * 8;
}
size_t pairwise_extra_bytes(int K) {
    const size_t a = gram_partials_bytes(K) + 3 * gram_matrix_bytes(K), b = bucketed_extra_bytes();
    return a > b ? a : b;
}

// The driver's tensor-map encoder, fetched once through the runtime (the library does not link the driver).
using TensorMapEncodeFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                       const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                       CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
TensorMapEncodeFn tensor_map_encoder() {
    static std::atomic<void *> fn{nullptr};
    static std::atomic<int> tried{0};
    if (!tried.load(std::memory_order_acquire)) {
        std::lock_guard<std::mutex> lock(g_plan_mutex);
        if (!tried.load(std::memory_order_relaxed)) {
            void *p = nullptr;
            cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
            if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
                q != cudaDriverEntryPointSuccess)
                p = nullptr;
            cudaGetLastError();
            fn.store(p, std::memory_order_relaxed);
            tried.store(1, std::memory_order_release);
        }
    }
    return reinterpret_cast<TensorMapEncodeFn>(fn.load(std::memory_order_relaxed));
}

constexpr int kTcTensorCopyMaxWideK = 42;

#ifndef GAF_TC_L2_PROMOTION
#define GAF_TC_L2_PROMOTION CU_TENSOR_MAP_L2_PROMOTION_L2_128B
#endif

// The K bfloat16 gradients as one tensor for tensor copies: possible when they are rows of one matrix (equal,
// positive distances between their addresses, multiples of 128 bytes), at least one whole 64-element chunk long,
// and every element coordinate a tile can ask for fits 32 bits.  `tile_map` sees {64 elements, D / 64 chunks, K
// gradients} and copies boxes of {64, R, K}: R consecutive chunks (R x 128 contiguous bytes) of each gradient;
// `row_map` sees {D elements, K gradients} and copies one 64-element row at a time (the ragged last chunk).  Both
// with the 128-byte swizzle; what lies outside reads as zero.
bool stacked_tensor_maps(const void *const *grads, int K, int Kp, int R, int box_k, int64_t D, int64_t tile_elems,
                         CUtensorMap *tile_map, CUtensorMap *row_map) {
    if (K < 2 || Kp < 32 || D < 64 || !aligned16(grads[0])) return false;
    // From 43 gradients on only two chunks fit the 128 rows, a box then has 256 contiguous bytes per gradient, and
    // the copy engine's rate falls with the number of separate pieces: measured at D = 11.2 M against the 16-byte
    // copies, 228 / 240 / 252 us against 219 / 228 / 236 us at 44 / 48 / 52 gradients (three chunks, up to 42
    // gradients: 149 / 170 us against 204 / 224 us at 33 / 40).
    if (Kp == 64 && K > kTcTensorCopyMaxWideK) return false;
    const intptr_t base = reinterpret_cast<intptr_t>(grads[0]);
    const intptr_t stride = reinterpret_cast<intptr_t>(grads[1]) - base;
    if (stride < intptr_t(D) * 2 || (stride & 127) != 0 || stride >= (intptr_t(1) << 40)) return false;
    for (int i = 2; i < K; ++i)
        if (reinterpret_cast<intptr_t>(grads[i]) != base + intptr_t(i) * stride) return false;
    if (D + tile_elems >= (int64_t(1) << 31)) return false;
    const TensorMapEncodeFn encode = tensor_map_encoder();
    if (!encode) return false;
    void *const origin = const_cast<void *>(grads[0]);
    {
        const cuuint64_t dims[3] = {64u, cuuint64_t(D / 64), cuuint64_t(K)};
        const cuuint64_t strides[2] = {128u, cuuint64_t(stride)};
        const cuuint32_t box[3] = {64u, cuuint32_t(R), cuuint32_t(box_k)};
        const cuuint32_t elem_strides[3] = {1u, 1u, 1u};
        if (encode(tile_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, origin, dims, strides, box, elem_strides,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, GAF_TC_L2_PROMOTION,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return false;
    }
    const cuuint64_t dims[2] = {cuuint64_t(D), cuuint64_t(K)};
    const cuuint64_t strides[1] = {cuuint64_t(stride)};
    const cuuint32_t box[2] = {64u, 1u};
    const cuuint32_t elem_strides[2] = {1u, 1u};
    return encode(row_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, origin, dims, strides, box, elem_strides,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, GAF_TC_L2_PROMOTION,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tiled Gram matrix of K gradients (by original index) into the workspace; optional
// distance matrix.  Two launches.
int launch_gram_tiles(const void *const *grads, int K, int64_t D, int dtype, float *dist_out,
                      double *gram_out, unsigned char *base, const DeviceInfo &di, cudaStream_t st) {
    const int sms = di.sms;
    GramArgs a{};
    for (int i = 0; i < K; ++i) a.g[i] = grads[i];
    a.K = K; a.D = D;
    a.tiles = (K + kGramTile - 1) / kGramTile;
    const int pairs = a.tiles * (a.tiles + 1) / 2;
    a.partials = reinterpret_cast<double *>(base + kExtraOffset);
    a.gram = reinterpret_cast<double *>(base + kExtraOffset + gram_partials_bytes(K));
    a.dist_out = dist_out ? dist_out
                          : reinterpret_cast<float *>(base + kExtraOffset + gram_partials_bytes(K) +
                                                      2 * gram_matrix_bytes(K));
    a.gram_out = gram_out;
    a.ctl = reinterpret_cast<Control *>(base);
    if (use_tensor_gram(K, D, dtype) && K <= kWideMaxK) {
        // 9..16 bfloat16 gradients: warp-level MMAs fed straight from the global loads, two CTAs per SM
        GramWideArgs w{};
        for (int i = 0; i < K; ++i) w.g[i] = grads[i];
        w.K = K; w.D = D; w.keep_from = D; w.partials = a.partials; w.ctl = a.ctl;
        const int64_t per_cta = int64_t(kWideThreads / 32) * kMmaTileElems;      // elements per trip of one CTA
        int64_t grid = int64_t(sms) * 2;
        if (grid > kGramMaxSlices) grid = kGramMaxSlices;
        const int64_t work = (D + per_cta - 1) / per_cta;
        if (grid > work) grid = work;
        if (grid < 1) grid = 1;
        a.slices = int(grid);
        // runs of 8 trips per CTA on long vectors (address-translation locality), one trip at a time otherwise
        w.run = D >= int64_t(32) * kMmaLongRun * per_cta * grid ? kMmaLongRun : 1;
        void (*kernel)(GramWideArgs) = gram_mma_wide_kernel;
        const int dyn = (kWideThreads / 32) * 2 * 128 * int(sizeof(double));       // [warp][tile][lane][4] doubles: 32 KB
        kernel<<<int(grid), kWideThreads, dyn, st>>>(w);
        ++g_launches;
    } else if (use_tensor_gram(K, D, dtype)) {
        // tensor cores: one CTA per SM, each with a contiguous slice of D
        GramTcArgs t{};
        for (int i = 0; i < K; ++i) t.g[i] = grads[i];
        t.K = K; t.Kp = K <= 8 ? 8 : (K <= 16 ? 16 : (K <= 32 ? 32 : 64)); t.D = D;
        t.partials = a.partials; t.tiles = a.tiles; t.ctl = a.ctl;
        const int dyn = kTcStages * kTcStageBytes + 1024;
        // gradients that are rows of one matrix are fetched by tensor copies, any others by 16-byte copies
        alignas(64) CUtensorMap tmap, tmap_row;
        std::memset(&tmap, 0, sizeof tmap);
        std::memset(&tmap_row, 0, sizeof tmap_row);
        // (tensor copies stack floor(128 / K) chunks of D in the 128 rows, the 16-byte copies 128 / Kp)
        t.R = 128 / K;
        t.box_k = t.R == 128 / t.Kp ? t.Kp : K;
        const int64_t unit_tma = int64_t(t.R) * 64 * kTcSub;
        const bool tma = stacked_tensor_maps(grads, K, t.Kp, t.R, t.box_k, D, unit_tma, &tmap, &tmap_row);
        // the 16-byte copies write the same gradient-major rows where those stack more chunks per tile than the padded
        // order (17..25 and 33..42 gradients); elsewhere the padded order's epilogue is the cheaper one
        const bool gm = tma || 128 / K > 128 / t.Kp;
        if (!gm) t.R = 128 / t.Kp;
        const int64_t unit = int64_t(t.R) * 64 * kTcSub;   // elements of D per tile
        const int64_t units = (D + unit - 1) / unit;
        int64_t slices = sms < kGramMaxSlices ? sms : kGramMaxSlices;
        if (slices > units) slices = units;
        if (slices < 1) slices = 1;
        a.slices = int(slices);
        g_gram_loader = tma ? 2 : 1;
        void (*kernel)(GramTcArgs, CUtensorMap, CUtensorMap) =
            t.Kp == 64 ? (tma ? gram_tc_kernel<true, true, true>
                              : (gm ? gram_tc_kernel<true, false, true> : gram_tc_kernel<true, false, false>))
                       : (tma ? gram_tc_kernel<false, true, true>
                              : (gm ? gram_tc_kernel<false, false, true> : gram_tc_kernel<false, false, false>));
        {
            static PerDevice<DynSmemPlan> table[6];
            const int w = (t.Kp == 64 ? 1 : 0) + (tma ? 2 : 0) + (gm && !tma ? 4 : 0);
            if (int rc = plan_once(table[w].plan[di.dev], table[w].ready[di.dev], [&](DynSmemPlan &pl) {
                    pl.dyn = dyn;
                    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn) == cudaSuccess
                        ? GAF_OK : GAF_ERR_CUDA;
                }))
                return rc;
        }
        t.spin_limit = g_test_wait_limit ? g_test_wait_limit : kTcSpinLimit;
        t.test_extra_arrival = g_test_withhold;
        // (a programmatic dependent of whatever precedes it on the stream: barriers and tensor memory are set up
        // while that grid winds down, and the kernel waits for it before it touches global memory)
        const cudaError_t err = launch_dependent_smem(kernel, a.slices, tc_threads(t.Kp == 64, tma), size_t(dyn), st,
                                                      t, tmap, tmap_row);
        ++g_launches;
        if (err != cudaSuccess) { cudaGetLastError(); return GAF_ERR_CUDA; }
    } else {
        // CUDA cores, every gradient read once: one warp per tile pair, panels of D through shared memory
        GramPanelArgs pa{};
        for (int i = 0; i < K; ++i) pa.g[i] = grads[i];
        pa.K = K; pa.D = D; pa.tiles = a.tiles; pa.pairs = pairs;
        const int groups = (pairs + kPanelMaxWarps - 1) / kPanelMaxWarps;
        pa.pairs_per_cta = (pairs + groups - 1) / groups;
        // A panel is at most 32 KB: 2 KB of every row up to 16 (padded) rows, 1 KB up to 32, 512 bytes
        // beyond.  With 3 or 6 tile pairs, 4 or 2 warps share a pair.
        const int shift = a.tiles <= 2 ? 7 : (a.tiles <= 4 ? 6 : 5);
        const int wpp = a.tiles <= 2 ? 4 : (a.tiles == 3 ? 2 : 1);
        pa.partials = a.partials; pa.ctl = a.ctl;
        const int threads = 32 * pa.pairs_per_cta * wpp;
        const int row_bytes = 16 << shift;
        const int dyn = kPanelStages * a.tiles * 8 * row_bytes;
        // (bfloat16 comes here with a single gradient only: 2 to 8 take the register-tiled kernel, up to 64
        // the tensor cores)
        void (*kernel)(GramPanelArgs) = nullptr;
        if (dtype == GAF_F32)
            kernel = shift == 7 ? gram_panel_kernel<float, 7, 4>
                   : (shift == 6 ? (wpp == 2 ? gram_panel_kernel<float, 6, 2> : gram_panel_kernel<float, 6, 1>)
                                 : gram_panel_kernel<float, 5, 1>);
        else
            kernel = shift == 7 ? gram_panel_kernel<__nv_bfloat16, 7, 4>
                   : (shift == 6 ? (wpp == 2 ? gram_panel_kernel<__nv_bfloat16, 6, 2> : gram_panel_kernel<__nv_bfloat16, 6, 1>)
                                 : gram_panel_kernel<__nv_bfloat16, 5, 1>);
        {
            // (the kernel pointer is the key: six instantiations per input type)
            static PerDevice<DynSmemPlan> table[2][4];
            const int v = shift == 7 ? 0 : (shift == 6 ? (wpp == 2 ? 1 : 2) : 3);
            auto &tb = table[dtype == GAF_F32 ? 0 : 1][v];
            if (int rc = plan_once(tb.plan[di.dev], tb.ready[di.dev], [&](DynSmemPlan &pl) {
                    // the largest panel this instantiation is ever launched with
                    pl.dyn = kPanelStages * (shift == 7 ? 2 : (shift == 6 ? 4 : 8)) * 8 * row_bytes;
                    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.dyn) == cudaSuccess
                        ? GAF_OK : GAF_ERR_CUDA;
                }))
                return rc;
        }
        const int64_t chunk_elems = row_bytes / int64_t(elem_bytes(dtype));
        const int64_t work = (D + chunk_elems - 1) / chunk_elems;
        int64_t slices = sms < kGramMaxSlices ? sms : kGramMaxSlices;      // one CTA per SM
        if (slices > work) slices = work;
        if (slices < 1) slices = 1;
        a.slices = int(slices);
        kernel<<<dim3(a.slices, groups), threads, dyn, st>>>(pa);
        ++g_launches;
    }
    {
        // the finishing blocks are placed while the Gram kernel winds down
        const cudaError_t err = launch_dependent(gram_finish_kernel, pairs, 64 * kFinishParts, st, a);
        ++g_launches;
        if (err != cudaSuccess) { cudaGetLastError(); return GAF_ERR_CUDA; }
    }
    return cudaGetLastError() == cudaSuccess ? GAF_OK : GAF_ERR_CUDA;
}

template <typename T, int KT>
int launch_gram_small_kt(GramSmallArgs a, const DeviceInfo &di, cudaStream_t st) {
    // 7 or 8 bfloat16 gradients go through the warp-level tensor-core kernel (with fewer, the lanes of the
    // absent rows fetch nothing and too few bytes are in flight: measured slower than the register tile)
    constexpr bool kMma = std::is_same<T, __nv_bfloat16>::value && KT >= 7;
    void (*kernel)(GramSmallArgs) = nullptr;
    if constexpr (kMma) kernel = gram_mma_kernel<KT>;
    else kernel = gram_small_kernel<T, KT>;
    static PerDevice<OccPlan> table;
    plan_once(table.plan[di.dev], table.ready[di.dev], [kernel](OccPlan &pl) {
        int occ = 1;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, kGsThreads, 0) != cudaSuccess || occ < 1)
            occ = 1;
        pl.occ = occ > 2 ? 2 : occ;
        return GAF_OK;
    });
    const int occ = table.plan[di.dev].occ;
    int64_t grid = int64_t(di.sms) * occ;
    if (grid > kGsMaxCtas) grid = kGsMaxCtas;
    // elements one CTA consumes per trip of its loop
    const int64_t per_cta = kMma ? int64_t(kGsThreads / 32) * kMmaTileElems * 2 : int64_t(kGsThreads) * GsVec<T>::N;
    const int64_t work = (a.D + per_cta - 1) / per_cta;
    if (grid > work) grid = work;
    if (grid < 1) grid = 1;
    // long vectors: runs of several trips per CTA (address-translation locality), once every CTA gets
    // at least eight such runs; otherwise one trip at a time
    a.mma_run = (kMma && a.D >= int64_t(8) * kMmaLongRun / 2 * per_cta * grid) ? kMmaLongRun : 2;
    kernel<<<int(grid), kGsThreads, 0, st>>>(a);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? GAF_OK : GAF_ERR_CUDA;
}

template <typename T>
int launch_gram_small(const GramSmallArgs &a, int K, const DeviceInfo &di, cudaStream_t st) {
    switch (K) {
        case 2: return launch_gram_small_kt<T, 2>(a, di, st);
        case 3: return launch_gram_small_kt<T, 3>(a, di, st);
        case 4: return launch_gram_small_kt<T, 4>(a, di, st);
        case 5: return launch_gram_small_kt<T, 5>(a, di, st);
        case 6: return launch_gram_small_kt<T, 6>(a, di, st);
        case 7: return launch_gram_small_kt<T, 7>(a, di, st);
        case 8: return launch_gram_small_kt<T, 8>(a, di, st);
        default: return GAF_ERR_ARG;
    }
}

// One-launch form of the Gram-first schedule (gaf_fused.cuh).  Returns GAF_OK when it was
// launched, GAF_ERR_UNSUPPORTED when this device or K does not allow it, or an error code.
constexpr int kKeepL2Pct = 10;          // share of L2 the Gram pass asks to keep for the second pass
                                        // ("evict last" lines live in the persisting part of L2, 24.9 MB by
                                        // default on this GPU; larger shares slow both passes down)
// Shared memory of one SM given to parked rounds.  The rest of the L1/shared array stays L1, which the
// loads in flight need: beyond about 60 % shared memory both passes lose more than parking gains.
constexpr int kParkBytesPerSm = 128 << 10;
// AUTO takes the one-launch form for binary32 inputs up to this many bytes in all: beyond, what stays
// on chip between the passes is a negligible share and the two-launch form is as fast or slightly
// faster.  For bfloat16 with up to 6 gradients the one-launch form stays ahead at every length measured;
// with 7 or 8 the two-launch form on the warp-level MMA Gram kernel overtakes it near 1 GB of inputs.
constexpr int64_t kFusedMaxInputBytesF32 = int64_t(512) << 20;
constexpr int64_t kFusedMaxInputBytesBf16Mma = int64_t(1) << 30;

// A one-launch call needs the whole device: its CTAs wait for one another, so two such grids in flight at once
// (two streams) could each hold part of the SMs and wait for the rest until their bounded waits run out.  Calls on
// one stream are ordered and safe.  The library therefore remembers, per device, the stream of its latest
// one-launch call, and refuses another one on a DIFFERENT stream while that stream still has work pending
// (GAF_ERR_UNSUPPORTED: the library's own choice then takes the two-launch form, which has no such need).
struct FusedGuard {
    std::mutex m;
    cudaStream_t last = nullptr;
    bool any = false;
};
FusedGuard g_fused_guard[kMaxDevices];

template <typename T, int KT>
int launch_gram_fused_kt(GramFusedArgs &a, const DeviceInfo &di, cudaStream_t st) {
    auto kernel = gram_fused_kernel<T, KT>;
    // The plan of this instantiation on this device: CTAs per SM by registers alone, then as many parked
    // rounds as shared memory allows; the kernel's shared-memory attributes are set on the way.
    static PerDevice<FusedPlan> table;
    if (int rc = plan_once(table.plan[di.dev], table.ready[di.dev], [&](FusedPlan &pl) {
            int occ = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, kGsThreads, 0) != cudaSuccess || occ < 1)
                return GAF_ERR_UNSUPPORTED;
            if (occ > 2) occ = 2;
            cudaFuncAttributes fa{};
            if (cudaFuncGetAttributes(&fa, kernel) != cudaSuccess) return GAF_ERR_CUDA;
            const int round_bytes = KT * kGsThreads * 16;
            int64_t budget = di.smem_per_sm / occ - 1024 - int64_t(fa.sharedSizeBytes);
            if (budget > di.smem_per_cta_max - int64_t(fa.sharedSizeBytes))
                budget = di.smem_per_cta_max - int64_t(fa.sharedSizeBytes);
            if (budget > kParkBytesPerSm / occ) budget = kParkBytesPerSm / occ;
            const int park = budget > 0 ? int(budget / round_bytes) : 0;
            const int dyn = park * round_bytes;
            if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn) != cudaSuccess)
                return GAF_ERR_CUDA;
            // shared memory share of the L1/shared array: what the CTAs of one SM need, no more (the rest is L1)
            int pct = int((int64_t(dyn + fa.sharedSizeBytes + 1024) * occ * 100 + di.smem_per_sm - 1) / di.smem_per_sm);
            if (pct > 100) pct = 100;
            if (cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, pct) != cudaSuccess)
                return GAF_ERR_CUDA;
            int occ2 = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ2, kernel, kGsThreads, dyn) != cudaSuccess || occ2 < 1)
                return GAF_ERR_UNSUPPORTED;
            pl.occ = occ2 < occ ? occ2 : occ;
            pl.park = park;
            pl.dyn = dyn;
            return GAF_OK;
        }))
        return rc;
    const FusedPlan &pl = table.plan[di.dev];
    int64_t grid = int64_t(di.sms) * pl.occ;
    if (grid > kGsMaxCtas) grid = kGsMaxCtas;
    const int64_t work = (a.D / FusedVec<T>::N + kGsThreads - 1) / kGsThreads;
    if (grid > work) grid = work;
    if (grid < 1) grid = 1;
    a.park_rounds = pl.park;
    a.spin_limit = g_test_wait_limit ? g_test_wait_limit : kFusedSpinLimit;
    a.test_withhold = g_test_withhold;
    // the last stretch is asked to stay in L2 for the second pass
    const int64_t per_elem = int64_t(KT) * int64_t(sizeof(T));
    const int64_t keep_elems = int64_t(di.l2_bytes) * kKeepL2Pct / 100 / per_elem;
    a.keep_from = a.D > keep_elems ? a.D - keep_elems : 0;
    // The grid is no larger than what the device holds at once (occupancy above), so all its CTAs become
    // resident and the one wait on other CTAs ends; it is bounded in any case.  Programmatic stream
    // serialisation: the kernel waits for its predecessor on the stream itself (griddepcontrol.wait, first
    // thing) and releases its successor once its decisions are taken.
    // Not while the stream is being captured into a graph: where the node will run, and beside what, is decided
    // at replay, out of this library's sight (and the query below is not allowed during a capture).
    {
        cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(st, &capturing) != cudaSuccess) { cudaGetLastError(); return GAF_ERR_CUDA; }
        if (capturing != cudaStreamCaptureStatusNone) return GAF_ERR_UNSUPPORTED;
    }
    FusedGuard &guard = g_fused_guard[di.dev];
    std::lock_guard<std::mutex> lock(guard.m);          // (check and launch are one step for other host threads)
    if (guard.any && guard.last != st) {
        const cudaError_t q = cudaStreamQuery(guard.last);
        if (q == cudaErrorNotReady) return GAF_ERR_UNSUPPORTED;
        if (q != cudaSuccess) cudaGetLastError();       // that stream no longer exists: nothing of it is in flight
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(unsigned(grid)); cfg.blockDim = dim3(kGsThreads);
    cfg.dynamicSmemBytes = size_t(pl.dyn); cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, kernel, a);
    if (err != cudaSuccess) { cudaGetLastError(); return GAF_ERR_CUDA; }
    guard.last = st;
    guard.any = true;
    ++g_launches;
    return GAF_OK;
}

template <typename T>
int launch_gram_fused(GramFusedArgs &a, int K, const DeviceInfo &di, cudaStream_t st) {
    switch (K) {
        case 2: return launch_gram_fused_kt<T, 2>(a, di, st);
        case 3: return launch_gram_fused_kt<T, 3>(a, di, st);
        case 4: return launch_gram_fused_kt<T, 4>(a, di, st);
        case 5: return launch_gram_fused_kt<T, 5>(a, di, st);
        case 6: return launch_gram_fused_kt<T, 6>(a, di, st);
        case 7: return launch_gram_fused_kt<T, 7>(a, di, st);
        case 8: return launch_gram_fused_kt<T, 8>(a, di, st);
        default: return GAF_ERR_UNSUPPORTED;
    }
}

// Gram-first schedule: Gram matrix, scalar walk of Algorithm 1, masked mean.
// `seed_out` non-null selects the any-seed variant (ord must then be the identity).
template <typename T>
int launch_gram_first(const void *const *g, int K, int64_t D, int dtype, double tau, const int32_t *ord,
                      float *macro_out, uint8_t *mask_out, float *dist_out, int32_t *count_out,
                      int32_t *seed_out, unsigned char *base, const DeviceInfo &di, bool one_launch,
                      cudaStream_t st) {
    const int sms = di.sms;
    Control *ctl = reinterpret_cast<Control *>(base);
    RingArgs ring{};
    if (seed_out) {
        ring.K = K; ring.tau = tau; ring.mask_out = mask_out; ring.dist_out = dist_out;
        ring.count_out = count_out; ring.seed_out = seed_out; ring.ctl = ctl;
    }
    ReplayArgs r{};
    r.K = K; r.tau = tau; r.mask_out = mask_out; r.dist_out = dist_out; r.count_out = count_out; r.ctl = ctl;
    for (int t = 0; t < K; ++t) r.idx[t] = ord[t];
    double *gram_by_index = reinterpret_cast<double *>(base + kExtraOffset + gram_partials_bytes(K));
    double *gram_by_step = reinterpret_cast<double *>(base + kExtraOffset + gram_partials_bytes(K) +
                                                      gram_matrix_bytes(K));
    if (one_launch) {
        if (K < 2 || K > kGsMaxK) return GAF_ERR_UNSUPPORTED;
        GramFusedArgs f{};
        for (int t = 0; t < K; ++t) f.g[t] = g[ord[t]];
        f.D = D; f.out = macro_out;
        f.partials = reinterpret_cast<double *>(base + kExtraOffset);
        f.gram = gram_by_step;
        f.replay = r;
        f.ring = ring;
        return launch_gram_fused<T>(f, K, di, st);
    }
    if (use_small_gram(K, D, dtype)) {
        GramSmallArgs a{};
        for (int t = 0; t < K; ++t) a.g[t] = g[ord[t]];
        a.D = D;
        // how much of the tail of the Gram pass should stay in L2 for the masked-mean pass
        const int64_t per_elem = int64_t(K) * int64_t(sizeof(T));
        const int64_t keep_elems = int64_t(di.l2_bytes) * kKeepL2Pct / 100 / per_elem;
        a.keep_from = D > keep_elems ? D - keep_elems : 0;
        a.partials = reinterpret_cast<double *>(base + kExtraOffset);
        a.gram = gram_by_step;
        a.replay = r;
        a.ring = ring;
        if (int rc = launch_gram_small<T>(a, K, di, st)) return rc;
    } else {
        if (int rc = launch_gram_tiles(g, K, D, dtype, nullptr, nullptr, base, di, st)) return rc;
        if (seed_out) gram_ring_replay_kernel<<<1, GAF_MAX_K, 0, st>>>(ring, gram_by_index);
        else gram_replay_kernel<<<1, 256, 0, st>>>(r, gram_by_index, gram_by_step);
        ++g_launches;
    }
    MaskedMeanArgs m{};
    for (int t = 0; t < K; ++t) m.g[t] = g[ord[t]];
    m.K = K; m.D = D; m.out = macro_out; m.ctl = ctl;
    const int grid = stream_grid(D, kMsThreads, sms);
    {
        // runs of 8 chunks per CTA once every CTA gets at least eight such runs, else one trip at a time
        const int per_trip = sizeof(T) == 2 ? 2 : 1;
        const int64_t chunks = (D / kOct + kMsThreads - 1) / kMsThreads;
        m.run = chunks >= int64_t(8) * kMsLongRun * grid ? kMsLongRun : per_trip;
    }
    // the blocks may be placed while the Gram pass winds down (its last CTA is still totalling partials)
    const cudaError_t err = launch_dependent(masked_mean_kernel<T>, grid, kMsThreads, st, m);
    ++g_launches;
    if (err != cudaSuccess) { cudaGetLastError(); return GAF_ERR_CUDA; }
    return cudaGetLastError() == cudaSuccess ? GAF_OK : GAF_ERR_CUDA;
}

// Whether the library's own choice is the one-launch form of the Gram-first schedule.
bool auto_one_launch(int K, int64_t D, int dtype) {
    if (!use_small_gram(K, D, dtype)) return false;
    // two gradients: the one-launch kernel writes their mean during its only pass over them, at any length
    if (K == 2) return true;
    if (dtype == GAF_F32) return int64_t(K) * 4 * D <= kFusedMaxInputBytesF32;
    return K < 7 || int64_t(K) * 2 * D <= kFusedMaxInputBytesBf16Mma;
}

int check_workspace(const void *ws, size_t have, size_t need) {
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0 || have < need) return GAF_ERR_WORKSPACE;
    return GAF_OK;
}

template <typename T>
int launch_stepwise(const void *const *g, int K, int64_t D, double tau, const int32_t *ord,
                    float *macro_out, uint8_t *mask_out, float *dist_out, int32_t *count_out,
                    Control *ctl, double *partials, int sms, cudaStream_t st) {
    const int grid = stream_grid(D, kStepThreads, sms);
    StepArgs a{};
    a.acc = macro_out; a.D = D; a.ctl = ctl; a.partials = partials; a.tau = tau;
    a.mask_out = mask_out; a.dist_out = dist_out; a.count_out = count_out; a.K = K;
    a.seed_index = ord[0];
    a.g_seed = g[ord[0]];
    if (K == 1) {
        step_kernel<T, kOnly><<<grid, kStepThreads, 0, st>>>(a);
        ++g_launches;
        return cudaGetLastError() == cudaSuccess ? GAF_OK : GAF_ERR_CUDA;
    }
    a.t = 0; a.g_next = g[ord[1]]; a.i_next = ord[1];
    step_kernel<T, kFirst><<<grid, kStepThreads, 0, st>>>(a);
    ++g_launches;
    for (int t = 1; t <= K - 2; ++t) {
        a.t = t; a.g_cur = g[ord[t]]; a.g_next = g[ord[t + 1]]; a.i_next = ord[t + 1];
        if (launch_dependent(step_kernel<T, kMid>, grid, kStepThreads, st, a) != cudaSuccess) {
            cudaGetLastError();
            return GAF_ERR_CUDA;
        }
        ++g_launches;
    }
    a.t = K - 1; a.g_cur = g[ord[K - 1]]; a.g_next = nullptr; a.i_next = -1;
    if (launch_dependent(step_kernel<T, kLast>, grid, kStepThreads, st, a) != cudaSuccess) {
        cudaGetLastError();
        return GAF_ERR_CUDA;
    }
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? GAF_OK : GAF_ERR_CUDA;
}

int check_grads(const void *const *grads, int K, int64_t D, int dtype) {
    if (!grads || K < 1 || K > GAF_MAX_K || D < 0) return GAF_ERR_ARG;
    if (dtype != GAF_F32 && dtype != GAF_BF16) return GAF_ERR_ARG;
    for (int i = 0; i < K; ++i) {
        if (!grads[i] && D > 0) return GAF_ERR_ARG;       // an empty buffer may be NULL
        if (!aligned16(grads[i])) return GAF_ERR_ALIGN;
    }
    return GAF_OK;
}

template <typename T, int KT>
void launch_bucket_gram_kt(const BucketGramArgs &a, const BucketTable &bt, int grid, cudaStream_t st) {
    bucket_gram_kernel<T, KT><<<grid, kBkThreads, 0, st>>>(a, bt);
}
template <typename T>
int launch_bucket_gram(const BucketGramArgs &a, const BucketTable &bt, int K, int grid, cudaStream_t st) {
    switch (K) {
        case 1: launch_bucket_gram_kt<T, 1>(a, bt, grid, st); break;
        case 2: launch_bucket_gram_kt<T, 2>(a, bt, grid, st); break;
        case 3: launch_bucket_gram_kt<T, 3>(a, bt, grid, st); break;
        case 4: launch_bucket_gram_kt<T, 4>(a, bt, grid, st); break;
        case 5: launch_bucket_gram_kt<T, 5>(a, bt, grid, st); break;
        case 6: launch_bucket_gram_kt<T, 6>(a, bt, grid, st); break;
        case 7: launch_bucket_gram_kt<T, 7>(a, bt, grid, st); break;
        case 8: launch_bucket_gram_kt<T, 8>(a, bt, grid, st); break;
        default: return GAF_ERR_ARG;
    }
    return GAF_OK;
}

}  // namespace

void gaf::set_last_launch_count(int launches) { g_launches = launches; }

extern "C" {

const char *gaf_error_string(int code) {
    switch (code) {
        case GAF_OK: return "ok";
        case GAF_ERR_ARG: return "invalid argument";
        case GAF_ERR_ALIGN: return "device pointer not 16-byte aligned";
        case GAF_ERR_ALIAS: return "macro_out overlaps an input gradient";
        case GAF_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case GAF_ERR_CUDA: return "CUDA runtime error";
        case GAF_ERR_RESERVED: return "reserved";
        case GAF_ERR_UNSUPPORTED: return "schedule not available for this call on this device";
        case GAF_ERR_TOO_LARGE: return "size beyond the fixed limit of the no-allocation entry point";
        default: return "unknown error code";
    }
}

int gaf_last_launch_count(void) { return g_launches; }
int gaf_last_schedule(void) { return g_schedule; }
int gaf_last_gram_loader(void) { return g_gram_loader; }

int gaf_test_set_wait_fault(unsigned int wait_limit, int withhold) {
    g_test_wait_limit = wait_limit;
    g_test_withhold = withhold ? 1 : 0;
    return GAF_OK;
}

int gaf_workspace_bytes(int K, int64_t D, int dtype, size_t *bytes_out) {
    if (!bytes_out || K < 1 || K > GAF_MAX_K || D < 0) return GAF_ERR_ARG;
    if (dtype != GAF_F32 && dtype != GAF_BF16) return GAF_ERR_ARG;
    *bytes_out = round_up(kExtraOffset + pairwise_extra_bytes(K), 256);
    return GAF_OK;
}

int gaf_workspace_init(void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (int rc = check_workspace(workspace, workspace_bytes, kExtraOffset)) return rc;
    g_launches = 0; g_gram_loader = 0;
    if (cudaMemsetAsync(workspace, 0, kControlBytes, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return GAF_ERR_CUDA;
    return GAF_OK;
}

int gaf_cosdist(const void *x, const void *y, int64_t D, int dtype, float *dist_out,
                double *stats_out, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    g_launches = 0; g_gram_loader = 0;
    if (((!x || !y) && D > 0) || !dist_out || D < 0) return GAF_ERR_ARG;
    if (dtype != GAF_F32 && dtype != GAF_BF16) return GAF_ERR_ARG;
    if (!aligned16(x) || !aligned16(y)) return GAF_ERR_ALIGN;
    if (int rc = check_workspace(workspace, workspace_bytes, kExtraOffset)) return rc;
    DeviceInfo di;
    if (!device_info(&di)) return GAF_ERR_CUDA;
    auto *base = static_cast<unsigned char *>(workspace);
    CosArgs a{x, y, D, reinterpret_cast<Control *>(base),
              reinterpret_cast<double *>(base + kPartialsOffset), dist_out, stats_out};
    const int grid = stream_grid(D, kStepThreads, di.sms);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // (the kernel waits for its predecessor on the stream itself and releases its successor when its streaming part ends)
    const cudaError_t err = dtype == GAF_F32 ? launch_dependent(cosdist_kernel<float>, grid, kStepThreads, st, a)
                                             : launch_dependent(cosdist_kernel<__nv_bfloat16>, grid, kStepThreads, st, a);
    if (err != cudaSuccess) { cudaGetLastError(); return GAF_ERR_CUDA; }
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? GAF_OK : GAF_ERR_CUDA;
}

int gaf_filter_accumulate(const void *const *grads, int K, int64_t D, int dtype, double tau,
                          const int32_t *order, float *macro_out, uint8_t *mask_out,
                          float *dist_out, int32_t *count_out, void *workspace,
                          size_t workspace_bytes, int schedule, void *cuda_stream) {
    g_launches = 0; g_gram_loader = 0;
    if (int rc = check_grads(grads, K, D, dtype)) return rc;
    if ((!macro_out && D > 0) || !mask_out || !count_out) return GAF_ERR_ARG;
    if (schedule < GAF_SCHED_AUTO || schedule > GAF_SCHED_GRAM_FUSED) return GAF_ERR_ARG;
    if (tau != tau) return GAF_ERR_ARG;
    if (!aligned16(macro_out)) return GAF_ERR_ALIGN;
    int32_t ord[GAF_MAX_K];
    if (!read_order(order, K, ord)) return GAF_ERR_ARG;
    if (overlaps_inputs(macro_out, grads, K, D, dtype)) return GAF_ERR_ALIAS;
    if (int rc = check_workspace(workspace, workspace_bytes, kExtraOffset)) return rc;
    DeviceInfo di;
    if (!device_info(&di)) return GAF_ERR_CUDA;
    auto *base = static_cast<unsigned char *>(workspace);
    Control *ctl = reinterpret_cast<Control *>(base);
    double *partials = reinterpret_cast<double *>(base + kPartialsOffset);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

    const bool library_choice = schedule == GAF_SCHED_AUTO;
    if (schedule == GAF_SCHED_AUTO) {
        // Gram-first moves fewer bytes whenever its one-pass Gram kernel applies
        const bool ws_ok = workspace_bytes >= kExtraOffset + pairwise_extra_bytes(K);
        // (the general CUDA-core Gram kernel beats the stepwise schedule up to 32 binary32 gradients)
        const bool fast_gram = K >= 2 && (K <= kGsMaxK || use_tensor_gram(K, D, dtype) ||
                                          (dtype == GAF_F32 && K <= kPanelAutoMaxK));
        schedule = (fast_gram && ws_ok) ? (auto_one_launch(K, D, dtype) ? GAF_SCHED_GRAM_FUSED : GAF_SCHED_GRAM)
                                        : GAF_SCHED_STEPWISE;
    }
    if (K == 1) schedule = GAF_SCHED_STEPWISE;          // one gradient: it is the seed and the result
    g_schedule = schedule;
    if (schedule == GAF_SCHED_GRAM || schedule == GAF_SCHED_GRAM_FUSED) {
        if (int rc = check_workspace(workspace, workspace_bytes, kExtraOffset + pairwise_extra_bytes(K)))
            return rc;
        auto run = [&](bool one_launch) {
            return dtype == GAF_F32
                ? launch_gram_first<float>(grads, K, D, dtype, tau, ord, macro_out, mask_out, dist_out,
                                           count_out, nullptr, base, di, one_launch, st)
                : launch_gram_first<__nv_bfloat16>(grads, K, D, dtype, tau, ord, macro_out, mask_out, dist_out,
                                                   count_out, nullptr, base, di, one_launch, st);
        };
        int rc = run(schedule == GAF_SCHED_GRAM_FUSED);
        if (rc != GAF_OK && library_choice && schedule == GAF_SCHED_GRAM_FUSED) {
            // the launch was refused (for example no CTA of this kernel fits an SM of this device): the
            // library's own choice falls back to the two-launch form, an explicit request does not
            g_launches = 0; g_gram_loader = 0;
            g_schedule = GAF_SCHED_GRAM;
            rc = run(false);
        }
        return rc;
    }
    return dtype == GAF_F32
        ? launch_stepwise<float>(grads, K, D, tau, ord, macro_out, mask_out, dist_out, count_out,
                                 ctl, partials, di.sms, st)
        : launch_stepwise<__nv_bfloat16>(grads, K, D, tau, ord, macro_out, mask_out, dist_out,
                                         count_out, ctl, partials, di.sms, st);
}

int gaf_filter_accumulate_repeat(int repeats, int n_sets, const void *const *grads, int K, int64_t D,
                                 int dtype, double tau, const int32_t *order, float *macro_out,
                                 uint8_t *mask_out, float *dist_out, int32_t *count_out, void *workspace,
                                 size_t workspace_bytes, int schedule, void *cuda_stream) {
    g_launches = 0; g_gram_loader = 0;
    if (repeats < 0 || n_sets < 1 || !grads || K < 1 || K > GAF_MAX_K) return GAF_ERR_ARG;
    int launches = 0;
    for (int r = 0; r < repeats; ++r) {
        const int rc = gaf_filter_accumulate(grads + size_t(r % n_sets) * K, K, D, dtype, tau, order, macro_out,
                                             mask_out, dist_out, count_out, workspace, workspace_bytes,
                                             schedule, cuda_stream);
        if (rc != GAF_OK) return rc;
        launches += g_launches;
    }
    g_launches = launches;
    return GAF_OK;
}

int gaf_filter_accumulate_any_seed(const void *const *grads, int K, int64_t D, int dtype, double tau,
                                   float *macro_out, uint8_t *mask_out, float *dist_out,
                                   int32_t *count_out, int32_t *seed_out, void *workspace,
                                   size_t workspace_bytes, void *cuda_stream) {
    g_launches = 0; g_gram_loader = 0;
    if (int rc = check_grads(grads, K, D, dtype)) return rc;
    if ((!macro_out && D > 0) || !mask_out || !count_out || !seed_out) return GAF_ERR_ARG;
    if (tau != tau) return GAF_ERR_ARG;
    if (!aligned16(macro_out)) return GAF_ERR_ALIGN;
    if (overlaps_inputs(macro_out, grads, K, D, dtype)) return GAF_ERR_ALIAS;
    if (int rc = check_workspace(workspace, workspace_bytes, kExtraOffset + pairwise_extra_bytes(K))) return rc;
    DeviceInfo di;
    if (!device_info(&di)) return GAF_ERR_CUDA;
    auto *base = static_cast<unsigned char *>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int32_t ord[GAF_MAX_K];
    for (int t = 0; t < K; ++t) ord[t] = t;
    if (K == 1) {
        // one gradient: it is the seed and the result
        Control *ctl = reinterpret_cast<Control *>(base);
        double *partials = reinterpret_cast<double *>(base + kPartialsOffset);
        int rc = dtype == GAF_F32
            ? launch_stepwise<float>(grads, K, D, tau, ord, macro_out, mask_out, dist_out, count_out, ctl,
                                     partials, di.sms, st)
            : launch_stepwise<__nv_bfloat16>(grads, K, D, tau, ord, macro_out, mask_out, dist_out, count_out,
                                             ctl, partials, di.sms, st);
        if (rc != GAF_OK) return rc;
        return cudaMemsetAsync(seed_out, 0, sizeof(int32_t), st) == cudaSuccess ? GAF_OK : GAF_ERR_CUDA;
    }
    auto run = [&](bool one_launch) {
        return dtype == GAF_F32
            ? launch_gram_first<float>(grads, K, D, dtype, tau, ord, macro_out, mask_out, dist_out, count_out,
                                       seed_out, base, di, one_launch, st)
            : launch_gram_first<__nv_bfloat16>(grads, K, D, dtype, tau, ord, macro_out, mask_out, dist_out,
                                               count_out, seed_out, base, di, one_launch, st);
    };
    const bool one_launch = auto_one_launch(K, D, dtype);
    int rc = run(one_launch);
    if (rc != GAF_OK && one_launch) {       // launch refused: two launches
        g_launches = 0; g_gram_loader = 0;
        rc = run(false);
    }
    return rc;
}

int gaf_filter_accumulate_bucketed(const void *const *grads, int K, int64_t D, int dtype, double tau,
                                   const int32_t *order, int S, const int64_t *offsets, float *macro_out,
                                   uint8_t *mask_out, float *dist_out, int32_t *count_out, void *workspace,
                                   size_t workspace_bytes, void *cuda_stream) {
    g_launches = 0; g_gram_loader = 0;
    if (int rc = check_grads(grads, K, D, dtype)) return rc;
    if (K > kGsMaxK) return GAF_ERR_UNSUPPORTED;
    if ((!macro_out && D > 0) || !mask_out || !count_out || !offsets || tau != tau) return GAF_ERR_ARG;
    if (S < 1 || S > GAF_MAX_BUCKETS || offsets[0] != 0 || offsets[S] != D) return GAF_ERR_ARG;
    for (int b = 0; b < S; ++b) {
        if (offsets[b + 1] < offsets[b]) return GAF_ERR_ARG;
        if (b > 0 && (offsets[b] & 7) != 0) return GAF_ERR_ALIGN;
    }
    if (!aligned16(macro_out)) return GAF_ERR_ALIGN;
    int32_t ord[GAF_MAX_K];
    if (!read_order(order, K, ord)) return GAF_ERR_ARG;
    if (overlaps_inputs(macro_out, grads, K, D, dtype)) return GAF_ERR_ALIAS;
    if (int rc = check_workspace(workspace, workspace_bytes, kExtraOffset + bucketed_extra_bytes())) return rc;
    DeviceInfo di;
    if (!device_info(&di)) return GAF_ERR_CUDA;
    auto *base = static_cast<unsigned char *>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

    BucketTable bt{};
    bt.S = S;
    for (int b = 0; b <= S; ++b) bt.off[b] = offsets[b];
    double *partials = reinterpret_cast<double *>(base + kExtraOffset);
    unsigned long long *bits = reinterpret_cast<unsigned long long *>(
        base + kExtraOffset + size_t(kBkMaxCtas + kBkMaxBuckets) * 64 * sizeof(double));
    // one wave: as many CTAs as are resident at once (two per SM up to 4 gradients, one beyond: registers)
    int grid = di.sms * (K <= 4 ? 2 : 1);
    if (grid > kBkMaxCtas) grid = kBkMaxCtas;
    const int64_t n_oct = D / kOct;
    if (n_oct < grid) grid = n_oct > 0 ? int(n_oct) : 1;

    BucketGramArgs ga{};
    for (int t = 0; t < K; ++t) ga.g[t] = grads[ord[t]];
    ga.D = D; ga.partials = partials; ga.ctl = reinterpret_cast<Control *>(base);
    // the end of every CTA's range, kKeepL2Pct of L2 in all, is asked to stay in L2 for the mean pass
    ga.keep_elems = int64_t(di.l2_bytes) * kKeepL2Pct / 100 / (int64_t(K) * int64_t(elem_bytes(dtype))) / grid;
    ga.keep_elems = (ga.keep_elems + 7) / 8 * 8;
    int rc = dtype == GAF_F32 ? launch_bucket_gram<float>(ga, bt, K, grid, st)
                              : launch_bucket_gram<__nv_bfloat16>(ga, bt, K, grid, st);
    if (rc != GAF_OK) return rc;
    ++g_launches;

    BucketWalkArgs wa{};
    wa.K = K; wa.D = D; wa.ctas = grid; wa.tau = tau; wa.partials = partials; wa.mask_out = mask_out;
    wa.dist_out = dist_out; wa.count_out = count_out; wa.bits = bits; wa.ctl = ga.ctl;
    for (int t = 0; t < K; ++t) wa.idx[t] = ord[t];
    if (launch_dependent(bucket_walk_kernel, S, 64 * kWalkChains, st, wa, bt) != cudaSuccess) {
        cudaGetLastError();
        return GAF_ERR_CUDA;
    }
    ++g_launches;

    BucketMeanArgs ma{};
    for (int t = 0; t < K; ++t) ma.g[t] = grads[ord[t]];
    ma.K = K; ma.D = D; ma.out = macro_out; ma.bits = bits;
    {
        // (its own grid, two CTAs per SM: the ranges need not be those of the Gram pass)
        int mean_grid = di.sms * 2;
        if (mean_grid > kBkMaxCtas) mean_grid = kBkMaxCtas;
        if (n_oct < mean_grid) mean_grid = n_oct > 0 ? int(n_oct) : 1;
        const cudaError_t err = dtype == GAF_F32
            ? launch_dependent(bucket_mean_kernel<float>, mean_grid, kBkThreads, st, ma, bt)
            : launch_dependent(bucket_mean_kernel<__nv_bfloat16>, mean_grid, kBkThreads, st, ma, bt);
        if (err != cudaSuccess) { cudaGetLastError(); return GAF_ERR_CUDA; }
    }
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? GAF_OK : GAF_ERR_CUDA;
}

int gaf_stream_begin(const void *seed, int64_t D, int dtype, float *acc, void *workspace,
                     size_t workspace_bytes, void *cuda_stream) {
    g_launches = 0; g_gram_loader = 0;
    if ((!seed && D > 0) || (!acc && D > 0) || D < 0) return GAF_ERR_ARG;
    if (dtype != GAF_F32 && dtype != GAF_BF16) return GAF_ERR_ARG;
    if (!aligned16(seed) || !aligned16(acc)) return GAF_ERR_ALIGN;
    if (int rc = check_workspace(workspace, workspace_bytes, kExtraOffset)) return rc;
    DeviceInfo di;
    if (!device_info(&di)) return GAF_ERR_CUDA;
    auto *base = static_cast<unsigned char *>(workspace);
    Control *ctl = reinterpret_cast<Control *>(base);
    // g <- seed, c <- 1: the one-gradient form of the stepwise kernel (its mask, distance and
    // count outputs go to the control block)
    StepArgs a{};
    a.acc = acc; a.D = D; a.ctl = ctl; a.partials = reinterpret_cast<double *>(base + kPartialsOffset);
    a.g_seed = seed; a.seed_index = 0; a.K = 1;
    a.mask_out = ctl->stream_mask; a.dist_out = ctl->stream_dist; a.count_out = &ctl->count;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int grid = stream_grid(D, kStepThreads, di.sms);
    if (dtype == GAF_F32) step_kernel<float, kOnly><<<grid, kStepThreads, 0, st>>>(a);
    else step_kernel<__nv_bfloat16, kOnly><<<grid, kStepThreads, 0, st>>>(a);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? GAF_OK : GAF_ERR_CUDA;
}

int gaf_stream_push(const void *g, int t, int64_t D, int dtype, double tau, float *acc, void *workspace,
                    size_t workspace_bytes, void *cuda_stream) {
    g_launches = 0; g_gram_loader = 0;
    if ((!g && D > 0) || (!acc && D > 0) || D < 0 || t < 1 || t >= GAF_MAX_K || tau != tau) return GAF_ERR_ARG;
    if (dtype != GAF_F32 && dtype != GAF_BF16) return GAF_ERR_ARG;
    if (!aligned16(g) || !aligned16(acc)) return GAF_ERR_ALIGN;
    {
        const uintptr_t o0 = reinterpret_cast<uintptr_t>(acc), o1 = o0 + size_t(D) * 4;
        const uintptr_t g0 = reinterpret_cast<uintptr_t>(g), g1 = g0 + size_t(D) * elem_bytes(dtype);
        if (o0 < g1 && g0 < o1) return GAF_ERR_ALIAS;
    }
    if (int rc = check_workspace(workspace, workspace_bytes, kExtraOffset)) return rc;
    DeviceInfo di;
    if (!device_info(&di)) return GAF_ERR_CUDA;
    auto *base = static_cast<unsigned char *>(workspace);
    StreamArgs a{g, acc, D, reinterpret_cast<Control *>(base),
                 reinterpret_cast<double *>(base + kPartialsOffset), tau, t};
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int grid = stream_grid(D, kStreamThreads, di.sms);
    if (dtype == GAF_F32) {
        stream_test_kernel<float><<<grid, kStreamThreads, 0, st>>>(a);
        if (launch_dependent(stream_add_kernel<float>, grid, kStreamThreads, st, a) != cudaSuccess) {
            cudaGetLastError();
            return GAF_ERR_CUDA;
        }
    } else {
        stream_test_kernel<__nv_bfloat16><<<grid, kStreamThreads, 0, st>>>(a);
        if (launch_dependent(stream_add_kernel<__nv_bfloat16>, grid, kStreamThreads, st, a) != cudaSuccess) {
            cudaGetLastError();
            return GAF_ERR_CUDA;
        }
    }
    g_launches += 2;
    return cudaGetLastError() == cudaSuccess ? GAF_OK : GAF_ERR_CUDA;
}

int gaf_stream_end(int K, int64_t D, float *acc, uint8_t *mask_out, float *dist_out, int32_t *count_out,
                   void *workspace, size_t workspace_bytes, void *cuda_stream) {
    g_launches = 0; g_gram_loader = 0;
    if (K < 1 || K > GAF_MAX_K || D < 0 || (!acc && D > 0) || !mask_out || !count_out) return GAF_ERR_ARG;
    if (!aligned16(acc)) return GAF_ERR_ALIGN;
    if (int rc = check_workspace(workspace, workspace_bytes, kExtraOffset)) return rc;
    DeviceInfo di;
    if (!device_info(&di)) return GAF_ERR_CUDA;
    StreamEndArgs a{acc, D, K, static_cast<const Control *>(workspace), mask_out, dist_out, count_out};
    const int grid = stream_grid(D, kStreamThreads, di.sms);
    stream_end_kernel<<<grid, kStreamThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(a);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? GAF_OK : GAF_ERR_CUDA;
}

int gaf_host_staging_bytes(int K, int64_t D, int dtype, size_t *bytes_out) {
    if (!bytes_out || K < 1 || K > GAF_MAX_K || D < 0) return GAF_ERR_ARG;
    if (dtype != GAF_F32 && dtype != GAF_BF16) return GAF_ERR_ARG;
    const size_t g = round_up(size_t(D) * elem_bytes(dtype), 256);
    *bytes_out = size_t(K) * g + round_up(size_t(D) * 4, 256) + 3 * 256;
    return GAF_OK;
}

int gaf_filter_accumulate_host(const void *const *grads_host, int K, int64_t D, int dtype,
                               double tau, const int32_t *order, float *macro_out_host,
                               uint8_t *mask_out_host, float *dist_out_host,
                               int32_t *count_out_host, void *staging, size_t staging_bytes,
                               void *workspace, size_t workspace_bytes, int schedule,
                               void *cuda_stream) {
    g_launches = 0; g_gram_loader = 0;
    size_t need = 0;
    if (int rc = gaf_host_staging_bytes(K, D, dtype, &need)) return rc;
    if (!grads_host || (!macro_out_host && D > 0) || !mask_out_host || !count_out_host) return GAF_ERR_ARG;
    for (int i = 0; i < K; ++i) if (!grads_host[i] && D > 0) return GAF_ERR_ARG;
    if (int rc = check_workspace(staging, staging_bytes, need)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    auto *base = static_cast<unsigned char *>(staging);
    const size_t gbytes = size_t(D) * elem_bytes(dtype), gstride = round_up(gbytes, 256);
    const void *dev[GAF_MAX_K];
    for (int i = 0; i < K; ++i) {
        dev[i] = base + size_t(i) * gstride;
        if (gbytes && cudaMemcpyAsync(base + size_t(i) * gstride, grads_host[i], gbytes,
                                      cudaMemcpyHostToDevice, st) != cudaSuccess)
            return GAF_ERR_CUDA;
    }
    unsigned char *p = base + size_t(K) * gstride;
    float *d_out = reinterpret_cast<float *>(p); p += round_up(size_t(D) * 4, 256);
    uint8_t *d_mask = p; p += 256;
    float *d_dist = reinterpret_cast<float *>(p); p += 256;
    int32_t *d_count = reinterpret_cast<int32_t *>(p);
    int rc = gaf_filter_accumulate(dev, K, D, dtype, tau, order, d_out, d_mask, d_dist, d_count,
                                   workspace, workspace_bytes, schedule, cuda_stream);
    if (rc != GAF_OK) return rc;
    bool ok = true;
    if (D) ok &= cudaMemcpyAsync(macro_out_host, d_out, size_t(D) * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(mask_out_host, d_mask, K, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    if (dist_out_host)
        ok &= cudaMemcpyAsync(dist_out_host, d_dist, size_t(K) * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(count_out_host, d_count, 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok &= cudaStreamSynchronize(st) == cudaSuccess;
    return ok ? GAF_OK : GAF_ERR_CUDA;
}

int gaf_pairwise_cosdist(const void *const *grads, int K, int64_t D, int dtype, float *dist_out,
                         double *gram_out, void *workspace, size_t workspace_bytes,
                         void *cuda_stream) {
    g_launches = 0; g_gram_loader = 0;
    if (int rc = check_grads(grads, K, D, dtype)) return rc;
    if (!dist_out) return GAF_ERR_ARG;
    if (int rc = check_workspace(workspace, workspace_bytes, kExtraOffset + pairwise_extra_bytes(K)))
        return rc;
    DeviceInfo di;
    if (!device_info(&di)) return GAF_ERR_CUDA;
    auto *base = static_cast<unsigned char *>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (use_small_gram(K, D, dtype)) {
        // few gradients: the one-pass register-tiled Gram kernel, distances in its last CTA
        GramSmallArgs a{};
        for (int i = 0; i < K; ++i) a.g[i] = grads[i];
        a.D = D;
        a.keep_from = D;                                    // nothing is read again: stream everything
        a.partials = reinterpret_cast<double *>(base + kExtraOffset);
        a.gram = reinterpret_cast<double *>(base + kExtraOffset + gram_partials_bytes(K));
        a.replay.ctl = reinterpret_cast<Control *>(base);
        a.pair_dist_out = dist_out;
        a.pair_gram_out = gram_out;
        return dtype == GAF_F32 ? launch_gram_small<float>(a, K, di, st)
                                : launch_gram_small<__nv_bfloat16>(a, K, di, st);
    }
    return launch_gram_tiles(grads, K, D, dtype, dist_out, gram_out, base, di, st);
}

int gaf_read_status(const void *workspace, void *cuda_stream, int *status_out) {
    if (!workspace || !status_out) return GAF_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const Control *ctl = static_cast<const Control *>(workspace);
    int status = 0;
    if (cudaMemcpyAsync(&status, &ctl->status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return GAF_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return GAF_ERR_CUDA;
    *status_out = status;
    return GAF_OK;
}

}  // extern "C"
