// gaf_cosdist_static: the cosine distance of two buffers for callers that cannot
// allocate device memory.
//
// Every other entry point of this library takes a caller-allocated workspace.
// Some callers have no way to get one: code running inside another framework's
// memory pool with allocation switched off, a plug-in invoked where cudaMalloc
// would synchronise the whole device in the middle of a training step, or a
// host program that must not touch the allocator after start-up.  For them the
// scratch memory of the reduction (one ticket, one status word, one partial
// triple per CTA) lives in a fixed array in this module's device image.  The
// price: the array is reserved on every GPU that loads the library, for the
// life of the process; its size fixes an upper limit on D; and all calls share
// it, so two calls that overlap on the GPU race.
#include <cuda_runtime.h>

#include <cstdint>
#include <mutex>

#include "../../include/gaf.h"
#include "gaf_host.h"
#include "gaf_stepwise.cuh"

namespace {

using namespace gaf;

constexpr int kStaticMaxCtas = 512;                               // partial triples in the array
constexpr size_t kStaticControlBytes = 256;                       // ticket + status live here
constexpr size_t kStaticScratchBytes = kStaticControlBytes + size_t(kStaticMaxCtas) * 3 * sizeof(double);
constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a handle for the runtime;
// the address the kernel needs comes from cudaGetSymbolAddress, per device.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_setup_mutex;
void *g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the array on the current device, looked up once per device.
int static_scratch(void **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GAF_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return GAF_ERR_CUDA;
        }
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return GAF_OK;
}

}  // namespace

extern "C" int gaf_cosdist_static(const void *x, const void *y, int64_t D, int dtype,
                                  float *dist_out, double *stats_out, void *cuda_stream) {
    set_last_launch_count(0);
    if (D < 0 || ((!x || !y) && D > 0) || !dist_out) return GAF_ERR_ARG;
    if (dtype != GAF_F32 && dtype != GAF_BF16) return GAF_ERR_ARG;
    if (D > GAF_STATIC_MAX_D) return GAF_ERR_TOO_LARGE;
    if ((reinterpret_cast<uintptr_t>(x) & 15u) || (reinterpret_cast<uintptr_t>(y) & 15u)) return GAF_ERR_ALIGN;

    void *scratch = nullptr;
    if (int rc = static_scratch(&scratch)) return rc;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return GAF_ERR_CUDA;

    // CTAs: two per SM, fewer for short inputs, never more than the array has slots for
    int64_t grid = (D / kOct + kStepThreads - 1) / kStepThreads;
    if (grid > int64_t(sms) * 2) grid = int64_t(sms) * 2;
    if (grid > kStaticMaxCtas) grid = kStaticMaxCtas;
    if (grid < 1) grid = 1;

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // The array keeps whatever the previous call left: the ticket and the status
    // word must start at zero.  (The partial slots are written before they are read.)
    if (cudaMemsetAsync(scratch, 0, kStaticControlBytes, st) != cudaSuccess) return GAF_ERR_CUDA;

    auto *base = static_cast<unsigned char *>(scratch);
    // The kernel uses only the first words of a Control block (ticket, status); they
    // fit in the 256 bytes reserved in front of the partial slots.
    static_assert(offsetof(Control, status) + sizeof(int) <= kStaticControlBytes, "control words");
    CosArgs a{x, y, D, reinterpret_cast<Control *>(base),
              reinterpret_cast<double *>(base + kStaticControlBytes), dist_out, stats_out};
    if (dtype == GAF_F32) cosdist_kernel<float><<<int(grid), kStepThreads, 0, st>>>(a);
    else cosdist_kernel<__nv_bfloat16><<<int(grid), kStepThreads, 0, st>>>(a);
    set_last_launch_count(1);
    return cudaGetLastError() == cudaSuccess ? GAF_OK : GAF_ERR_CUDA;
}
