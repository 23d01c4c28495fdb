// replace_sample for callers that cannot allocate device memory: the per-call scratch lives in
// a fixed array that is part of the library image on every GPU that loads it.
#include <string.h>

#include <atomic>

#include "common.cuh"
#include "launch.h"

using namespace spr;

namespace {

// Limits of the built-in scratch (see include/sprinter.h).
constexpr int kMaxDraws = SPR_STATIC_MAX_DRAWS;
constexpr int kMaxDrawSteps = SPR_STATIC_MAX_DRAW_STEPS;
constexpr size_t kOffCounters = kHeaderBytes;
constexpr size_t kOffPart = kOffCounters + sizeof(int32_t) * (size_t)kMaxDraws;
constexpr size_t kScratchBytes = kOffPart + sizeof(float2) * (size_t)kMaxDrawSteps;
static_assert(kOffCounters % 256 == 0 && kOffPart % 256 == 0, "scratch regions must stay 256-byte aligned");

// ~516 KB of device memory per GPU, held from library load until process exit.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

// Device address of g_static_scratch per device ordinal.  In host code the array's name is
// only a handle for the runtime, never something a kernel may dereference; the address a
// kernel needs comes from cudaGetSymbolAddress, asked once per device while it is current.
// Host threads that make their first call on a device at the same time all look the address
// up and store the same value; the atomic only keeps that free of a data race.
constexpr int kMaxDevices = 64;
std::atomic<void *> g_scratch_addr[kMaxDevices];

int scratch_for_current_device(void **out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return report_cuda_error(e);
    if (dev < 0 || dev >= kMaxDevices) return SPR_ERR_UNSUPPORTED;
    void *ptr = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (!ptr) {
        e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return report_cuda_error(e);
        if (!ptr) return SPR_ERR_CUDA;
        g_scratch_addr[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
    return SPR_OK;
}

}  // namespace

extern "C" int replace_sample_static(const void *target_logits, int64_t ldv, int V, int64_t R,
                                     const int32_t *rows, const int32_t *first_reject, int K,
                                     int seq_stride, int n, const float *uniforms, int dt,
                                     int32_t *tokens, void *cuda_stream)
{
    if (dt != SPR_F32 && dt != SPR_BF16) return SPR_ERR_UNSUPPORTED;
    if (V <= 0 || ldv < V || R < 0 || n < 0 || seq_stride < 0) return SPR_ERR_INVALID_ARG;
    if (n == 0) return SPR_OK;
    if (!target_logits || !uniforms || !tokens || R == 0) return SPR_ERR_INVALID_ARG;
    if (first_reject && K <= 0) return SPR_ERR_INVALID_ARG;
    if (first_reject && !rows && n > 1 && seq_stride < K) return SPR_ERR_INVALID_ARG;
    const size_t es = elem_size(dt);
    if (reinterpret_cast<uintptr_t>(target_logits) % es || reinterpret_cast<uintptr_t>(uniforms) % 4 ||
        reinterpret_cast<uintptr_t>(tokens) % 4 || (rows && reinterpret_cast<uintptr_t>(rows) % 4) ||
        (first_reject && reinterpret_cast<uintptr_t>(first_reject) % 4))
        return SPR_ERR_INVALID_ARG;
    DrawParams dp = replace_params(target_logits, ldv, V, R, rows, first_reject, K, seq_stride, n, uniforms, dt,
                                   tokens);
    // the built-in scratch has room for kMaxDraws tickets and kMaxDrawSteps step partials
    if (n > kMaxDraws || (int64_t)n * dp.steps > kMaxDrawSteps) return SPR_ERR_WORKSPACE;

    int major = 0, dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return report_cuda_error(e);
    if (major != 10) return SPR_ERR_UNSUPPORTED;

    void *base = nullptr;
    int rc = scratch_for_current_device(&base);
    if (rc != SPR_OK) return rc;
    char *scratch = static_cast<char *>(base);
    dp.status = reinterpret_cast<int *>(scratch);
    dp.counters = reinterpret_cast<int *>(scratch + kOffCounters);
    dp.part = reinterpret_cast<float2 *>(scratch + kOffPart);

    // The array keeps whatever the previous call left: the tickets must start at zero (the
    // partials are always written before they are read, and the status word is not reported).
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    e = cudaMemsetAsync(dp.counters, 0, sizeof(int32_t) * (size_t)n, st);
    if (e == cudaSuccess) e = launch_draw(dp, dt, st);
    return e == cudaSuccess ? SPR_OK : report_cuda_error(e);
}
