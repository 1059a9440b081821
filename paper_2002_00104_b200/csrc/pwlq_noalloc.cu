// Breakpoint search for callers that cannot allocate device memory.
//
// pwlq_search needs a caller-provided workspace (status word, internally computed ranges, the
// partial sums of rows longer than one tile).  Some callers have no way to obtain one: a plugin
// inside a host application whose memory pool already owns the whole device, so that cudaMalloc
// fails or is forbidden by the host's rules; a latency-critical loop that must not hit
// cudaMalloc's implicit device-wide synchronisation; a component that is only handed input and
// output buffers.  For them the workspace lives in a fixed array in device global memory that is
// part of the library image: every GPU on which the library is used holds
// PWLQ_NOALLOC_SCRATCH_BYTES of it from the moment the module is loaded until the process exits.
#include <mutex>

#include "../../include/pwlq.h"
#include "pwlq_kernels.h"

namespace {

// The scratch itself.  In host code this name is only a handle for the runtime, NOT a device
// address: the address the kernels need is obtained with cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_noalloc_scratch[PWLQ_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the scratch on the current device; resolved once per device, with that
// device current, on the first call made there.
int scratch_for_current_device(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PWLQ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_addr[dev]) {
        void* ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
        if (e != cudaSuccess || !ptr) return PWLQ_ERR_CUDA;
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return PWLQ_OK;
}

inline bool misaligned(const void* p, size_t a) {
    return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0;
}

}  // namespace

extern "C" int pwlq_search_noalloc(const float* x, int64_t C, int64_t n, int bits,
                                   const float* ratios, int K, const float* m, float* p_out,
                                   float* err_out, int32_t* idx_out, float* sse_all,
                                   int32_t* status_out, void* stream) {
    if (C < 1 || n < 1 || !x || !ratios || !p_out || !idx_out || bits < 2 || bits > 8 || K < 1)
        return PWLQ_ERR_INVALID_ARG;
    if (misaligned(x, 4) || misaligned(ratios, 4) || misaligned(m, 4) || misaligned(p_out, 4) ||
        misaligned(err_out, 4) || misaligned(idx_out, 4) || misaligned(sse_all, 4) ||
        misaligned(status_out, 4))
        return PWLQ_ERR_INVALID_ARG;
    if (K > PWLQ_MAX_K || C > ((int64_t)1 << 31) - 1 || n > ((int64_t)1 << 40) / C)
        return PWLQ_ERR_UNSUPPORTED;
    const pwlq::SearchPlan plan = pwlq::plan_search(C, n, K);
    if (plan.bytes > (size_t)PWLQ_NOALLOC_SCRATCH_BYTES || C * plan.tiles > ((int64_t)1 << 31) - 1)
        return PWLQ_ERR_UNSUPPORTED;      // the problem does not fit the built-in scratch
    void* scratch = nullptr;
    if (int rc = scratch_for_current_device(&scratch)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // launch_search clears the status word and writes every range and partial sum it later
    // reads, so nothing of the previous call's contents is consumed.
    cudaError_t e = pwlq::launch_search(x, nullptr, C, n, C * n, bits, ratios, K, m, nullptr, p_out,
                                        err_out, idx_out, sse_all, scratch, plan, st);
    if (e != cudaSuccess) return PWLQ_ERR_CUDA;
    if (status_out) {
        e = cudaMemcpyAsync(status_out, scratch, sizeof(int32_t), cudaMemcpyDeviceToDevice, st);
        if (e != cudaSuccess) return PWLQ_ERR_CUDA;
    }
    return PWLQ_OK;
}

extern "C" size_t pwlq_search_noalloc_max_bytes(void) { return PWLQ_NOALLOC_SCRATCH_BYTES; }
