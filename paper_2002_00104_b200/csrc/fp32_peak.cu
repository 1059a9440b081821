// FP32 pipe micro-benchmark: the denominator of the search kernels' roofline, measured on the
// device the benchmark runs on instead of derived from the data sheet.
//
// Every thread runs kChains independent dependency chains of one packed instruction
// (fma.rn.f32x2, add.rn.f32x2: two binary32 lanes per thread and instruction) or of the scalar
// fma.rn.f32, long enough to hide the pipe's latency with eight warps per scheduler; nothing
// else is in the loop.  The library proper does not use this file: it is built into a shared
// object of its own that only the benchmark loads.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

typedef unsigned long long u64;
constexpr int kChains = 8;
constexpr int kUnroll = 4;
constexpr int kThreads = 256;

__device__ __forceinline__ u64 pack2(float lo, float hi) {
    u64 r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi)); return r;
}
__device__ __forceinline__ u64 fma2(u64 a, u64 b, u64 c) {
    u64 d; asm volatile("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c)); return d;
}
__device__ __forceinline__ u64 add2(u64 a, u64 b) {
    u64 d; asm volatile("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d;
}

// MODE 0: scalar fma, 1: packed fma, 2: packed add.
template <int MODE>
__global__ void __launch_bounds__(kThreads) fp32_chain_kernel(float* out, int iters, float scale) {
    float a[kChains];
    u64 p[kChains];
#pragma unroll
    for (int i = 0; i < kChains; ++i) {
        a[i] = threadIdx.x * 1e-3f + i;
        p[i] = pack2(a[i], a[i] + 0.5f);
    }
    const u64 ss = pack2(scale, scale), cc = pack2(1e-3f, 1e-3f);
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
#pragma unroll
            for (int i = 0; i < kChains; ++i) {
                if (MODE == 0) a[i] = __fmaf_rn(a[i], scale, 1e-3f);
                else if (MODE == 1) p[i] = fma2(p[i], ss, cc);
                else p[i] = add2(p[i], cc);
            }
        }
    }
    float r = 0.0f;
#pragma unroll
    for (int i = 0; i < kChains; ++i)
        r += a[i] + __uint_as_float((unsigned)p[i]) + __uint_as_float((unsigned)(p[i] >> 32));
    out[(size_t)blockIdx.x * kThreads + threadIdx.x] = r;        // keeps the chains alive
}

}  // namespace

// Enqueues one launch of `blocks` CTAs of 256 threads, `iters` loop trips each, on `stream`.
// out: device buffer of blocks * 256 floats.  Returns 0, or a CUDA error code.  The launch
// executes blocks * 256 * iters * 32 thread-instructions, each worth pwlq_peak_lanes(mode) FP32
// lane-operations (one fma, or one add, per lane counts as one).
extern "C" int pwlq_peak_launch(int mode, int blocks, int iters, float* out, void* stream) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (mode == 0) fp32_chain_kernel<0><<<blocks, kThreads, 0, st>>>(out, iters, 1.0001f);
    else if (mode == 1) fp32_chain_kernel<1><<<blocks, kThreads, 0, st>>>(out, iters, 1.0001f);
    else if (mode == 2) fp32_chain_kernel<2><<<blocks, kThreads, 0, st>>>(out, iters, 1.0001f);
    else return -1;
    return (int)cudaGetLastError();
}
extern "C" int pwlq_peak_lanes(int mode) { return mode == 0 ? 1 : 2; }
extern "C" int pwlq_peak_instr_per_trip(void) { return kChains * kUnroll; }
extern "C" int pwlq_peak_threads(void) { return kThreads; }
