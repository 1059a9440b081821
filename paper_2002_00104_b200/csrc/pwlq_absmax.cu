// Range m of every row: m_c = max_i |x_{c,i}|  (Sec. 3.2: quantization range [-m, m]).
//
// HBM-bound streaming reduction.  The flat storage is cut into spans of kSpan values, one CTA
// per span; a thread reads 128-bit vectors that lie inside one row and folds the magnitude bit
// patterns with an integer maximum (exact and order-free), and hands its result to the row's
// slot with atomicMax -- after a warp-shuffle and a block-level merge whenever the whole warp /
// CTA worked on the same row, so that a long row costs one atomic per CTA.
#include "pwlq_common.cuh"
#include "pwlq_kernels.h"

namespace pwlq {

constexpr int kAbsThreads = 256;
constexpr int kAbsUnroll = 8;
constexpr int kAbsSpan = kAbsThreads * 4 * kAbsUnroll;  // values per CTA

__global__ void __launch_bounds__(kAbsThreads)
absmax_kernel(const float* __restrict__ x, Rows rows, int64_t total, uint32_t* __restrict__ m_bits,
              int vec_ok) {
    const int64_t span_base = (int64_t)blockIdx.x * kAbsSpan;
    int64_t row = -1, row_beg = 0, row_end = 0;   // row currently accumulated by this thread
    uint32_t mx = 0;

    auto flush = [&]() {
        if (row >= 0 && mx != 0) atomicMax(m_bits + row, mx);
    };
    auto enter_row_of = [&](int64_t i) {
        flush();
        row = rows.row_of(i);
        row_beg = rows.begin(row);
        row_end = rows.begin(row + 1);
        mx = 0;
    };

#pragma unroll
    for (int j = 0; j < kAbsUnroll; ++j) {
        const int64_t i = span_base + ((int64_t)j * kAbsThreads + threadIdx.x) * 4;
        if (i >= total) break;
        if (vec_ok && i + 4 <= total) {
            const float4 v = __ldg(reinterpret_cast<const float4*>(x + i));
            if (!(i >= row_beg && i + 4 <= row_end)) {
                enter_row_of(i);
            }
            if (i + 4 <= row_end) {
                mx = max(max(mx, abs_bits(v.x)), max(abs_bits(v.y), max(abs_bits(v.z), abs_bits(v.w))));
            } else {                                   // the vector straddles a row boundary
                const float e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    if (i + t >= row_end) enter_row_of(i + t);
                    mx = max(mx, abs_bits(e[t]));
                }
            }
        } else {
            for (int t = 0; t < 4 && i + t < total; ++t) {
                if (!(i + t >= row_beg && i + t < row_end)) enter_row_of(i + t);
                mx = max(mx, abs_bits(x[i + t]));
            }
        }
    }

    // Merge within the warp, then within the CTA, when everybody holds the same row.
    const unsigned full = 0xffffffffu;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row0 = __shfl_sync(full, row, 0);
    const bool warp_uniform = __all_sync(full, row == row0);
    __shared__ int64_t s_row[kAbsThreads / 32];
    __shared__ uint32_t s_max[kAbsThreads / 32];
    if (warp_uniform) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(full, mx, o));
        if (lane == 0) { s_row[warp] = row; s_max[warp] = mx; }
    } else {
        flush();
        if (lane == 0) { s_row[warp] = -1; s_max[warp] = 0; }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        // consecutive warps with the same row are merged before touching global memory
        int64_t r = -1;
        uint32_t v = 0;
        for (int w = 0; w < kAbsThreads / 32; ++w) {
            if (s_row[w] != r) {
                if (r >= 0 && v != 0) atomicMax(m_bits + r, v);
                r = s_row[w];
                v = 0;
            }
            v = max(v, s_max[w]);
        }
        if (r >= 0 && v != 0) atomicMax(m_bits + r, v);
    }
}

cudaError_t launch_absmax(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                          int64_t total, float* m_out, cudaStream_t stream) {
    cudaError_t e = cudaMemsetAsync(m_out, 0, sizeof(float) * (size_t)C, stream);
    if (e != cudaSuccess) return e;
    if (total == 0) return cudaSuccess;
    Rows rows{row_offsets, C, n};
    const int64_t grid = (total + kAbsSpan - 1) / kAbsSpan;
    const int vec_ok = (reinterpret_cast<uintptr_t>(x) & 15u) == 0;
    absmax_kernel<<<(unsigned)grid, kAbsThreads, 0, stream>>>(
        x, rows, total, reinterpret_cast<uint32_t*>(m_out), vec_ok);
    return cudaGetLastError();
}

}  // namespace pwlq
