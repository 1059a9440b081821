// Row maps of a layout, built ahead of time (see pwlq_rowmap.cuh).  The streaming kernels
// (abs-max, quantize, dequantize) describe, per span of 4096 values, which rows overlap the span;
// that description depends on the row offsets only.  A caller that runs several such calls over
// one layout -- abs-max, then quantize, then dequantize of the same weights, or the same layout
// batch after batch -- has the maps built once here and passes them to the *_mapped entry points.
#include <algorithm>

#include "pwlq_kernels.h"
#include "pwlq_rowmap.cuh"

namespace pwlq {

constexpr int kBuildWarps = 4;

// One warp per span: finds the span's first row (a 32-ary search over the offsets), writes the
// map into shared memory with the code the kernels' own producers use, and copies it out.
__global__ void __launch_bounds__(kBuildWarps * 32)
rowmap_build_kernel(Rows rows, int64_t total, unsigned char* __restrict__ out) {
    __shared__ SpanRowMap maps[kBuildWarps];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t nspans = (total + kMapSpan - 1) / kMapSpan;
    const int64_t span = (int64_t)blockIdx.x * kBuildWarps + warp;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        RowMapHeader* h = reinterpret_cast<RowMapHeader*>(out);
        h->magic = kRowMapMagic;
        h->C = rows.C;
        h->total = total;
        h->n = rows.offsets ? 0 : rows.n;
    }
    if (span >= nspans) return;
    const int64_t span_beg = span * kMapSpan, span_end = min(span_beg + kMapSpan, total);
    MapProducer<false, false> prod;
    prod.rows = rows;
    prod.in = RowInputs{nullptr, nullptr, nullptr, nullptr, nullptr};
    prod.Lf = 0.0f;
    prod.request(warp_row_of(rows, span_beg), true);
    prod.build(maps[warp], nullptr, nullptr, span_beg, span_end, false);
    __syncwarp();
    const uint4* src = reinterpret_cast<const uint4*>(&maps[warp]);
    uint4* dst = reinterpret_cast<uint4*>(out + kRowMapHeaderBytes + (size_t)span * sizeof(SpanRowMap));
    for (int i = lane; i < (int)(sizeof(SpanRowMap) / 16); i += 32) dst[i] = src[i];
}

size_t rowmap_bytes(int64_t total) {
    const int64_t nspans = (total + kMapSpan - 1) / kMapSpan;
    return kRowMapHeaderBytes + (size_t)nspans * sizeof(SpanRowMap);
}

cudaError_t launch_rowmap_build(const int64_t* row_offsets, int64_t C, int64_t n, int64_t total,
                                void* rowmap, cudaStream_t stream) {
    // the header goes first, so that maps of an empty layout are recognised too
    Rows rows{row_offsets, C, n, n > 0 ? 1.0 / (double)n : 0.0, 0};
    const int64_t nspans = (total + kMapSpan - 1) / kMapSpan;
    const unsigned grid = (unsigned)std::max<int64_t>((nspans + kBuildWarps - 1) / kBuildWarps, 1);
    rowmap_build_kernel<<<grid, kBuildWarps * 32, 0, stream>>>(
        rows, total, static_cast<unsigned char*>(rowmap));
    return cudaGetLastError();
}

}  // namespace pwlq
