// Range m of every row: m_c = max_i |x_{c,i}|  (Sec. 3.2: quantization range [-m, m]).
//
// HBM-bound streaming reduction, 4 bytes read per value.  The flat storage is cut into spans of
// kAbsSpan values that persistent CTAs walk; the spans arrive in a ring of shared-memory slots
// filled by bulk asynchronous copies, three spans ahead.
// A thread folds the magnitude bit patterns with an integer maximum (exact and order-free).  The
// rows that overlap the span are staged in shared memory together with one maximum per row;
// threads merge into those with shared-memory atomics (once per row they touch, after a warp
// shuffle when the whole warp sits in one row), and the CTA issues one global atomicMax per row
// of its span.
#include "pwlq_common.cuh"
#include "pwlq_kernels.h"
#include "pwlq_pipeline.cuh"

namespace pwlq {

constexpr int kAbsThreads = 256;
constexpr int kAbsUnroll = 4;
constexpr int kAbsSpan = kAbsThreads * 4 * kAbsUnroll;  // values per span
constexpr int kAbsRows = 1024;                           // staged rows per span
constexpr int kAbsStages = 3;                            // spans in flight per CTA

static __device__ int g_absmax_timeout;                  // set when a bounded wait expired

struct AbsSmem {
    BulkRing<kAbsStages, kAbsSpan * 4> ring;
    RowTable<kAbsRows> T;
    uint32_t s_max[kAbsRows];
};

// Bytes of span `span` if it can be fetched by a bulk copy (aligned base, whole 16-byte units).
__device__ __forceinline__ unsigned abs_bulk_bytes(int64_t span, int64_t total, int vec_ok) {
    const int64_t beg = span * kAbsSpan;
    const int64_t cnt = min((int64_t)kAbsSpan, total - beg);
    return (vec_ok && (cnt & 3) == 0) ? (unsigned)(cnt * 4) : 0u;
}

__global__ void __launch_bounds__(kAbsThreads)
absmax_kernel(const float* __restrict__ x, Rows rows, int64_t total, uint32_t* __restrict__ m_bits,
              int vec_ok) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    AbsSmem& S = *reinterpret_cast<AbsSmem*>(smem_raw);
    __shared__ int s_abort;
    const int64_t nspans = (total + kAbsSpan - 1) / kAbsSpan;
    const bool ragged = rows.offsets != nullptr;
    if (threadIdx.x == 0) s_abort = 0;
    S.ring.init();
    for (int it = 0; it < kAbsStages; ++it) {
        const int64_t span = blockIdx.x + (int64_t)it * gridDim.x;
        if (span < nspans)
            S.ring.issue(it, x + span * kAbsSpan, abs_bulk_bytes(span, total, vec_ok));
    }

    // The row a thread is accumulating; it survives from span to span, so a long row costs one
    // atomic per warp for the whole kernel.  loc >= 0: the row has a slot in S.s_max.
    int loc = -1;
    int64_t grow = -1, row_beg = 0, row_end = 0;
    uint32_t mx = 0;
    auto flush = [&]() {
        if (mx == 0) return;
        if (loc >= 0) atomicMax(&S.s_max[loc], mx);
        else if (grow >= 0) atomicMax(m_bits + grow, mx);
        mx = 0;
    };

    // Same, after merging inside the warp when all of its lanes carry the same long row (every
    // lane of the warp must call this).
    auto flush_merged = [&]() {
        const unsigned full = 0xffffffffu;
        const int64_t g0 = __shfl_sync(full, grow, 0);
        if (__all_sync(full, grow == g0 && loc < 0)) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(full, mx, o));
            if ((threadIdx.x & 31) != 0) mx = 0;
        }
        flush();
    };

    int64_t it = 0;
    for (int64_t span = blockIdx.x; span < nspans; span += gridDim.x, ++it) {
        const int64_t span_beg = span * kAbsSpan;
        const int64_t span_end = min(span_beg + kAbsSpan, total);
        // Does the span lie inside one row?  Dense: arithmetic.  Ragged: after staging the rows.
        bool single;
        int64_t first_row = 0;
        if (ragged) {
            S.T.load(rows, span_beg);                 // two barriers
            first_row = S.T.row0;
            single = S.T.off[1] >= span_end;
        } else {
            first_row = span_beg / rows.n;
            single = (first_row + 1) * rows.n >= span_end;
        }
        if (!single) {                                 // several rows: merge through shared memory
            flush_merged();
            loc = -1; grow = -1; row_beg = row_end = 0;
            for (int r = threadIdx.x; r < kAbsRows; r += kAbsThreads) S.s_max[r] = 0;
            __syncthreads();
        } else if (grow != first_row) {                // a new long row begins
            flush_merged();
            loc = -1;
            grow = first_row;
            row_beg = rows.begin(grow);
            row_end = rows.begin(grow + 1);
        }
        auto enter = [&](int64_t i) {                  // only reached when the span has several rows
            flush();
            if (ragged) {
                const int l = S.T.find(i);
                if (l >= 0) { loc = l; grow = S.T.row0 + l; row_beg = S.T.off[l]; row_end = S.T.off[l + 1]; }
                else { loc = -1; grow = rows.row_of(i); row_beg = rows.begin(grow); row_end = rows.begin(grow + 1); }
            } else {
                grow = i / rows.n;
                row_beg = grow * rows.n;
                row_end = row_beg + rows.n;
                loc = (grow - first_row < kAbsRows) ? (int)(grow - first_row) : -1;
            }
        };

        float* xs = reinterpret_cast<float*>(S.ring.slot(it));
        if (abs_bulk_bytes(span, total, vec_ok) != 0) {
            if (!S.ring.wait(it, (unsigned)(it / kAbsStages))) s_abort = 1;   // never expected
        } else {                                       // unaligned base or ragged tail: plain loads
            for (int i = threadIdx.x; i < (int)(span_end - span_beg); i += kAbsThreads)
                xs[i] = x[span_beg + i];
            __syncthreads();
        }
#pragma unroll
        for (int j = 0; j < kAbsUnroll; ++j) {
            const int li = (j * kAbsThreads + threadIdx.x) * 4;
            const int64_t i = span_beg + li;
            if (i < total) {
                const float4 v = *reinterpret_cast<const float4*>(xs + li);
                const float e[4] = {v.x, v.y, v.z, v.w};
                if (i >= row_beg && i + 4 <= row_end) {    // still inside the current row
                    mx = max(max(mx, abs_bits(e[0])),
                             max(abs_bits(e[1]), max(abs_bits(e[2]), abs_bits(e[3]))));
                } else {
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        if (i + t < total) {
                            if (!(i + t >= row_beg && i + t < row_end)) enter(i + t);
                            mx = max(mx, abs_bits(e[t]));
                        }
                    }
                }
            }
        }
        if (!single) {
            flush();
            loc = -1; grow = -1; row_beg = row_end = 0;
            __syncthreads();
            for (int r = threadIdx.x; r < kAbsRows; r += kAbsThreads)
                if (S.s_max[r] != 0) atomicMax(m_bits + first_row + r, S.s_max[r]);
        }
        __syncthreads();                              // slot, table and maxima are free again
        if (s_abort) {                                 // a wait ran out: report and leave
            if (threadIdx.x == 0) atomicExch(&g_absmax_timeout, 1);
            return;
        }
        const int64_t ahead = span + (int64_t)kAbsStages * gridDim.x;
        if (ahead < nspans)
            S.ring.issue(it + kAbsStages, x + ahead * kAbsSpan, abs_bulk_bytes(ahead, total, vec_ok));
    }
    flush_merged();                                   // what is still carried at the end
}

int absmax_timeout_flag() {
    int v = 0;
    cudaMemcpyFromSymbol(&v, g_absmax_timeout, sizeof(int));
    return v;
}

cudaError_t launch_absmax(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                          int64_t total, float* m_out, cudaStream_t stream) {
    cudaError_t e = cudaMemsetAsync(m_out, 0, sizeof(float) * (size_t)C, stream);
    if (e != cudaSuccess) return e;
    if (total == 0) return cudaSuccess;
    Rows rows{row_offsets, C, n};
    const int64_t nspans = (total + kAbsSpan - 1) / kAbsSpan;
    static int cached[64] = {0};                       // CTAs that fit the device at once
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) dev = 0;
    if (cached[dev] == 0) {
        e = cudaFuncSetAttribute(absmax_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)sizeof(AbsSmem));
        if (e != cudaSuccess) return e;
        int sms = 0, per_sm = 0;
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, absmax_kernel, kAbsThreads,
                                                      sizeof(AbsSmem));
        cached[dev] = (sms > 0 && per_sm > 0) ? sms * per_sm : 148;
    }
    const unsigned grid = (unsigned)(nspans < cached[dev] ? nspans : cached[dev]);
    const int vec_ok = (reinterpret_cast<uintptr_t>(x) & 15u) == 0;
    absmax_kernel<<<grid, kAbsThreads, sizeof(AbsSmem), stream>>>(
        x, rows, total, reinterpret_cast<uint32_t*>(m_out), vec_ok);
    return cudaGetLastError();
}

}  // namespace pwlq
