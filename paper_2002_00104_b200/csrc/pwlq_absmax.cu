// Range m of every row: m_c = max_i |x_{c,i}|  (Sec. 3.2: quantization range [-m, m]).
//
// HBM-bound streaming reduction, 4 bytes read per value.  The flat storage is cut into spans of
// kAbsSpan values that persistent CTAs walk; the spans arrive in a ring of shared-memory slots
// filled by bulk asynchronous copies, three spans ahead.
// Magnitude bit patterns are folded with an integer maximum (exact and order-free).  A span that
// lies inside one row is folded into per-thread registers that live on from span to span (one
// atomic per warp when the row ends); a span that holds several rows is cut into one slice per
// warp, and the warp walks the rows overlapping its slice (offsets staged in shared memory) with
// a strided read, a shuffle reduction and one atomicMax per piece.
#include <algorithm>

#include "pwlq_common.cuh"
#include "pwlq_kernels.h"
#include "pwlq_pipeline.cuh"

namespace pwlq {

constexpr int kAbsThreads = 256;
constexpr int kAbsUnroll = 4;
constexpr int kAbsSpan = kAbsThreads * 4 * kAbsUnroll;  // values per span
constexpr int kAbsStages = 3;                            // spans in flight per CTA
constexpr int kAbsTableRows = 512;                       // staged rows per span (rows of >= 8 values fit)

static __device__ int g_absmax_timeout;                  // set when a bounded wait expired

struct AbsSmem {
    BulkRing<kAbsStages, kAbsSpan * 4> ring;
    SpanTable<false, kAbsTableRows> T;
};

// Bytes of span `span` if it can be fetched by a bulk copy (aligned base, whole 16-byte units).
__device__ __forceinline__ unsigned abs_bulk_bytes(int64_t span, int64_t total, int vec_ok) {
    const int64_t beg = span * kAbsSpan;
    const int64_t cnt = min((int64_t)kAbsSpan, total - beg);
    return (vec_ok && (cnt & 3) == 0) ? (unsigned)(cnt * 4) : 0u;
}

__global__ void __launch_bounds__(kAbsThreads)
absmax_kernel(const float* __restrict__ x, Rows rows, int64_t total, uint32_t* __restrict__ m_bits,
              int vec_ok, int64_t spans_per_cta) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    AbsSmem& S = *reinterpret_cast<AbsSmem*>(smem_raw);
    __shared__ int s_abort;
    const int64_t nspans = (total + kAbsSpan - 1) / kAbsSpan;
    // this CTA's consecutive spans
    const int64_t s0 = blockIdx.x * spans_per_cta, s1 = min(s0 + spans_per_cta, nspans);
    const bool use_table = rows.offsets != nullptr || rows.n < kAbsSpan;   // several rows per span
    if (threadIdx.x == 0) s_abort = 0;
    S.ring.init();
    for (int it = 0; it < kAbsStages; ++it)
        if (s0 + it < s1)
            S.ring.issue(it, x + (s0 + it) * kAbsSpan, abs_bulk_bytes(s0 + it, total, vec_ok));

    int64_t row0 = 0;                                  // first staged row of the current span
    RowFetch<kAbsTableRows> nf;
    if (use_table && s0 < s1) {
        row0 = cta_row_near(rows, s0 * kAbsSpan);
        S.T.fetch(rows, nullptr, nullptr, row0, nf);
        S.T.commit(nf, 0.0f);
        __syncthreads();
    }

    // The long row the CTA is inside of (the same for all of its threads) and this thread's
    // maximum over it; both survive from span to span, so a long row costs one atomic per warp
    // for the whole kernel.
    int64_t grow = -1;
    uint32_t mx = 0;
    auto flush_merged = [&]() {                        // every lane of the warp calls this
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        if ((threadIdx.x & 31) == 0 && mx != 0 && grow >= 0) atomicMax(m_bits + grow, mx);
        mx = 0;
    };

    for (int64_t span = s0; span < s1; ++span) {
        const int64_t it = span - s0;
        const int64_t span_beg = span * kAbsSpan;
        const int64_t span_end = min(span_beg + kAbsSpan, total);
        // Does the span lie inside one row?
        bool single;
        int64_t first_row;
        if (use_table) {
            const int l0 = S.T.find(span_beg);          // -1: more rows than the window holds
            first_row = row0 + l0;
            single = l0 >= 0 && S.T.off[l0 + 1] >= span_end;
        } else {
            first_row = rows.dense_row(span_beg);
            single = (first_row + 1) * rows.n >= span_end;
        }
        // the staged rows end before the next span does: request the window that starts in the
        // row in which this span ends
        int64_t next_row0 = 0;
        const bool has_next = use_table && span + 1 < s1 &&
                              !S.T.covers(min(span_end + kAbsSpan, total));
        if (has_next) {
            const int l = S.T.find(span_end);
            next_row0 = (l >= 0) ? row0 + l : warp_row_of(rows, span_end);
            S.T.fetch(rows, nullptr, nullptr, next_row0, nf);
        }
        if (!single) {                                 // several rows: nothing is carried across
            flush_merged();
            grow = -1;
        } else if (grow != first_row) {                // a new long row begins
            flush_merged();
            grow = first_row;
        }

        float* xs = reinterpret_cast<float*>(S.ring.slot(it));
        if (abs_bulk_bytes(span, total, vec_ok) != 0) {
            if (!S.ring.wait(it, (unsigned)(it / kAbsStages))) s_abort = 1;   // never expected
        } else {                                       // unaligned base or ragged tail: plain loads
            for (int i = threadIdx.x; i < (int)(span_end - span_beg); i += kAbsThreads)
                xs[i] = x[span_beg + i];
            __syncthreads();
        }
        if (single) {
            // the whole span belongs to the carried row: registers only
#pragma unroll
            for (int j = 0; j < kAbsUnroll; ++j) {
                const int li = (j * kAbsThreads + threadIdx.x) * 4;
                if (span_beg + li + 4 <= span_end) {
                    const float4 v = *reinterpret_cast<const float4*>(xs + li);
                    mx = max(max(mx, abs_bits(v.x)),
                             max(abs_bits(v.y), max(abs_bits(v.z), abs_bits(v.w))));
                } else {
                    for (int t = 0; t < 4; ++t)
                        if (span_beg + li + t < span_end) mx = max(mx, abs_bits(xs[li + t]));
                }
            }
        } else {
            // several rows: every warp takes a contiguous slice of the span and walks it in
            // windows of 128 values (one 128-bit read per lane).  The maximum of the row the warp
            // is in stays in per-lane registers from window to window; when the row ends inside a
            // window the lanes' values are split at the boundary, the finished row is reduced with
            // one warp-wide maximum and one atomic, and the next row starts.  All control flow is
            // warp-uniform.
            const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
            constexpr int kSlice = kAbsSpan / (kAbsThreads / 32);
            const int sl_beg = warp * kSlice;                              // relative to the span
            const int sl_end = min(sl_beg + kSlice, (int)(span_end - span_beg));
            if (sl_beg < sl_end) {
                int l = use_table ? S.T.find(span_beg + sl_beg) : -1;
                int64_t r_glob = 0;
                int r_end = 0;                                             // relative to the span
                auto enter_row = [&](int pos) {            // the row that contains / follows pos
                    int64_t e;
                    if (l >= 0 && l < kAbsTableRows) {     // staged row
                        r_glob = row0 + l;
                        e = S.T.off[l + 1];
                        ++l;
                    } else {                               // long dense rows, or beyond the table
                        r_glob = rows.row_of(span_beg + pos);
                        e = rows.begin(r_glob + 1);
                        l = -1;
                    }
                    r_end = (int)min(e - span_beg, (int64_t)kAbsSpan);
                };
                enter_row(sl_beg);
                uint32_t v = 0;
                for (int wb = sl_beg; wb < sl_end; wb += 128) {
                    const int we = min(wb + 128, sl_end);
                    const int i0 = wb + 4 * lane;
                    uint32_t b[4] = {0u, 0u, 0u, 0u};
                    if (i0 + 4 <= we) {
                        const float4 f = *reinterpret_cast<const float4*>(xs + i0);
                        b[0] = abs_bits(f.x); b[1] = abs_bits(f.y);
                        b[2] = abs_bits(f.z); b[3] = abs_bits(f.w);
                    } else {
#pragma unroll
                        for (int t = 0; t < 4; ++t)
                            if (i0 + t < we) b[t] = abs_bits(xs[i0 + t]);
                    }
                    if (r_end >= we) {                     // the window lies inside the current row
                        v = max(max(v, b[0]), max(b[1], max(b[2], b[3])));
                        continue;
                    }
                    int pos = wb;                          // values before pos are accounted for
                    while (true) {
                        const int e = min(r_end, we);
#pragma unroll
                        for (int t = 0; t < 4; ++t)
                            if (i0 + t >= pos && i0 + t < e) v = max(v, b[t]);
                        if (r_end > we) break;             // the row continues in the next window
                        v = __reduce_max_sync(0xffffffffu, v);
                        if (lane == 0 && v != 0) atomicMax(m_bits + r_glob, v);
                        v = 0;
                        pos = e;
                        if (pos >= sl_end) break;          // the slice ends with this row
                        enter_row(pos);
                        if (pos >= we) break;              // the new row starts with the next window
                    }
                }
                v = __reduce_max_sync(0xffffffffu, v);     // the row the slice ends in
                if (lane == 0 && v != 0) atomicMax(m_bits + r_glob, v);
            }
        }
        __syncthreads();                              // slot and table are no longer read
        if (s_abort) {                                 // a wait ran out: report and leave
            if (threadIdx.x == 0) atomicExch(&g_absmax_timeout, 1);
            return;
        }
        if (has_next) { S.T.commit(nf, 0.0f); row0 = next_row0; }
        if (span + kAbsStages < s1)
            S.ring.issue(it + kAbsStages, x + (span + kAbsStages) * kAbsSpan,
                         abs_bulk_bytes(span + kAbsStages, total, vec_ok));
        if (has_next) __syncthreads();                // the next window is published
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
    Rows rows{row_offsets, C, n, n > 0 ? 1.0 / (double)n : 0.0};
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
    // Long dense rows cost the same everywhere: one CTA per slot of the device, equal shares.
    // Where spans hold several rows the cost per span depends on the row lengths, so the spans are
    // handed out in small blocks (about four per slot) and the hardware scheduler balances them.
    const int64_t slots = cached[dev];
    const bool several_rows = row_offsets != nullptr || n < kAbsSpan;
    int64_t per_cta = (nspans + slots - 1) / slots;
    if (several_rows) per_cta = std::min<int64_t>(std::max<int64_t>((nspans + 4 * slots - 1) / (4 * slots), 4), 32);
    const unsigned grid = (unsigned)((nspans + per_cta - 1) / per_cta);
    const int vec_ok = (reinterpret_cast<uintptr_t>(x) & 15u) == 0;
    absmax_kernel<<<grid, kAbsThreads, sizeof(AbsSmem), stream>>>(
        x, rows, total, reinterpret_cast<uint32_t*>(m_out), vec_ok, per_cta);
    return cudaGetLastError();
}

}  // namespace pwlq
