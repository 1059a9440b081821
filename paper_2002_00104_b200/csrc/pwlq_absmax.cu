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

// Order-preserving map of binary32 values onto unsigned integers (and back), so that minima and
// maxima of signed values can use integer atomics.
__device__ __forceinline__ uint32_t ordered_key(float x) {
    const uint32_t b = __float_as_uint(x);
    return b ^ ((uint32_t)((int32_t)b >> 31) | 0x80000000u);
}
__device__ __forceinline__ float from_ordered_key(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k ^ 0x80000000u) : ~k);
}

// What is folded over a row.  MINMAX = false: the maximum of the magnitude bit patterns (exact and
// order-free).  MINMAX = true: the maximum of the ordered keys and the maximum of the inverted
// keys (i.e. the minimum); 0 means "nothing seen" in both.
template <bool MINMAX>
struct Fold {
    uint32_t a = 0, b = 0;
    __device__ __forceinline__ void add(float x) {
        if (MINMAX) {
            const uint32_t k = ordered_key(x);
            a = max(a, k);
            b = max(b, ~k);
        } else {
            a = max(a, abs_bits(x));
        }
    }
    __device__ __forceinline__ void add4(const float4 v) { add(v.x); add(v.y); add(v.z); add(v.w); }
    __device__ __forceinline__ void reduce_warp() {
        a = __reduce_max_sync(0xffffffffu, a);
        if (MINMAX) b = __reduce_max_sync(0xffffffffu, b);
    }
    __device__ __forceinline__ void store(uint32_t* hi, uint32_t* lo, int64_t row) const {
        if (a != 0) atomicMax(hi + row, a);
        if (MINMAX && b != 0) atomicMax(lo + row, b);
    }
    __device__ __forceinline__ void clear() { a = b = 0; }
};

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

template <bool MINMAX>
__global__ void __launch_bounds__(kAbsThreads)
absmax_kernel(const float* __restrict__ x, Rows rows, int64_t total, uint32_t* __restrict__ m_bits,
              uint32_t* __restrict__ lo_bits, int vec_ok, int64_t spans_per_cta) {
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
        S.T.fetch(rows, nullptr, nullptr, nullptr, row0, nf);
        S.T.commit(nf, 0, 0.0f);
        __syncthreads();
    }

    // The long row the CTA is inside of (the same for all of its threads) and this thread's
    // maximum over it; both survive from span to span, so a long row costs one atomic per warp
    // for the whole kernel.
    int64_t grow = -1;
    Fold<MINMAX> mx;
    auto flush_merged = [&]() {                        // every lane of the warp calls this
        mx.reduce_warp();
        if ((threadIdx.x & 31) == 0 && grow >= 0) mx.store(m_bits, lo_bits, grow);
        mx.clear();
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
            S.T.fetch(rows, nullptr, nullptr, nullptr, next_row0, nf);
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
                    mx.add4(*reinterpret_cast<const float4*>(xs + li));
                } else {
                    for (int t = 0; t < 4; ++t)
                        if (span_beg + li + t < span_end) mx.add(xs[li + t]);
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
                Fold<MINMAX> v;
                for (int wb = sl_beg; wb < sl_end; wb += 128) {
                    const int we = min(wb + 128, sl_end);
                    const int i0 = wb + 4 * lane;
                    float f[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                    const bool whole = i0 + 4 <= we;       // all four values lie inside the window
                    if (whole) {
                        const float4 q = *reinterpret_cast<const float4*>(xs + i0);
                        f[0] = q.x; f[1] = q.y; f[2] = q.z; f[3] = q.w;
                    } else {
#pragma unroll
                        for (int t = 0; t < 4; ++t)
                            if (i0 + t < we) f[t] = xs[i0 + t];
                    }
                    if (r_end >= we) {                     // the window lies inside the current row
                        if (whole) {
                            v.add4(make_float4(f[0], f[1], f[2], f[3]));
                        } else {
#pragma unroll
                            for (int t = 0; t < 4; ++t)
                                if (i0 + t < we) v.add(f[t]);
                        }
                        continue;
                    }
                    int pos = wb;                          // values before pos are accounted for
                    while (true) {
                        const int e = min(r_end, we);
#pragma unroll
                        for (int t = 0; t < 4; ++t)
                            if (i0 + t >= pos && i0 + t < e) v.add(f[t]);
                        if (r_end > we) break;             // the row continues in the next window
                        v.reduce_warp();
                        if (lane == 0) v.store(m_bits, lo_bits, r_glob);
                        v.clear();
                        pos = e;
                        if (pos >= sl_end) break;          // the slice ends with this row
                        enter_row(pos);
                        if (pos >= we) break;              // the new row starts with the next window
                    }
                }
                v.reduce_warp();                           // the row the slice ends in
                if (lane == 0) v.store(m_bits, lo_bits, r_glob);
            }
        }
        __syncthreads();                              // slot and table are no longer read
        if (s_abort) {                                 // a wait ran out: report and leave
            if (threadIdx.x == 0) atomicExch(&g_absmax_timeout, 1);
            return;
        }
        if (has_next) { S.T.commit(nf, 0, 0.0f); row0 = next_row0; }
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

// Turns the folded keys of minmax into values, in place.  A row in which nothing was seen (an
// empty row) gets lo = hi = 0; zeros are delivered as +0.
__global__ void minmax_finalize_kernel(uint32_t* __restrict__ lo_bits,
                                       uint32_t* __restrict__ hi_bits, int64_t C) {
    const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    const uint32_t kh = hi_bits[c], kl = lo_bits[c];
    float hi = 0.0f, lo = 0.0f;
    if (kh != 0 || kl != 0) {
        hi = from_ordered_key(kh);
        lo = from_ordered_key(~kl);
    }
    if (hi == 0.0f) hi = 0.0f;
    if (lo == 0.0f) lo = 0.0f;
    hi_bits[c] = __float_as_uint(hi);
    lo_bits[c] = __float_as_uint(lo);
}

// Launches the folding kernel: MINMAX = false writes the abs-max bit patterns to out_a;
// MINMAX = true folds ordered keys of the maxima into out_a and of the minima into out_b.
template <bool MINMAX>
static cudaError_t launch_fold(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                               int64_t total, float* out_a, float* out_b, cudaStream_t stream,
                               int64_t shift) {
    cudaError_t e = cudaMemsetAsync(out_a, 0, sizeof(float) * (size_t)C, stream);
    if (e != cudaSuccess) return e;
    if (MINMAX) {
        e = cudaMemsetAsync(out_b, 0, sizeof(float) * (size_t)C, stream);
        if (e != cudaSuccess) return e;
    }
    if (total == 0) return cudaSuccess;
    Rows rows{row_offsets, C, n, n > 0 ? 1.0 / (double)n : 0.0, row_offsets ? shift : 0};
    const int64_t nspans = (total + kAbsSpan - 1) / kAbsSpan;
    static int cached[64] = {0};                       // CTAs that fit the device at once
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) dev = 0;
    if (cached[dev] == 0) {
        e = cudaFuncSetAttribute(absmax_kernel<MINMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)sizeof(AbsSmem));
        if (e != cudaSuccess) return e;
        int sms = 0, per_sm = 0;
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, absmax_kernel<MINMAX>, kAbsThreads,
                                                      sizeof(AbsSmem));
        cached[dev] = (sms > 0 && per_sm > 0) ? sms * per_sm : 148;
    }
    // Long dense rows cost the same everywhere: one CTA per slot of the device, equal shares.
    // Where spans hold several rows the cost per span depends on the row lengths, so the spans are
    // handed out in small blocks (about four per slot) and the hardware scheduler balances them.
    const int64_t slots = cached[dev];
    const bool several_rows = row_offsets != nullptr || n < kAbsSpan;
    int64_t per_cta = (nspans + slots - 1) / slots;
    if (several_rows)
        per_cta = std::min<int64_t>(std::max<int64_t>((nspans + 4 * slots - 1) / (4 * slots), 4), 32);
    const unsigned grid = (unsigned)((nspans + per_cta - 1) / per_cta);
    const int vec_ok = (reinterpret_cast<uintptr_t>(x) & 15u) == 0;
    absmax_kernel<MINMAX><<<grid, kAbsThreads, sizeof(AbsSmem), stream>>>(
        x, rows, total, reinterpret_cast<uint32_t*>(out_a), reinterpret_cast<uint32_t*>(out_b),
        vec_ok, per_cta);
    return cudaGetLastError();
}

cudaError_t launch_absmax(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                          int64_t total, float* m_out, cudaStream_t stream, int64_t shift) {
    return launch_fold<false>(x, row_offsets, C, n, total, m_out, nullptr, stream, shift);
}

cudaError_t launch_minmax(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                          int64_t total, float* lo_out, float* hi_out, cudaStream_t stream) {
    cudaError_t e = launch_fold<true>(x, row_offsets, C, n, total, hi_out, lo_out, stream, 0);
    if (e != cudaSuccess) return e;
    minmax_finalize_kernel<<<(unsigned)((C + 255) / 256), 256, 0, stream>>>(
        reinterpret_cast<uint32_t*>(lo_out), reinterpret_cast<uint32_t*>(hi_out), C);
    return cudaGetLastError();
}

}  // namespace pwlq
