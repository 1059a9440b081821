// Range m of every row: m_c = max_i |x_{c,i}|  (Sec. 3.2: quantization range [-m, m]).
//
// HBM-bound streaming reduction, 4 bytes read per value.  The flat storage is cut into spans of
// kMapSpan values; a CTA walks consecutive spans, which arrive in a ring of shared-memory stages
// filled by bulk asynchronous copies together with a map of the rows that start in them.
// Magnitude bit patterns are folded with an integer maximum (exact and order-free).
#include <algorithm>
#include <mutex>

#include "pwlq_common.cuh"
#include "pwlq_kernels.h"
#include "pwlq_pipeline.cuh"
#include "pwlq_rowmap.cuh"

namespace pwlq {

constexpr int kAbsConsumers = 8;                         // folding warps per CTA
constexpr int kAbsThreads = (kAbsConsumers + 1) * 32;    // + the producer warp
constexpr int kAbsStages = 2;                            // spans in flight per CTA
static_assert(kAbsStages <= 4, "MapProducer tracks at most four stages");

static __device__ int g_absmax_timeout;   // bit 0: a bounded wait expired; bit 1: row maps of another layout

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
    // keys as add() forms them (0: nothing)
    __device__ __forceinline__ void add_keys(uint32_t ka, uint32_t kb) {
        a = max(a, ka);
        if (MINMAX) b = max(b, kb);
    }
    __device__ __forceinline__ void merge(const Fold& o) { add_keys(o.a, o.b); }
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

// One stage of the producer / consumer pipeline: a span's values and its row map.
struct AbsStage {
    alignas(128) float data[kMapSpan];
    SpanRowMap map;
};

// Bytes of span `span` if it can be fetched by a bulk copy (aligned base, whole 16-byte units).
__device__ __forceinline__ unsigned abs_bulk_bytes(int64_t span, int64_t total, int vec_ok) {
    const int64_t beg = span * kMapSpan;
    const int64_t cnt = min((int64_t)kMapSpan, total - beg);
    return (vec_ok && (cnt & 3) == 0) ? (unsigned)(cnt * 4) : 0u;
}

// Warp kAbsConsumers produces (bulk copy of the span's values + row map, see pwlq_rowmap.cuh);
// the other warps fold.  A consumer warp owns a contiguous eighth of the span and walks it in
// windows of 256 values, eight consecutive values per lane.  The fold of the row the warp is in
// stays in per-lane registers from window to window and from span to span (a long row costs one
// atomic per warp for the whole kernel).  A window in which rows start is handled without a
// loop over the rows: every lane splits its values at its start, a segmented scan over the lanes
// joins the pieces of every row, and the lane in which a row ends issues the row's atomic.
// LONG: dense rows of at least a span (the maps follow from the row length).
// PRE: the maps were built ahead of time (premap: header, then one map per span); the producer
// only requests copies.
template <bool MINMAX, bool LONG, bool PRE>
__global__ void __launch_bounds__(kAbsThreads)
absmax_kernel(const float* __restrict__ x, Rows rows, int64_t total, uint32_t* __restrict__ m_bits,
              uint32_t* __restrict__ lo_bits, int vec_ok, int64_t spans_per_cta,
              const unsigned char* __restrict__ premap) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    if (PRE && !rowmap_matches(premap, rows, total)) {        // maps of another layout: no work
        if (threadIdx.x == 0) atomicOr(&g_absmax_timeout, 2);
        return;
    }
    AbsStage* st = reinterpret_cast<AbsStage*>(smem_raw);
    __shared__ uint64_t full_bar[kAbsStages], empty_bar[kAbsStages];
    const unsigned full = 0xffffffffu;
    const int64_t nspans = (total + kMapSpan - 1) / kMapSpan;
    const int64_t first = blockIdx.x * spans_per_cta, last = min(first + spans_per_cta, nspans);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kAbsStages; ++s) {
            mbar_init(&full_bar[s], 2);            // the data (or its stand-in) and the map
            mbar_init(&empty_bar[s], kAbsConsumers);
        }
        fence_barrier_init();
    }
    __syncthreads();
    if (first >= last) return;

    if (PRE && warp == kAbsConsumers) {
        // ---- producer, maps built ahead of time: two bulk copies per span
        const SpanRowMap* maps = reinterpret_cast<const SpanRowMap*>(premap + kRowMapHeaderBytes);
        int64_t it = 0;
        for (int64_t span = first; span < last; ++span, ++it) {
            const int s = (int)(it % kAbsStages);
            const unsigned use = (unsigned)(it / kAbsStages);
            if (use > 0 && !mbar_wait(&empty_bar[s], (use - 1) & 1u)) {
                if (lane == 0) atomicOr(&g_absmax_timeout, 1);
                for (int64_t j = it - 1; j >= 0 && j > it - 1 - kAbsStages; --j)
                    mbar_wait(&full_bar[j % kAbsStages], (unsigned)(j / kAbsStages) & 1u);
                return;
            }
            const int64_t span_beg = span * kMapSpan, span_end = min(span_beg + kMapSpan, total);
            const unsigned bytes = abs_bulk_bytes(span, total, vec_ok);
            if (bytes != 0) {
                if (lane == 0) {
                    mbar_expect_tx(&full_bar[s], bytes);
                    bulk_copy_g2s(st[s].data, x + span_beg, bytes, &full_bar[s]);
                }
            } else {                               // unaligned base or ragged tail: plain loads
                for (int i = lane; i < (int)(span_end - span_beg); i += 32) st[s].data[i] = x[span_beg + i];
                __syncwarp();
                if (lane == 0) mbar_arrive(&full_bar[s]);
            }
            if (lane == 0) {
                mbar_expect_tx(&full_bar[s], (unsigned)sizeof(SpanRowMap));
                bulk_copy_g2s(&st[s].map, maps + span, (unsigned)sizeof(SpanRowMap), &full_bar[s]);
            }
        }
        return;
    }
    if (warp == kAbsConsumers) {
        // ---- producer
        MapProducer<false, false> prod;
        prod.rows = rows;
        prod.in = RowInputs{nullptr, nullptr, nullptr};
        prod.Lf = 0.0f;
        // the values of the first spans do not depend on the rows: request them before the search
        for (int64_t span = first; span < last && span < first + kAbsStages; ++span) {
            const unsigned bytes = abs_bulk_bytes(span, total, vec_ok);
            if (bytes != 0 && lane == 0) {
                mbar_expect_tx(&full_bar[span - first], bytes);
                bulk_copy_g2s(st[span - first].data, x + span * kMapSpan, bytes, &full_bar[span - first]);
            }
        }
        if (LONG) prod.request_long(rows.dense_row(first * kMapSpan));
        else prod.request(warp_row_of(rows, first * kMapSpan), true);
        int64_t it = 0;
        for (int64_t span = first; span < last; ++span, ++it) {
            const int s = (int)(it % kAbsStages);
            const unsigned use = (unsigned)(it / kAbsStages);
            if (use > 0 && !mbar_wait(&empty_bar[s], (use - 1) & 1u)) {
                // never expected: report, let the copies of the earlier spans land (their stages'
                // barriers have this warp's arrivals already), and leave
                if (lane == 0) atomicOr(&g_absmax_timeout, 1);
                for (int64_t j = it - 1; j >= 0 && j > it - 1 - kAbsStages; --j)
                    mbar_wait(&full_bar[j % kAbsStages], (unsigned)(j / kAbsStages) & 1u);
                return;
            }
            const int64_t span_beg = span * kMapSpan, span_end = min(span_beg + kMapSpan, total);
            const unsigned bytes = abs_bulk_bytes(span, total, vec_ok);
            if (bytes != 0) {
                if (lane == 0 && use > 0) {        // (first round: requested above)
                    // the stage was last read (by the consumers, whose arrivals this warp has
                    // waited for), not written, through the generic proxy: no proxy fence needed
                    mbar_expect_tx(&full_bar[s], bytes);
                    bulk_copy_g2s(st[s].data, x + span_beg, bytes, &full_bar[s]);
                }
            } else {                               // unaligned base or ragged tail: plain loads
                for (int i = lane; i < (int)(span_end - span_beg); i += 32) st[s].data[i] = x[span_beg + i];
                __syncwarp();
                if (lane == 0) mbar_arrive(&full_bar[s]);
            }
            if (LONG) prod.build_long(st[s].map, nullptr, nullptr, s, span_beg, span_end, span + 1 < last);
            else prod.build(st[s].map, nullptr, nullptr, span_beg, span_end, span + 1 < last);
            __syncwarp();
            if (lane == 0) mbar_arrive(&full_bar[s]);
        }
        return;
    }

    // ---- consumers
    Fold<MINMAX> acc;                              // this lane's share of the row the warp is in
    int64_t acc_row = -1;                          // that row (the same for all lanes)
    auto flush_acc = [&]() {                       // every lane of the warp calls this
        acc.reduce_warp();
        if (lane == 0 && acc_row >= 0) acc.store(m_bits, lo_bits, acc_row);
        acc.clear();
    };
    constexpr int kSlice = kMapSpan / kAbsConsumers;
    int64_t it = 0;
    for (int64_t span = first; span < last; ++span, ++it) {
        const int s = (int)(it % kAbsStages);
        const unsigned use = (unsigned)(it / kAbsStages);
        if (!mbar_wait_relaxed(&full_bar[s], use & 1u)) {
            if (lane == 0) atomicOr(&g_absmax_timeout, 1);
            return;
        }
        const int64_t span_beg = span * kMapSpan;
        const int span_len = (int)min((int64_t)kMapSpan, total - span_beg);
        const AbsStage& S = st[s];
        const float* xs = S.data;
        const int sl_beg = warp * kSlice;
        if (sl_beg < span_len) {
            const bool slow = S.map.slow != 0;
            const int64_t first_row = S.map.first_row;
            if (!slow) {
                // the row that is open where the slice begins (a row that starts exactly there
                // is opened by the window below)
                uint32_t w0;
                const int sl_slot = map_slot(S.map, sl_beg, w0);
                const int64_t r_open = first_row + sl_slot - (int)((w0 >> (sl_beg & 31)) & 1u);
                if (r_open != acc_row) { flush_acc(); acc_row = r_open; }
            } else {
                flush_acc();
                acc_row = -1;
            }
#pragma unroll 1
            for (int win = 0; win < kSlice / 256; ++win) {
                const int li = sl_beg + win * 256 + lane * 8;
                const int cnt = max(0, min(8, span_len - li));
                uint32_t ka[8], kb[8];
                if (cnt == 8) {
                    const float4 xa = *reinterpret_cast<const float4*>(xs + li);
                    const float4 xb = *reinterpret_cast<const float4*>(xs + li + 4);
                    const float v[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        ka[j] = MINMAX ? ordered_key(v[j]) : abs_bits(v[j]);
                        kb[j] = MINMAX ? ~ka[j] : 0u;
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        ka[j] = kb[j] = 0u;                      // 0: nothing
                        if (j < cnt) {
                            ka[j] = MINMAX ? ordered_key(xs[li + j]) : abs_bits(xs[li + j]);
                            kb[j] = MINMAX ? ~ka[j] : 0u;
                        }
                    }
                }
                if (slow) {
                    // no usable map: every value finds its row in global memory
                    for (int j = 0; j < cnt; ++j) {
                        Fold<MINMAX> one;
                        one.a = ka[j]; one.b = kb[j];
                        one.store(m_bits, lo_bits, rows.row_of(span_beg + li + j));
                    }
                    continue;
                }
                uint32_t word;
                const int slot0 = map_slot(S.map, li, word);     // row of my first value
                const uint32_t nib = (word >> (li & 31)) & 0xFFu;   // bit j: a row starts at li + j
                const unsigned starts = __ballot_sync(full, nib != 0);
                if (starts == 0) {                               // the window lies inside the open row
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc.add_keys(ka[j], kb[j]);
                    continue;
                }
                if (__any_sync(full, (nib & (nib - 1)) != 0)) {
                    // a lane holds more than one start (rows of fewer than eight values): every
                    // lane walks its values on its own
                    flush_acc();
                    Fold<MINMAX> cur;
                    int cur_slot = slot0 - (int)(nib & 1u);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if ((nib >> j) & 1u) {
                            cur.store(m_bits, lo_bits, first_row + cur_slot);
                            cur.clear();
                            ++cur_slot;
                        }
                        cur.add_keys(ka[j], kb[j]);
                    }
                    cur.store(m_bits, lo_bits, first_row + cur_slot);
                    acc_row = first_row + __shfl_sync(full, cur_slot, 31);
                    continue;
                }
                // at most one start per lane: split my values at it
                const bool flag = nib != 0;
                const int fpos = flag ? __ffs(nib) - 1 : 8;
                const uint32_t low = (1u << fpos) - 1u;          // bit j: value j lies before my start
                Fold<MINMAX> h, t;
                if (!__any_sync(full, (nib & 0xFEu) != 0)) {
                    // every start is at a lane's first value (row lengths that are multiples of
                    // eight): a lane's values all go one way
#pragma unroll
                    for (int j = 0; j < 8; ++j) t.add_keys(ka[j], kb[j]);
                    if (!flag) { h = t; t.clear(); }
                } else {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const uint32_t hm = 0u - ((low >> j) & 1u);
                        h.add_keys(ka[j] & hm, kb[j] & hm);
                        t.add_keys(ka[j] & ~hm, kb[j] & ~hm);
                    }
                }
                // inclusive scan over the lanes, restarted at every lane with a start
                Fold<MINMAX> sc = flag ? t : h;
                const unsigned below = starts & (0xFFFFFFFFu >> (31 - lane));
                const int ss = below ? 31 - __clz(below) : 0;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    Fold<MINMAX> y;
                    y.a = __shfl_up_sync(full, sc.a, d);
                    y.b = MINMAX ? __shfl_up_sync(full, sc.b, d) : 0u;
                    if (lane - d >= ss) sc.merge(y);
                }
                Fold<MINMAX> left;                               // the lanes between the previous start and me
                left.a = __shfl_up_sync(full, sc.a, 1);
                left.b = MINMAX ? __shfl_up_sync(full, sc.b, 1) : 0u;
                if (lane == 0) left.clear();
                Fold<MINMAX> carry = acc;                        // the open row so far
                carry.reduce_warp();
                if (flag) {                                      // a row ends before my start
                    Fold<MINMAX> closed = h;
                    closed.merge(left);
                    if ((starts & ((1u << lane) - 1u)) == 0) closed.merge(carry);
                    closed.store(m_bits, lo_bits, first_row + slot0 - (int)(nib & 1u));
                }
                const int last_flag = 31 - __clz(starts);
                acc.clear();
                if (lane > last_flag) acc = h;
                else if (lane == last_flag) acc = t;
                acc_row = first_row + __shfl_sync(full, slot0 + __popc(nib >> 1), last_flag);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[s]);
    }
    flush_acc();                                      // what is still carried at the end
}

int take_absmax_timeout_flag() {
    int v = 0;
    const int zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_absmax_timeout, sizeof(int)) != cudaSuccess) return -1;
    if (v != 0 && cudaMemcpyToSymbol(g_absmax_timeout, &zero, sizeof(int)) != cudaSuccess) return -1;
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
                               int64_t shift, const void* rowmap) {
    cudaError_t e = cudaMemsetAsync(out_a, 0, sizeof(float) * (size_t)C, stream);
    if (e != cudaSuccess) return e;
    if (MINMAX) {
        e = cudaMemsetAsync(out_b, 0, sizeof(float) * (size_t)C, stream);
        if (e != cudaSuccess) return e;
    }
    if (total == 0) return cudaSuccess;
    Rows rows{row_offsets, C, n, n > 0 ? 1.0 / (double)n : 0.0, row_offsets ? shift : 0};
    const int64_t nspans = (total + kMapSpan - 1) / kMapSpan;
    const bool long_rows = row_offsets == nullptr && n >= kMapSpan;   // the maps follow from n
    const size_t smem = sizeof(AbsStage) * kAbsStages;
    // (maps built ahead of time are of no use where the map follows from the row length)
    const unsigned char* premap = long_rows ? nullptr : static_cast<const unsigned char*>(rowmap);
    const void* kernel = long_rows ? (const void*)absmax_kernel<MINMAX, true, false>
                         : premap  ? (const void*)absmax_kernel<MINMAX, false, true>
                                   : (const void*)absmax_kernel<MINMAX, false, false>;
    static int cached[2][3][64] = {{{0}}};             // CTAs that fit the device at once
    static std::mutex cached_mu;
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) dev = 0;
    std::lock_guard<std::mutex> lock(cached_mu);
    int& slots_dev = cached[MINMAX ? 1 : 0][long_rows ? 1 : (premap ? 2 : 0)][dev];
    if (slots_dev == 0) {
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        int sms = 0, per_sm = 0;
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kAbsThreads, smem);
        slots_dev = (sms > 0 && per_sm > 0) ? sms * per_sm : 148;
    }
    // Consecutive spans are handed out in blocks of at most kSpansPerBlockMax, about two per slot
    // of the device when the input is small: long enough to pay for the producer's start, short
    // enough for the hardware scheduler to even out what differs between spans (row starts per
    // span).  (Measured on B200, ragged rows: blocks of 11 spans beat blocks of 6, 22 and 32 on
    // 408 MB; on 102 MB blocks of 6 or 11 beat blocks of 3.)
    const int64_t slots = slots_dev;
    const int64_t per_cta = std::min<int64_t>(
        std::max<int64_t>((nspans + 2 * slots - 1) / (2 * slots), 1), kSpansPerBlockMax);
    const unsigned grid = (unsigned)((nspans + per_cta - 1) / per_cta);
    const int vec_ok = (reinterpret_cast<uintptr_t>(x) & 15u) == 0;
    uint32_t* a_bits = reinterpret_cast<uint32_t*>(out_a);
    uint32_t* b_bits = reinterpret_cast<uint32_t*>(out_b);
    if (long_rows)
        absmax_kernel<MINMAX, true, false><<<grid, kAbsThreads, smem, stream>>>(
            x, rows, total, a_bits, b_bits, vec_ok, per_cta, nullptr);
    else if (premap)
        absmax_kernel<MINMAX, false, true><<<grid, kAbsThreads, smem, stream>>>(
            x, rows, total, a_bits, b_bits, vec_ok, per_cta, premap);
    else
        absmax_kernel<MINMAX, false, false><<<grid, kAbsThreads, smem, stream>>>(
            x, rows, total, a_bits, b_bits, vec_ok, per_cta, nullptr);
    return cudaGetLastError();
}

cudaError_t launch_absmax(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                          int64_t total, float* m_out, cudaStream_t stream, int64_t shift,
                          const void* rowmap) {
    return launch_fold<false>(x, row_offsets, C, n, total, m_out, nullptr, stream, shift, rowmap);
}

cudaError_t launch_minmax(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                          int64_t total, float* lo_out, float* hi_out, cudaStream_t stream,
                          int64_t shift) {
    cudaError_t e = launch_fold<true>(x, row_offsets, C, n, total, hi_out, lo_out, stream, shift, nullptr);
    if (e != cudaSuccess) return e;
    minmax_finalize_kernel<<<(unsigned)((C + 255) / 256), 256, 0, stream>>>(
        reinterpret_cast<uint32_t*>(lo_out), reinterpret_cast<uint32_t*>(hi_out), C);
    return cudaGetLastError();
}

}  // namespace pwlq
