// Row maps for the streaming kernels when a span of the flat storage holds several rows (ragged
// rows, and dense rows shorter than a span).
//
// A CTA is one producer warp and a number of consumer warps.  For every span of kMapSpan values
// the producer describes the rows that overlap it in a stage of shared memory: a bitmap with one
// bit per position at which a row starts, the number of starts before every 32-bit word of the
// bitmap, and the rows' constants in the order in which the rows appear ("slots"; slot 0 is the
// row that holds the span's first value).  A consumer lane then finds the slot of any position
// with two shared-memory reads and a population count, and sees the row starts among the values
// it owns directly in the bitmap; it never searches and never touches the row arrays in global
// memory.  The producer walks the spans in order, so the first row of a span is where the previous
// span ended.  It keeps the offsets and inputs of the 33 to 64 rows from that row on in registers
// (two chunks of 32 consecutive rows, one row per lane) and requests a new chunk as soon as the
// walk has left an old one, so that with rows of a few hundred values or more its loads are
// several spans ahead of their use.  Stages are handed over through mbarriers (full: producer ->
// consumers, empty: consumers -> producer), which keeps the producer's global round trips off the
// consumers' path.
//
// Spans the map cannot describe (more than kMapSlots rows, or empty rows inside the span) are
// marked `slow`; consumers then look every value's row up in global memory.
//
// The maps depend on the row layout only, not on the values or on the rows' inputs.  A caller
// that runs several streaming calls over one layout can have them built once, into memory of its
// own (rowmap_build_kernel, RowMapHeader); the producer of a kernel that is given such maps
// fetches each span's map with one more bulk copy and only computes the rows' constants, from
// inputs it requested a span earlier.
#pragma once

#include "pwlq_common.cuh"
#include "pwlq_multi.cuh"
#include "pwlq_pipeline.cuh"

namespace pwlq {

constexpr int kMapSpan = 4096;                 // values per span
constexpr int kSpansPerBlockMax = 11;          // consecutive spans one CTA walks, at most
constexpr int kMapWords = kMapSpan / 32;
constexpr int kMapRounds = 17;                 // rounds of 32 rows the producer looks at per span
constexpr int kMapSlots = kMapRounds * 32;     // rows a map can describe (rows of >= 8 values fit)

struct SpanRowMap {
    uint32_t bits[kMapWords];     // bit i: a row starts at position i of the span (i > 0)
    uint16_t before[kMapWords];   // number of set bits in the words before this one
    int64_t first_row;            // row of slot 0
    int32_t slow;                 // 1: the map does not describe the span
    int32_t nrows;                // rows (slots) the map describes; 0 when slow
};
static_assert(sizeof(SpanRowMap) % 16 == 0, "maps are moved with bulk copies");

// Maps built ahead of time: a header, then one SpanRowMap per span.
constexpr uint64_t kRowMapMagic = 0x70776c7170616d31ull;
constexpr size_t kRowMapHeaderBytes = 256;
struct RowMapHeader {
    uint64_t magic;
    int64_t C, total, n;          // the layout the maps describe (n = 0: ragged rows)
};

// Whether maps built ahead of time describe this layout (every thread of a CTA asks before it
// does anything else; the header is 32 bytes that stay in L2).
__device__ __forceinline__ bool rowmap_matches(const unsigned char* premap, const Rows& rows,
                                               int64_t total) {
    const RowMapHeader* h = reinterpret_cast<const RowMapHeader*>(premap);
    return __ldg(&h->magic) == kRowMapMagic && __ldg(&h->C) == rows.C &&
           __ldg(&h->total) == total && __ldg(&h->n) == (rows.offsets ? 0 : rows.n);
}

// Slot of the row that holds position li of the span; `word` returns the bitmap word of li.
__device__ __forceinline__ int map_slot(const SpanRowMap& M, int li, uint32_t& word) {
    word = M.bits[li >> 5];
    return (int)M.before[li >> 5] + __popc(word & (0xFFFFFFFFu >> (31 - (li & 31))));
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

// Per-row inputs of the quantizer: m = abs-max and lo = nullptr (signed scheme), or m = upper and
// lo = lower bound of a one-sided range; p = breakpoint.
struct RowInputs {
    const float* __restrict__ m;
    const float* __restrict__ lo;
    const float* __restrict__ p;
    const float* __restrict__ xi;      // bias correction (dequantize only): scale and offset
    const float* __restrict__ beta;    // per row, or nullptr
};

// Constants of one row as the consumers read them; m is the range width (abs-max, or upper -
// lower bound).  Quantize (DEQ = false): qa = (m, p, L/p, L/(m-p)), qb = (p/L, (m-p)/L, lo, 0);
// a row whose L/p or L/(m-p) is not finite (a breakpoint or tail range near the smallest binary32
// magnitudes) is stored with -m: the branch-free quantizer, which has no saturation, must not see
// it, and the consumers send every row with m <= 0 to the value-by-value path.
// Dequantize (DEQ = true): qa = (m, p, p/L, (m-p)/L), qb = (lo, xi, beta, 0) with the scale and
// offset of the bias correction (1 and 0 without it).
template <bool DEQ>
__device__ __forceinline__ void store_row_consts(float4* qa, float4* qb, int slot, float m, float p,
                                                 float lo, float xi, float beta, float Lf) {
    const PieceParams P = make_params(m, p, Lf);
    if (DEQ) {
        qa[slot] = make_float4(m, P.p, P.s1, P.s2);
        if (qb) qb[slot] = make_float4(lo, xi, beta, 0.0f);
    } else {
        const bool finite = P.inv1 <= 3.402823466e38f && P.inv2 <= 3.402823466e38f;
        qa[slot] = make_float4(m > 0.0f ? (finite ? m : -m) : 0.0f, P.p, P.inv1, P.inv2);
        if (qb) qb[slot] = make_float4(P.s1, P.s2, lo, 0.0f);
    }
}

// The producer warp's view of the rows.  Rows are looked at in chunks of 32 consecutive rows
// (chunk c = rows 32 c .. 32 c + 31, lane = row % 32); the two chunks from the current first row
// on are held in registers.  Every member function is called by all 32 lanes.
// NBP > 1: rows with two or three breakpoints.  in.p, in.lo and in.xi then point to p1, p2 and p3
// (BC: a third breakpoint exists), read with stride pstride; the constants of a row are four
// 128-bit records in qa (store_row_consts_multi), for at most kMultiSlots rows per span.
template <bool PARAMS, bool UNS, bool DEQ = false, bool BC = false, int NBP = 1>
struct MapProducer {
    Rows rows;
    RowInputs in;
    float Lf;
    int pstride;                // NBP > 1 only
    int64_t rf;                 // row that holds the first value of the next span
    int64_t ch0, ch1;           // chunk held in (o0, m0, p0, lo0): even chunks; (o1, ...): odd chunks
    int64_t o0, o1;             // offset of row 32 ch + lane (INT64_MAX past the last offset)
    float m0, p0, lo0, m1, p1, lo1;
    float x0, b0, x1, b1;       // BC: scale and offset of the bias correction

    __device__ __forceinline__ void load_inputs(int64_t r, float& mv, float& pv, float& lov,
                                                float& xv, float& bv) const {
        mv = __ldg(in.m + r);
        if (NBP > 1) {                              // (p1, p2, p3) in (pv, lov, xv); p3 = m without one
            pv = __ldg(in.p + r * pstride);
            lov = __ldg(in.lo + r * pstride);
            xv = BC ? __ldg(in.xi + r * pstride) : mv;
            bv = 0.0f;
            return;
        }
        pv = __ldg(in.p + r);
        lov = 0.0f;
        if (UNS) lov = __ldg(in.lo + r);            // m stays the upper bound until it is used
        xv = 1.0f;
        bv = 0.0f;
        if (BC) { xv = __ldg(in.xi + r); bv = __ldg(in.beta + r); }
    }
    __device__ __forceinline__ void load_chunk(int64_t c, int64_t& o, float& mv, float& pv,
                                               float& lov, float& xv, float& bv) const {
        const int64_t r = 32 * c + (threadIdx.x & 31);
        // as stored (ragged: before the slice's shift is taken off), so that nothing here waits
        // for the load
        o = (r <= rows.C) ? (rows.offsets ? __ldg(rows.offsets + r) : r * rows.n) : INT64_MAX;
        mv = pv = lov = bv = 0.0f;
        xv = 1.0f;
        if (PARAMS && r < rows.C) load_inputs(r, mv, pv, lov, xv, bv);
    }
    // Makes the registers hold the two chunks from row `first_row` on; chunks already held are
    // kept, nothing is waited for.
    __device__ __forceinline__ void request(int64_t first_row, bool fresh) {
        rf = first_row;
        const int64_t c = rf >> 5;
        const int64_t want0 = (c & 1) ? c + 1 : c, want1 = (c & 1) ? c : c + 1;
        if (fresh || ch0 != want0) { ch0 = want0; load_chunk(want0, o0, m0, p0, lo0, x0, b0); }
        if (fresh || ch1 != want1) { ch1 = want1; load_chunk(want1, o1, m1, p1, lo1, x1, b1); }
    }
    // Writes the map of the span [span_beg, span_end), whose first value lies in row rf, and the
    // constants of its rows; then moves on to the first row of the next span (more == true).
    __device__ __forceinline__ void build(SpanRowMap& M, float4* qa, float4* qb, int64_t span_beg,
                                          int64_t span_end, bool more) {
        const unsigned full = 0xffffffffu;
        const int lane = threadIdx.x & 31;
        reinterpret_cast<uint4*>(M.bits)[lane] = make_uint4(0u, 0u, 0u, 0u);
        __syncwarp();
        const int64_t this_rf = rf;
        const int64_t c0 = this_rf >> 5;
        const int l0 = (int)(this_rf & 31);        // slot s = 32 k + lane - l0 in round k
        int total_in = 0;
        bool open = true;                          // every row seen so far starts in the span
        // offsets of the first two rows that do not start inside the span
        int64_t os = 0, os1 = 0;
        bool have_os = false, have_os1 = false;
        for (int k = 0; open && k < kMapRounds; ++k) {
            const int64_t c = c0 + k;
            const int s = 32 * k + lane - l0;
            const int64_t r = 32 * c + lane;
            int64_t off;
            float mv, pv, lov, xv, bv;
            if (k < 2) {                           // held in registers
                const bool odd = (c & 1) != 0;
                off = odd ? o1 : o0;
                mv = odd ? m1 : m0; pv = odd ? p1 : p0; lov = odd ? lo1 : lo0;
                xv = odd ? x1 : x0; bv = odd ? b1 : b0;
            } else {                               // short rows: fetched now
                off = (r <= rows.C) ? (rows.offsets ? __ldg(rows.offsets + r) : r * rows.n) : INT64_MAX;
                mv = pv = lov = bv = 0.0f;
                xv = 1.0f;
            }
            if (off != INT64_MAX) off -= rows.shift;
            const bool inside = s >= 0 && r < rows.C && (s == 0 || off < span_end);
            if (inside) {
                if (s > 0) {
                    const int pos = (int)(off - span_beg);
                    const uint32_t bit = 1u << (pos & 31);
                    atomicOr(&M.bits[pos >> 5], bit);
                }
                if (PARAMS) {
                    if (k >= 2) load_inputs(r, mv, pv, lov, xv, bv);
                    if (NBP > 1) {
                        if (s < kMultiSlots) store_row_consts_multi(qa, s, mv, pv, lov, xv, Lf);
                    } else {
                        if (UNS) mv = __fsub_rn(mv, lov);          // range width
                        store_row_consts<DEQ>(qa, qb, s, mv, pv, lov, xv, bv, Lf);
                    }
                }
            }
            const unsigned in_mask = __ballot_sync(full, inside);
            const int cnt = __popc(in_mask);
            total_in += cnt;
            // the rows inside are the lanes from (k == 0 ? l0 : 0) up to some lane
            const int first_out = (k == 0 ? l0 : 0) + cnt;
            open = first_out == 32;
            if (!open) {
                os = __shfl_sync(full, off, first_out);
                have_os = true;
                if (first_out < 31) {
                    os1 = __shfl_sync(full, off, first_out + 1);
                    have_os1 = true;
                }
            }
        }
        const bool overflow = open;                // all rounds full: there may be more rows
        if (more) {
            // the row that holds position span_end (the last row that starts at or before it)
            int64_t rn;
            if (overflow) {
                rn = warp_row_of(rows, span_end);
            } else {
                const int64_t rs = this_rf + total_in;              // first row not inside, <= C
                if (!have_os) os = rows.begin(rs);
                if (rs < rows.C && os == span_end) {
                    if (!have_os1) os1 = (rs + 1 <= rows.C) ? rows.begin(rs + 1) : INT64_MAX;
                    const bool empty_next = rs + 1 < rows.C && os1 == span_end;
                    rn = empty_next ? warp_row_of(rows, span_end) : rs;
                } else {
                    rn = rs - 1;
                }
            }
            request(rn, false);
        }
        __syncwarp();
        const uint4 w = reinterpret_cast<const uint4*>(M.bits)[lane];
        const int c0b = __popc(w.x), c1b = __popc(w.y), c2b = __popc(w.z), c3b = __popc(w.w);
        const int tot = c0b + c1b + c2b + c3b;
        int incl = tot;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int t = __shfl_up_sync(full, incl, d);
            if (lane >= d) incl += t;
        }
        const uint32_t e0 = (uint32_t)(incl - tot), e1 = e0 + c0b, e2 = e1 + c1b, e3 = e2 + c2b;
        reinterpret_cast<uint2*>(M.before)[lane] = make_uint2(e0 | (e1 << 16), e2 | (e3 << 16));
        // rows that start at the same position (empty rows) set one bit between them
        const bool dup = __shfl_sync(full, incl, 31) != total_in - 1;
        if (lane == 0) {
            const bool unusable = dup || overflow || (NBP > 1 && total_in > kMultiSlots);
            M.first_row = this_rf;
            M.slow = unusable ? 1 : 0;
            M.nrows = unusable ? 0 : total_in;
        }
    }

    // ---- dense rows of at least kMapSpan values: a span holds one row, or the end of one and
    // the beginning of the next.  Everything follows from the row length; the inputs of the
    // current and the next row are held in registers (every lane the same), and a stage whose
    // slot 0 already belongs to the row is left as it is.
    static constexpr int kMaxStages = 4;
    int64_t long_end;                    // end of row rf
    int64_t stage_first[kMaxStages];     // per stage: the row its slot 0 was written for, or -1
    bool stage_plain[kMaxStages];        // per stage: the map says "one row, no start"

    __device__ __forceinline__ void request_long(int64_t first_row) {
        rf = first_row;
        long_end = (rf + 1) * rows.n;
        m0 = p0 = lo0 = m1 = p1 = lo1 = b0 = b1 = 0.0f;
        x0 = x1 = 1.0f;
        if (PARAMS) {
            load_inputs(rf, m0, p0, lo0, x0, b0);
            if (rf + 1 < rows.C) load_inputs(rf + 1, m1, p1, lo1, x1, b1);
        }
#pragma unroll
        for (int i = 0; i < kMaxStages; ++i) { stage_first[i] = -1; stage_plain[i] = false; }
    }
    __device__ __forceinline__ void build_long(SpanRowMap& M, float4* qa, float4* qb, int stage,
                                               int64_t span_beg, int64_t span_end, bool more) {
        const int lane = threadIdx.x & 31;
        const bool starts = long_end < span_end;          // row rf + 1 begins inside the span
        // (selected with constant indices: the arrays stay in registers; stage < kMaxStages)
        bool have_first = false, plain = false;
#pragma unroll
        for (int i = 0; i < kMaxStages; ++i)
            if (stage == i) { have_first = stage_first[i] == rf; plain = stage_plain[i]; }
        if (PARAMS && !have_first && lane == 0)
            store_row_consts<DEQ>(qa, qb, 0, UNS ? __fsub_rn(m0, lo0) : m0, p0, lo0, x0, b0, Lf);
        if (PARAMS && starts && lane == 1)
            store_row_consts<DEQ>(qa, qb, 1, UNS ? __fsub_rn(m1, lo1) : m1, p1, lo1, x1, b1, Lf);
        if (starts || !plain || !have_first) {
            const int pos = starts ? (int)(long_end - span_beg) : -1;      // > 0 when it exists
            const int wpos = pos >> 5;                                     // -1: no start
            uint32_t w[4], e[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int wi = 4 * lane + j;
                w[j] = (wi == wpos) ? (1u << (pos & 31)) : 0u;
                e[j] = (starts && wi > wpos) ? 1u : 0u;
            }
            reinterpret_cast<uint4*>(M.bits)[lane] = make_uint4(w[0], w[1], w[2], w[3]);
            reinterpret_cast<uint2*>(M.before)[lane] = make_uint2(e[0] | (e[1] << 16), e[2] | (e[3] << 16));
            if (lane == 0) { M.first_row = rf; M.slow = 0; }
        }
#pragma unroll
        for (int i = 0; i < kMaxStages; ++i)
            if (stage == i) { stage_first[i] = rf; stage_plain[i] = !starts; }
        if (more && long_end <= span_end) {               // the next span begins in row rf + 1
            rf += 1;
            long_end += rows.n;
            m0 = m1; p0 = p1; lo0 = lo1; x0 = x1; b0 = b1;
            if (PARAMS && rf + 1 < rows.C) load_inputs(rf + 1, m1, p1, lo1, x1, b1);
        }
    }
};

// The producer warp's work when the maps were built ahead of time: it fetches each span's map
// with a bulk copy (issued by the kernel) and computes the constants of the span's rows.  Lane l
// holds the first row and the row count of span pre_batch + l; (mn, pn, ...) are the inputs of
// row (first row of the span that is built next) + lane, requested while the span before it was
// being built.  Every member function is called by all 32 lanes.
template <bool PARAMS, bool UNS, bool DEQ = false, bool BC = false>
struct PreProducer {
    RowInputs in;
    float Lf;
    const SpanRowMap* pre;
    int64_t pre_batch, pre_first;
    int pre_rows;
    float mn, pn, lon, xn, bn;

    __device__ __forceinline__ void load_inputs(int64_t r, float& mv, float& pv, float& lov,
                                                float& xv, float& bv) const {
        mv = __ldg(in.m + r);
        pv = __ldg(in.p + r);
        lov = 0.0f;
        if (UNS) lov = __ldg(in.lo + r);
        xv = 1.0f;
        bv = 0.0f;
        if (BC) { xv = __ldg(in.xi + r); bv = __ldg(in.beta + r); }
    }
    __device__ __forceinline__ void load_batch(int64_t span0, int64_t last) {
        const int64_t sp = span0 + (threadIdx.x & 31);
        pre_batch = span0;
        pre_first = 0;
        pre_rows = 0;
        if (PARAMS && sp < last) {
            pre_first = __ldg(&pre[sp].first_row);
            pre_rows = __ldg(&pre[sp].nrows);
        }
    }
    __device__ __forceinline__ void fetch(int64_t span) {
        if (!PARAMS) return;
        const int j = (int)(span - pre_batch);
        const int64_t fr = __shfl_sync(0xffffffffu, pre_first, j);
        const int nr = __shfl_sync(0xffffffffu, pre_rows, j);
        const int lane = threadIdx.x & 31;
        mn = pn = lon = bn = 0.0f;
        xn = 1.0f;
        if (lane < nr) load_inputs(fr + lane, mn, pn, lon, xn, bn);
    }
    __device__ __forceinline__ void begin(const SpanRowMap* maps, int64_t first, int64_t last) {
        pre = maps;
        load_batch(first, last);
        fetch(first);
    }
    // Constants of the rows of `span`; then the inputs of the next span's rows are requested.
    __device__ __forceinline__ void build(float4* qa, float4* qb, int64_t span, int64_t last) {
        if (!PARAMS) return;
        const int lane = threadIdx.x & 31;
        const int j = (int)(span - pre_batch);
        const int64_t fr = __shfl_sync(0xffffffffu, pre_first, j);
        const int nr = __shfl_sync(0xffffffffu, pre_rows, j);
        if (lane < nr)
            store_row_consts<DEQ>(qa, qb, lane, UNS ? __fsub_rn(mn, lon) : mn, pn, lon, xn, bn, Lf);
        // many short rows: fetched now, four rows per lane in flight (one row at a time, every 32
        // rows exposed a round trip: MobileNetV2 rows, quantize 0.61 -> 0.67 of the copy peak)
        constexpr int kB = 4;
        for (int k0 = 32 + lane; k0 < nr; k0 += 32 * kB) {
            float mv[kB], pv[kB], lov[kB], xv[kB], bv[kB];
#pragma unroll
            for (int u = 0; u < kB; ++u)
                if (k0 + 32 * u < nr) load_inputs(fr + k0 + 32 * u, mv[u], pv[u], lov[u], xv[u], bv[u]);
#pragma unroll
            for (int u = 0; u < kB; ++u)
                if (k0 + 32 * u < nr)
                    store_row_consts<DEQ>(qa, qb, k0 + 32 * u, UNS ? __fsub_rn(mv[u], lov[u]) : mv[u],
                                          pv[u], lov[u], xv[u], bv[u], Lf);
        }
        if (span + 1 < last) {
            if (span + 1 - pre_batch == 32) load_batch(span + 1, last);
            fetch(span + 1);
        }
    }
};

}  // namespace pwlq
