// Quantizer of Eq. 3 (integer code + region bit, Sec. 4) and its inverse (Eq. 1, first line).
//
// Both are single streaming passes bound by HBM.  A thread owns 8 consecutive values: two
// 128-bit reads of x, then one 64-bit store of byte codes (or one 32-bit store of nibble-packed
// codes) and one region-mask byte, so that a warp writes contiguous 256 / 128 / 32-byte runs.
// The flat storage is cut into spans of 4096 values.  A CTA is a producer warp, which requests
// the spans' values with bulk asynchronous copies and describes the rows of every span (row map
// and row constants, see pwlq_rowmap.cuh), and eight consumer warps, which quantize.
#include <algorithm>
#include <mutex>

#include "pwlq_common.cuh"
#include "pwlq_kernels.h"
#include "pwlq_pipeline.cuh"
#include "pwlq_multi.cuh"
#include "pwlq_rowmap.cuh"

namespace pwlq {

constexpr int kQThreads = 256;
constexpr int kQChunk = kQThreads * 8;           // values one pass of the CTA covers
constexpr int kQChunks = 2;                      // passes per span
constexpr int kQSpan = kQChunk * kQChunks;       // values per span
static_assert(kQSpan == kMapSpan, "the spans of the row maps");

static __device__ int g_quantize_timeout;   // bit 0: a bounded wait expired; bit 1: row maps of another layout

// Offset inside the span of the eight values a thread handles in pass c.  A warp owns one
// contiguous eighth of the span and walks it in passes of 256 values, so that a thread's
// successive passes mostly stay inside one row (its row constants stay in registers) while a
// warp's reads and writes of one pass remain contiguous.
__device__ __forceinline__ int chunk_offset(int c) {
    return ((int)threadIdx.x >> 5) * (kQSpan / (kQThreads / 32)) + c * 256 + ((int)threadIdx.x & 31) * 8;
}

// Per-row inputs: m = abs-max and lo = nullptr (signed scheme), or m = upper and lo = lower
// bound of a one-sided range; p = breakpoint.
struct RowArrays {
    const float* __restrict__ m;
    const float* __restrict__ lo;
    const float* __restrict__ p;
    const float* __restrict__ xi;      // bias correction (dequantize): per-row scale and offset,
    const float* __restrict__ beta;    // or nullptr
};

// The row a thread is currently in, with its constants in registers, looked up in global memory
// (spans without a usable row map, and the tensor's last, partial span).
struct RowState {
    int64_t beg = 0, end = 0;
    float m = 0.0f;                                // range width (abs-max, or hi - lo)
    float lo = 0.0f;                               // lower bound of a one-sided range, else 0
    PieceParams P;
    int64_t row = -1;

    // Range width and lower bound of `row` straight from global memory.
    static __device__ __forceinline__ void load_range(const RowArrays& A, int64_t row, float& m,
                                                      float& lo) {
        m = __ldg(A.m + row);
        lo = 0.0f;
        if (A.lo) { lo = __ldg(A.lo + row); m = __fsub_rn(m, lo); }
    }
    __device__ __forceinline__ void seek(const Rows& rows, const RowArrays& A, float Lf, int64_t i) {
        if (i >= beg && i < end) return;
        row = rows.row_of(i);
        beg = rows.begin(row);
        end = rows.begin(row + 1);
        load_range(A, row, m, lo);
        P = make_params(m, __ldg(A.p + row), Lf);
    }
};

// Bytes of span `span` if it can be fetched by a bulk copy (aligned base, whole 16-byte units).
__device__ __forceinline__ unsigned q_bulk_bytes(int64_t span, int64_t total, int vec_in) {
    const int64_t beg = span * kQSpan;
    const int64_t cnt = min((int64_t)kQSpan, total - beg);
    return (vec_in && (cnt & 3) == 0) ? (unsigned)(cnt * 4) : 0u;
}

// Bit t of x moved to bit 4 t (t < 8) resp. to bit 8 t (t < 4).
__device__ __forceinline__ uint32_t spread_to_nibbles(uint32_t x) {
    x = (x | (x << 12)) & 0x000F000Fu;
    x = (x | (x << 6)) & 0x03030303u;
    x = (x | (x << 3)) & 0x11111111u;
    return x;
}
__device__ __forceinline__ uint32_t spread_to_bytes(uint32_t x) {
    return ((x & 0xFu) * 0x00204081u) & 0x01010101u;
}

// Eight consecutive values, the first `split` of them in row A and the rest in row B (TWO = false:
// all in row A), both rows with m > 0.  The sequence of quantize_mag without a branch, a compare
// or a select per value:
//   - both pieces are evaluated, r_c = a L/p + 1.5 * 2^23 and r_t = (a - p) L/(m-p) + 1.5 * 2^23
//     (the latter as (p - a) * -(L/(m-p)), the same value), and the one that applies is kept with
//     a bitwise blend under the sign of p - a (negative exactly when a > p: p - a is never -0);
//   - the level sits in the low mantissa bits of r (it never exceeds L, since a - z <= Delta), so
//     r's bit patterns are summed at their code positions and the constant the eight exponent
//     fields add up to is taken off once;
//   - region bits and sign flags (x < 0, false for -0.0: the sign bit of x + 0.0) are gathered
//     with one funnel shift each and spread to their positions once per eight values;
//   - the magnitude is formed negated (-a = max(-|x|, -m), one instruction), so that p - a and
//     x + 0.0 are plain additions, done for two values at a time (add.rn.f32x2).
// UNS: one-sided range, a = min(max(x - lo, 0), m), the code is the level itself and the delivered
// value is v + lo.
template <bool PACKED, bool WANT_FAKE, bool TWO, bool UNS>
__device__ __forceinline__ void quantize8(const float (&xv)[8], int split, float mA, float loA,
                                          const PieceParams& A, float mB, float loB,
                                          const PieceParams& B, float Lf, int Li,
                                          uint32_t sign_unit, int sign_shift, uint32_t& w0,
                                          uint32_t& w1, uint32_t& mb, float (&yv)[8]) {
    constexpr uint32_t kR = 0x4B400000u;                  // bit pattern of 1.5 * 2^23
    uint32_t acc0 = 0, acc1 = 0, tails = 0, signs = 0;
    // Two values at a time where only additions are involved: p - a as p + (-a) and x + 0.0 are
    // packed additions (one issue slot for two values, each lane rounded as the scalar operation
    // rounds); the products and the additions that follow them stay scalar, so that no product is
    // ever fused with its addition.
#pragma unroll
    for (int u = 0; u < 8; u += 2) {
        const int t1 = 7 - u, t0 = 6 - u;                 // descending: bit t of tails / signs
        float na[2], pp[2], nuv[2], sbv[2] = {0.0f, 0.0f};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int t = h ? t1 : t0;
            const bool second = TWO && t >= split;
            const float m = second ? mB : mA;
            const float lo = second ? loB : loA;
            pp[h] = second ? B.p : A.p;
            const float xi = xv[t];
            // -a, a = min(|x|, m) resp. min(max(x - lo, 0), m)
            na[h] = UNS ? -fminf(fmaxf(__fsub_rn(xi, lo), 0.0f), m) : fmaxf(-fabsf(xi), -m);
        }
        unpack2(add2(pack2(pp[0], pp[1]), pack2(na[0], na[1])), nuv[0], nuv[1]);   // -(a - p)
        if (!UNS) unpack2(add2(pack2(xv[t0], xv[t1]), pack2(0.0f, 0.0f)), sbv[0], sbv[1]);
#pragma unroll
        for (int h = 1; h >= 0; --h) {
            const int t = h ? t1 : t0;
            const bool second = TWO && t >= split;
            const float lo = second ? loB : loA;
            const float p = pp[h];
            const float ninv1 = -(second ? B.inv1 : A.inv1);
            const float ninv2 = -(second ? B.inv2 : A.inv2);
            const float nu = nuv[h];                      // negative: tail piece
            const uint32_t T = (uint32_t)((int32_t)__float_as_uint(nu) >> 31);   // all ones: tail
            const uint32_t rc = __float_as_uint(__fadd_rn(__fmul_rn(na[h], ninv1), 12582912.0f));
            const uint32_t rt = __float_as_uint(__fadd_rn(__fmul_rn(nu, ninv2), 12582912.0f));
            const uint32_t r = (rt & T) | (rc & ~T);
            if (PACKED) acc0 += r << (4 * t);
            else if (t < 4) acc0 += r << (8 * t);
            else acc1 += r << (8 * (t - 4));
            tails = __funnelshift_l(__float_as_uint(nu), tails, 1);
            uint32_t sb = 0;
            if (!UNS) {
                sb = __float_as_uint(sbv[h]);
                signs = __funnelshift_l(sb, signs, 1);
            }
            if (WANT_FAKE) {
                const uint32_t s1 = __float_as_uint(second ? B.s1 : A.s1);
                const uint32_t s2 = __float_as_uint(second ? B.s2 : A.s2);
                const float s = __uint_as_float((s2 & T) | (s1 & ~T));
                const float z = __uint_as_float(__float_as_uint(p) & T);
                const float qf = __fsub_rn(__uint_as_float(r), 12582912.0f);
                const float v = __fadd_rn(__fmul_rn(qf, s), z);
                yv[t] = UNS ? __fadd_rn(v, lo)
                            : __uint_as_float(__float_as_uint(v) | (sb & 0x80000000u));
            }
        }
    }
    mb = tails;
    if (PACKED) {
        constexpr uint32_t kGarbage = (uint32_t)(0x4B400000ull * 0x11111111ull);
        w0 = (acc0 - kGarbage) | (UNS ? 0u : spread_to_nibbles(signs) * sign_unit);
        w1 = 0;
    } else {
        constexpr uint32_t kGarbage = (uint32_t)(0x4B400000ull * 0x01010101ull);
        w0 = (acc0 - kGarbage) | (UNS ? 0u : spread_to_bytes(signs) * sign_unit);
        w1 = (acc1 - kGarbage) | (UNS ? 0u : spread_to_bytes(signs >> 4) * sign_unit);
    }
    (void)kR;
}

// ------------------------------------------------------------------ several rows per span
// Producer / consumer form of the quantizer for ragged rows and dense rows shorter than a span
// (see pwlq_rowmap.cuh): warp kMapConsumers fills the stages (bulk copy of the span's values, row
// map, row constants), the other warps quantize.  A consumer warp owns a contiguous eighth of the
// span and walks it in passes of 256 values, a lane owns eight consecutive values of a pass.
constexpr int kMapConsumers = 8;
constexpr int kMapThreads = (kMapConsumers + 1) * 32;
constexpr int kMapStages = 2;
static_assert(kMapStages <= 4, "MapProducer tracks at most four stages");

template <bool DATA, bool QB>
struct MapStage {
    alignas(128) float data[DATA ? kMapSpan : 4];
    SpanRowMap map;
    alignas(16) float4 qa[kMapSlots];
    alignas(16) float4 qb[QB ? kMapSlots : 1];
};

__device__ __forceinline__ PieceParams params_of(const float4 qa, const float4 qb) {
    PieceParams P;
    P.p = qa.y; P.inv1 = qa.z; P.inv2 = qa.w; P.s1 = qb.x; P.s2 = qb.y;
    return P;
}

// What a consumer's pass needs besides the stage.
template <bool UNS>
struct QuantizeCtx {
    Rows rows;
    RowArrays A;
    int64_t total;
    int bits, Li;
    float Lf;
    uint32_t sign_unit;
    int sign_shift;
    uint8_t* __restrict__ codes;
    uint8_t* __restrict__ mask;
    float* __restrict__ fake;
    int vec_fake, vec_codes;
};

// One pass of a consumer lane: the eight values at offset li of the span that begins at flat
// index span_beg.  FULL: the span is complete, its map is usable and every output can be stored
// with vector stores (the common case: no value counts, no 64-bit indices, no byte-wise stores).
template <bool PACKED, bool WANT_FAKE, bool UNS, bool QB, bool FULL>
__device__ __forceinline__ void quantize_pass(const QuantizeCtx<UNS>& g, const float* data,
                                              const SpanRowMap& M, const float4* qa,
                                              const float4* qb, int64_t span_beg, int li) {
    const unsigned full = 0xffffffffu;
    const int64_t i0 = span_beg + li;
    const int cnt = FULL ? 8 : (int)max((int64_t)0, min((int64_t)8, g.total - i0));
    const float4 xa = *reinterpret_cast<const float4*>(data + li);
    const float4 xb = *reinterpret_cast<const float4*>(data + li + 4);
    const float xv[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
    uint32_t w0 = 0, w1 = 0, mb = 0;
    float yv[8];
    if (FULL || M.slow == 0) {
        uint32_t word;
        const int l = map_slot(M, li, word);
        const uint32_t inner = (word >> ((li & 31) + 1)) & 0x7Fu;   // starts at li+1 .. li+7
        const float4 ca = qa[l];
        const float4 cb = QB ? qb[l] : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        const bool simple = inner == 0 && ca.x > 0.0f && cnt == 8;
        if (__all_sync(full, simple)) {
            const PieceParams P = params_of(ca, cb);
            quantize8<PACKED, WANT_FAKE, false, UNS>(xv, 8, ca.x, cb.z, P, ca.x, cb.z, P, g.Lf, g.Li,
                                                     g.sign_unit, g.sign_shift, w0, w1, mb, yv);
        } else {
            const bool one = inner != 0 && (inner & (inner - 1)) == 0 && ca.x > 0.0f && cnt == 8;
            float4 da = ca, db = cb;
            int split = 8;
            if (one) {
                da = qa[l + 1];
                if (QB) db = qb[l + 1];
                split = __ffs(inner);
            }
            if (__all_sync(full, simple || (one && da.x > 0.0f))) {
                quantize8<PACKED, WANT_FAKE, true, UNS>(xv, split, ca.x, cb.z, params_of(ca, cb), da.x,
                                                        db.z, params_of(da, db), g.Lf, g.Li, g.sign_unit,
                                                        g.sign_shift, w0, w1, mb, yv);
            } else {
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    yv[t] = 0.0f;
                    if (t < cnt) {
                        const int lt = l + __popc(inner & ((1u << t) - 1u));
                        const float4 ea = qa[lt];
                        const float4 eb = QB ? qb[lt] : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                        if (UNS) yv[t] = eb.z;                 // a constant row delivers lo
                        const float em = fabsf(ea.x);          // (-m marks a row kept off the fast paths)
                        if (em > 0.0f) {
                            const float xi = xv[t];
                            const int neg = !UNS && xi < 0.0f;
                            int q, tail;
                            float v;
                            const float a = UNS ? fminf(fmaxf(__fsub_rn(xi, eb.z), 0.0f), em)
                                                : fminf(fabsf(xi), em);
                            quantize_mag(a, params_of(ea, eb), g.Lf, q, tail, v);
                            const uint32_t code = (uint32_t)((neg << (g.bits - 1)) | q);
                            if (PACKED) w0 |= code << (4 * t);
                            else if (t < 4) w0 |= code << (8 * t);
                            else w1 |= code << (8 * (t - 4));
                            mb |= (uint32_t)tail << t;
                            yv[t] = UNS ? __fadd_rn(v, eb.z) : (neg ? -v : v);
                        }
                    }
                }
            }
        }
    } else {
        RowState rs;
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            yv[t] = 0.0f;
            if (t < cnt) {
                rs.seek(g.rows, g.A, g.Lf, i0 + t);
                if (UNS) yv[t] = rs.lo;
                if (rs.m > 0.0f) {
                    const float xi = xv[t];
                    const int neg = !UNS && xi < 0.0f;
                    int q, tail;
                    float v;
                    const float a = UNS ? fminf(fmaxf(__fsub_rn(xi, rs.lo), 0.0f), rs.m)
                                        : fminf(fabsf(xi), rs.m);
                    quantize_mag(a, rs.P, g.Lf, q, tail, v);
                    const uint32_t code = (uint32_t)((neg << (g.bits - 1)) | q);
                    if (PACKED) w0 |= code << (4 * t);
                    else if (t < 4) w0 |= code << (8 * t);
                    else w1 |= code << (8 * (t - 4));
                    mb |= (uint32_t)tail << t;
                    yv[t] = UNS ? __fadd_rn(v, rs.lo) : (neg ? -v : v);
                }
            }
        }
    }
    if (FULL) {
        // span_beg is a multiple of the span: the span's slices of the outputs start at
        // multiples of 512 / 2048 / 4096 bytes, so 32-bit offsets inside them suffice
        uint8_t* mask_s = g.mask + (span_beg >> 3);
        mask_s[li >> 3] = (uint8_t)mb;
        if (PACKED) {
            reinterpret_cast<uint32_t*>(g.codes + (span_beg >> 1))[li >> 3] = w0;
        } else {
            reinterpret_cast<uint2*>(g.codes + span_beg)[li >> 3] = make_uint2(w0, w1);
        }
        if (WANT_FAKE) {
            float4* f = reinterpret_cast<float4*>(g.fake + span_beg) + (li >> 2);
            __stcs(f, make_float4(yv[0], yv[1], yv[2], yv[3]));
            __stcs(f + 1, make_float4(yv[4], yv[5], yv[6], yv[7]));
        }
        return;
    }
    if (cnt == 0) return;
    g.mask[i0 >> 3] = (uint8_t)mb;
    if (PACKED) {
        uint8_t* dst = g.codes + (i0 >> 1);
        if (g.vec_codes && cnt == 8) {
            *reinterpret_cast<uint32_t*>(dst) = w0;
        } else {
            const int nb = (cnt + 1) >> 1;
            for (int b = 0; b < nb; ++b) dst[b] = (uint8_t)(w0 >> (8 * b));
        }
    } else {
        uint8_t* dst = g.codes + i0;
        if (g.vec_codes && cnt == 8) {
            *reinterpret_cast<uint2*>(dst) = make_uint2(w0, w1);
        } else {
            for (int t = 0; t < cnt; ++t)
                dst[t] = (uint8_t)((t < 4 ? w0 : w1) >> (8 * (t & 3)));
        }
    }
    if (WANT_FAKE) {
        if (g.vec_fake && cnt == 8) {
            __stcs(reinterpret_cast<float4*>(g.fake + i0), make_float4(yv[0], yv[1], yv[2], yv[3]));
            __stcs(reinterpret_cast<float4*>(g.fake + i0 + 4), make_float4(yv[4], yv[5], yv[6], yv[7]));
        } else {
            for (int t = 0; t < cnt; ++t) g.fake[i0 + t] = yv[t];
        }
    }
}

// PRE: the row maps were built ahead of time (premap: header, then one map per span).
template <bool PACKED, bool WANT_FAKE, bool UNS, bool LONG, bool PRE>
__global__ void __launch_bounds__(kMapThreads, (WANT_FAKE || UNS) ? 3 : 4)
quantize_map_kernel(const float* __restrict__ x, Rows rows, int64_t total, int bits, RowArrays A,
                    uint8_t* __restrict__ codes, uint8_t* __restrict__ mask,
                    float* __restrict__ fake, int vec_in, int vec_fake, int vec_codes,
                    int64_t spans_per_cta, const unsigned char* __restrict__ premap) {
    constexpr bool QB = WANT_FAKE || UNS;
    typedef MapStage<true, QB> Stage;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    if (PRE && !rowmap_matches(premap, rows, total)) {        // maps of another layout: no work
        if (threadIdx.x == 0) atomicOr(&g_quantize_timeout, 2);
        return;
    }
    Stage* st = reinterpret_cast<Stage*>(smem_raw);
    __shared__ uint64_t full_bar[kMapStages], empty_bar[kMapStages];
    const int Li = UNS ? (1 << bits) - 1 : (1 << (bits - 1)) - 1;    // largest level of a piece
    const float Lf = (float)Li;
    const uint32_t sign_unit = 1u << (bits - 1);
    const int sign_shift = 32 - bits;
    const int64_t nspans = (total + kMapSpan - 1) / kMapSpan;
    const int64_t first = blockIdx.x * spans_per_cta, last = min(first + spans_per_cta, nspans);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kMapStages; ++s) {
            // the data (or its stand-in) and the map; PRE: and the rows' constants
            mbar_init(&full_bar[s], PRE ? 3 : 2);
            mbar_init(&empty_bar[s], kMapConsumers);
        }
        fence_barrier_init();
    }
    __syncthreads();
    if (first >= last) return;

    if (PRE && warp == kMapConsumers) {
        // ---- producer, maps built ahead of time: the values and the map of a span arrive by
        // bulk copies; the warp computes the constants of the span's rows
        const SpanRowMap* maps = reinterpret_cast<const SpanRowMap*>(premap + kRowMapHeaderBytes);
        PreProducer<true, UNS> prod;
        prod.in = RowInputs{A.m, A.lo, A.p, A.xi, A.beta};
        prod.Lf = Lf;
        prod.begin(maps, first, last);
        int64_t it = 0;
        for (int64_t span = first; span < last; ++span, ++it) {
            const int s = (int)(it % kMapStages);
            const unsigned use = (unsigned)(it / kMapStages);
            if (use > 0 && !mbar_wait(&empty_bar[s], (use - 1) & 1u)) {
                if (lane == 0) atomicOr(&g_quantize_timeout, 1);
                for (int64_t j = it - 1; j >= 0 && j > it - 1 - kMapStages; --j)
                    mbar_wait(&full_bar[j % kMapStages], (unsigned)(j / kMapStages) & 1u);
                return;
            }
            const int64_t span_beg = span * kMapSpan, span_end = min(span_beg + kMapSpan, total);
            const unsigned bytes = q_bulk_bytes(span, total, vec_in);
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
            // the map travels while the constants are computed
            if (lane == 0) {
                mbar_expect_tx(&full_bar[s], (unsigned)sizeof(SpanRowMap));
                bulk_copy_g2s(&st[s].map, maps + span, (unsigned)sizeof(SpanRowMap), &full_bar[s]);
            }
            prod.build(st[s].qa, QB ? st[s].qb : nullptr, span, last);
            __syncwarp();
            if (lane == 0) mbar_arrive(&full_bar[s]);
        }
        return;
    }
    if (warp == kMapConsumers) {
        // ---- producer
        MapProducer<true, UNS> prod;
        prod.rows = rows;
        prod.in = RowInputs{A.m, A.lo, A.p, A.xi, A.beta};
        prod.Lf = Lf;
        // LONG: dense rows of at least a span, the map follows from the row length
        constexpr bool long_rows = LONG;
        // the values of the first spans do not depend on the rows: request them before the search
        for (int64_t span = first; span < last && span < first + kMapStages; ++span) {
            const unsigned bytes = q_bulk_bytes(span, total, vec_in);
            if (bytes != 0 && lane == 0) {
                mbar_expect_tx(&full_bar[span - first], bytes);
                bulk_copy_g2s(st[span - first].data, x + span * kMapSpan, bytes, &full_bar[span - first]);
            }
        }
        if (long_rows) prod.request_long(rows.dense_row(first * kMapSpan));
        else prod.request(warp_row_of(rows, first * kMapSpan), true);
        int64_t it = 0;
        for (int64_t span = first; span < last; ++span, ++it) {
            const int s = (int)(it % kMapStages);
            const unsigned use = (unsigned)(it / kMapStages);
            if (use > 0 && !mbar_wait(&empty_bar[s], (use - 1) & 1u)) {
                // never expected: report, let the copies of the earlier spans land (their stages'
                // barriers have this warp's arrivals already), and leave
                if (lane == 0) atomicOr(&g_quantize_timeout, 1);
                for (int64_t j = it - 1; j >= 0 && j > it - 1 - kMapStages; --j)
                    mbar_wait(&full_bar[j % kMapStages], (unsigned)(j / kMapStages) & 1u);
                return;
            }
            const int64_t span_beg = span * kMapSpan, span_end = min(span_beg + kMapSpan, total);
            const unsigned bytes = q_bulk_bytes(span, total, vec_in);
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
            if (long_rows)
                prod.build_long(st[s].map, st[s].qa, QB ? st[s].qb : nullptr, s, span_beg, span_end,
                                span + 1 < last);
            else
                prod.build(st[s].map, st[s].qa, QB ? st[s].qb : nullptr, span_beg, span_end,
                           span + 1 < last);
            __syncwarp();
            if (lane == 0) mbar_arrive(&full_bar[s]);
        }
        return;
    }

    // ---- consumers
    QuantizeCtx<UNS> ctx{rows, A, total, bits, Li, Lf, sign_unit, sign_shift, codes, mask, fake,
                         vec_fake, vec_codes};
    const int li0 = warp * (kMapSpan / kMapConsumers) + lane * 8;     // pass c: li0 + 256 c
    const bool vec_all = vec_codes && (!WANT_FAKE || vec_fake);
    int64_t it = 0;
    for (int64_t span = first; span < last; ++span, ++it) {
        const int s = (int)(it % kMapStages);
        const unsigned use = (unsigned)(it / kMapStages);
        if (!mbar_wait_relaxed(&full_bar[s], use & 1u)) {
            if (lane == 0) atomicOr(&g_quantize_timeout, 1);
            return;
        }
        const int64_t span_beg = span * kMapSpan;
        const Stage& S = st[s];
        // a whole span with a usable map and vector-aligned outputs: no counts, no 64-bit
        // indices, no byte-wise stores in the passes
        if (S.map.slow == 0 && span_beg + kMapSpan <= total && vec_all) {
#pragma unroll
            for (int c = 0; c < 2; ++c)
                quantize_pass<PACKED, WANT_FAKE, UNS, QB, true>(ctx, S.data, S.map, S.qa, S.qb,
                                                                span_beg, li0 + c * 256);
        } else {
#pragma unroll 1
            for (int c = 0; c < 2; ++c)
                quantize_pass<PACKED, WANT_FAKE, UNS, QB, false>(ctx, S.data, S.map, S.qa, S.qb,
                                                                 span_beg, li0 + c * 256);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[s]);
    }
}

// One span's worth of a thread's codes and region bits, requested ahead of use.
template <bool PACKED>
struct CodeRegs {
    uint32_t w0[kQChunks], w1[kQChunks], mb[kQChunks];
    __device__ __forceinline__ void load(const uint8_t* __restrict__ codes,
                                         const uint8_t* __restrict__ mask, int64_t span_beg,
                                         int64_t total, int vec_codes) {
#pragma unroll
        for (int c = 0; c < kQChunks; ++c) {
            const int64_t i0 = span_beg + chunk_offset(c);
            const int cnt = (int)max((int64_t)0, min((int64_t)8, total - i0));
            w0[c] = w1[c] = mb[c] = 0;
            if (cnt == 0) continue;
            if (PACKED) {
                const uint8_t* src = codes + (i0 >> 1);
                if (vec_codes && cnt == 8) {
                    w0[c] = __ldcs(reinterpret_cast<const unsigned int*>(src));
                } else {
                    const int nb = (cnt + 1) >> 1;
                    for (int b = 0; b < nb; ++b) w0[c] |= (uint32_t)src[b] << (8 * b);
                }
            } else {
                const uint8_t* src = codes + i0;
                if (vec_codes && cnt == 8) {
                    const uint2 w = __ldcs(reinterpret_cast<const uint2*>(src));
                    w0[c] = w.x; w1[c] = w.y;
                } else {
                    for (int t = 0; t < cnt; ++t) {
                        if (t < 4) w0[c] |= (uint32_t)src[t] << (8 * t);
                        else       w1[c] |= (uint32_t)src[t] << (8 * (t - 4));
                    }
                }
            }
            mb[c] = mask[i0 >> 3];
        }
    }
};

template <bool PACKED>
__device__ __forceinline__ uint32_t code_of(uint32_t w0, uint32_t w1, int t) {
    if (PACKED) return (w0 >> (4 * t)) & 0xFu;
    return ((t < 4 ? w0 : w1) >> (8 * (t & 3))) & 0xFFu;
}

// Eight consecutive codes, the first `split` of them in row A and the rest in row B (TWO = false:
// all in row A), both rows with m > 0.  The levels are masked out of the code words once per
// eight values and spread to one byte each; a byte permute then puts a level straight under the
// exponent of 1.5 * 2^23, whose subtraction leaves the level as a float (exact for q < 2^22)
// without an integer conversion.  The sign bit is shifted from its place in the code word to
// bit 31.
// UNS: one-sided range, the code is the level and the delivered value is v + lo.
template <bool PACKED, bool TWO, bool UNS>
__device__ __forceinline__ void dequantize8(uint32_t w0, uint32_t w1, uint32_t mb, int split,
                                            const PieceParams& A, float loA, const PieceParams& B,
                                            float loB, int qmask, int sign_shift, float (&yv)[8]) {
    // byte j of e0 / e1: level of value 2j / 2j + 1 (packed nibbles), or of value j / 4 + j
    const uint32_t rep = (uint32_t)qmask * 0x01010101u;
    const uint32_t e0 = w0 & rep;
    const uint32_t e1 = (PACKED ? (w0 >> 4) : w1) & rep;
    // the sign bit of the word's last code moved to bit 31 (sign_shift >= 28 for nibble codes,
    // >= 24 for byte codes)
    const uint32_t sw0 = w0 << (sign_shift - (PACKED ? 28 : 24));
    const uint32_t sw1 = w1 << (sign_shift - (PACKED ? 28 : 24));
    // the levels as floats, two at a time (the subtraction of 1.5 * 2^23 is a packed addition)
    float qv[8];
#pragma unroll
    for (int t = 0; t < 8; t += 2) {
        float r[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int tt = t + h;
            const uint32_t src = PACKED ? ((tt & 1) ? e1 : e0) : (tt < 4 ? e0 : e1);
            const uint32_t sel = 0x7650u | (uint32_t)(PACKED ? (tt >> 1) : (tt & 3));
            r[h] = __uint_as_float(__byte_perm(src, 0x4B400000u, sel));
        }
        unpack2(add2(pack2(r[0], r[1]), pack2(-12582912.0f, -12582912.0f)), qv[t], qv[t + 1]);
    }
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        const bool second = TWO && t >= split;
        const float lo = second ? loB : loA;
        const float p = second ? B.p : A.p;
        const float s1 = second ? B.s1 : A.s1;
        const float s2 = second ? B.s2 : A.s2;
        const bool tail = (mb & (1u << t)) != 0;
        const float q = qv[t];
        // both pieces, then one select (q s1 + 0 is q s1: nothing here is negative)
        const float vt = __fadd_rn(__fmul_rn(q, s2), p);
        const float v = tail ? vt : __fmul_rn(q, s1);
        // signed scheme: the code's sign bit, at bit 4 t + b - 1 (8 (t mod 4) + b - 1 for byte
        // codes) of its word, moved to bit 31
        // (the run-time part of the shift is applied once per word, sw0 / sw1 below; what is left
        // per value is a shift by a constant)
        const uint32_t sw = PACKED ? sw0 : (t < 4 ? sw0 : sw1);
        constexpr int kTop = PACKED ? 28 : 24;
        const int up = kTop - (PACKED ? 4 * t : 8 * (t & 3));
        yv[t] = UNS ? __fadd_rn(v, lo)
                    : __uint_as_float(__float_as_uint(v) | ((sw << up) & 0x80000000u));
    }
}

// ------------------------------------------------------------------ several rows per span
// What a consumer's pass of the inverse needs besides the stage.
struct DequantizeCtx {
    Rows rows;
    RowArrays A;
    int64_t total;
    int bits, qmask, sign_shift;
    float Lf;
    float* __restrict__ y;
    int vec_out;
};

// One pass of a consumer lane of the inverse: the eight codes (w0, w1) and region bits (mb) at
// offset li of the span that begins at flat index span_beg.  FULL: the span is complete, its map
// is usable and y can be stored with vector stores (no value counts, no 64-bit indices).
template <bool PACKED, bool UNS, bool BC, bool FULL>
__device__ __forceinline__ void dequantize_pass(const DequantizeCtx& g, uint32_t w0, uint32_t w1,
                                                uint32_t mb, const SpanRowMap& M, const float4* qa,
                                                const float4* qb, int64_t span_beg, int li) {
    constexpr bool QB = UNS || BC;
    const unsigned full = 0xffffffffu;
    const int64_t i0 = span_beg + li;
    const int cnt = FULL ? 8 : (int)max((int64_t)0, min((int64_t)8, g.total - i0));
    float yv[8];
    if (FULL || M.slow == 0) {
        uint32_t word;
        const int l = map_slot(M, li, word);
        const uint32_t inner = (word >> ((li & 31) + 1)) & 0x7Fu;   // starts at li+1 .. li+7
        const float4 ca = qa[l];
        const float4 ba = QB ? qb[l] : make_float4(0.0f, 1.0f, 0.0f, 0.0f);
        const float loA = UNS ? ba.x : 0.0f;
        const bool simple = inner == 0 && ca.x > 0.0f && cnt == 8;
        PieceParams PA;
        PA.p = ca.y; PA.s1 = ca.z; PA.s2 = ca.w; PA.inv1 = PA.inv2 = 0.0f;
        if (__all_sync(full, simple)) {
            dequantize8<PACKED, false, UNS>(w0, w1, mb, 8, PA, loA, PA, loA, g.qmask, g.sign_shift, yv);
            if (BC) {
#pragma unroll
                for (int t = 0; t < 8; ++t) yv[t] = __fadd_rn(__fmul_rn(ba.y, yv[t]), ba.z);
            }
        } else {
            const bool one = inner != 0 && (inner & (inner - 1)) == 0 && ca.x > 0.0f && cnt == 8;
            float4 da = ca, bb = ba;
            int split = 8;
            if (one) {
                da = qa[l + 1];
                if (QB) bb = qb[l + 1];
                split = __ffs(inner);
            }
            const float loB = UNS ? bb.x : 0.0f;
            if (__all_sync(full, simple || (one && da.x > 0.0f))) {
                PieceParams PB;
                PB.p = da.y; PB.s1 = da.z; PB.s2 = da.w; PB.inv1 = PB.inv2 = 0.0f;
                dequantize8<PACKED, true, UNS>(w0, w1, mb, split, PA, loA, PB, loB, g.qmask,
                                               g.sign_shift, yv);
                if (BC) {
#pragma unroll
                    for (int t = 0; t < 8; ++t)
                        yv[t] = __fadd_rn(__fmul_rn(t < split ? ba.y : bb.y, yv[t]),
                                          t < split ? ba.z : bb.z);
                }
            } else {
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    yv[t] = 0.0f;
                    if (t < cnt) {
                        const int lt = l + __popc(inner & ((1u << t) - 1u));
                        const float4 ea = qa[lt];
                        const float4 eb = QB ? qb[lt] : make_float4(0.0f, 1.0f, 0.0f, 0.0f);
                        const float loE = UNS ? eb.x : 0.0f;
                        if (UNS) yv[t] = loE;                  // a constant row delivers lo
                        if (ea.x > 0.0f) {
                            const uint32_t code = code_of<PACKED>(w0, w1, t);
                            const int tail = (mb >> t) & 1;
                            const int neg = !UNS && ((code >> (g.bits - 1)) & 1);
                            const float q = (float)(code & g.qmask);
                            float v = __fmul_rn(q, tail ? ea.w : ea.z);
                            v = __fadd_rn(v, tail ? ea.y : 0.0f);
                            yv[t] = UNS ? __fadd_rn(v, loE) : (neg ? -v : v);
                        }
                        if (BC) yv[t] = __fadd_rn(__fmul_rn(eb.y, yv[t]), eb.z);
                    }
                }
            }
        }
    } else {
        RowState rs;
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            yv[t] = 0.0f;
            if (t < cnt) {
                rs.seek(g.rows, g.A, g.Lf, i0 + t);
                if (UNS) yv[t] = rs.lo;
                if (rs.m > 0.0f) {
                    const uint32_t code = code_of<PACKED>(w0, w1, t);
                    const int tail = (mb >> t) & 1;
                    const int neg = !UNS && ((code >> (g.bits - 1)) & 1);
                    const float q = (float)(code & g.qmask);
                    float v = __fmul_rn(q, tail ? rs.P.s2 : rs.P.s1);
                    v = __fadd_rn(v, tail ? rs.P.p : 0.0f);
                    yv[t] = UNS ? __fadd_rn(v, rs.lo) : (neg ? -v : v);
                }
                if (BC) yv[t] = __fadd_rn(__fmul_rn(__ldg(g.A.xi + rs.row), yv[t]), __ldg(g.A.beta + rs.row));
            }
        }
    }
    if (FULL) {
        float4* dst = reinterpret_cast<float4*>(g.y + span_beg) + (li >> 2);
        __stcs(dst, make_float4(yv[0], yv[1], yv[2], yv[3]));
        __stcs(dst + 1, make_float4(yv[4], yv[5], yv[6], yv[7]));
        return;
    }
    if (cnt == 0) return;
    if (g.vec_out && cnt == 8) {
        __stcs(reinterpret_cast<float4*>(g.y + i0), make_float4(yv[0], yv[1], yv[2], yv[3]));
        __stcs(reinterpret_cast<float4*>(g.y + i0 + 4), make_float4(yv[4], yv[5], yv[6], yv[7]));
    } else {
        for (int t = 0; t < cnt; ++t) g.y[i0 + t] = yv[t];
    }
}

// A thread's codes and region bits of one span, requested ahead of use.  A complete span whose
// code words can be read whole takes 32-bit offsets from the span's slices of the two streams.
template <bool PACKED>
__device__ __forceinline__ void load_codes(CodeRegs<PACKED>& r, const uint8_t* __restrict__ codes,
                                           const uint8_t* __restrict__ mask, int64_t span_beg,
                                           int64_t total, int vec_codes, int li0) {
    if (vec_codes && span_beg + kMapSpan <= total) {
        const uint8_t* ms = mask + (span_beg >> 3);
#pragma unroll
        for (int c = 0; c < kQChunks; ++c) {
            const int g8 = (li0 + c * 256) >> 3;
            if (PACKED) {
                r.w0[c] = __ldcs(reinterpret_cast<const unsigned int*>(codes + (span_beg >> 1)) + g8);
                r.w1[c] = 0;
            } else {
                const uint2 w = __ldcs(reinterpret_cast<const uint2*>(codes + span_beg) + g8);
                r.w0[c] = w.x; r.w1[c] = w.y;
            }
            r.mb[c] = ms[g8];
        }
    } else {
        r.load(codes, mask, span_beg, total, vec_codes);
    }
}

// Producer / consumer form of the inverse (see quantize_map_kernel and pwlq_rowmap.cuh).  The
// producer writes row maps and constants only; the consumers request the codes and region bits
// of the next span into registers before they wait for the current span's map.
// BC: the bias-corrected value xi * y + beta (one multiply, one add) instead of y.
// PRE: the row maps were built ahead of time (premap: header, then one map per span).
template <bool PACKED, bool UNS, bool LONG, bool BC, bool PRE>
__global__ void __launch_bounds__(kMapThreads, 4)
dequantize_map_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ mask, Rows rows,
                      int64_t total, int bits, RowArrays A, float* __restrict__ y, int vec_codes,
                      int vec_out, int64_t spans_per_cta, const unsigned char* __restrict__ premap) {
    constexpr bool QB = UNS || BC;                    // the stages hold the second half of the constants
    typedef MapStage<false, QB> Stage;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    if (PRE && !rowmap_matches(premap, rows, total)) {        // maps of another layout: no work
        if (threadIdx.x == 0) atomicOr(&g_quantize_timeout, 2);
        return;
    }
    Stage* st = reinterpret_cast<Stage*>(smem_raw);
    __shared__ uint64_t full_bar[kMapStages], empty_bar[kMapStages];
    const int qmask = UNS ? (1 << bits) - 1 : (1 << (bits - 1)) - 1;   // the level inside a code
    const float Lf = (float)qmask;
    const int sign_shift = 32 - bits;                 // moves a code's sign bit to bit 31
    const int64_t nspans = (total + kMapSpan - 1) / kMapSpan;
    const int64_t first = blockIdx.x * spans_per_cta, last = min(first + spans_per_cta, nspans);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kMapStages; ++s) {
            mbar_init(&full_bar[s], PRE ? 2 : 1);  // PRE: the map and the rows' constants
            mbar_init(&empty_bar[s], kMapConsumers);
        }
        fence_barrier_init();
    }
    __syncthreads();
    if (first >= last) return;

    if (PRE && warp == kMapConsumers) {
        // ---- producer, maps built ahead of time: the map arrives by a bulk copy, the warp
        // computes the constants of the span's rows
        const SpanRowMap* maps = reinterpret_cast<const SpanRowMap*>(premap + kRowMapHeaderBytes);
        PreProducer<true, UNS, true, BC> prod;
        prod.in = RowInputs{A.m, A.lo, A.p, A.xi, A.beta};
        prod.Lf = Lf;
        prod.begin(maps, first, last);
        int64_t it = 0;
        for (int64_t span = first; span < last; ++span, ++it) {
            const int s = (int)(it % kMapStages);
            const unsigned use = (unsigned)(it / kMapStages);
            if (use > 0 && !mbar_wait(&empty_bar[s], (use - 1) & 1u)) {
                if (lane == 0) atomicOr(&g_quantize_timeout, 1);
                for (int64_t j = it - 1; j >= 0 && j > it - 1 - kMapStages; --j)
                    mbar_wait(&full_bar[j % kMapStages], (unsigned)(j / kMapStages) & 1u);
                return;
            }
            if (lane == 0) {                       // the map travels while the constants are computed
                mbar_expect_tx(&full_bar[s], (unsigned)sizeof(SpanRowMap));
                bulk_copy_g2s(&st[s].map, maps + span, (unsigned)sizeof(SpanRowMap), &full_bar[s]);
            }
            prod.build(st[s].qa, QB ? st[s].qb : nullptr, span, last);
            __syncwarp();
            if (lane == 0) mbar_arrive(&full_bar[s]);
        }
        return;
    }
    if (warp == kMapConsumers) {
        // ---- producer
        MapProducer<true, UNS, true, BC> prod;
        prod.rows = rows;
        prod.in = RowInputs{A.m, A.lo, A.p, A.xi, A.beta};
        prod.Lf = Lf;
        if (LONG) prod.request_long(rows.dense_row(first * kMapSpan));
        else prod.request(warp_row_of(rows, first * kMapSpan), true);
        int64_t it = 0;
        for (int64_t span = first; span < last; ++span, ++it) {
            const int s = (int)(it % kMapStages);
            const unsigned use = (unsigned)(it / kMapStages);
            if (use > 0 && !mbar_wait(&empty_bar[s], (use - 1) & 1u)) {
                if (lane == 0) atomicOr(&g_quantize_timeout, 1);
                return;
            }
            const int64_t span_beg = span * kMapSpan, span_end = min(span_beg + kMapSpan, total);
            if (LONG)
                prod.build_long(st[s].map, st[s].qa, QB ? st[s].qb : nullptr, s, span_beg, span_end,
                                span + 1 < last);
            else
                prod.build(st[s].map, st[s].qa, QB ? st[s].qb : nullptr, span_beg, span_end,
                           span + 1 < last);
            __syncwarp();
            if (lane == 0) mbar_arrive(&full_bar[s]);
        }
        return;
    }

    // ---- consumers
    const DequantizeCtx ctx{rows, A, total, bits, qmask, sign_shift, Lf, y, vec_out};
    const int li0 = warp * (kMapSpan / kMapConsumers) + lane * 8;     // pass c: li0 + 256 c
    CodeRegs<PACKED> cur, nxt;
    load_codes<PACKED>(cur, codes, mask, first * kMapSpan, total, vec_codes, li0);
    int64_t it = 0;
    for (int64_t span = first; span < last; ++span, ++it) {
        const int s = (int)(it % kMapStages);
        const unsigned use = (unsigned)(it / kMapStages);
        const int64_t span_beg = span * kMapSpan;
        if (span + 1 < last) load_codes<PACKED>(nxt, codes, mask, span_beg + kMapSpan, total, vec_codes, li0);
        if (!mbar_wait_relaxed(&full_bar[s], use & 1u)) {
            if (lane == 0) atomicOr(&g_quantize_timeout, 1);
            return;
        }
        const Stage& S = st[s];
        if (S.map.slow == 0 && span_beg + kMapSpan <= total && vec_out) {
#pragma unroll
            for (int c = 0; c < kQChunks; ++c)
                dequantize_pass<PACKED, UNS, BC, true>(ctx, cur.w0[c], cur.w1[c], cur.mb[c], S.map, S.qa,
                                                       S.qb, span_beg, li0 + c * 256);
        } else {
#pragma unroll
            for (int c = 0; c < kQChunks; ++c)
                dequantize_pass<PACKED, UNS, BC, false>(ctx, cur.w0[c], cur.w1[c], cur.mb[c], S.map, S.qa,
                                                        S.qb, span_beg, li0 + c * 256);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[s]);
        cur = nxt;
    }
}

// ------------------------------------------------ two or three breakpoints per row (Sec. 5.1)
// The same producer / consumer structure for rows with three or four regions: the producer
// describes the rows of every span (row map, and per row one record of constants per region, see
// store_row_consts_multi), the consumers quantize or expand eight consecutive values per lane and
// pass; a value's constants are one shared-memory read indexed by its region.  The region index 0..3 takes two bits per value (16 bits per lane and pass).
// Whole spans with a usable map take the form below; the tensor's last, partial span and spans
// the map cannot describe go value by value with a lookup in global memory.
// Two stages and four CTAs per SM (three stages were no faster: 0.41 / 0.36 of the copy peak with
// three / two CTAs per SM against 0.45).
constexpr int kMultiStages = 2;
constexpr int kMultiCtasPerSm = 4;
template <bool DATA>
struct MultiStage {
    alignas(128) float data[DATA ? kMapSpan : 4];
    SpanRowMap map;
    alignas(16) float4 q[4 * kMultiSlots];
};

// Region, offset, L / range and step of magnitude a in a row with breakpoints z = (p1, p2, p3, m).
__device__ __forceinline__ int region_of(float a, const float4& z) {
    return (a > z.x) + (a > z.y) + (a > z.z);
}
__device__ __forceinline__ float pick4(int r, float v0, const float4& v) {
    return r == 0 ? v0 : (r == 1 ? v.x : (r == 2 ? v.y : v.z));
}
__device__ __forceinline__ float pick4(int r, const float4& v) {
    return r == 0 ? v.x : (r == 1 ? v.y : (r == 2 ? v.z : v.w));
}

// One value of a row with constants (z, inv, s): code, region and delivered value; the sequence
// of the element-wise kernel (every product and sum rounded on its own).  A row with m <= 0
// delivers zeros.
__device__ __forceinline__ void quantize_multi_value(float xi, const float4& z, const float4& inv,
                                                     const float4& s, float Lf, int bits,
                                                     uint32_t& code, uint32_t& reg, float& y) {
    const float m = z.w;
    const float a = fminf(fabsf(xi), m);
    const int r = region_of(a, z);
    const float zr = pick4(r, 0.0f, z);
    const float rr = __fadd_rn(__fmul_rn(__fsub_rn(a, zr), pick4(r, inv)), 12582912.0f);
    const float q = fminf(__fsub_rn(rr, 12582912.0f), Lf);
    const float v = __fadd_rn(__fmul_rn(q, pick4(r, s)), zr);
    const int neg = xi < 0.0f;
    const bool ok = m > 0.0f;
    code = ok ? (uint32_t)((neg << (bits - 1)) | (int)q) : 0u;
    reg = ok ? (uint32_t)r : 0u;
    y = ok ? (neg ? -v : v) : 0.0f;
}

struct QuantizeMultiCtx {
    Rows rows;
    const float* __restrict__ m;
    BreakPts bp;
    int64_t total;
    int bits;
    float Lf;
    uint8_t* __restrict__ codes;
    uint8_t* __restrict__ region2;
    float* __restrict__ fake;
};

// The constants of the row in slot l that a lane keeps in registers: the three breakpoints, the
// range and the sign mask (0 for a row that delivers zeros).
struct MultiRow {
    const float4* rec;
    float p1, p2, p3, m;
    uint32_t smask;
    __device__ __forceinline__ void load(const float4* q, int l) {
        rec = q + 4 * l;
        const float4 c0 = rec[0], c1 = rec[1];
        m = c0.w;
        p1 = c1.x;
        smask = __float_as_uint(c1.w);
        p2 = rec[2].x;
        p3 = rec[3].x;
    }
};

// One pass of a consumer lane over the eight values at offset li of a whole span with a usable
// map (all outputs vector-aligned).  Per value the sequence of the element-wise kernel, every
// product and sum rounded on its own; the sign is the sign bit of x + 0.0 (so that -0.0 is not
// negative) under the row's mask.
template <bool PACKED, bool WANT_FAKE>
__device__ __forceinline__ void quantize_multi_pass(const QuantizeMultiCtx& g, const float* data,
                                                    const SpanRowMap& M, const float4* q,
                                                    int64_t span_beg, int li) {
    const float4 xa = *reinterpret_cast<const float4*>(data + li);
    const float4 xb = *reinterpret_cast<const float4*>(data + li + 4);
    const float xv[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
    uint32_t word;
    const int l = map_slot(M, li, word);
    const uint32_t inner = (word >> ((li & 31) + 1)) & 0x7Fu;       // starts at li+1 .. li+7
    MultiRow R;
    R.load(q, l);
    // As in quantize8: the level sits in the low mantissa bits of rr (clamped to L as a float:
    // 1.5 * 2^23 + L), so the rr patterns are summed at their code positions and the constant
    // their exponent fields add up to is taken off once; the sign flags (sign bit of x + 0.0 under
    // the row's mask) are gathered with one funnel shift each and spread to their positions once.
    const uint32_t sign_unit = 1u << (g.bits - 1);
    const float top = __fadd_rn(12582912.0f, g.Lf);                 // exact: L < 2^22
    uint32_t acc0 = 0, acc1 = 0, rw = 0, signs = 0;
    float yv[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        if (t > 0 && (inner & (1u << (t - 1))))                     // a row starts at this value
            R.load(q, l + __popc(inner & ((1u << t) - 1u)));
        const float xi = xv[t];
        const float a = fminf(fabsf(xi), R.m);
        const int r = (a > R.p1) + (a > R.p2) + (a > R.p3);
        const float4 c = R.rec[r];                                  // (z, L / range, step, -)
        const float rr = fminf(__fadd_rn(__fmul_rn(__fsub_rn(a, c.x), c.y), 12582912.0f), top);
        const uint32_t sign = __float_as_uint(__fadd_rn(xi, 0.0f)) & R.smask;
        signs = __funnelshift_l(sign, signs, 1);                    // value t ends up at bit 7 - t
        if (PACKED) acc0 += __float_as_uint(rr) << (4 * t);
        else if (t < 4) acc0 += __float_as_uint(rr) << (8 * t);
        else acc1 += __float_as_uint(rr) << (8 * (t - 4));
        if (WANT_FAKE) {
            const float qf = __fsub_rn(rr, 12582912.0f);
            const float v = __fadd_rn(__fmul_rn(qf, c.z), c.x);
            yv[t] = __uint_as_float(__float_as_uint(v) | sign);
        }
        rw |= (uint32_t)r << (2 * t);
    }
    signs = __brev(signs) >> 24;                                    // value t at bit t
    uint32_t w0, w1 = 0;
    if (PACKED) {
        constexpr uint32_t kGarbage = (uint32_t)(0x4B400000ull * 0x11111111ull);
        w0 = (acc0 - kGarbage) | spread_to_nibbles(signs) * sign_unit;
    } else {
        constexpr uint32_t kGarbage = (uint32_t)(0x4B400000ull * 0x01010101ull);
        w0 = (acc0 - kGarbage) | spread_to_bytes(signs) * sign_unit;
        w1 = (acc1 - kGarbage) | spread_to_bytes(signs >> 4) * sign_unit;
    }
    // span_beg is a multiple of the span: 32-bit offsets inside the span's slices of the outputs
    reinterpret_cast<uint16_t*>(g.region2 + (span_beg >> 2))[li >> 3] = (uint16_t)rw;
    if (PACKED) reinterpret_cast<uint32_t*>(g.codes + (span_beg >> 1))[li >> 3] = w0;
    else        reinterpret_cast<uint2*>(g.codes + span_beg)[li >> 3] = make_uint2(w0, w1);
    if (WANT_FAKE) {
        float4* f = reinterpret_cast<float4*>(g.fake + span_beg) + (li >> 2);
        __stcs(f, make_float4(yv[0], yv[1], yv[2], yv[3]));
        __stcs(f + 1, make_float4(yv[4], yv[5], yv[6], yv[7]));
    }
}

// The same value by value, rows looked up in global memory: the tensor's last span, and spans
// without a usable map.
template <bool PACKED, bool WANT_FAKE>
__device__ __forceinline__ void quantize_multi_slow(const QuantizeMultiCtx& g, const float* data,
                                                    int64_t span_beg, int li) {
    const int64_t i0 = span_beg + li;
    const int cnt = (int)max((int64_t)0, min((int64_t)8, g.total - i0));
    if (cnt == 0) return;
    Row3 rs;
    rs.whole(g.rows);
    uint32_t code[8], reg[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        code[t] = reg[t] = 0;
        if (t < cnt) {
            rs.seek(g.rows, g.m, g.bp, g.Lf, i0 + t);
            const float4 z = make_float4(rs.P.z[1], rs.P.z[2], rs.P.z[3], rs.m);
            const float4 inv = make_float4(rs.P.inv[0], rs.P.inv[1], rs.P.inv[2], rs.P.inv[3]);
            const float4 s = make_float4(rs.P.s[0], rs.P.s[1], rs.P.s[2], rs.P.s[3]);
            float y;
            quantize_multi_value(data[li + t], z, inv, s, g.Lf, g.bits, code[t], reg[t], y);
            if (WANT_FAKE) g.fake[i0 + t] = y;
        }
    }
#pragma unroll
    for (int b = 0; b < 2; ++b)
        if (4 * b < cnt)
            g.region2[(i0 >> 2) + b] = (uint8_t)(reg[4 * b] | (reg[4 * b + 1] << 2) |
                                                 (reg[4 * b + 2] << 4) | (reg[4 * b + 3] << 6));
    if (PACKED) {
#pragma unroll
        for (int b = 0; b < 4; ++b)
            if (2 * b < cnt) g.codes[(i0 >> 1) + b] = (uint8_t)(code[2 * b] | (code[2 * b + 1] << 4));
    } else {
#pragma unroll
        for (int t = 0; t < 8; ++t)
            if (t < cnt) g.codes[i0 + t] = (uint8_t)code[t];
    }
}

// P3: the rows have a third breakpoint.  x, codes, region2 and fake are vector-aligned (the
// launcher sends everything else to the element-wise kernel).
template <bool PACKED, bool WANT_FAKE, bool P3>
__global__ void __launch_bounds__(kMapThreads, kMultiCtasPerSm)
quantize_multi_kernel(const float* __restrict__ x, Rows rows, int64_t total, int bits,
                      const float* __restrict__ m, BreakPts bp, uint8_t* __restrict__ codes,
                      uint8_t* __restrict__ region2, float* __restrict__ fake,
                      int64_t spans_per_cta) {
    typedef MultiStage<true> Stage;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Stage* st = reinterpret_cast<Stage*>(smem_raw);
    __shared__ uint64_t full_bar[kMultiStages], empty_bar[kMultiStages];
    const float Lf = (float)((1 << (bits - 1)) - 1);
    const int64_t nspans = (total + kMapSpan - 1) / kMapSpan;
    const int64_t first = blockIdx.x * spans_per_cta, last = min(first + spans_per_cta, nspans);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kMultiStages; ++s) {
            mbar_init(&full_bar[s], 2);            // the data (or its stand-in) and the map
            mbar_init(&empty_bar[s], kMapConsumers);
        }
        fence_barrier_init();
    }
    __syncthreads();
    if (first >= last) return;

    if (warp == kMapConsumers) {
        // ---- producer
        MapProducer<true, false, false, P3, 2> prod;
        prod.rows = rows;
        prod.in = RowInputs{m, bp.p2, bp.p1, bp.p3, nullptr};
        prod.Lf = Lf;
        prod.pstride = bp.stride;
        for (int64_t span = first; span < last && span < first + kMultiStages; ++span) {
            const unsigned bytes = q_bulk_bytes(span, total, 1);
            if (bytes != 0 && lane == 0) {
                mbar_expect_tx(&full_bar[span - first], bytes);
                bulk_copy_g2s(st[span - first].data, x + span * kMapSpan, bytes, &full_bar[span - first]);
            }
        }
        prod.request(warp_row_of(rows, first * kMapSpan), true);
        int64_t it = 0;
        for (int64_t span = first; span < last; ++span, ++it) {
            const int s = (int)(it % kMultiStages);
            const unsigned use = (unsigned)(it / kMultiStages);
            if (use > 0 && !mbar_wait(&empty_bar[s], (use - 1) & 1u)) {
                // never expected: report, let the copies of the earlier spans land, and leave
                if (lane == 0) atomicOr(&g_quantize_timeout, 1);
                for (int64_t j = it - 1; j >= 0 && j > it - 1 - kMultiStages; --j)
                    mbar_wait(&full_bar[j % kMultiStages], (unsigned)(j / kMultiStages) & 1u);
                return;
            }
            const int64_t span_beg = span * kMapSpan, span_end = min(span_beg + kMapSpan, total);
            const unsigned bytes = q_bulk_bytes(span, total, 1);
            if (bytes != 0) {
                if (lane == 0 && use > 0) {        // (first round: requested above)
                    mbar_expect_tx(&full_bar[s], bytes);
                    bulk_copy_g2s(st[s].data, x + span_beg, bytes, &full_bar[s]);
                }
            } else {                               // ragged tail: plain loads
                for (int i = lane; i < (int)(span_end - span_beg); i += 32) st[s].data[i] = x[span_beg + i];
                __syncwarp();
                if (lane == 0) mbar_arrive(&full_bar[s]);
            }
            prod.build(st[s].map, st[s].q, nullptr, span_beg, span_end, span + 1 < last);
            __syncwarp();
            if (lane == 0) mbar_arrive(&full_bar[s]);
        }
        return;
    }

    // ---- consumers
    const QuantizeMultiCtx ctx{rows, m, bp, total, bits, Lf, codes, region2, fake};
    const int li0 = warp * (kMapSpan / kMapConsumers) + lane * 8;     // pass c: li0 + 256 c
    int64_t it = 0;
    for (int64_t span = first; span < last; ++span, ++it) {
        const int s = (int)(it % kMultiStages);
        const unsigned use = (unsigned)(it / kMultiStages);
        if (!mbar_wait_relaxed(&full_bar[s], use & 1u)) {
            if (lane == 0) atomicOr(&g_quantize_timeout, 1);
            return;
        }
        const int64_t span_beg = span * kMapSpan;
        const Stage& S = st[s];
        if (S.map.slow == 0 && span_beg + kMapSpan <= total) {
#pragma unroll
            for (int c = 0; c < 2; ++c)
                quantize_multi_pass<PACKED, WANT_FAKE>(ctx, S.data, S.map, S.q, span_beg, li0 + c * 256);
        } else {
#pragma unroll 1
            for (int c = 0; c < 2; ++c)
                quantize_multi_slow<PACKED, WANT_FAKE>(ctx, S.data, span_beg, li0 + c * 256);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[s]);
    }
}

// A thread's codes and region bits of one span, requested ahead of use (whole spans: one load
// per stream and pass; the tensor's last span byte by byte).
template <bool PACKED>
struct MultiCodeRegs {
    uint32_t w0[kQChunks], w1[kQChunks], rw[kQChunks];
    __device__ __forceinline__ void load(const uint8_t* __restrict__ codes,
                                         const uint8_t* __restrict__ region2, int64_t span_beg,
                                         int64_t total, int li0) {
#pragma unroll
        for (int c = 0; c < kQChunks; ++c) {
            const int li = li0 + c * 256;
            w0[c] = w1[c] = rw[c] = 0;
            if (span_beg + kMapSpan <= total) {
                const int g8 = li >> 3;
                rw[c] = __ldcs(reinterpret_cast<const unsigned short*>(region2 + (span_beg >> 2)) + g8);
                if (PACKED) {
                    w0[c] = __ldcs(reinterpret_cast<const unsigned int*>(codes + (span_beg >> 1)) + g8);
                } else {
                    const uint2 w = __ldcs(reinterpret_cast<const uint2*>(codes + span_beg) + g8);
                    w0[c] = w.x; w1[c] = w.y;
                }
            } else {
                const int64_t i0 = span_beg + li;
                const int cnt = (int)max((int64_t)0, min((int64_t)8, total - i0));
                for (int t = 0; t < cnt; ++t) {
                    const int64_t i = i0 + t;
                    const uint32_t code = PACKED ? ((codes[i >> 1] >> ((i & 1) * 4)) & 0xFu) : codes[i];
                    if (PACKED) w0[c] |= code << (4 * t);
                    else if (t < 4) w0[c] |= code << (8 * t);
                    else w1[c] |= code << (8 * (t - 4));
                    rw[c] |= (uint32_t)((region2[i >> 2] >> ((i & 3) * 2)) & 3u) << (2 * t);
                }
            }
        }
    }
};

// Delivered value of one code in a row with breakpoints z = (p1, p2, p3, m) and steps s.
__device__ __forceinline__ float dequantize_multi_value(uint32_t code, int r, const float4& z,
                                                        const float4& s, int bits, int qmask) {
    const float v = __fadd_rn(__fmul_rn((float)(int)(code & (uint32_t)qmask), pick4(r, s)),
                              pick4(r, 0.0f, z));
    const bool neg = ((code >> (bits - 1)) & 1u) != 0;
    return z.w > 0.0f ? (neg ? -v : v) : 0.0f;
}

template <bool PACKED, bool P3>
__global__ void __launch_bounds__(kMapThreads, kMultiCtasPerSm)
dequantize_multi_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ region2,
                        Rows rows, int64_t total, int bits, const float* __restrict__ m,
                        BreakPts bp, float* __restrict__ y, int64_t spans_per_cta) {
    typedef MultiStage<false> Stage;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Stage* st = reinterpret_cast<Stage*>(smem_raw);
    __shared__ uint64_t full_bar[kMultiStages], empty_bar[kMultiStages];
    const int qmask = (1 << (bits - 1)) - 1;
    const float Lf = (float)qmask;
    const int rmax = P3 ? 3 : 2;
    const int sign_shift = 32 - bits;                 // moves a code's sign bit to bit 31
    const int64_t nspans = (total + kMapSpan - 1) / kMapSpan;
    const int64_t first = blockIdx.x * spans_per_cta, last = min(first + spans_per_cta, nspans);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kMultiStages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], kMapConsumers);
        }
        fence_barrier_init();
    }
    __syncthreads();
    if (first >= last) return;

    if (warp == kMapConsumers) {
        // ---- producer: row maps and constants only
        MapProducer<true, false, true, P3, 2> prod;
        prod.rows = rows;
        prod.in = RowInputs{m, bp.p2, bp.p1, bp.p3, nullptr};
        prod.Lf = Lf;
        prod.pstride = bp.stride;
        prod.request(warp_row_of(rows, first * kMapSpan), true);
        int64_t it = 0;
        for (int64_t span = first; span < last; ++span, ++it) {
            const int s = (int)(it % kMultiStages);
            const unsigned use = (unsigned)(it / kMultiStages);
            if (use > 0 && !mbar_wait(&empty_bar[s], (use - 1) & 1u)) {
                if (lane == 0) atomicOr(&g_quantize_timeout, 1);
                return;
            }
            const int64_t span_beg = span * kMapSpan, span_end = min(span_beg + kMapSpan, total);
            prod.build(st[s].map, st[s].q, nullptr, span_beg, span_end, span + 1 < last);
            __syncwarp();
            if (lane == 0) mbar_arrive(&full_bar[s]);
        }
        return;
    }

    // ---- consumers
    const int li0 = warp * (kMapSpan / kMapConsumers) + lane * 8;     // pass c: li0 + 256 c
    MultiCodeRegs<PACKED> cur, nxt;
    cur.load(codes, region2, first * kMapSpan, total, li0);
    int64_t it = 0;
    for (int64_t span = first; span < last; ++span, ++it) {
        const int s = (int)(it % kMultiStages);
        const unsigned use = (unsigned)(it / kMultiStages);
        const int64_t span_beg = span * kMapSpan;
        if (span + 1 < last) nxt.load(codes, region2, span_beg + kMapSpan, total, li0);
        if (!mbar_wait_relaxed(&full_bar[s], use & 1u)) {
            if (lane == 0) atomicOr(&g_quantize_timeout, 1);
            return;
        }
        const Stage& S = st[s];
        const bool whole = S.map.slow == 0 && span_beg + kMapSpan <= total;
#pragma unroll
        for (int c = 0; c < kQChunks; ++c) {
            const int li = li0 + c * 256;
            const uint32_t w0 = cur.w0[c], w1 = cur.w1[c], rw = cur.rw[c];
            if (whole) {
                uint32_t word;
                const int l = map_slot(S.map, li, word);
                const uint32_t inner = (word >> ((li & 31) + 1)) & 0x7Fu;
                const float4* rec = S.q + 4 * l;
                uint32_t smask = __float_as_uint(rec[1].w);
                float yv[8];
                // the levels as floats without an integer conversion, two at a time, and the
                // sign bits moved with one run-time shift per code word (as in dequantize8)
                const uint32_t rep = (uint32_t)qmask * 0x01010101u;
                const uint32_t e0 = w0 & rep;
                const uint32_t e1 = (PACKED ? (w0 >> 4) : w1) & rep;
                const uint32_t sw0 = w0 << (sign_shift - (PACKED ? 28 : 24));
                const uint32_t sw1 = w1 << (sign_shift - (PACKED ? 28 : 24));
                float qv[8];
#pragma unroll
                for (int t = 0; t < 8; t += 2) {
                    float r[2];
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int tt = t + h;
                        const uint32_t src = PACKED ? ((tt & 1) ? e1 : e0) : (tt < 4 ? e0 : e1);
                        const uint32_t sel = 0x7650u | (uint32_t)(PACKED ? (tt >> 1) : (tt & 3));
                        r[h] = __uint_as_float(__byte_perm(src, 0x4B400000u, sel));
                    }
                    unpack2(add2(pack2(r[0], r[1]), pack2(-12582912.0f, -12582912.0f)), qv[t], qv[t + 1]);
                }
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    if (t > 0 && (inner & (1u << (t - 1)))) {
                        rec = S.q + 4 * (l + __popc(inner & ((1u << t) - 1u)));
                        smask = __float_as_uint(rec[1].w);
                    }
                    const float4 c = rec[min((int)((rw >> (2 * t)) & 3u), rmax)];   // (z, -, step, -)
                    const float v = __fadd_rn(__fmul_rn(qv[t], c.z), c.x);
                    const uint32_t sw = PACKED ? sw0 : (t < 4 ? sw0 : sw1);
                    const int up = (PACKED ? 28 : 24) - (PACKED ? 4 * t : 8 * (t & 3));
                    yv[t] = __uint_as_float(__float_as_uint(v) | ((sw << up) & smask));
                }
                float4* f = reinterpret_cast<float4*>(y + span_beg) + (li >> 2);
                __stcs(f, make_float4(yv[0], yv[1], yv[2], yv[3]));
                __stcs(f + 1, make_float4(yv[4], yv[5], yv[6], yv[7]));
            } else {
                const int64_t i0 = span_beg + li;
                const int cnt = (int)max((int64_t)0, min((int64_t)8, total - i0));
                Row3 rs;
                rs.whole(rows);
                for (int t = 0; t < cnt; ++t) {
                    rs.seek(rows, m, bp, Lf, i0 + t);
                    const float4 z = make_float4(rs.P.z[1], rs.P.z[2], rs.P.z[3], rs.m);
                    const float4 sv = make_float4(rs.P.s[0], rs.P.s[1], rs.P.s[2], rs.P.s[3]);
                    y[i0 + t] = dequantize_multi_value(code_of<PACKED>(w0, w1, t),
                                                       min((int)((rw >> (2 * t)) & 3u), rmax), z, sv,
                                                       bits, qmask);
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[s]);
        cur = nxt;
    }
}

static inline bool aligned(const void* p, size_t a) {
    return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0;
}

// CTAs of `kernel` that fit the device at once.  Looked up once per (kernel, device); the first
// lookup also opts the kernel in to its dynamic shared memory size.
static int64_t device_slots(const void* kernel, int threads, size_t smem) {
    struct Entry { const void* kernel; int dev; int ctas; };
    static Entry table[64];
    static int used = 0;
    static std::mutex mu;
    int dev = 0;
    cudaGetDevice(&dev);
    int ctas = 0;
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < used; ++i)
        if (table[i].kernel == kernel && table[i].dev == dev) ctas = table[i].ctas;
    if (ctas == 0) {
        if (smem > 0)
            cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        int sms = 0, per_sm = 0;
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, smem);
        ctas = (sms > 0 && per_sm > 0) ? sms * per_sm : 148;
        if (used < 64) table[used++] = Entry{kernel, dev, ctas};
    }
    return ctas;
}

// Grid and spans per CTA.  The producer / consumer kernels walk consecutive spans, handed out in
// blocks of at most kSpansPerBlockMax, about two per slot when the input is small: a block should
// be long enough to pay for the producer's start (finding its first row), and short enough for
// the hardware scheduler to even out what differs between spans.
struct SpanGrid { unsigned grid; int64_t per_cta; };
static SpanGrid span_grid(const void* kernel, int threads, size_t smem, int64_t nspans) {
    const int64_t slots = device_slots(kernel, threads, smem);
    const int64_t per_cta = std::min<int64_t>(
        std::max<int64_t>((nspans + 2 * slots - 1) / (2 * slots), 1), kSpansPerBlockMax);
    return SpanGrid{(unsigned)((nspans + per_cta - 1) / per_cta), per_cta};
}

int take_quantize_timeout_flag() {
    int v = 0;
    const int zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_quantize_timeout, sizeof(int)) != cudaSuccess) return -1;
    if (v != 0 && cudaMemcpyToSymbol(g_quantize_timeout, &zero, sizeof(int)) != cudaSuccess) return -1;
    return v;
}

// Self-test of the expiry path: one warp initialises a barrier that expects one arrival which
// nobody makes, polls it `polls` times through the helper the streaming kernels use, reports the
// expiry exactly as they do, and returns.  No copy is in flight and nothing is left waiting.
__global__ void expire_wait_kernel(int polls) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        fence_barrier_init();
    }
    __syncwarp();
    if (!mbar_wait(&bar, 0u, polls) && threadIdx.x == 0) atomicOr(&g_quantize_timeout, 1);
}
cudaError_t launch_expire_wait(int polls, cudaStream_t stream) {
    expire_wait_kernel<<<1, 32, 0, stream>>>(polls);
    return cudaGetLastError();
}

// lo == nullptr: signed scheme, m = abs-max.  lo != nullptr: one-sided ranges [lo, m].
cudaError_t launch_quantize(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                            int64_t total, int bits, const float* m, const float* lo,
                            const float* p, uint8_t* codes, uint8_t* mask, float* fake, int layout,
                            cudaStream_t stream, int64_t shift, const void* rowmap) {
    const float* xi = nullptr;
    const float* beta = nullptr;
    if (total == 0) return cudaSuccess;
    Rows rows{row_offsets, C, n, n > 0 ? 1.0 / (double)n : 0.0, row_offsets ? shift : 0};
    const RowArrays A{m, lo, p, xi, beta};
    const bool packed = (layout == 1 && bits <= 4);
    const int64_t nspans = (total + kQSpan - 1) / kQSpan;
    const int vec_in = aligned(x, 16), vec_fake = fake ? aligned(fake, 16) : 0;
    const int vec_codes = packed ? aligned(codes, 4) : aligned(codes, 8);
    const bool long_rows = row_offsets == nullptr && n >= kMapSpan;   // the map follows from n
    // (maps built ahead of time are of no use where the map follows from the row length)
    const unsigned char* premap = long_rows ? nullptr : static_cast<const unsigned char*>(rowmap);
#define PWLQ_LAUNCH_QUANTIZE_AS(PK, FK, UN, LG, PR)                                                \
    do {                                                                                          \
        const size_t msmem = sizeof(MapStage<true, FK || UN>) * kMapStages;                       \
        const SpanGrid g = span_grid((const void*)quantize_map_kernel<PK, FK, UN, LG, PR>,        \
                                     kMapThreads, msmem, nspans);                                 \
        quantize_map_kernel<PK, FK, UN, LG, PR><<<g.grid, kMapThreads, msmem, stream>>>(          \
            x, rows, total, bits, A, codes, mask, fake, vec_in, vec_fake, vec_codes, g.per_cta,   \
            premap);                                                                              \
    } while (0)
#define PWLQ_LAUNCH_QUANTIZE(PK, FK, UN)                                                          \
    do {                                                                                          \
        if (long_rows)   PWLQ_LAUNCH_QUANTIZE_AS(PK, FK, UN, true, false);                        \
        else if (premap) PWLQ_LAUNCH_QUANTIZE_AS(PK, FK, UN, false, true);                        \
        else             PWLQ_LAUNCH_QUANTIZE_AS(PK, FK, UN, false, false);                       \
    } while (0)
#define PWLQ_LAUNCH_QUANTIZE_UN(PK, FK) \
    do { if (lo) PWLQ_LAUNCH_QUANTIZE(PK, FK, true); else PWLQ_LAUNCH_QUANTIZE(PK, FK, false); } while (0)
    if (packed) { if (fake) PWLQ_LAUNCH_QUANTIZE_UN(true, true); else PWLQ_LAUNCH_QUANTIZE_UN(true, false); }
    else        { if (fake) PWLQ_LAUNCH_QUANTIZE_UN(false, true); else PWLQ_LAUNCH_QUANTIZE_UN(false, false); }
#undef PWLQ_LAUNCH_QUANTIZE_UN
#undef PWLQ_LAUNCH_QUANTIZE
#undef PWLQ_LAUNCH_QUANTIZE_AS
    return cudaGetLastError();
}

cudaError_t launch_dequantize(const uint8_t* codes, const uint8_t* mask,
                              const int64_t* row_offsets, int64_t C, int64_t n, int64_t total,
                              int bits, const float* m, const float* lo, const float* p, float* y,
                              int layout, cudaStream_t stream, int64_t shift, const float* xi,
                              const float* beta, const void* rowmap) {
    if (total == 0) return cudaSuccess;
    Rows rows{row_offsets, C, n, n > 0 ? 1.0 / (double)n : 0.0, row_offsets ? shift : 0};
    const RowArrays A{m, lo, p, xi, beta};
    const bool packed = (layout == 1 && bits <= 4);
    const int64_t nspans = (total + kQSpan - 1) / kQSpan;
#define PWLQ_LAUNCH_DEQUANTIZE_AS(PK, UN, LG, BCF, PR)                                             \
    do {                                                                                          \
        const int vc = aligned(codes, PK ? 4 : 8), vo = aligned(y, 16);                           \
        const size_t msmem = sizeof(MapStage<false, UN || BCF>) * kMapStages;                     \
        const SpanGrid g = span_grid((const void*)dequantize_map_kernel<PK, UN, LG, BCF, PR>,     \
                                     kMapThreads, msmem, nspans);                                 \
        dequantize_map_kernel<PK, UN, LG, BCF, PR><<<g.grid, kMapThreads, msmem, stream>>>(       \
            codes, mask, rows, total, bits, A, y, vc, vo, g.per_cta, premap);                     \
    } while (0)
#define PWLQ_LAUNCH_DEQUANTIZE(PK, UN, BCF)                                                       \
    do {                                                                                          \
        if (long_rows)   PWLQ_LAUNCH_DEQUANTIZE_AS(PK, UN, true, BCF, false);                     \
        else if (premap) PWLQ_LAUNCH_DEQUANTIZE_AS(PK, UN, false, BCF, true);                     \
        else             PWLQ_LAUNCH_DEQUANTIZE_AS(PK, UN, false, BCF, false);                    \
    } while (0)
    // Every layout goes through the producer / consumer kernel; for dense rows of at least a span
    // the map follows from the row length (LONG).  (A register-only kernel with a persistent grid
    // used to take dense rows of 16 spans or more; once the per-value work of the inverse had
    // shrunk, the producer / consumer kernel was faster there too: 0.89 against 0.73-0.82 of the
    // copy peak on one row of 25.7 M values.)
    const bool bc = xi != nullptr;
    const bool long_rows = row_offsets == nullptr && n >= kMapSpan;   // the map follows from n
    const unsigned char* premap = long_rows ? nullptr : static_cast<const unsigned char*>(rowmap);
    if (bc) {
        if (packed) PWLQ_LAUNCH_DEQUANTIZE(true, false, true); else PWLQ_LAUNCH_DEQUANTIZE(false, false, true);
    } else if (lo) {
        if (packed) PWLQ_LAUNCH_DEQUANTIZE(true, true, false); else PWLQ_LAUNCH_DEQUANTIZE(false, true, false);
    } else {
        if (packed) PWLQ_LAUNCH_DEQUANTIZE(true, false, false); else PWLQ_LAUNCH_DEQUANTIZE(false, false, false);
    }
#undef PWLQ_LAUNCH_DEQUANTIZE
#undef PWLQ_LAUNCH_DEQUANTIZE_AS
    return cudaGetLastError();
}

// Two or three breakpoints per row (p3 == nullptr: two).  Vector-aligned buffers go through the
// producer / consumer kernels; anything else, and layouts whose rows are so short that most spans
// would have no usable map, through the element-wise kernels.
static bool multi_by_maps(int64_t C, int64_t total, bool vec_ok) {
    return vec_ok && total >= 32 * C;
}
cudaError_t launch_quantize2(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                             int64_t total, int bits, const float* m, const float* p1,
                             const float* p2, const float* p3, int p_stride, uint8_t* codes,
                             uint8_t* region2, float* fake, int layout, cudaStream_t stream) {
    if (total == 0) return cudaSuccess;
    const bool vec_ok = aligned(x, 16) && aligned(codes, 16) && aligned(region2, 4) &&
                        (!fake || aligned(fake, 16));
    if (!multi_by_maps(C, total, vec_ok))
        return launch_quantize2_plain(x, row_offsets, C, n, total, bits, m, p1, p2, p3, p_stride,
                                      codes, region2, fake, layout, stream);
    const BreakPts bp{p1, p2, p3, p_stride};
    Rows rows{row_offsets, C, n, n > 0 ? 1.0 / (double)n : 0.0, 0};
    const bool packed = (layout == 1 && bits <= 4);
    const int64_t nspans = (total + kQSpan - 1) / kQSpan;
    const size_t msmem = sizeof(MultiStage<true>) * kMultiStages;
#define PWLQ_LAUNCH_QM(PK, FK, P3)                                                                \
    do {                                                                                          \
        const SpanGrid g = span_grid((const void*)quantize_multi_kernel<PK, FK, P3>, kMapThreads, \
                                     msmem, nspans);                                              \
        quantize_multi_kernel<PK, FK, P3><<<g.grid, kMapThreads, msmem, stream>>>(                \
            x, rows, total, bits, m, bp, codes, region2, fake, g.per_cta);                        \
    } while (0)
#define PWLQ_LAUNCH_QM3(PK, FK) \
    do { if (p3) PWLQ_LAUNCH_QM(PK, FK, true); else PWLQ_LAUNCH_QM(PK, FK, false); } while (0)
    if (packed) { if (fake) PWLQ_LAUNCH_QM3(true, true); else PWLQ_LAUNCH_QM3(true, false); }
    else        { if (fake) PWLQ_LAUNCH_QM3(false, true); else PWLQ_LAUNCH_QM3(false, false); }
#undef PWLQ_LAUNCH_QM3
#undef PWLQ_LAUNCH_QM
    return cudaGetLastError();
}

cudaError_t launch_dequantize2(const uint8_t* codes, const uint8_t* region2,
                               const int64_t* row_offsets, int64_t C, int64_t n, int64_t total,
                               int bits, const float* m, const float* p1, const float* p2,
                               const float* p3, int p_stride, float* y, int layout,
                               cudaStream_t stream) {
    if (total == 0) return cudaSuccess;
    const bool vec_ok = aligned(y, 16) && aligned(codes, 16) && aligned(region2, 4);
    if (!multi_by_maps(C, total, vec_ok))
        return launch_dequantize2_plain(codes, region2, row_offsets, C, n, total, bits, m, p1, p2,
                                        p3, p_stride, y, layout, stream);
    const BreakPts bp{p1, p2, p3, p_stride};
    Rows rows{row_offsets, C, n, n > 0 ? 1.0 / (double)n : 0.0, 0};
    const bool packed = (layout == 1 && bits <= 4);
    const int64_t nspans = (total + kQSpan - 1) / kQSpan;
    const size_t msmem = sizeof(MultiStage<false>) * kMultiStages;
#define PWLQ_LAUNCH_DM(PK, P3)                                                                    \
    do {                                                                                          \
        const SpanGrid g = span_grid((const void*)dequantize_multi_kernel<PK, P3>, kMapThreads,   \
                                     msmem, nspans);                                              \
        dequantize_multi_kernel<PK, P3><<<g.grid, kMapThreads, msmem, stream>>>(                  \
            codes, region2, rows, total, bits, m, bp, y, g.per_cta);                              \
    } while (0)
    if (packed) { if (p3) PWLQ_LAUNCH_DM(true, true); else PWLQ_LAUNCH_DM(true, false); }
    else        { if (p3) PWLQ_LAUNCH_DM(false, true); else PWLQ_LAUNCH_DM(false, false); }
#undef PWLQ_LAUNCH_DM
    return cudaGetLastError();
}

}  // namespace pwlq
