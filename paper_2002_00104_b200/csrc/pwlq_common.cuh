// Device helpers shared by the PWLQ kernels (sm_100a).
//
// The element arithmetic restates Eq. 1 and Eq. 3 of arXiv 2002.00104 in IEEE binary32 with one
// rounding per operation; the explicit __f*_rn intrinsics are never contracted into FMAs.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace pwlq {

constexpr int kWarp = 32;
constexpr int kStatusNonFinite = 1 << 5;   // device status bit: 1 << PWLQ_ERR_NONFINITE
constexpr int kStatusBadGrid = 1 << 1;     // device status bit: 1 << PWLQ_ERR_INVALID_ARG

struct PieceParams {
    float p;     // breakpoint (offset z of the tail pieces, Eq. 3)
    float s1;    // step of the center pieces, p / L        (Eq. 1: s = Delta / (N - 1))
    float inv1;  // L / p
    float s2;    // step of the tail pieces, (m - p) / L
    float inv2;  // L / (m - p)
};

// Per-(row, candidate) constants.  A piece with a non-positive range gets step 0.
__device__ __forceinline__ PieceParams make_params(float m, float p, float Lf) {
    PieceParams P;
    P.p = p;
    if (p > 0.0f) { P.s1 = __fdiv_rn(p, Lf); P.inv1 = __fdiv_rn(Lf, p); }
    else          { P.s1 = 0.0f;             P.inv1 = 0.0f; }
    const float d = __fsub_rn(m, p);
    if (d > 0.0f) { P.s2 = __fdiv_rn(d, Lf); P.inv2 = __fdiv_rn(Lf, d); }
    else          { P.s2 = 0.0f;             P.inv2 = 0.0f; }
    return P;
}

// Eq. 3 for one magnitude a = min(|x|, m): level q, region, reconstructed magnitude v.
__device__ __forceinline__ void quantize_mag(float a, const PieceParams& P, float Lf,
                                             int& q_out, int& tail_out, float& v_out) {
    const bool tail = a > P.p;                       // R2 = (p, m]
    const float z = tail ? P.p : 0.0f;
    const float inv = tail ? P.inv2 : P.inv1;
    const float s = tail ? P.s2 : P.s1;
    const float u = __fsub_rn(a, z);
    const float t = __fmul_rn(u, inv);
    // t + 1.5 * 2^23 rounds t (0 <= t < 2^22) to the nearest integer, ties to even, exactly like
    // rintf; the integer then sits in the low mantissa bits of r
    const float r = __fadd_rn(t, 12582912.0f);
    const float q = fminf(__fsub_rn(r, 12582912.0f), Lf);     // saturate
    float v = __fmul_rn(q, s);
    v = __fadd_rn(v, z);
    q_out = min(__float_as_int(r) - 0x4B400000, (int)Lf);
    tail_out = tail ? 1 : 0;
    v_out = v;
}

// ---------------------------------------------------------------------------- packed fp32x2
// Two binary32 lanes in one 64-bit register; fma.rn.f32x2 / add.rn.f32x2 take one issue slot for
// both lanes.  (The assembler contracts a packed multiply followed by a packed add into one packed
// FMA, so code that needs the product's own rounding uses the scalar __f*_rn intrinsics instead.)
typedef unsigned long long u64;
__device__ __forceinline__ u64 pack2(float lo, float hi) {
    u64 r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi)); return r;
}
__device__ __forceinline__ void unpack2(u64 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ u64 fma2(u64 a, u64 b, u64 c) {
    u64 d; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c)); return d;
}
__device__ __forceinline__ u64 add2(u64 a, u64 b) {
    u64 d; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d;
}

// Row lookup: dense rows have length n, ragged rows are given by ascending offsets.
struct Rows {
    const int64_t* offsets;  // [C + 1] or nullptr (dense)
    int64_t C;
    int64_t n;               // dense row length (unused when ragged)
    double inv_n;            // 1 / n (dense), so that i / n costs a multiply and a correction
    int64_t shift;           // ragged: subtracted from every offset (a slice of a longer list of
                             // rows whose data pointer was advanced by `shift` values); else 0

    // i / n for dense rows without a 64-bit integer division (exact for i < 2^52).
    __device__ __forceinline__ int64_t dense_row(int64_t i) const {
        int64_t r = (int64_t)((double)i * inv_n);
        if (r * n > i) --r;
        else if ((r + 1) * n <= i) ++r;
        return r;
    }

    __device__ __forceinline__ int64_t begin(int64_t c) const {
        return offsets ? offsets[c] - shift : c * n;
    }
    // Row that contains flat index i (0 <= i < total); empty rows are skipped.
    __device__ __forceinline__ int64_t row_of(int64_t i) const {
        if (!offsets) return dense_row(i);
        const int64_t key = i + shift;
        int64_t lo = 0, hi = C;                      // offsets[lo] <= key < offsets[hi]
        while (hi - lo > 1) {
            const int64_t mid = (lo + hi) >> 1;
            if (offsets[mid] <= key) lo = mid; else hi = mid;
        }
        return lo;
    }
};

__device__ __forceinline__ uint32_t abs_bits(float x) { return __float_as_uint(x) & 0x7fffffffu; }

// Row that contains flat index i, found by one warp together (every lane passes the same i and
// gets the same answer): a 32-ary search, three dependent rounds of loads for up to 32768 rows
// instead of fifteen.
__device__ __forceinline__ int64_t warp_row_of(const Rows& rows, int64_t i) {
    if (!rows.offsets) return rows.dense_row(i);
    const int lane = threadIdx.x & 31;
    int64_t lo = 0, hi = rows.C;                     // offsets[lo] <= i < offsets[hi]
    while (hi - lo > 1) {
        const int64_t step = (hi - lo + 31) / 32;
        const int64_t q = lo + (int64_t)(lane + 1) * step;
        const bool le = (q < hi) && (rows.offsets[q] - rows.shift <= i);   // true for a prefix of the lanes
        const int cnt = __popc(__ballot_sync(0xffffffffu, le));
        const int64_t new_lo = lo + (int64_t)cnt * step;
        hi = min(hi, new_lo + step);
        lo = new_lo;
    }
    return lo;
}

// A row at or shortly before the row that contains flat index i (at most three rows before it),
// found by a whole CTA together in rounds of blockDim.x-way search: two dependent rounds of loads
// for up to 65536 rows with 256 threads.  Every thread calls it with the same i (it contains CTA
// barriers) and gets the same answer.
__device__ __forceinline__ int64_t cta_row_near(const Rows& rows, int64_t i) {
    if (!rows.offsets) return rows.dense_row(i);
    const int64_t T = blockDim.x;
    int64_t lo = 0, hi = rows.C;                     // offsets[lo] <= i < offsets[hi]
    while (hi - lo > 4) {
        const int64_t step = (hi - lo + T - 1) / T;
        const int64_t q = lo + (int64_t)(threadIdx.x + 1) * step;
        const int le = (q < hi) && (rows.offsets[q] - rows.shift <= i);    // true for a prefix of the threads
        const int cnt = __syncthreads_count(le);
        const int64_t new_lo = lo + (int64_t)cnt * step;
        hi = min(hi, new_lo + step);
        lo = new_lo;
    }
    return lo;
}

// A window of CAP consecutive rows of the flat storage, staged in shared memory so that the
// per-thread row lookups of a CTA never touch global memory.  The CTA walks consecutive spans and
// keeps the window for as long as it reaches to the end of the next span: with long
// rows it is filled once per CTA.  When the next span will run past it, the window that starts at
// the row in which the current span ends is requested into registers before the current span is
// processed and written to shared memory after it, which keeps the global round trip off the
// critical path.  Values that lie beyond the last staged row (spans with more than CAP rows) use
// the global search.
constexpr int kTableThreads = 256;        // CTA size the fetch / commit pattern is written for

template <int CAP>
struct RowFetch {                          // what one thread holds of the next window
    static constexpr int kPerThread = CAP / kTableThreads;
    int64_t off[kPerThread + 1];           // rows tid + u * 256, and (thread 0) the entry CAP
    float m[kPerThread], p[kPerThread], lo[kPerThread];
};

template <bool PARAMS, int CAP>
struct SpanTable {
    static constexpr int kPerThread = CAP / kTableThreads;
    static_assert(CAP % kTableThreads == 0, "whole rounds of the CTA");
    int64_t off[CAP + 1];     // off[r] = first flat index of row row0 + r (INT64_MAX past the last row)
    float m[PARAMS ? CAP : 1];    // range width: abs-max, or hi - lo for one-sided ranges
    float lo[PARAMS ? CAP : 1];   // lower bound of a one-sided range (0 otherwise)
    PieceParams P[PARAMS ? CAP : 1];

    // True when every flat index below `end` lies in a staged row (or past the last row).
    __device__ __forceinline__ bool covers(int64_t end) const { return off[CAP] >= end; }

    // Local index of the staged row containing i, or -1 when i lies beyond the staged rows.
    // Neighbouring rows are mostly equally long (one layer), so a proportional guess is tried
    // first and corrected by a few neighbour steps; irregular windows fall back to bisection.
    __device__ __forceinline__ int find(int64_t i) const {
        const int64_t last = off[CAP];
        if (i >= last) return -1;
        int lo = 0, hi = CAP;                         // off[lo] <= i < off[hi]
        if (last != INT64_MAX) {
            const float scale = (float)CAP / (float)(last - off[0]);
            int g = min(max((int)((float)(i - off[0]) * scale), 0), CAP - 1);
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                if (off[g] > i) { hi = g; g = max(g - 1, 0); }
                else if (off[g + 1] <= i) { lo = g + 1; g = min(g + 1, CAP - 1); }
                else return g;
            }
        }
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (off[mid] <= i) lo = mid; else hi = mid;
        }
        return lo;
    }
    // Requests the window that starts at row r0 (no barrier; the values stay in registers).
    // lo_arr != nullptr: one-sided ranges, m_arr holds the upper bounds.  (All loads are
    // independent of each other, so that none of them is waited for here.)
    __device__ __forceinline__ void fetch(const Rows& rows, const float* __restrict__ m_arr,
                                          const float* __restrict__ p_arr,
                                          const float* __restrict__ lo_arr, int64_t r0,
                                          RowFetch<CAP>& f) const {
#pragma unroll
        for (int u = 0; u < kPerThread; ++u) {
            const int64_t row = r0 + (int)threadIdx.x + u * kTableThreads;
            f.off[u] = (row <= rows.C) ? rows.begin(row) : INT64_MAX;
            f.m[u] = f.p[u] = f.lo[u] = 0.0f;
            if (PARAMS && row < rows.C) {
                f.m[u] = __ldg(m_arr + row);
                f.p[u] = __ldg(p_arr + row);
                if (lo_arr) {
                    f.lo[u] = __ldg(lo_arr + row);
                    f.m[u] = __fsub_rn(f.m[u], f.lo[u]);
                }
            }
        }
        f.off[kPerThread] = (threadIdx.x == 0 && r0 + CAP <= rows.C) ? rows.begin(r0 + CAP)
                                                                     : INT64_MAX;
    }
    // Writes what fetch() requested, with the constants of the rows that start before `limit`
    // (the end of the CTA's share of the storage; later rows are staged with their offsets
    // alone); call between the barrier that retires the previous window and the barrier that
    // publishes this one.
    __device__ __forceinline__ void commit(const RowFetch<CAP>& f, int64_t limit, float Lf) {
#pragma unroll
        for (int u = 0; u < kPerThread; ++u) {
            const int r = (int)threadIdx.x + u * kTableThreads;
            off[r] = f.off[u];
            if (PARAMS && f.off[u] < limit) {
                m[r] = f.m[u];
                lo[r] = f.lo[u];
                P[r] = make_params(f.m[u], f.p[u], Lf);
            }
        }
        if (threadIdx.x == 0) off[CAP] = f.off[kPerThread];
    }
};

}  // namespace pwlq
