// Two and three breakpoints per row (Sec. 5.1 "Multiple Breakpoints"): the rows' breakpoints and
// the constants of a row's three or four regions, shared by the element-wise kernels and by the
// producer / consumer kernels (see pwlq_rowmap.cuh).
#pragma once

#include "pwlq_common.cuh"

namespace pwlq {

// Breakpoints of the rows: two arrays (p3 == nullptr: three regions) or three, read with a stride
// (1 for separate arrays, 3 for one [C, 3] array).
struct BreakPts {
    const float* p1;
    const float* p2;
    const float* p3;
    int stride;
};
// Constants of the regions of one row.  Without a third breakpoint the fourth region starts at m
// and is never entered (a <= m).
struct Params3 {
    float z[4], s[4], inv[4];
};
__device__ __forceinline__ Params3 make_params3(float m, float p1, float p2, float p3, float Lf) {
    Params3 P;
    P.z[0] = 0.0f; P.z[1] = p1; P.z[2] = p2; P.z[3] = p3;
    const float d[4] = {p1, __fsub_rn(p2, p1), __fsub_rn(p3, p2), __fsub_rn(m, p3)};
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        if (d[r] > 0.0f) { P.s[r] = __fdiv_rn(d[r], Lf); P.inv[r] = __fdiv_rn(Lf, d[r]); }
        else             { P.s[r] = 0.0f;                P.inv[r] = 0.0f; }
    }
    return P;
}

// Rows a span's stage holds constants for in the producer / consumer kernels; spans with more
// rows -- rows of fewer than 26 values on average -- are marked slow.  A row takes four 128-bit
// records, one per region r: (z_r, L / range_r, step_r, aux_r) with aux_0 = m and aux_1 = the
// sign mask 0x80000000, so that a consumer fetches what a value needs with one shared-memory read
// indexed by the value's region.  A row with m <= 0 (or a NaN) is stored as zeros: every value
// then comes out as level 0 of region 0, magnitude 0, no sign -- the zeros such a row delivers.
constexpr int kMultiSlots = 160;
__device__ __forceinline__ void store_row_consts_multi(float4* q, int slot, float m, float p1,
                                                       float p2, float p3, float Lf) {
    const Params3 P = make_params3(m, p1, p2, p3, Lf);
    const bool ok = m > 0.0f;
    const float4 zero = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    q[4 * slot] = ok ? make_float4(0.0f, P.inv[0], P.s[0], m) : zero;
    q[4 * slot + 1] = ok ? make_float4(p1, P.inv[1], P.s[1], __uint_as_float(0x80000000u)) : zero;
    q[4 * slot + 2] = ok ? make_float4(p2, P.inv[2], P.s[2], 0.0f) : zero;
    q[4 * slot + 3] = ok ? make_float4(p3, P.inv[3], P.s[3], 0.0f) : zero;
}

// Row state of a thread that walks consecutive values.
struct Row3 {
    int64_t row = -1, end = 0;
    int64_t first = 0, last = 0;       // the rows of the warp's values: bounds of the first lookup
    float m = 0.0f;
    Params3 P;
    // The rows that hold the first and the last of the `count` consecutive values a warp
    // handles, found by the warp together (a few dependent loads instead of a bisection over all
    // rows per thread).  Every lane of the warp calls this, before any lane leaves.
    __device__ __forceinline__ void bracket(const Rows& rows, int64_t warp_beg, int count,
                                            int64_t total) {
        if (warp_beg >= total) return;
        first = warp_row_of(rows, warp_beg);
        last = warp_row_of(rows, min(warp_beg + (int64_t)count, total) - 1);
    }
    // No bracket: the first lookup bisects over all rows.
    __device__ __forceinline__ void whole(const Rows& rows) { first = 0; last = rows.C - 1; }
    __device__ __forceinline__ void seek(const Rows& rows, const float* m_arr, const BreakPts& bp,
                                         float Lf, int64_t i) {
        if (row >= 0 && i < end) return;
        if (row < 0) {                                    // last row of [first, last] that begins at or before i
            int64_t lo = first, hi = last;
            while (hi > lo) {
                const int64_t mid = (lo + hi + 1) >> 1;
                if (rows.begin(mid) <= i) lo = mid; else hi = mid - 1;
            }
            row = lo;
        } else {
            row = row + 1;
        }
        while (rows.begin(row + 1) <= i) ++row;              // skips empty rows
        end = rows.begin(row + 1);
        m = __ldg(m_arr + row);
        P = make_params3(m, __ldg(bp.p1 + row * bp.stride), __ldg(bp.p2 + row * bp.stride),
                         bp.p3 ? __ldg(bp.p3 + row * bp.stride) : m, Lf);
    }
};

}  // namespace pwlq
