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

}  // namespace pwlq
