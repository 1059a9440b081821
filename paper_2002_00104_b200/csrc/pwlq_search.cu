// Breakpoint search: for every row and each of K candidate breakpoints p_k = m * ratio_k,
// SSE_k = sum_i (pw(x_i; b, m, p_k) - x_i)^2 with the quantizer of Eq. 3, then the first minimal
// k (grid form of Eq. 6).  Bound by the FP32 pipe: n * K evaluations per row, 4 bytes of HBM
// traffic per value.
//
// One CTA per (row, tile of at most kSearchTile values).
//   1. The candidates are taken in groups of cw consecutive ones (4 to 32, by tile length).  The
//      tile's magnitudes a = min(|x|, m) are bucketed by group (c(a) = number of groups whose
//      lowest breakpoint is below a) and counting-sorted into shared memory, with a deterministic
//      placement (per-warp histograms + in-warp ranks), so that for group g the values that are
//      center values under every one of its candidates are exactly the first entries (buckets
//      0 .. g) and the values that are tail values under every one of them the last (buckets
//      g + 2 and up).
//   2. Every lane owns one candidate; a warp works on one group at a time and walks the sorted
//      tile with 128-bit shared-memory broadcasts.  The first entries run a select-free center
//      loop, the last a select-free tail loop, both on packed fp32x2 FMAs (two values per
//      instruction); only the entries of bucket g + 1 need the per-lane region select.  No
//      per-candidate cross-lane reduction exists.
//   3. Sums run in binary32 over at most 256 terms per accumulator, are then carried in binary64,
//      always in the same order: results are bit-reproducible.
// Grids that are not ascending skip the sort and evaluate the region select for every (value,
// candidate); grids with more than kSortMaxK candidates take a kernel that only does that.
//
// Fused arithmetic (per value and candidate; r, q, e in binary32):
//     r = fma(u, inv, 1.5 * 2^23); q = r - 1.5 * 2^23      round-half-even of u * inv
//     e = fma(q, -s, u)                                      u = a - z;  e = -(v - a) up to rounding
// which differs from the operation-by-operation sequence of Eq. 1 only in rounding; the relative
// effect on a sum is about 3 L 2^-23 / sqrt(n).  Rows shorter than L^2 / 4, and all rows of fewer
// than 32 values (few terms average the effect out; and when most of a short row's values sit on
// levels -- the zeros of a ReLU output -- the sum is carried by two or three small errors whose
// own rounding then shows at 1e-5 and more) therefore use the unfused reconstruction
// v = (q * s) + z, e = v - a instead; measured against binary64 sums of the
// operation-by-operation values, the fused form then stays within 2e-6 relative.
#include <algorithm>
#include <cstdint>

#include "pwlq_common.cuh"
#include "pwlq_kernels.h"

namespace pwlq {

constexpr int kSThreads = 256;            // largest CTA; short rows run with fewer warps
constexpr int kSWarps = kSThreads / 32;
constexpr int kChunkVec = 256;     // float4 vectors per binary32 accumulation run
constexpr int kSortMaxK = 1024;    // largest K handled by the sorted kernel
constexpr float kMagic = 12582912.0f;   // 1.5 * 2^23: adding it rounds to the nearest integer

// Rows for which the fused error is accurate enough (see the file comment).
__host__ __device__ inline bool fused_ok(int64_t n_row, int64_t L) {
    return 4 * n_row >= L * L && n_row >= 32;
}

struct SearchArgs {
    const float* x;
    Rows rows;
    const float* m;     // per-row abs-max (signed scheme) or upper bound (one-sided ranges)
    const float* lo;    // per-row lower bound of a one-sided range; nullptr: signed scheme
    const float* ratios;
    int K;
    int levels;         // L: largest level of a piece, 2^(b-1) - 1 signed, 2^b - 1 one-sided
    int cap;            // tile capacity in values (multiple of 4, <= kSearchTile)
    int64_t n_min, n_max;   // this launch handles the rows with n_min <= length <= n_max
    int64_t grid_tiles;     // blockIdx.x = row * grid_tiles + tile
    int64_t tiles;          // tiles per row in the partial-sum layout
    double* partials;
    float* p_out;
    float* err_out;
    int32_t* idx_out;
    float* sse_all;
    double* sums64;     // not null: deliver the binary64 sums [C][K] only (no argmin, no p / err / idx)
    int* status;
};

// Unfused reconstruction error of a pair of values: e = ((q * s) + z) - a, one rounding per
// operation.  Done with scalar intrinsics: the assembler contracts a packed mul.rn.f32x2 followed
// by add.rn.f32x2 into one packed FMA (observed on the device: the pair loses the product's
// rounding, also when the product is written as fma(q, s, -0)), which the scalar forms never do.
template <bool WITH_Z>
__device__ __forceinline__ u64 exact_err2(u64 q, float s, float z, u64 a) {
    float q0, q1, a0, a1;
    unpack2(q, q0, q1);
    unpack2(a, a0, a1);
    float v0 = __fmul_rn(q0, s), v1 = __fmul_rn(q1, s);
    if (WITH_Z) { v0 = __fadd_rn(v0, z); v1 = __fadd_rn(v1, z); }
    return pack2(__fsub_rn(v0, a0), __fsub_rn(v1, a1));
}

// ------------------------------------------------------------------------------ reductions
// First minimal (value, index) over K sums held in shared memory; result valid in thread 0.
__device__ __forceinline__ void block_argmin(const double* sse, int K, double* red_val,
                                             int* red_idx, double& best_out, int& idx_out) {
    double best = 0.0;
    int bk = 0x7fffffff;
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        const double v = sse[k];
        if (bk == 0x7fffffff || v < best) { best = v; bk = k; }
    }
    const unsigned full = 0xffffffffu;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double ov = __shfl_xor_sync(full, best, o);
        const int ok = __shfl_xor_sync(full, bk, o);
        if (ok != 0x7fffffff && (bk == 0x7fffffff || ov < best || (ov == best && ok < bk))) {
            best = ov; bk = ok;
        }
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { red_val[warp] = best; red_idx[warp] = bk; }
    __syncthreads();
    if (threadIdx.x == 0) {
        best = red_val[0]; bk = red_idx[0];
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w) {
            const double ov = red_val[w];
            const int ok = red_idx[w];
            if (ok != 0x7fffffff && (bk == 0x7fffffff || ov < best || (ov == best && ok < bk))) {
                best = ov; bk = ok;
            }
        }
        best_out = best;
        idx_out = bk;
    }
}

__device__ __forceinline__ void write_degenerate_row(const SearchArgs& a, int64_t row) {
    // m == 0 (or not finite): nothing to search.
    if (a.sums64) {
        for (int k = threadIdx.x; k < a.K; k += blockDim.x) a.sums64[row * a.K + k] = 0.0;
        return;
    }
    if (threadIdx.x == 0) {
        a.idx_out[row] = 0;
        a.p_out[row] = 0.0f;
        if (a.err_out) a.err_out[row] = 0.0f;
    }
    if (a.sse_all)
        for (int k = threadIdx.x; k < a.K; k += blockDim.x) a.sse_all[row * a.K + k] = 0.0f;
}

__device__ __forceinline__ void write_row_result(const SearchArgs& a, int64_t row, float m,
                                                 double best, int idx) {
    a.idx_out[row] = idx;
    a.p_out[row] = __fmul_rn(m, a.ratios[idx]);
    if (a.err_out) a.err_out[row] = (float)best;
}

// Sums the element slices of every candidate, then either stores the tile's partial sums or
// finishes the row (all sums, argmin).  part: [E][K] binary64 in shared memory.
__device__ __forceinline__ void finish_tile(const SearchArgs& a, int64_t row, int64_t tile,
                                            float m, double* part, int E, double* red_val,
                                            int* red_idx) {
    const int K = a.K;
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        double tot = part[k];
        for (int e = 1; e < E; ++e) tot += part[e * K + k];
        if (a.tiles > 1) {
            a.partials[((size_t)row * a.tiles + tile) * K + k] = tot;
        } else if (a.sums64) {
            a.sums64[row * K + k] = tot;
        } else {
            if (E > 1) part[k] = tot;
            if (a.sse_all) a.sse_all[row * K + k] = (float)tot;
        }
    }
    if (a.tiles > 1 || a.sums64) return;
    if (E > 1) __syncthreads();                      // E == 1: part[] already holds the sums
    double best; int idx;
    block_argmin(part, K, red_val, red_idx, best, idx);
    if (threadIdx.x == 0) write_row_result(a, row, m, best, idx);
}

// ------------------------------------------------------------------- per-value evaluations
// Region select for one (value, candidate); EXACT_V chooses the unfused reconstruction.
template <bool EXACT_V>
__device__ __forceinline__ float sq_err_select(float a, const PieceParams& P, float acc) {
    const bool tail = a > P.p;
    const float z = tail ? P.p : 0.0f;
    const float inv = tail ? P.inv2 : P.inv1;
    const float s = tail ? P.s2 : P.s1;
    const float u = __fsub_rn(a, z);
    if (EXACT_V) {
        const float t = __fmul_rn(u, inv);
        const float q = __fsub_rn(__fadd_rn(t, kMagic), kMagic);   // rint(t), 0 <= t < 2^22
        float v = __fmul_rn(q, s);
        v = __fadd_rn(v, z);
        const float e = __fsub_rn(v, a);
        return __fmaf_rn(e, e, acc);
    } else {
        const float q = __fsub_rn(__fmaf_rn(u, inv, kMagic), kMagic);
        const float e = __fmaf_rn(q, -s, u);
        return __fmaf_rn(e, e, acc);
    }
}

struct Acc {
    u64 v0, v1;            // packed accumulators of the select-free loops
    float s0, s1, s2, s3;  // scalar accumulators of the select loop
    double d;              // binary64 carry
    __device__ __forceinline__ void clear() { v0 = v1 = 0ull; s0 = s1 = s2 = s3 = 0.0f; }
    __device__ __forceinline__ void flush() {
        float a, b, c, e;
        unpack2(v0, a, b);
        unpack2(v1, c, e);
        d += ((double)a + (double)b) + ((double)c + (double)e);
        d += ((double)s0 + (double)s1) + ((double)s2 + (double)s3);
        clear();
    }
};

// Candidate constants as fp32x2 pairs for the packed loops.
struct Pairs {
    u64 inv1, ns1, inv2, ns2, np, magic, nmagic;
};

// u * inv + 1.5 * 2^23 for a pair of values.  EXACT_V: product and sum rounded one after the
// other, as Eq. 3 is evaluated operation by operation -- where the rounded product is an exact
// tie (x.5) and the unrounded one is not, the fused form rounds to the other level, and in a row
// of few values at many levels that one level shows in the sum (one-sided 8-bit rows of about a
// hundred values: 1.3e-5 relative).
template <bool EXACT_V>
__device__ __forceinline__ u64 level_pattern2(u64 u, u64 inv_pair, float inv, const Pairs& c) {
    if (!EXACT_V) return fma2(u, inv_pair, c.magic);
    float u0, u1;
    unpack2(u, u0, u1);
    return add2(pack2(__fmul_rn(u0, inv), __fmul_rn(u1, inv)), c.magic);   // scalar products
}

template <bool EXACT_V>
__device__ __forceinline__ void center_vec(const ulonglong2 v, const Pairs& c,
                                           const PieceParams& P, Acc& A) {
    const u64 r0 = level_pattern2<EXACT_V>(v.x, c.inv1, P.inv1, c);
    const u64 r1 = level_pattern2<EXACT_V>(v.y, c.inv1, P.inv1, c);
    const u64 q0 = add2(r0, c.nmagic), q1 = add2(r1, c.nmagic);
    u64 e0, e1;
    if (EXACT_V) {
        e0 = exact_err2<false>(q0, P.s1, 0.0f, v.x);
        e1 = exact_err2<false>(q1, P.s1, 0.0f, v.y);
    } else {
        e0 = fma2(q0, c.ns1, v.x);
        e1 = fma2(q1, c.ns1, v.y);
    }
    A.v0 = fma2(e0, e0, A.v0);
    A.v1 = fma2(e1, e1, A.v1);
}

template <bool EXACT_V>
__device__ __forceinline__ void tail_vec(const ulonglong2 v, const Pairs& c,
                                         const PieceParams& P, Acc& A) {
    const u64 u0 = add2(v.x, c.np), u1 = add2(v.y, c.np);
    const u64 r0 = level_pattern2<EXACT_V>(u0, c.inv2, P.inv2, c);
    const u64 r1 = level_pattern2<EXACT_V>(u1, c.inv2, P.inv2, c);
    const u64 q0 = add2(r0, c.nmagic), q1 = add2(r1, c.nmagic);
    u64 e0, e1;
    if (EXACT_V) {
        e0 = exact_err2<true>(q0, P.s2, P.p, v.x);
        e1 = exact_err2<true>(q1, P.s2, P.p, v.y);
    } else {
        e0 = fma2(q0, c.ns2, u0);
        e1 = fma2(q1, c.ns2, u1);
    }
    A.v0 = fma2(e0, e0, A.v0);
    A.v1 = fma2(e1, e1, A.v1);
}

template <bool EXACT_V>
__device__ __forceinline__ void select_vec(const float4 v, const PieceParams& P, Acc& A) {
    A.s0 = sq_err_select<EXACT_V>(v.x, P, A.s0);
    A.s1 = sq_err_select<EXACT_V>(v.y, P, A.s1);
    A.s2 = sq_err_select<EXACT_V>(v.z, P, A.s2);
    A.s3 = sq_err_select<EXACT_V>(v.w, P, A.s3);
}

// Walks float4 vectors first, first + step, ... (< hi) of the tile with one of the three bodies.
// A binary32 accumulation run is closed after kChunkVec vectors; the last, shorter run stays open
// for the caller to close (an accumulator therefore never sums more than 3 * kChunkVec terms).
// MODE 0: center, 1: tail, 2: select.
template <int MODE, bool EXACT_V>
__device__ __forceinline__ void walk(const float* tile_s, int first, int hi, int step,
                                     const Pairs& c, const PieceParams& P, Acc& A) {
    const ulonglong2* t2 = reinterpret_cast<const ulonglong2*>(tile_s);
    const float4* t4 = reinterpret_cast<const float4*>(tile_s);
    for (int base = first; base < hi; base += kChunkVec * step) {
        const int stop = min(base + kChunkVec * step, hi);
        if (MODE == 2) {
#pragma unroll 2
            for (int j = base; j < stop; j += step) select_vec<EXACT_V>(t4[j], P, A);
        } else {
#pragma unroll 4
            for (int j = base; j < stop; j += step) {
                if (MODE == 0) center_vec<EXACT_V>(t2[j], c, P, A);
                else tail_vec<EXACT_V>(t2[j], c, P, A);
            }
        }
        if (stop < hi) A.flush();
    }
}

__host__ __device__ inline int slices_for(int K, int warps) {
    const int G = (K + 31) / 32;
    return (G >= warps) ? 1 : (warps / G);
}

// Region select for every (value, candidate) of an unsorted tile (zero-padded to whole vectors).
__device__ __forceinline__ void eval_unsorted(const SearchArgs& a, const float* tile_s,
                                              double* part, int cnt4, float m, int E) {
    const int K = a.K;
    const int G = (K + 31) / 32;
    const float Lf = (float)a.levels;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const Pairs unused = {};
    for (int item = warp; item < G * E; item += (int)(blockDim.x >> 5)) {
        const int g = item % G, e = item / G;
        const int k = g * 32 + lane;
        const int lo = (int)((int64_t)cnt4 * e / E), hi = (int)((int64_t)cnt4 * (e + 1) / E);
        if (k < K) {
            const PieceParams P = make_params(m, __fmul_rn(m, a.ratios[k]), Lf);
            Acc A;
            A.clear();
            A.d = 0.0;
            walk<2, true>(tile_s, lo, hi, 1, unused, P, A);
            A.flush();
            part[e * K + k] = A.d;
        }
    }
}

// Range width of a row (abs-max, or hi - lo) and its lower bound (0 for the signed scheme).
__device__ __forceinline__ float row_range(const SearchArgs& a, int64_t row, float& lo) {
    float m = a.m[row];
    lo = 0.0f;
    if (a.lo) { lo = a.lo[row]; m = __fsub_rn(m, lo); }
    return m;
}
// Magnitude the quantizer sees: min(|x|, m), or min(max(x - lo, 0), m) for a one-sided range.
__device__ __forceinline__ float mag_of(const SearchArgs& a, float x, float m, float lo) {
    return a.lo ? fminf(fmaxf(__fsub_rn(x, lo), 0.0f), m) : fminf(fabsf(x), m);
}

__device__ __forceinline__ bool row_setup(const SearchArgs& a, int64_t& row, int64_t& tile,
                                          int64_t& t_beg, int& cnt, float& m, float& lo) {
    row = blockIdx.x / a.grid_tiles;
    tile = blockIdx.x - row * a.grid_tiles;
    const int64_t beg = a.rows.begin(row), end = a.rows.begin(row + 1);
    if (end - beg < a.n_min || end - beg > a.n_max) return false;   // another launch's row
    t_beg = beg + tile * (int64_t)a.cap;
    if (t_beg >= end && tile > 0) return false;      // this row has fewer tiles than the longest
    cnt = (int)min((int64_t)a.cap, end - t_beg);
    m = row_range(a, row, lo);
    const bool finite = (__float_as_uint(m) & 0x7fffffffu) < 0x7f800000u &&
                        (__float_as_uint(lo) & 0x7fffffffu) < 0x7f800000u;
    if (!finite || !(m > 0.0f) || cnt <= 0) {
        if (!finite && threadIdx.x == 0 && tile == 0) atomicOr(a.status, kStatusNonFinite);
        if (a.tiles == 1) write_degenerate_row(a, row);
        return false;                                // tiles > 1: the combine kernel handles it
    }
    return true;
}

// ------------------------------------------------------------------------- sorted kernel
// A warp works on kCW consecutive candidates at a time; its 32 / kCW lane groups ("phases") take
// every (32 / kCW)-th vector of the tile.  Fewer candidates per warp means fewer entries between
// the lowest and the highest boundary, i.e. less work in the select loop.
// Short tiles use wider groups: per work item there is a fixed cost (fetching the item, loading
// the constants, closing the sums) that a handful of vectors per lane cannot amortise.
constexpr int kCwLongTile = 8, kCwMidTile = 16, kCwShortTile = 32;
constexpr int kLongTileMin = 3072, kMidTileMin = 768;     // values per tile
// Few candidates on a long tile: groups of four keep as many (group, slice) items as there are
// warps without slicing the tile, and halve the entries between a group's boundaries.
constexpr int kCwFewCand = 4;
#ifndef PWLQ_FEW_CAND_K
#define PWLQ_FEW_CAND_K 64
#endif
__host__ __device__ inline int group_width(int cnt, int K) {
    if (cnt >= kLongTileMin && K <= PWLQ_FEW_CAND_K) return kCwFewCand;
    return cnt >= kLongTileMin ? kCwLongTile : (cnt >= kMidTileMin ? kCwMidTile : kCwShortTile);
}

// Element slices per candidate group: enough (group, slice) work items to keep the warps busy.
// Sized for the narrowest group so that one shared-memory layout serves every width.
// (two work items per warp: every item recomputes its candidates' constants, so more, smaller
// items cost more than the better balance gains -- measured at K = 64)
constexpr int kItemsPerWarp = 2;
__host__ __device__ inline int slices_sorted(int K, int cw, int warps) {
    const int G = (K + cw - 1) / cw;
    const int E = (kItemsPerWarp * warps + G - 1) / G;
    return E < 1 ? 1 : (E > 8 ? 8 : E);
}
__host__ __device__ inline int max_slices_sorted(int K, int warps) {
    return slices_sorted(K, kCwShortTile, warps);      // fewest groups: most slices
}

// Shared memory: sorted tile | bucket ids | candidate breakpoints | candidate constants | bucket
// starts | per-warp histograms | per-slice sums.
struct SortedSmem {
    float* tile;        // [cap + 4]
    uint32_t* jr;       // [cap]  bucket | rank << 11
    float* ps;          // [K]
    float* qs;          // [G]  qs[g] = ps[g * cw]: the lowest breakpoint of group g
    int* start;         // [K + 2]
    uint16_t* hist;     // [kSWarps][K + 2]
    double* part;       // [E][K]
};
__host__ __device__ inline size_t sorted_smem_layout(int cap, int K, int warps, size_t off[7]) {
    const int E = max_slices_sorted(K, warps);
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t r = o; o = (o + bytes + 15) & ~(size_t)15; return r; };
    off[0] = take(sizeof(float) * (size_t)(cap + 4));
    off[1] = take(sizeof(uint32_t) * (size_t)cap);
    off[2] = take(sizeof(float) * (size_t)K);
    off[3] = take(sizeof(float) * (size_t)((K + 3) / 4));       // group boundaries (groups of >= 4)
    off[4] = take(sizeof(int) * (size_t)(K + 2));
    off[5] = take(sizeof(uint16_t) * (size_t)warps * (size_t)(K + 2));
    off[6] = take(sizeof(double) * (size_t)E * (size_t)K);
    return o;
}

// j(a) = number of candidates with p_k < a, for ascending ps[0..K).  A linear-grid guess is
// verified against its two neighbours; a guess that is off (rounding at a boundary, a grid that
// is not linear) is replaced by a binary search, kept out of line so that the common path stays
// a dozen instructions without branches.  Exact for every ascending grid.
__device__ __noinline__ int bucket_search(const float* ps, int K, float a) {
    int lo = 0, hi = K;                               // the answer lies in [lo, hi]
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (ps[mid] < a) lo = mid + 1; else hi = mid;
    }
    return lo;
}
__device__ __forceinline__ int bucket_of(const float* ps, int K, float a, float p_first,
                                         float hint_scale) {
    const int j = min((int)ceilf(fmaxf((a - p_first) * hint_scale, 0.0f)), K);
    const float below = ps[max(j - 1, 0)], at = ps[min(j, K - 1)];
    const bool ok = (j == 0 || below < a) && (j == K || !(at < a));
    return ok ? j : bucket_search(ps, K, a);
}

template <int kCW, bool EXACT_V>
__device__ __forceinline__ void eval_sorted(const SearchArgs& a, const SortedSmem& S, float m,
                                            int n4, int pad, int E, int* next_item) {
    constexpr int kPhases = 32 / kCW;
    const int K = a.K;
    const float Lf = (float)a.levels;
    const int G = (K + kCW - 1) / kCW;
    const int lane = threadIdx.x & 31;
    const int ci = lane % kCW, ph = lane / kCW;
    const unsigned full = 0xffffffffu;
    for (;;) {
        // work items are handed out in order (low candidates first: for bell-shaped data their
        // boundaries lie in the dense part of the tile, so they carry the longest select loops)
        int item = 0;
        if (lane == 0) item = atomicAdd(next_item, 1);
        item = __shfl_sync(full, item, 0);
        if (item >= G * E) break;
        const int g = item / E, e = item - g * E;
        const int k0 = g * kCW;
        const int k = min(k0 + ci, K - 1);
        const int lo = (int)((int64_t)n4 * e / E), hi = (int)((int64_t)n4 * (e + 1) / E);
        // the tile is sorted by group bucket c(a) = number of groups whose lowest breakpoint is
        // below a: buckets 0 .. g hold the values a <= p_k0, center values of every candidate of
        // group g; buckets g + 2 and up hold values a > p_(k0 + kCW), tail values of all of them
        const int c_hi = min(hi, (pad + S.start[g + 1]) >> 2);      // vectors below every boundary
        const int t_lo = max(lo, (pad + S.start[g + 2] + 3) >> 2);  // vectors above every boundary
        // the candidate's constants (four divisions) are computed here, by the lanes that use
        // them, while other warps keep the FP32 pipe busy -- not in a serial phase of the CTA
        const PieceParams P = make_params(m, S.ps[k], Lf);
        Pairs c;
        c.inv1 = pack2(P.inv1, P.inv1); c.ns1 = pack2(-P.s1, -P.s1);
        c.inv2 = pack2(P.inv2, P.inv2); c.ns2 = pack2(-P.s2, -P.s2);
        c.np = pack2(-P.p, -P.p);
        c.magic = pack2(kMagic, kMagic); c.nmagic = pack2(-kMagic, -kMagic);
        Acc A;
        A.clear();
        A.d = 0.0;
        walk<0, EXACT_V>(S.tile, lo + ph, c_hi, kPhases, c, P, A);
        walk<2, EXACT_V>(S.tile, max(lo, c_hi) + ph, min(hi, t_lo), kPhases, c, P, A);
        walk<1, EXACT_V>(S.tile, t_lo + ph, hi, kPhases, c, P, A);
        A.flush();
        double d = A.d;                               // phases combined in a fixed order
#pragma unroll
        for (int o = kCW; o < 32; o <<= 1) d += __shfl_xor_sync(full, d, o);
        if (ph == 0 && k0 + ci < K) S.part[e * K + k0 + ci] = d;
    }
}

__global__ void __launch_bounds__(kSThreads)
search_sorted_kernel(SearchArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ double red_val[kSWarps];
    __shared__ int red_idx[kSWarps];
    __shared__ int warp_sums[kSWarps];
    __shared__ int next_item;
    // The launches of the other row-length classes touch other rows only: let the next one start
    // filling the SMs as soon as every CTA of this grid is resident or done.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    int64_t row, tile, t_beg;
    int cnt;
    float m, lo;
    if (!row_setup(a, row, tile, t_beg, cnt, m, lo)) return;

    const int K = a.K;
    const int nwarps = (int)(blockDim.x >> 5), nthreads = (int)blockDim.x;
    const int cw = group_width(cnt, K);
    const int E = min(slices_sorted(K, cw, nwarps), max(1, cnt / 512));   // a slice is worth >= 128 vectors
    size_t off[7];
    sorted_smem_layout(a.cap, K, nwarps, off);
    SortedSmem S;
    S.tile = reinterpret_cast<float*>(smem_raw + off[0]);
    S.jr = reinterpret_cast<uint32_t*>(smem_raw + off[1]);
    S.ps = reinterpret_cast<float*>(smem_raw + off[2]);
    S.qs = reinterpret_cast<float*>(smem_raw + off[3]);
    S.start = reinterpret_cast<int*>(smem_raw + off[4]);
    S.hist = reinterpret_cast<uint16_t*>(smem_raw + off[5]);
    S.part = reinterpret_cast<double*>(smem_raw + off[6]);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned full = 0xffffffffu;
    // The sort's keys are group buckets (one per group of cw candidates and one above the last
    // group), not candidate intervals: all the evaluation needs, a shorter table to look a value
    // up in and fewer distinct keys for the in-warp ranking.  (The entries that need the per-lane
    // region select grow by one candidate interval per group; measured, the cheaper sort wins on
    // rows of up to a few thousand values -- ResNet-50 shapes +1.3 %, MobileNetV2 +2 %, K = 64
    // +2.3 % -- and loses 2 % on the 25.7 M-value activation at K = 1024.)
    const int G = (K + cw - 1) / cw;
    const int HS = G + 2;                           // histogram stride; bucket G + 1 = "no value"

    // candidate breakpoints p_k = m * ratio_k; they ascend exactly when the ratios do (m > 0 and
    // the multiplication rounds monotonically)
    int unordered = 0;
    for (int k = threadIdx.x; k < K; k += nthreads) {
        const float rk = __ldg(a.ratios + k);
        if (k > 0) unordered |= (rk < __ldg(a.ratios + k - 1));
        S.ps[k] = __fmul_rn(m, rk);
    }
    for (int g = threadIdx.x; g < G; g += nthreads) S.qs[g] = __fmul_rn(m, __ldg(a.ratios + g * cw));
    for (int i = threadIdx.x; i < nwarps * HS; i += nthreads) S.hist[i] = 0;
    if (threadIdx.x == 0) next_item = 0;
    if (__syncthreads_or(unordered)) {
        // the grid is not ascending: no sorted structure to exploit
        const int cnt4 = (cnt + 3) >> 2;
        for (int i = threadIdx.x; i < cnt4 * 4; i += nthreads)
            S.tile[i] = (i < cnt) ? mag_of(a, a.x[t_beg + i], m, lo) : 0.0f;
        __syncthreads();
        const int Eu = slices_for(K, nwarps);         // never more slices than the sorted layout
        eval_unsorted(a, S.tile, S.part, cnt4, m, Eu);
        __syncthreads();
        finish_tile(a, row, tile, m, S.part, Eu, red_val, red_idx);
        return;
    }

    // ---- pass 1: group bucket j and rank of every value (each warp owns a contiguous segment, which
    // it walks four groups of 32 at a time so that the four lookups overlap); jr = j | rank << 11,
    // rank = number of earlier values of this warp's segment in the same bucket
    const int seg = (((cnt + nwarps - 1) / nwarps) + 31) & ~31;
    const int w_beg = min(warp * seg, cnt), w_end = min(w_beg + seg, cnt);
    uint16_t* myhist = S.hist + warp * HS;
    const float p_first = S.qs[0];
    const float span = S.qs[G - 1] - p_first;
    const float hint_scale = span > 0.0f ? (float)(G - 1) / span : 0.0f;
    float nxt[4];                                   // values of the next iteration, already in flight
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int i = w_beg + u * 32 + lane;
        nxt[u] = (i < w_end) ? __ldg(a.x + t_beg + i) : 0.0f;
    }
    for (int base = w_beg; base < w_end; base += 128) {
        float av[4];
        int jv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            av[u] = mag_of(a, nxt[u], m, lo);
            const int i = base + 128 + u * 32 + lane;
            nxt[u] = (i < w_end) ? __ldg(a.x + t_beg + i) : 0.0f;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            jv[u] = (base + u * 32 + lane < w_end) ? bucket_of(S.qs, G, av[u], p_first, hint_scale)
                                                   : G + 1;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = base + u * 32 + lane;
            const int j = jv[u];
            const unsigned peers = __match_any_sync(full, j);
            int before = 0;
            if (j <= G) before = myhist[j];
            __syncwarp();
            if (j <= G) {
                if (lane == __ffs(peers) - 1) myhist[j] = (uint16_t)(before + __popc(peers));
                S.jr[i] = (uint32_t)j | ((uint32_t)(before + __popc(peers & ((1u << lane) - 1u))) << 11);
            }
            __syncwarp();
        }
    }
    __syncthreads();

    // ---- exclusive scan over buckets (and over warps inside a bucket)
    {
        const int per = (G + 1 + nthreads - 1) / nthreads;
        const int j0 = min(threadIdx.x * per, G + 1), j1 = min(j0 + per, G + 1);
        int local = 0;
        for (int j = j0; j < j1; ++j)
            for (int w = 0; w < nwarps; ++w) local += S.hist[w * HS + j];
        int incl = local;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(full, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) warp_sums[warp] = incl;
        __syncthreads();
        int run = incl - local;
        for (int w = 0; w < warp; ++w) run += warp_sums[w];
        for (int j = j0; j < j1; ++j) {
            S.start[j] = run;
            for (int w = 0; w < nwarps; ++w) {
                const int c = S.hist[w * HS + j];
                S.hist[w * HS + j] = (uint16_t)run;
                run += c;
            }
        }
        if (threadIdx.x == 0) S.start[G + 1] = cnt;
    }
    const int pad = (4 - (cnt & 3)) & 3;            // zeros in front: error 0 under every candidate
    if (threadIdx.x < pad) S.tile[threadIdx.x] = 0.0f;
    __syncthreads();

    // ---- pass 2: stable placement (bucket, then warp segment, then order inside the segment)
    for (int base = w_beg; base < w_end; base += 128) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = base + u * 32 + lane;
            if (i < w_end) {
                const uint32_t jr = S.jr[i];
                S.tile[pad + myhist[jr & 0x7ffu] + (jr >> 11)] = mag_of(a, a.x[t_beg + i], m, lo);
            }
        }
    }
    __syncthreads();

    // ---- evaluation
    const int n4 = (pad + cnt) >> 2;
    const int64_t n_row = a.rows.begin(row + 1) - a.rows.begin(row);
    const int64_t L = a.levels;
    const bool fused = fused_ok(n_row, L);
    if (cw == kCwFewCand) {
        if (fused) eval_sorted<kCwFewCand, false>(a, S, m, n4, pad, E, &next_item);
        else       eval_sorted<kCwFewCand, true>(a, S, m, n4, pad, E, &next_item);
    } else if (cw == kCwLongTile) {
        if (fused) eval_sorted<kCwLongTile, false>(a, S, m, n4, pad, E, &next_item);
        else       eval_sorted<kCwLongTile, true>(a, S, m, n4, pad, E, &next_item);
    } else if (cw == kCwMidTile) {
        if (fused) eval_sorted<kCwMidTile, false>(a, S, m, n4, pad, E, &next_item);
        else       eval_sorted<kCwMidTile, true>(a, S, m, n4, pad, E, &next_item);
    } else {
        if (fused) eval_sorted<kCwShortTile, false>(a, S, m, n4, pad, E, &next_item);
        else       eval_sorted<kCwShortTile, true>(a, S, m, n4, pad, E, &next_item);
    }
    __syncthreads();
    finish_tile(a, row, tile, m, S.part, E, red_val, red_idx);
}

// --------------------------------------------------------------------------- tiny rows
// Rows of at most kTinyMax values (depthwise 3x3 channels have 9): one warp per row, eight rows
// per CTA.  The row's magnitudes sit in two registers per lane and are broadcast with shuffles;
// a lane owns kTinyBatch candidates at a time (candidate k0 + 32 j + lane, so that a warp's
// stores of the sums are contiguous) and evaluates the region select for every value -- with a
// handful of values there is nothing to sort, and no cross-lane reduction exists.  Sums: binary32
// over the row's at most kTinyMax terms, compared in binary64; first minimum.
constexpr int kTinyMax = 64;
constexpr int kTinyBatch = 4;
constexpr int kTinyWarps = 8;

template <bool EXACT_V>
__device__ __forceinline__ void tiny_row(const SearchArgs& a, int64_t row, int cnt, float m,
                                         float a0, float a1) {
    const unsigned full = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const int K = a.K;
    const float Lf = (float)a.levels;
    double best = 0.0;
    int bk = 0x7fffffff;
    for (int k0 = 0; k0 < K; k0 += 32 * kTinyBatch) {
        PieceParams P[kTinyBatch];
        float acc[kTinyBatch];
#pragma unroll
        for (int j = 0; j < kTinyBatch; ++j) {
            const int k = min(k0 + 32 * j + lane, K - 1);
            P[j] = make_params(m, __fmul_rn(m, __ldg(a.ratios + k)), Lf);
            acc[j] = 0.0f;
        }
        for (int i = 0; i < cnt; ++i) {
            const float v = __shfl_sync(full, i < 32 ? a0 : a1, i & 31);
#pragma unroll
            for (int j = 0; j < kTinyBatch; ++j) acc[j] = sq_err_select<EXACT_V>(v, P[j], acc[j]);
        }
#pragma unroll
        for (int j = 0; j < kTinyBatch; ++j) {
            const int k = k0 + 32 * j + lane;
            if (k < K) {
                const double tot = (double)acc[j];
                if (a.tiles > 1) {
                    a.partials[((size_t)row * a.tiles) * K + k] = tot;    // tile 0 of the row
                } else if (a.sums64) {
                    a.sums64[row * K + k] = tot;
                } else {
                    if (a.sse_all) a.sse_all[row * K + k] = (float)tot;
                    if (bk == 0x7fffffff || tot < best) { best = tot; bk = k; }   // k ascends
                }
            }
        }
    }
    if (a.tiles > 1 || a.sums64) return;              // the combine kernels finish the row
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double ov = __shfl_xor_sync(full, best, o);
        const int ok = __shfl_xor_sync(full, bk, o);
        if (ok != 0x7fffffff && (bk == 0x7fffffff || ov < best || (ov == best && ok < bk))) {
            best = ov; bk = ok;
        }
    }
    if (lane == 0) write_row_result(a, row, m, best, bk);
}

__global__ void __launch_bounds__(kTinyWarps * 32)
search_tiny_kernel(SearchArgs a) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row = (int64_t)blockIdx.x * kTinyWarps + warp;
    if (row >= a.rows.C) return;
    const int64_t beg = a.rows.begin(row), end = a.rows.begin(row + 1);
    if (end - beg > a.n_max || end - beg < a.n_min) return;          // another launch's row
    const int cnt = (int)(end - beg);
    float lo;
    const float m = row_range(a, row, lo);
    const bool finite = (__float_as_uint(m) & 0x7fffffffu) < 0x7f800000u &&
                        (__float_as_uint(lo) & 0x7fffffffu) < 0x7f800000u;
    if (!finite || !(m > 0.0f) || cnt <= 0) {
        // m == 0 (or not finite): nothing to search; with several tiles per row the combine
        // kernels write the row
        if (!finite && lane == 0) atomicOr(a.status, kStatusNonFinite);
        if (a.tiles == 1 && a.sums64) {
            for (int k = lane; k < a.K; k += 32) a.sums64[row * a.K + k] = 0.0;
        } else if (a.tiles == 1) {
            if (lane == 0) {
                a.idx_out[row] = 0;
                a.p_out[row] = 0.0f;
                if (a.err_out) a.err_out[row] = 0.0f;
            }
            if (a.sse_all)
                for (int k = lane; k < a.K; k += 32) a.sse_all[row * a.K + k] = 0.0f;
        }
        return;
    }
    const float a0 = lane < cnt ? mag_of(a, __ldg(a.x + beg + lane), m, lo) : 0.0f;
    const float a1 = lane + 32 < cnt ? mag_of(a, __ldg(a.x + beg + lane + 32), m, lo) : 0.0f;
    const int64_t L = a.levels;
    if (fused_ok(cnt, L)) tiny_row<false>(a, row, cnt, m, a0, a1);
    else tiny_row<true>(a, row, cnt, m, a0, a1);
}

// ------------------------------------------------------------------------ generic kernel
// More than kSortMaxK candidates: region select for every (value, candidate).
__global__ void __launch_bounds__(kSThreads)
search_generic_kernel(SearchArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ double red_val[kSWarps];
    __shared__ int red_idx[kSWarps];
    int64_t row, tile, t_beg;
    int cnt;
    float m, lo;
    if (!row_setup(a, row, tile, t_beg, cnt, m, lo)) return;
    const int E = slices_for(a.K, kSWarps);
    const int cnt4 = (cnt + 3) >> 2;
    float* tile_s = reinterpret_cast<float*>(smem_raw);
    double* part = reinterpret_cast<double*>(smem_raw + (((size_t)a.cap * 4 + 15) & ~(size_t)15));
    for (int i = threadIdx.x; i < cnt4 * 4; i += kSThreads)
        tile_s[i] = (i < cnt) ? mag_of(a, a.x[t_beg + i], m, lo) : 0.0f;   // zero padding: error 0
    __syncthreads();
    eval_unsorted(a, tile_s, part, cnt4, m, E);
    __syncthreads();
    finish_tile(a, row, tile, m, part, E, red_val, red_idx);
}

// Long rows, step 1: sums the tiles' partial sums of 32 candidates of one row.  The tiles are cut
// into kCombineWarps consecutive segments, one per warp, each summed in ascending tile order; the
// segment sums are then added in ascending order.  Fixed order, hence reproducible.
constexpr int kCombineWarps = 32;
__global__ void __launch_bounds__(kCombineWarps * 32)
search_combine_kernel(SearchArgs a, double* __restrict__ sums) {
    __shared__ double seg[kCombineWarps][32];
    const int chunks = (a.K + 31) / 32;
    const int64_t row = blockIdx.x / chunks;
    const int chunk = (int)(blockIdx.x - row * chunks);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int k = chunk * 32 + lane;
    const int64_t n_row = a.rows.begin(row + 1) - a.rows.begin(row);
    float lo;
    const float m = row_range(a, row, lo);
    const bool finite = (__float_as_uint(m) & 0x7fffffffu) < 0x7f800000u &&
                        (__float_as_uint(lo) & 0x7fffffffu) < 0x7f800000u;
    const bool degenerate = !finite || !(m > 0.0f) || n_row <= 0;
    const int64_t nt = degenerate ? 0 : (n_row + a.cap - 1) / a.cap;
    const int64_t t0 = nt * warp / kCombineWarps, t1 = nt * (warp + 1) / kCombineWarps;
    double tot = 0.0;
    if (k < a.K) {
        const double* src = a.partials + (size_t)row * a.tiles * a.K + k;
        for (int64_t t = t0; t < t1; ++t) tot += src[(size_t)t * a.K];
    }
    seg[warp][lane] = tot;
    __syncthreads();
    if (warp == 0 && k < a.K) {
        double v = seg[0][lane];
        for (int w = 1; w < kCombineWarps; ++w) v += seg[w][lane];
        sums[row * a.K + k] = v;
        if (a.sse_all) a.sse_all[row * a.K + k] = (float)v;
    }
}

// Long rows, step 2: first minimal candidate of every row.
__global__ void __launch_bounds__(kSThreads)
search_argmin_kernel(SearchArgs a, const double* __restrict__ sums) {
    __shared__ double red_val[kSWarps];
    __shared__ int red_idx[kSWarps];
    const int64_t row = blockIdx.x;
    const int64_t n_row = a.rows.begin(row + 1) - a.rows.begin(row);
    float lo;
    const float m = row_range(a, row, lo);
    const bool finite = (__float_as_uint(m) & 0x7fffffffu) < 0x7f800000u &&
                        (__float_as_uint(lo) & 0x7fffffffu) < 0x7f800000u;
    if (!finite || !(m > 0.0f) || n_row <= 0) {
        if (threadIdx.x == 0) {
            a.idx_out[row] = 0;
            a.p_out[row] = 0.0f;
            if (a.err_out) a.err_out[row] = 0.0f;
        }
        return;
    }
    double best; int idx;
    block_argmin(sums + row * a.K, a.K, red_val, red_idx, best, idx);
    if (threadIdx.x == 0) write_row_result(a, row, m, best, idx);
}

// ------------------------------------------------------------------------------- host side
static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

SearchPlan plan_search(int64_t C, int64_t max_n, int K) {
    SearchPlan p;
    p.max_n = max_n;
    p.tile = kSearchTile;
    p.tiles = (max_n + kSearchTile - 1) / kSearchTile;
    if (p.tiles < 1) p.tiles = 1;
    // A few long rows (a per-tensor search) give few CTAs at full tiles: cut them finer, down to
    // kMinSplitTile values, until there are about two CTAs per SM.  (The extra tiles cost a
    // sort each, but they run side by side.)
    constexpr int64_t kMinSplitTile = 1024, kWantCtas = 2 * 148;
    if (max_n > kMinSplitTile && C * p.tiles < kWantCtas) {
        const int64_t per_row = (kWantCtas + C - 1) / C;                    // tiles wanted per row
        int64_t tile = (max_n + per_row - 1) / per_row;
        tile = std::min<int64_t>(std::max<int64_t>((tile + 255) / 256 * 256, kMinSplitTile), kSearchTile);
        const int64_t tiles = (max_n + tile - 1) / tile;
        if (tiles > 1) { p.tile = tile; p.tiles = tiles; }
    }
    p.off_m = 256;
    p.off_partials = align_up(p.off_m + sizeof(float) * (size_t)C, 256);
    p.off_sums = p.off_partials;
    p.bytes = p.off_partials;
    if (p.tiles > 1) {
        p.off_sums = align_up(p.off_partials +
                              sizeof(double) * (size_t)C * (size_t)p.tiles * (size_t)K, 256);
        p.bytes = p.off_sums + sizeof(double) * (size_t)C * (size_t)K;
    }
    p.bytes = align_up(p.bytes, 256);
    return p;
}

cudaError_t launch_search(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                          int64_t total, int bits, const float* ratios, int K, const float* m,
                          const float* lo, float* p_out, float* err_out, int32_t* idx_out,
                          float* sse_all, void* workspace, const SearchPlan& plan,
                          cudaStream_t stream, int64_t shift, bool clear_status, double* sums64) {
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    cudaError_t e = cudaSuccess;
    if (clear_status) e = cudaMemsetAsync(ws, 0, 256, stream);    // status word
    if (e != cudaSuccess) return e;
    if (!m && !lo) {
        float* m_ws = reinterpret_cast<float*>(ws + plan.off_m);
        e = launch_absmax(x, row_offsets, C, n, total, m_ws, stream, shift);
        if (e != cudaSuccess) return e;
        m = m_ws;
    }
    SearchArgs a;
    a.x = x;
    a.rows = Rows{row_offsets, C, n, n > 0 ? 1.0 / (double)n : 0.0, row_offsets ? shift : 0};
    a.m = m;
    a.ratios = ratios;
    a.K = K;
    a.lo = lo;
    a.levels = lo ? (1 << bits) - 1 : (1 << (bits - 1)) - 1;
    a.tiles = plan.tiles;
    a.cap = (plan.tiles > 1) ? (int)plan.tile : (int)((plan.max_n + 3) / 4 * 4);
    a.partials = reinterpret_cast<double*>(ws + plan.off_partials);
    a.p_out = p_out;
    a.err_out = err_out;
    a.idx_out = idx_out;
    a.sse_all = sse_all;
    a.sums64 = sums64;
    a.status = reinterpret_cast<int*>(ws);

    if (K <= kSortMaxK) {
        // Rows are served by CTAs sized to their length: the per-row latency of the sort and of
        // the final argmin is hidden by the number of rows in flight, and short rows fit many
        // more small CTAs per SM.  One launch per class; a CTA whose row belongs to another
        // class exits at once.  A dense tensor has one class.
        struct RowClass { int64_t n_min, n_max; int threads; };
        // (boundaries measured on B200: 128-thread CTAs beat 256-thread ones up to rows of about
        // 2300 values, 64-thread CTAs beat 128-thread ones up to about 500)
        RowClass classes[4] = {{2305, INT64_MAX, 256}, {513, 2304, 128},
                               {kTinyMax + 1, 512, 64}, {0, kTinyMax, 0}};   // 0: tiny rows
        if (plan.tile < kSearchTile) {
            // a few long rows cut into finer tiles (plan_search): every row longer than the tiny
            // ones is tiled the same way, in one launch, so that the combine kernel finds the
            // partial sums of all its tiles
            classes[0] = RowClass{kTinyMax + 1, INT64_MAX, plan.tile <= 2304 ? 128 : 256};
            classes[1] = classes[2] = RowClass{INT64_MAX, INT64_MAX, 64};   // never launched
        }
        size_t off[7];
        const size_t smem_max = sorted_smem_layout(a.cap, K, kSWarps, off);
        if (smem_max > 48 * 1024) {  // above the default limit: opt in (idempotent, per device)
            e = cudaFuncSetAttribute(search_sorted_kernel,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max);
            if (e != cudaSuccess) return e;
        }
        if (plan.tile == kSearchTile && total / C < 512) {
            // Mostly short rows (the library sees the mean length only): the small-CTA classes
            // hold the bulk of the work and go first, so that the stream does not end with their
            // long tail of half-empty SMs (MobileNetV2 shapes: 244 -> 236 us; with the longest
            // class first the ResNet-50 shapes are 0.5 % faster, hence the two orders).
            std::swap(classes[0], classes[2]);
        }
        const int full_cap = a.cap;
        int launched = 0;
        for (const RowClass& rc : classes) {
            if (plan.max_n < rc.n_min) continue;
            if (!row_offsets && n > rc.n_max) continue;           // dense: every row has length n
            const bool longest = rc.n_max == INT64_MAX;
            a.n_min = rc.n_min;
            a.n_max = rc.n_max;
            a.grid_tiles = longest ? plan.tiles : 1;
            a.cap = longest ? full_cap
                            : (int)((std::min<int64_t>(plan.max_n, rc.n_max) + 3) / 4 * 4);
            const bool tiny = rc.threads == 0;            // one warp per row, no shared memory
            const size_t smem = tiny ? 0 : sorted_smem_layout(a.cap, K, rc.threads / 32, off);
            // Launches after the first may overlap the tail of the one before (they are
            // independent of each other; all of them were ordered after the abs-max above by the
            // first, ordinary launch).
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(tiny ? (unsigned)((C + kTinyWarps - 1) / kTinyWarps)
                                    : (unsigned)(C * a.grid_tiles));
            cfg.blockDim = dim3(tiny ? (unsigned)(kTinyWarps * 32) : (unsigned)rc.threads);
            cfg.dynamicSmemBytes = smem;
            cfg.stream = stream;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = attr;
            cfg.numAttrs = launched > 0 ? 1 : 0;
            e = tiny ? cudaLaunchKernelEx(&cfg, search_tiny_kernel, a)
                     : cudaLaunchKernelEx(&cfg, search_sorted_kernel, a);
            if (e != cudaSuccess) return e;
            ++launched;
        }
        a.cap = full_cap;
    } else {
        const int E = slices_for(K, kSWarps);
        a.n_min = 0;
        a.n_max = INT64_MAX;
        a.grid_tiles = plan.tiles;
        const size_t smem = (((size_t)a.cap * 4 + 15) & ~(size_t)15) +
                            sizeof(double) * (size_t)E * (size_t)K;
        if (smem > 48 * 1024) {
            e = cudaFuncSetAttribute(search_generic_kernel,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
        }
        search_generic_kernel<<<(unsigned)(C * plan.tiles), kSThreads, smem, stream>>>(a);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (plan.tiles > 1) {
        double* sums = sums64 ? sums64 : reinterpret_cast<double*>(ws + plan.off_sums);
        const int64_t chunks = (K + 31) / 32;
        search_combine_kernel<<<(unsigned)(C * chunks), kCombineWarps * 32, 0, stream>>>(a, sums);
        e = cudaGetLastError();
        if (e != cudaSuccess || sums64) return e;
        search_argmin_kernel<<<(unsigned)C, kSThreads, 0, stream>>>(a, sums);
        e = cudaGetLastError();
    }
    return e;
}

// Rows cut across several devices or calls: adds the `parts` sets of per-candidate sums of every
// row in ascending part order (fixed order: reproducible), then takes the first minimum.
__global__ void __launch_bounds__(kSThreads)
search_finish_kernel(const double* __restrict__ sums, int parts, int64_t C, int K,
                     const float* __restrict__ m_in, const float* __restrict__ lo_in,
                     const float* __restrict__ ratios, float* __restrict__ p_out,
                     float* __restrict__ err_out, int32_t* __restrict__ idx_out,
                     float* __restrict__ sse_all, int* __restrict__ status) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ double red_val[kSWarps];
    __shared__ int red_idx[kSWarps];
    double* tot = reinterpret_cast<double*>(smem_raw);
    const int64_t row = blockIdx.x;
    float m = m_in[row];
    const float lo = lo_in ? lo_in[row] : 0.0f;
    if (lo_in) m = __fsub_rn(m, lo);
    const bool finite = (__float_as_uint(m) & 0x7fffffffu) < 0x7f800000u &&
                        (__float_as_uint(lo) & 0x7fffffffu) < 0x7f800000u;
    if (!finite || !(m > 0.0f)) {
        if (!finite && threadIdx.x == 0 && status) atomicOr(status, kStatusNonFinite);
        if (threadIdx.x == 0) {
            idx_out[row] = 0;
            p_out[row] = 0.0f;
            if (err_out) err_out[row] = 0.0f;
        }
        if (sse_all)
            for (int k = threadIdx.x; k < K; k += blockDim.x) sse_all[row * K + k] = 0.0f;
        return;
    }
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        double v = sums[(size_t)row * K + k];
        for (int part = 1; part < parts; ++part) v += sums[((size_t)part * C + row) * K + k];
        tot[k] = v;
        if (sse_all) sse_all[row * K + k] = (float)v;
    }
    __syncthreads();
    double best; int idx;
    block_argmin(tot, K, red_val, red_idx, best, idx);
    if (threadIdx.x == 0) {
        idx_out[row] = idx;
        p_out[row] = __fmul_rn(m, ratios[idx]);
        if (err_out) err_out[row] = (float)best;
    }
}

cudaError_t launch_search_finish(const double* sums, int parts, int64_t C, int K, const float* m,
                                 const float* lo, const float* ratios, float* p_out, float* err_out,
                                 int32_t* idx_out, float* sse_all, int* status,
                                 cudaStream_t stream) {
    cudaError_t e = cudaSuccess;
    if (status) e = cudaMemsetAsync(status, 0, sizeof(int), stream);
    if (e != cudaSuccess) return e;
    search_finish_kernel<<<(unsigned)C, kSThreads, sizeof(double) * (size_t)K, stream>>>(
        sums, parts, C, K, m, lo, ratios, p_out, err_out, idx_out, sse_all, status);
    return cudaGetLastError();
}

}  // namespace pwlq
