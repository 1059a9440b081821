// Two breakpoints (Sec. 5.1, "Multiple Breakpoints"): regions [0, p1], (p1, p2], (p2, m], each
// quantized like the regions of Eq. 3; search over all pairs i < j of a grid of K ratios.
//
// The squared error of a pair splits by region:
//     SSE(i, j) = C_i + M_ij + T_j
//     C_i  = error of the values a <= p_i        quantized on [0, p_i]
//     M_ij = error of the values p_i < a <= p_j  quantized on [p_i, p_j]
//     T_j  = error of the values a > p_j         quantized on [p_j, m]
// One CTA per row: the row's magnitudes are counting-sorted by candidate interval into shared
// memory (deterministic placement, per-warp counts and in-warp ranks), after which every term is a sum over a contiguous range of
// the sorted tile.  A warp takes one term at a time, its lanes stride over the range (per value
// the operation-by-operation sequence of Eq. 1, no fused multiply-add), and the lane sums are
// added in binary64 in a fixed order.  Work per row: the honest evaluation of every (value, pair)
// of the pair's middle region plus 2 K passes for the C and T terms.
#include <algorithm>

#include "pwlq_common.cuh"
#include "pwlq_kernels.h"
#include "pwlq_multi.cuh"

namespace pwlq {

constexpr int kS2Threads = 256;
constexpr int kS2Warps = kS2Threads / 32;
constexpr float kMagic2 = 12582912.0f;      // 1.5 * 2^23

struct Search2Args {
    const float* x;
    Rows rows;
    const float* m;
    const float* ratios;
    int K;
    int levels;
    int cap;              // tile capacity in values
    int nbp;              // breakpoints searched: 2 (pairs) or 3 (triples)
    int64_t tiles;        // tiles per row (by the longest row); > 1: partial terms go to `partials`
    double* partials;     // [C, tiles, 2 K + K (K - 1) / 2]: C_i, T_j, M_ij of every tile
    float* p_out[3];      // breakpoint t of row c: p_out[t][c * out_stride]
    int32_t* idx_out[3];
    int out_stride;
    float* err_out;
    float* sse_out;       // pairs: [C, K, K]; triples: [C, K, K, K]; or nullptr
    int* status;
};

__host__ __device__ inline size_t s2_align(size_t v) { return (v + 15) & ~(size_t)15; }

// Shared-memory layout: sorted tile | bucket+rank per value | breakpoints | bucket starts |
// per-warp bucket counts | C, T | M (triangular) | best left / right parts of the triple search.
__host__ __device__ inline size_t search2_smem(int cap, int K, size_t* off) {
    size_t o = 0;
    off[0] = o; o = s2_align(o + sizeof(float) * (size_t)cap);
    off[1] = o; o = s2_align(o + sizeof(uint32_t) * (size_t)cap);
    off[2] = o; o = s2_align(o + sizeof(float) * (size_t)K);
    off[3] = o; o = s2_align(o + sizeof(int) * (size_t)(K + 2));
    off[4] = o; o = s2_align(o + sizeof(uint16_t) * (size_t)(K + 1) * kS2Warps);
    off[5] = o; o = s2_align(o + sizeof(double) * (size_t)(2 * K));
    off[6] = o; o = s2_align(o + sizeof(double) * (size_t)(K * (K - 1) / 2));
    off[7] = o; o = s2_align(o + sizeof(double) * (size_t)(2 * K));      // triples: best left / right parts
    off[8] = o; o = s2_align(o + sizeof(int) * (size_t)(2 * K));
    return o;
}

__device__ __forceinline__ int pair_index(int i, int j, int K) {      // i < j, order (i, j)
    return i * (2 * K - i - 1) / 2 + (j - i - 1);
}

// Sum over sorted values [beg, end) of the squared error of Eq. 1 on the range [z, z + delta];
// every lane returns the warp's total.
__device__ __forceinline__ double range_error(const float* tile, int beg, int end, float z,
                                              float delta, float Lf) {
    float s = 0.0f, inv = 0.0f;
    if (delta > 0.0f) { s = __fdiv_rn(delta, Lf); inv = __fdiv_rn(Lf, delta); }
    const int lane = threadIdx.x & 31;
    float acc0 = 0.0f, acc1 = 0.0f;
    int i = beg + lane;
    for (; i + 32 < end; i += 64) {
        const float a0 = tile[i], a1 = tile[i + 32];
        const float r0 = __fadd_rn(__fmul_rn(__fsub_rn(a0, z), inv), kMagic2);
        const float r1 = __fadd_rn(__fmul_rn(__fsub_rn(a1, z), inv), kMagic2);
        const float q0 = fminf(__fsub_rn(r0, kMagic2), Lf), q1 = fminf(__fsub_rn(r1, kMagic2), Lf);
        const float e0 = __fsub_rn(__fadd_rn(__fmul_rn(q0, s), z), a0);
        const float e1 = __fsub_rn(__fadd_rn(__fmul_rn(q1, s), z), a1);
        acc0 = __fmaf_rn(e0, e0, acc0);
        acc1 = __fmaf_rn(e1, e1, acc1);
    }
    if (i < end) {
        const float a0 = tile[i];
        const float r0 = __fadd_rn(__fmul_rn(__fsub_rn(a0, z), inv), kMagic2);
        const float q0 = fminf(__fsub_rn(r0, kMagic2), Lf);
        const float e0 = __fsub_rn(__fadd_rn(__fmul_rn(q0, s), z), a0);
        acc0 = __fmaf_rn(e0, e0, acc0);
    }
    double d = (double)acc0 + (double)acc1;           // <= 256 terms per lane in binary32
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
    return d;
}

// Squared error of Eq. 1 for one value on the range [z, z + delta] (s = delta / L, inv = L / delta),
// added to acc; operation by operation, no fused multiply-add except the final square-and-add.
// (No saturation needed: a - z <= delta, so the level cannot exceed L.)
__device__ __forceinline__ float add_sq_err(float a, float z, float inv, float s, float acc) {
    const float r = __fadd_rn(__fmul_rn(__fsub_rn(a, z), inv), kMagic2);
    const float q = __fsub_rn(r, kMagic2);
    const float e = __fsub_rn(__fadd_rn(__fmul_rn(q, s), z), a);
    return __fmaf_rn(e, e, acc);
}

// Constants of one (i, j) middle region, replicated in both lanes of a packed register.
struct MidConst {
    float pi, pj, inv, s;
    u64 npi2, inv2, magic2, nmagic2, ns2;
};

// Error of two values, fused form: u = a - p_i, r = fma(u, inv, magic), q = r - magic,
// e = fma(q, -s, u).  It differs from the operation-by-operation form only in rounding.
__device__ __forceinline__ u64 fused_err2(u64 a, const MidConst& c) {
    const u64 u = add2(a, c.npi2);
    const u64 r = fma2(u, c.inv2, c.magic2);
    const u64 q = add2(r, c.nmagic2);
    return fma2(q, c.ns2, u);
}

// Middle terms M_ij for one first breakpoint i and eight consecutive second breakpoints
// j = jb .. jb + 7, by one warp: lane = (phase, sub) with sub = lane & 7 the candidate and
// phase = lane >> 3 taking every fourth 128-bit vector of the sorted tile (shared-memory
// broadcast reads: the eight candidates of a phase read the same vector).  All eight candidates
// need the values between B_i and the smallest B_j; only the vectors around B_i and between the
// smallest and the largest B_j need the per-value test p_i < a <= p_j.
// EXACT: the oracle's operation-by-operation arithmetic (short rows, where the rounding of the
// fused form would show in the sums); otherwise the fused form on packed pairs of values.
template <bool EXACT>
__device__ __forceinline__ void middle_terms(const float* tile, const int* start, const float* ps,
                                             int K, int i, int jb, float Lf, double* M) {
    const int lane = threadIdx.x & 31, sub = lane & 7, phase = lane >> 3;
    const int j = jb + sub;
    MidConst c;
    c.pi = ps[i];
    c.pj = (j < K) ? ps[j] : c.pi;                   // j >= K: empty range, contributes nothing
    const float delta = __fsub_rn(c.pj, c.pi);
    c.s = 0.0f; c.inv = 0.0f;
    if (delta > 0.0f) { c.s = __fdiv_rn(delta, Lf); c.inv = __fdiv_rn(Lf, delta); }
    c.npi2 = pack2(-c.pi, -c.pi);
    c.inv2 = pack2(c.inv, c.inv);
    c.magic2 = pack2(kMagic2, kMagic2);
    c.nmagic2 = pack2(-kMagic2, -kMagic2);
    c.ns2 = pack2(-c.s, -c.s);
    const int b_i = start[i + 1], b_first = start[jb + 1], b_last = start[min(jb + 7, K - 1) + 1];
    const int v_lo = b_i >> 2, v_in0 = (b_i + 3) >> 2, v_in1 = max(b_first >> 2, v_in0);
    const int v_hi = (b_last + 3) >> 2;
    const float4* t4 = reinterpret_cast<const float4*>(tile);
    const ulonglong2* t2 = reinterpret_cast<const ulonglong2*>(tile);
    double total = 0.0;
    float acc = 0.0f;                                 // EXACT, and the tested vectors
    u64 acc2a = 0, acc2b = 0;                         // fused interior: two packed accumulators
    // vectors that hold B_i (at most one) and those from the smallest B_j on: tested per value
    auto tested = [&](int v0, int v1) {
        int run = 0;
        for (int v = v0 + phase; v < v1; v += 4) {
            const float4 q = t4[v];
            const float a4[4] = {q.x, q.y, q.z, q.w};
            if (EXACT) {
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const float with = add_sq_err(a4[t], c.pi, c.inv, c.s, acc);
                    acc = (a4[t] > c.pi && a4[t] <= c.pj) ? with : acc;
                }
            } else {
                float e[4];
                unpack2(fused_err2(pack2(q.x, q.y), c), e[0], e[1]);
                unpack2(fused_err2(pack2(q.z, q.w), c), e[2], e[3]);
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const float et = (a4[t] > c.pi && a4[t] <= c.pj) ? e[t] : 0.0f;
                    acc = __fmaf_rn(et, et, acc);
                }
            }
            if (++run == 128) { total += (double)acc; acc = 0.0f; run = 0; }
        }
    };
    tested(v_lo, v_in0);
    {
        int run = 0;
        for (int v = v_in0 + phase; v < v_in1; v += 4) {
            if (EXACT) {
                const float4 q = t4[v];
                acc = add_sq_err(q.x, c.pi, c.inv, c.s, acc);
                acc = add_sq_err(q.y, c.pi, c.inv, c.s, acc);
                acc = add_sq_err(q.z, c.pi, c.inv, c.s, acc);
                acc = add_sq_err(q.w, c.pi, c.inv, c.s, acc);
            } else {
                const ulonglong2 q = t2[v];
                const u64 e0 = fused_err2(q.x, c), e1 = fused_err2(q.y, c);
                acc2a = fma2(e0, e0, acc2a);
                acc2b = fma2(e1, e1, acc2b);
            }
            if (++run == 128) {
                float f0, f1, f2, f3;
                unpack2(acc2a, f0, f1);
                unpack2(acc2b, f2, f3);
                total += (double)acc + ((double)f0 + (double)f1) + ((double)f2 + (double)f3);
                acc = 0.0f; acc2a = 0; acc2b = 0; run = 0;
            }
        }
    }
    tested(v_in1, v_hi);
    {
        float f0, f1, f2, f3;
        unpack2(acc2a, f0, f1);
        unpack2(acc2b, f2, f3);
        total += (double)acc + ((double)f0 + (double)f1) + ((double)f2 + (double)f3);
    }
    total += __shfl_xor_sync(0xffffffffu, total, 8);
    total += __shfl_xor_sync(0xffffffffu, total, 16);
    if (phase == 0 && j < K) M[pair_index(i, j, K)] = total;
}

__device__ __forceinline__ void write_degenerate2(const Search2Args& a, int64_t row) {
    if (threadIdx.x == 0) {
        for (int t = 0; t < a.nbp; ++t) {
            a.idx_out[t][row * a.out_stride] = t;
            a.p_out[t][row * a.out_stride] = 0.0f;
        }
        if (a.err_out) a.err_out[row] = 0.0f;
    }
    if (a.sse_out) {
        const int64_t per_row = (int64_t)a.K * a.K * (a.nbp == 3 ? a.K : 1);
        for (int64_t t = threadIdx.x; t < per_row; t += kS2Threads) a.sse_out[row * per_row + t] = 0.0f;
    }
}

// First minimum of (value, index) pairs over the CTA; the result is valid in thread 0.
__device__ __forceinline__ void cta_first_min(double& best, int& best_idx, double* red_val,
                                              int* red_idx) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double ov = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, best_idx, o);
        if (oi != 0x7fffffff && (best_idx == 0x7fffffff || ov < best || (ov == best && oi < best_idx))) {
            best = ov; best_idx = oi;
        }
    }
    if (lane == 0) { red_val[warp] = best; red_idx[warp] = best_idx; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kS2Warps; ++w) {
            const double ov = red_val[w];
            const int oi = red_idx[w];
            if (oi != 0x7fffffff && (best_idx == 0x7fffffff || ov < best || (ov == best && oi < best_idx))) {
                best = ov; best_idx = oi;
            }
        }
    }
}

// Totals and the first minimal pair in the order (i, j), from the terms of one row in shared
// memory (CT = C[0..K), T[K..2K); M triangular; ps = the row's breakpoints).  All threads call.
__device__ __forceinline__ void finish_pairs(const Search2Args& a, int64_t row, const float* ps,
                                             double* CT, double* M, double* red_val, int* red_idx) {
    const int K = a.K, tid = threadIdx.x;
    const int npairs = K * (K - 1) / 2;
    double best = 0.0;
    int best_idx = 0x7fffffff;
    {
        int i = 0, base = 0;                          // base = pair_index(i, i + 1)
        for (int t = tid; t < npairs; t += kS2Threads) {
            while (t >= base + (K - 1 - i)) { base += K - 1 - i; ++i; }
            const int j = i + 1 + (t - base);
            const double v = CT[i] + M[t] + CT[K + j];
            M[t] = v;
            if (best_idx == 0x7fffffff || v < best) { best = v; best_idx = t; }
        }
    }
    cta_first_min(best, best_idx, red_val, red_idx);
    if (tid == 0) {
        int i = 0, base = 0;
        while (best_idx >= base + (K - 1 - i)) { base += K - 1 - i; ++i; }
        const int j = i + 1 + (best_idx - base);
        a.idx_out[0][row * a.out_stride] = i;
        a.idx_out[1][row * a.out_stride] = j;
        a.p_out[0][row * a.out_stride] = ps[i];
        a.p_out[1][row * a.out_stride] = ps[j];
        if (a.err_out) a.err_out[row] = (float)best;
    }
    if (a.sse_out) {
        float* dst = a.sse_out + row * K * K;
        for (int t = tid; t < K * K; t += kS2Threads) {
            const int i = t / K, j = t - i * K;
            dst[t] = (i < j) ? (float)M[pair_index(i, j, K)] : 0.0f;
        }
    }
}

// Three breakpoints: SSE(i, j, k) = (C_i + M_ij) + (M_jk + T_k), the regions' errors being sums
// over disjoint sets of values.  For every middle breakpoint j the best left part (over i < j) and
// the best right part (over k > j) are independent, so the first minimal triple in the order
// (i, j, k) follows from K - 2 pairs of scans over the terms the pair search already has --
// O(K^2) per row instead of K^3 / 6 evaluations.  left / right: 2 K doubles and 2 K ints of
// shared memory.
__device__ __forceinline__ void finish_triples(const Search2Args& a, int64_t row, const float* ps,
                                               const double* CT, const double* M, double* lr_val,
                                               int* lr_idx, double* red_val, int* red_idx) {
    const int K = a.K, tid = threadIdx.x;
    for (int t = tid; t < 2 * K; t += kS2Threads) {
        const bool left = t < K;
        const int j = left ? t : t - K;
        double best = 0.0;
        int arg = -1;
        if (left) {
            for (int i = 0; i < j; ++i) {             // ascending i: the first minimum stays
                const double v = CT[i] + M[pair_index(i, j, K)];
                if (arg < 0 || v < best) { best = v; arg = i; }
            }
        } else {
            for (int k = j + 1; k < K; ++k) {
                const double v = M[pair_index(j, k, K)] + CT[K + k];
                if (arg < 0 || v < best) { best = v; arg = k; }
            }
        }
        lr_val[t] = best;
        lr_idx[t] = arg;
    }
    __syncthreads();
    // the triples of two middle breakpoints differ in j, so (total, i, j) orders them completely
    double best = 0.0;
    int best_idx = 0x7fffffff;
    for (int j = 1 + tid; j < K - 1; j += kS2Threads) {
        const double v = lr_val[j] + lr_val[K + j];
        const int key = lr_idx[j] * K + j;            // order (i, j)
        if (best_idx == 0x7fffffff || v < best || (v == best && key < best_idx)) { best = v; best_idx = key; }
    }
    cta_first_min(best, best_idx, red_val, red_idx);
    if (tid == 0) {
        const int i = best_idx / K, j = best_idx - i * K, k = lr_idx[K + j];
        const int idx[3] = {i, j, k};
        for (int t = 0; t < 3; ++t) {
            a.idx_out[t][row * a.out_stride] = idx[t];
            a.p_out[t][row * a.out_stride] = ps[idx[t]];
        }
        if (a.err_out) a.err_out[row] = (float)best;
    }
    if (a.sse_out) {
        float* dst = a.sse_out + row * (int64_t)K * K * K;
        for (int t = tid; t < K * K * K; t += kS2Threads) {
            const int i = t / (K * K), j = (t / K) % K, k = t % K;
            dst[t] = (i < j && j < k)
                         ? (float)((CT[i] + M[pair_index(i, j, K)]) + (M[pair_index(j, k, K)] + CT[K + k]))
                         : 0.0f;
        }
    }
}

// Shared memory of the row-closing step: breakpoints | C, T | M | best left / right parts.
__host__ __device__ inline size_t finish2_smem(int K, size_t* off) {
    size_t o = 0;
    off[0] = o; o = s2_align(o + sizeof(float) * (size_t)K);
    off[1] = o; o = s2_align(o + sizeof(double) * (size_t)(2 * K));
    off[2] = o; o = s2_align(o + sizeof(double) * (size_t)(K * (K - 1) / 2));
    off[3] = o; o = s2_align(o + sizeof(double) * (size_t)(2 * K));
    off[4] = o; o = s2_align(o + sizeof(int) * (size_t)(2 * K));
    return o;
}

// One CTA per (row, tile of at most a.cap values).  A row of one tile is closed here; the terms
// of a longer row's tiles go to a.partials and search2_finish_kernel closes the row.
__global__ void __launch_bounds__(kS2Threads)
search2_kernel(Search2Args a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ double red_val[kS2Warps];
    __shared__ int red_idx[kS2Warps];
    const int64_t row = blockIdx.x / a.tiles, tile_no = blockIdx.x - row * a.tiles;
    const int64_t row_beg = a.rows.begin(row), end = a.rows.begin(row + 1);
    const int64_t n_row = end - row_beg;
    const int64_t beg = row_beg + tile_no * (int64_t)a.cap;
    if (tile_no > 0 && beg >= end) return;            // this row has fewer tiles than the longest
    const int cnt = (int)min((int64_t)a.cap, end - beg);
    const int K = a.K;
    const float m = a.m[row];
    const float Lf = (float)a.levels;
    const bool finite = (__float_as_uint(m) & 0x7fffffffu) < 0x7f800000u;
    if (!finite || !(m > 0.0f) || cnt <= 0) {
        if (a.tiles > 1) return;                      // the row-closing kernel writes the row
        if (!finite && threadIdx.x == 0) atomicOr(a.status, kStatusNonFinite);
        write_degenerate2(a, row);
        return;
    }
    size_t off[9];
    search2_smem(a.cap, K, off);
    float* tile = reinterpret_cast<float*>(smem_raw + off[0]);
    uint32_t* jr = reinterpret_cast<uint32_t*>(smem_raw + off[1]);
    float* ps = reinterpret_cast<float*>(smem_raw + off[2]);
    int* start = reinterpret_cast<int*>(smem_raw + off[3]);
    uint16_t* hist = reinterpret_cast<uint16_t*>(smem_raw + off[4]);
    double* CT = reinterpret_cast<double*>(smem_raw + off[5]);       // C[0..K), T[K..2K)
    double* M = reinterpret_cast<double*>(smem_raw + off[6]);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    int unordered = 0;
    for (int k = tid; k < K; k += kS2Threads) {
        const float rk = __ldg(a.ratios + k);
        if (k > 0) unordered |= (rk < __ldg(a.ratios + k - 1));
        ps[k] = __fmul_rn(m, rk);
    }
    for (int t = tid; t < (K + 1) * kS2Warps; t += kS2Threads) hist[t] = 0;
    if (__syncthreads_or(unordered)) {               // the search needs an ascending grid
        if (a.tiles > 1) return;
        if (tid == 0) atomicOr(a.status, kStatusBadGrid);
        write_degenerate2(a, row);
        return;
    }

    // pass 1: bucket j = #{k : p_k < a} of every value and its rank among the earlier values of
    // the same bucket in this warp's segment (each warp owns a contiguous segment of the tile and
    // walks it 32 values at a time; ranks inside a group of 32 come from match.any)
    const unsigned full = 0xffffffffu;
    const int seg = (((cnt + kS2Warps - 1) / kS2Warps) + 31) & ~31;
    const int w_beg = min(warp * seg, cnt), w_end = min(w_beg + seg, cnt);
    uint16_t* myhist = hist + warp * (K + 1);
    for (int base = w_beg; base < w_end; base += 32) {
        const int i = base + lane;
        int j = K + 1;                                // "no value"
        if (i < w_end) {
            const float v = fminf(fabsf(__ldg(a.x + beg + i)), m);
            int lo = 0, hi = K;                       // p_k < v for k < lo; p_k >= v for k >= hi
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (ps[mid] < v) lo = mid + 1; else hi = mid;
            }
            j = lo;
        }
        const unsigned peers = __match_any_sync(full, j);
        int before = 0;
        if (j <= K) before = myhist[j];
        __syncwarp();
        if (j <= K) {
            if (lane == __ffs(peers) - 1) myhist[j] = (uint16_t)(before + __popc(peers));
            jr[i] = (uint32_t)j | ((uint32_t)(before + __popc(peers & ((1u << lane) - 1u))) << 7);
        }
        __syncwarp();
    }
    __syncthreads();
    // exclusive scan over buckets, then over the warps inside a bucket
    if (tid <= K) {
        int tot = 0;
        for (int w = 0; w < kS2Warps; ++w) tot += hist[w * (K + 1) + tid];
        start[tid] = tot;
    }
    __syncthreads();
    if (tid == 0) {
        int run = 0;
        for (int j = 0; j <= K; ++j) { const int c = start[j]; start[j] = run; run += c; }
        start[K + 1] = run;
    }
    __syncthreads();
    if (tid <= K) {
        int run = start[tid];
        for (int w = 0; w < kS2Warps; ++w) {
            const int c = hist[w * (K + 1) + tid];
            hist[w * (K + 1) + tid] = (uint16_t)run;
            run += c;
        }
    }
    __syncthreads();
    // pass 2: placement (bucket, then warp segment, then order inside the segment): deterministic
    for (int i = w_beg + lane; i < w_end; i += 32) {
        const uint32_t e = jr[i];
        tile[myhist[e & 0x7fu] + (e >> 7)] = fminf(fabsf(__ldg(a.x + beg + i)), m);
    }
    if (tid < ((4 - (cnt & 3)) & 3)) tile[cnt + tid] = 0.0f;     // whole vectors: zeros pass no test
    __syncthreads();

    // evaluation: values <= p_k are the first B_k = start[k + 1] entries of the sorted tile
    for (int k = warp; k < 2 * K; k += kS2Warps) {
        double d;
        if (k < K) d = range_error(tile, 0, start[k + 1], 0.0f, ps[k], Lf);
        else       d = range_error(tile, start[k - K + 1], cnt, ps[k - K], __fsub_rn(m, ps[k - K]), Lf);
        if (lane == 0) CT[k] = d;
    }
    // The fused form's rounding shows in the sums of short rows (it grows like L / sqrt(n)); rows
    // shorter than L^2 / 2, and all rows of fewer than 32 values, use the operation-by-operation
    // form.
    const bool fused = 2 * n_row >= (int64_t)a.levels * a.levels && n_row >= 32;
    {
        int item = 0;                                  // (i, group of eight j) in a fixed order
        for (int i = 0; i < K - 1; ++i)
            for (int jb = i + 1; jb < K; jb += 8, ++item)
                if ((item & (kS2Warps - 1)) == warp) {
                    if (fused) middle_terms<false>(tile, start, ps, K, i, jb, Lf, M);
                    else       middle_terms<true>(tile, start, ps, K, i, jb, Lf, M);
                }
    }
    __syncthreads();

    const int npairs = K * (K - 1) / 2;
    if (a.tiles > 1) {
        double* dst = a.partials + ((size_t)row * a.tiles + tile_no) * (size_t)(2 * K + npairs);
        for (int t = tid; t < 2 * K; t += kS2Threads) dst[t] = CT[t];
        for (int t = tid; t < npairs; t += kS2Threads) dst[2 * K + t] = M[t];
        return;
    }
    if (a.nbp == 3)
        finish_triples(a, row, ps, CT, M, reinterpret_cast<double*>(smem_raw + off[7]),
                       reinterpret_cast<int*>(smem_raw + off[8]), red_val, red_idx);
    else
        finish_pairs(a, row, ps, CT, M, red_val, red_idx);
}

// Closes the rows that were cut into tiles: adds the tiles' terms in ascending tile order (fixed
// order: reproducible) and takes the first minimal pair or triple.  One CTA per row.
__global__ void __launch_bounds__(kS2Threads)
search2_finish_kernel(Search2Args a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ double red_val[kS2Warps];
    __shared__ int red_idx[kS2Warps];
    const int64_t row = blockIdx.x;
    const int64_t n_row = a.rows.begin(row + 1) - a.rows.begin(row);
    const int K = a.K, tid = threadIdx.x;
    const float m = a.m[row];
    const bool finite = (__float_as_uint(m) & 0x7fffffffu) < 0x7f800000u;
    if (!finite || !(m > 0.0f) || n_row <= 0) {
        if (!finite && tid == 0) atomicOr(a.status, kStatusNonFinite);
        write_degenerate2(a, row);
        return;
    }
    size_t off[5];
    finish2_smem(K, off);
    float* ps = reinterpret_cast<float*>(smem_raw + off[0]);
    double* CT = reinterpret_cast<double*>(smem_raw + off[1]);
    double* M = reinterpret_cast<double*>(smem_raw + off[2]);
    int unordered = 0;
    for (int k = tid; k < K; k += kS2Threads) {
        const float rk = __ldg(a.ratios + k);
        if (k > 0) unordered |= (rk < __ldg(a.ratios + k - 1));
        ps[k] = __fmul_rn(m, rk);
    }
    if (__syncthreads_or(unordered)) {
        if (tid == 0) atomicOr(a.status, kStatusBadGrid);
        write_degenerate2(a, row);
        return;
    }
    const int npairs = K * (K - 1) / 2, nterms = 2 * K + npairs;
    const int64_t nt = (n_row + a.cap - 1) / a.cap;
    const double* src = a.partials + (size_t)row * a.tiles * (size_t)nterms;
    for (int t = tid; t < nterms; t += kS2Threads) {
        double v = 0.0;
        for (int64_t u = 0; u < nt; ++u) v += src[(size_t)u * nterms + t];
        if (t < 2 * K) CT[t] = v; else M[t - 2 * K] = v;
    }
    __syncthreads();
    if (a.nbp == 3)
        finish_triples(a, row, ps, CT, M, reinterpret_cast<double*>(smem_raw + off[3]),
                       reinterpret_cast<int*>(smem_raw + off[4]), red_val, red_idx);
    else
        finish_pairs(a, row, ps, CT, M, red_val, red_idx);
}

size_t search2_workspace_bytes(int64_t C, int64_t max_n, int K) {
    const int64_t tiles = (max_n + kSearchTile - 1) / kSearchTile;
    size_t bytes = 256;
    if (tiles > 1)
        bytes += sizeof(double) * (size_t)C * (size_t)tiles * (size_t)(2 * K + K * (K - 1) / 2);
    return (bytes + 255) / 256 * 256;
}

cudaError_t launch_search2(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                           int64_t max_n, int bits, const float* ratios, int K, const float* m,
                           int nbp, float* const* p_out, int32_t* const* idx_out, int out_stride,
                           float* err_out, float* sse_out, void* workspace, cudaStream_t stream) {
    cudaError_t e = cudaMemsetAsync(workspace, 0, 256, stream);          // status word
    if (e != cudaSuccess) return e;
    Search2Args a;
    a.x = x;
    a.rows = Rows{row_offsets, C, n, n > 0 ? 1.0 / (double)n : 0.0, 0};
    a.m = m;
    a.ratios = ratios;
    a.K = K;
    a.levels = (1 << (bits - 1)) - 1;
    a.nbp = nbp;
    a.tiles = (max_n + kSearchTile - 1) / kSearchTile;
    a.cap = a.tiles > 1 ? kSearchTile : (int)((max_n + 3) / 4 * 4);
    a.partials = reinterpret_cast<double*>(static_cast<unsigned char*>(workspace) + 256);
    for (int t = 0; t < 3; ++t) {
        a.p_out[t] = t < nbp ? p_out[t] : nullptr;
        a.idx_out[t] = t < nbp ? idx_out[t] : nullptr;
    }
    a.out_stride = out_stride;
    a.err_out = err_out;
    a.sse_out = sse_out;
    a.status = static_cast<int*>(workspace);
    size_t off[9];
    const size_t smem = search2_smem(a.cap, K, off);
    if (smem > 48 * 1024) {
        e = cudaFuncSetAttribute(search2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem);
        if (e != cudaSuccess) return e;
    }
    search2_kernel<<<(unsigned)(C * a.tiles), kS2Threads, smem, stream>>>(a);
    e = cudaGetLastError();
    if (e != cudaSuccess || a.tiles == 1) return e;
    size_t foff[5];
    search2_finish_kernel<<<(unsigned)C, kS2Threads, finish2_smem(K, foff), stream>>>(a);
    return cudaGetLastError();
}

// ------------------------------------------------ quantize / dequantize, three or four regions
constexpr int kQ2Threads = 256;
constexpr int kQ2PerThread = 16;      // consecutive values per thread: four region bytes

template <bool PACKED, bool WANT_FAKE>
__global__ void __launch_bounds__(kQ2Threads)
quantize2_kernel(const float* __restrict__ x, Rows rows, int64_t total, int bits,
                 const float* __restrict__ m_arr, BreakPts bp, uint8_t* __restrict__ codes,
                 uint8_t* __restrict__ region2, float* __restrict__ fake, int vec_ok) {
    const int64_t i0 = ((int64_t)blockIdx.x * kQ2Threads + threadIdx.x) * kQ2PerThread;
    Row3 rs;
    rs.bracket(rows, i0 - (int64_t)(threadIdx.x & 31) * kQ2PerThread, 32 * kQ2PerThread, total);
    if (i0 >= total) return;
    const float Lf = (float)((1 << (bits - 1)) - 1);
    const int cnt = (int)min((int64_t)kQ2PerThread, total - i0);
    uint32_t code[kQ2PerThread], reg[kQ2PerThread];
    // whole groups of 16 with aligned buffers: 128-bit loads, one store per output
    const bool vec = cnt == kQ2PerThread && vec_ok;
    float xv[kQ2PerThread], yv[kQ2PerThread];
    if (vec) {
#pragma unroll
        for (int v = 0; v < kQ2PerThread / 4; ++v) {
            const float4 q = __ldcs(reinterpret_cast<const float4*>(x + i0) + v);
            xv[4 * v] = q.x; xv[4 * v + 1] = q.y; xv[4 * v + 2] = q.z; xv[4 * v + 3] = q.w;
        }
    }
#pragma unroll
    for (int t = 0; t < kQ2PerThread; ++t) {
        code[t] = reg[t] = 0;
        yv[t] = 0.0f;
        if (t < cnt) {
            rs.seek(rows, m_arr, bp, Lf, i0 + t);
            const float xi = vec ? xv[t] : x[i0 + t];
            float y = 0.0f;
            if (rs.m > 0.0f) {
                const float a = fminf(fabsf(xi), rs.m);
                const int r = (a > rs.P.z[1]) + (a > rs.P.z[2]) + (a > rs.P.z[3]);
                const float z = r == 0 ? 0.0f : (r == 1 ? rs.P.z[1] : (r == 2 ? rs.P.z[2] : rs.P.z[3]));
                const float inv = r == 0 ? rs.P.inv[0] : (r == 1 ? rs.P.inv[1] : (r == 2 ? rs.P.inv[2] : rs.P.inv[3]));
                const float s = r == 0 ? rs.P.s[0] : (r == 1 ? rs.P.s[1] : (r == 2 ? rs.P.s[2] : rs.P.s[3]));
                const float rr = __fadd_rn(__fmul_rn(__fsub_rn(a, z), inv), kMagic2);
                const float q = fminf(__fsub_rn(rr, kMagic2), Lf);
                const float v = __fadd_rn(__fmul_rn(q, s), z);
                const int neg = xi < 0.0f;
                code[t] = (uint32_t)((neg << (bits - 1)) | (int)q);
                reg[t] = (uint32_t)r;
                y = neg ? -v : v;
            }
            yv[t] = y;
            if (WANT_FAKE && !vec) fake[i0 + t] = y;
        }
    }
    // i0 is a multiple of 16: region bytes i0/4 .. i0/4 + 3, code bytes i0 .. (or i0/2 ..)
    if (vec) {
        uint32_t rw = 0;
#pragma unroll
        for (int t = 0; t < kQ2PerThread; ++t) rw |= reg[t] << (2 * t);
        *reinterpret_cast<uint32_t*>(region2 + (i0 >> 2)) = rw;
        if (PACKED) {
            uint32_t w0 = 0, w1 = 0;
#pragma unroll
            for (int t = 0; t < 8; ++t) { w0 |= code[t] << (4 * t); w1 |= code[8 + t] << (4 * t); }
            *reinterpret_cast<uint2*>(codes + (i0 >> 1)) = make_uint2(w0, w1);
        } else {
            uint32_t w[4] = {0, 0, 0, 0};
#pragma unroll
            for (int t = 0; t < kQ2PerThread; ++t) w[t >> 2] |= code[t] << (8 * (t & 3));
            *reinterpret_cast<uint4*>(codes + i0) = make_uint4(w[0], w[1], w[2], w[3]);
        }
        if (WANT_FAKE) {
#pragma unroll
            for (int v = 0; v < kQ2PerThread / 4; ++v)
                __stcs(reinterpret_cast<float4*>(fake + i0) + v,
                       make_float4(yv[4 * v], yv[4 * v + 1], yv[4 * v + 2], yv[4 * v + 3]));
        }
        return;
    }
#pragma unroll
    for (int b = 0; b < 4; ++b)
        if (4 * b < cnt)
            region2[(i0 >> 2) + b] = (uint8_t)(reg[4 * b] | (reg[4 * b + 1] << 2) |
                                               (reg[4 * b + 2] << 4) | (reg[4 * b + 3] << 6));
    if (PACKED) {
#pragma unroll
        for (int b = 0; b < 8; ++b)
            if (2 * b < cnt) codes[(i0 >> 1) + b] = (uint8_t)(code[2 * b] | (code[2 * b + 1] << 4));
    } else {
#pragma unroll
        for (int t = 0; t < kQ2PerThread; ++t)
            if (t < cnt) codes[i0 + t] = (uint8_t)code[t];
    }
}

template <bool PACKED>
__global__ void __launch_bounds__(kQ2Threads)
dequantize2_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ region2,
                   Rows rows, int64_t total, int bits, const float* __restrict__ m_arr,
                   BreakPts bp, float* __restrict__ y, int vec_ok) {
    const int64_t i0 = ((int64_t)blockIdx.x * kQ2Threads + threadIdx.x) * kQ2PerThread;
    Row3 rs;
    rs.bracket(rows, i0 - (int64_t)(threadIdx.x & 31) * kQ2PerThread, 32 * kQ2PerThread, total);
    if (i0 >= total) return;
    const float Lf = (float)((1 << (bits - 1)) - 1);
    const int qmask = (1 << (bits - 1)) - 1;
    const int cnt = (int)min((int64_t)kQ2PerThread, total - i0);
    // whole groups of 16 with aligned buffers: one load per input, 128-bit stores
    const bool vec = cnt == kQ2PerThread && vec_ok;
    uint32_t cw[4] = {0, 0, 0, 0}, rw = 0;
    float yv[kQ2PerThread];
    if (vec) {
        rw = __ldcs(reinterpret_cast<const unsigned int*>(region2 + (i0 >> 2)));
        if (PACKED) {
            const uint2 q = __ldcs(reinterpret_cast<const uint2*>(codes + (i0 >> 1)));
            cw[0] = q.x; cw[1] = q.y;
        } else {
            const uint4 q = __ldcs(reinterpret_cast<const uint4*>(codes + i0));
            cw[0] = q.x; cw[1] = q.y; cw[2] = q.z; cw[3] = q.w;
        }
    }
#pragma unroll
    for (int t = 0; t < kQ2PerThread; ++t) {
        yv[t] = 0.0f;
        if (t < cnt) {
            rs.seek(rows, m_arr, bp, Lf, i0 + t);
            const int64_t i = i0 + t;
            int code, r;
            if (vec) {
                code = PACKED ? (int)((cw[t >> 3] >> (4 * (t & 7))) & 0xFu)
                              : (int)((cw[t >> 2] >> (8 * (t & 3))) & 0xFFu);
                r = (int)((rw >> (2 * t)) & 3u);
            } else {
                code = PACKED ? ((codes[i >> 1] >> ((i & 1) * 4)) & 0xF) : codes[i];
                r = (region2[i >> 2] >> ((i & 3) * 2)) & 3;
            }
            r = min(r, bp.p3 ? 3 : 2);
            const float s = r == 0 ? rs.P.s[0] : (r == 1 ? rs.P.s[1] : (r == 2 ? rs.P.s[2] : rs.P.s[3]));
            const float z = r == 0 ? 0.0f : (r == 1 ? rs.P.z[1] : (r == 2 ? rs.P.z[2] : rs.P.z[3]));
            float v = __fadd_rn(__fmul_rn((float)(code & qmask), s), z);
            int neg = (code >> (bits - 1)) & 1;
            if (!(rs.m > 0.0f)) { v = 0.0f; neg = 0; }
            yv[t] = neg ? -v : v;
            if (!vec) y[i] = yv[t];
        }
    }
    if (vec) {
#pragma unroll
        for (int v = 0; v < kQ2PerThread / 4; ++v)
            __stcs(reinterpret_cast<float4*>(y + i0) + v,
                   make_float4(yv[4 * v], yv[4 * v + 1], yv[4 * v + 2], yv[4 * v + 3]));
    }
}

cudaError_t launch_quantize2_plain(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                             int64_t total, int bits, const float* m, const float* p1,
                             const float* p2, const float* p3, int p_stride, uint8_t* codes,
                             uint8_t* region2, float* fake, int layout, cudaStream_t stream) {
    if (total == 0) return cudaSuccess;
    const BreakPts bp{p1, p2, p3, p_stride};
    Rows rows{row_offsets, C, n, n > 0 ? 1.0 / (double)n : 0.0, 0};
    const bool packed = (layout == 1 && bits <= 4);
    const int64_t per_cta = (int64_t)kQ2Threads * kQ2PerThread;
    const unsigned grid = (unsigned)((total + per_cta - 1) / per_cta);
    auto al = [](const void* q, size_t a) { return (reinterpret_cast<uintptr_t>(q) & (a - 1)) == 0; };
    const int vec_ok = al(x, 16) && al(codes, 16) && al(region2, 4) && (!fake || al(fake, 16));
    if (packed) {
        if (fake) quantize2_kernel<true, true><<<grid, kQ2Threads, 0, stream>>>(x, rows, total, bits, m, bp, codes, region2, fake, vec_ok);
        else      quantize2_kernel<true, false><<<grid, kQ2Threads, 0, stream>>>(x, rows, total, bits, m, bp, codes, region2, fake, vec_ok);
    } else {
        if (fake) quantize2_kernel<false, true><<<grid, kQ2Threads, 0, stream>>>(x, rows, total, bits, m, bp, codes, region2, fake, vec_ok);
        else      quantize2_kernel<false, false><<<grid, kQ2Threads, 0, stream>>>(x, rows, total, bits, m, bp, codes, region2, fake, vec_ok);
    }
    return cudaGetLastError();
}

cudaError_t launch_dequantize2_plain(const uint8_t* codes, const uint8_t* region2,
                               const int64_t* row_offsets, int64_t C, int64_t n, int64_t total,
                               int bits, const float* m, const float* p1, const float* p2,
                               const float* p3, int p_stride, float* y, int layout,
                               cudaStream_t stream) {
    if (total == 0) return cudaSuccess;
    const BreakPts bp{p1, p2, p3, p_stride};
    Rows rows{row_offsets, C, n, n > 0 ? 1.0 / (double)n : 0.0, 0};
    const bool packed = (layout == 1 && bits <= 4);
    const int64_t per_cta = (int64_t)kQ2Threads * kQ2PerThread;
    const unsigned grid = (unsigned)((total + per_cta - 1) / per_cta);
    auto al = [](const void* q, size_t a) { return (reinterpret_cast<uintptr_t>(q) & (a - 1)) == 0; };
    const int vec_ok = al(y, 16) && al(codes, 16) && al(region2, 4);
    if (packed) dequantize2_kernel<true><<<grid, kQ2Threads, 0, stream>>>(codes, region2, rows, total, bits, m, bp, y, vec_ok);
    else        dequantize2_kernel<false><<<grid, kQ2Threads, 0, stream>>>(codes, region2, rows, total, bits, m, bp, y, vec_ok);
    return cudaGetLastError();
}

}  // namespace pwlq
