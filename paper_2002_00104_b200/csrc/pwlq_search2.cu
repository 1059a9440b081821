// Two breakpoints (Sec. 5.1, "Multiple Breakpoints"): regions [0, p1], (p1, p2], (p2, m], each
// quantized like the regions of Eq. 3; search over all pairs i < j of a grid of K ratios.
//
// The squared error of a pair splits by region:
//     SSE(i, j) = C_i + M_ij + T_j
//     C_i  = error of the values a <= p_i        quantized on [0, p_i]
//     M_ij = error of the values p_i < a <= p_j  quantized on [p_i, p_j]
//     T_j  = error of the values a > p_j         quantized on [p_j, m]
// One CTA per row: the row's magnitudes are counting-sorted by candidate interval into shared
// memory (deterministic placement), after which every term is a sum over a contiguous range of
// the sorted tile.  A warp takes one term at a time, its lanes stride over the range (per value
// the operation-by-operation sequence of Eq. 1, no fused multiply-add), and the lane sums are
// added in binary64 in a fixed order.  Work per row: the honest evaluation of every (value, pair)
// of the pair's middle region plus 2 K passes for the C and T terms.
#include <algorithm>

#include "pwlq_common.cuh"
#include "pwlq_kernels.h"

namespace pwlq {

constexpr int kS2Threads = 256;
constexpr int kS2Warps = kS2Threads / 32;
constexpr int kS2HistStride = 258;          // u16 entries per bucket row (256 threads + padding)
constexpr float kMagic2 = 12582912.0f;      // 1.5 * 2^23

struct Search2Args {
    const float* x;
    Rows rows;
    const float* m;
    const float* ratios;
    int K;
    int levels;
    int cap;              // tile capacity in values
    float* p1_out;
    float* p2_out;
    float* err_out;
    int32_t* idx1_out;
    int32_t* idx2_out;
    float* sse_pairs;     // [C, K, K] or nullptr
    int* status;
};

__host__ __device__ inline size_t s2_align(size_t v) { return (v + 15) & ~(size_t)15; }

// Shared-memory layout: sorted tile | bucket+rank per value | breakpoints | bucket starts |
// per-thread bucket counts | C, T | M (triangular).
__host__ __device__ inline size_t search2_smem(int cap, int K, size_t* off) {
    size_t o = 0;
    off[0] = o; o = s2_align(o + sizeof(float) * (size_t)cap);
    off[1] = o; o = s2_align(o + sizeof(uint16_t) * (size_t)cap);
    off[2] = o; o = s2_align(o + sizeof(float) * (size_t)K);
    off[3] = o; o = s2_align(o + sizeof(int) * (size_t)(K + 2));
    off[4] = o; o = s2_align(o + sizeof(uint16_t) * (size_t)(K + 1) * kS2HistStride);
    off[5] = o; o = s2_align(o + sizeof(double) * (size_t)(2 * K));
    off[6] = o; o = s2_align(o + sizeof(double) * (size_t)(K * (K - 1) / 2));
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

__device__ __forceinline__ void write_degenerate2(const Search2Args& a, int64_t row) {
    if (threadIdx.x == 0) {
        a.idx1_out[row] = 0;
        a.idx2_out[row] = 1;
        a.p1_out[row] = 0.0f;
        a.p2_out[row] = 0.0f;
        if (a.err_out) a.err_out[row] = 0.0f;
    }
    if (a.sse_pairs)
        for (int t = threadIdx.x; t < a.K * a.K; t += kS2Threads)
            a.sse_pairs[row * a.K * a.K + t] = 0.0f;
}

__global__ void __launch_bounds__(kS2Threads)
search2_kernel(Search2Args a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ double red_val[kS2Warps];
    __shared__ int red_idx[kS2Warps];
    const int64_t row = blockIdx.x;
    const int64_t beg = a.rows.begin(row), end = a.rows.begin(row + 1);
    const int cnt = (int)(end - beg);
    const int K = a.K;
    const float m = a.m[row];
    const float Lf = (float)a.levels;
    const bool finite = (__float_as_uint(m) & 0x7fffffffu) < 0x7f800000u;
    if (!finite || !(m > 0.0f) || cnt <= 0) {
        if (!finite && threadIdx.x == 0) atomicOr(a.status, kStatusNonFinite);
        write_degenerate2(a, row);
        return;
    }
    size_t off[7];
    search2_smem(a.cap, K, off);
    float* tile = reinterpret_cast<float*>(smem_raw + off[0]);
    uint16_t* jr = reinterpret_cast<uint16_t*>(smem_raw + off[1]);
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
    for (int t = tid; t < (K + 1) * kS2HistStride; t += kS2Threads) hist[t] = 0;
    if (__syncthreads_or(unordered)) {               // the pair search needs an ascending grid
        if (tid == 0) atomicOr(a.status, kStatusBadGrid);
        write_degenerate2(a, row);
        return;
    }

    // pass 1: bucket j = #{k : p_k < a} and the value's rank among this thread's values of the
    // bucket (a thread takes values tid, tid + 256, ...: at most 32 of them)
    for (int i = tid; i < cnt; i += kS2Threads) {
        const float v = fminf(fabsf(__ldg(a.x + beg + i)), m);
        int lo = 0, hi = K;                           // p_k < v for k < lo; p_k >= v for k >= hi
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (ps[mid] < v) lo = mid + 1; else hi = mid;
        }
        const int rank = hist[lo * kS2HistStride + tid]++;
        jr[i] = (uint16_t)(lo | (rank << 7));
    }
    __syncthreads();
    // bucket totals, exclusive scan over buckets, then per (bucket, thread) start positions
    if (tid <= K) {
        int tot = 0;
        for (int t = 0; t < kS2Threads; ++t) tot += hist[tid * kS2HistStride + t];
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
        for (int t = 0; t < kS2Threads; ++t) {
            const int c = hist[tid * kS2HistStride + t];
            hist[tid * kS2HistStride + t] = (uint16_t)run;
            run += c;
        }
    }
    __syncthreads();
    // pass 2: placement (bucket, then thread, then the thread's own order): deterministic
    for (int i = tid; i < cnt; i += kS2Threads) {
        const int j = jr[i] & 0x7f, rank = jr[i] >> 7;
        tile[hist[j * kS2HistStride + tid] + rank] = fminf(fabsf(__ldg(a.x + beg + i)), m);
    }
    __syncthreads();

    // evaluation: values <= p_k are the first B_k = start[k + 1] entries of the sorted tile
    for (int k = warp; k < 2 * K; k += kS2Warps) {
        double d;
        if (k < K) d = range_error(tile, 0, start[k + 1], 0.0f, ps[k], Lf);
        else       d = range_error(tile, start[k - K + 1], cnt, ps[k - K], __fsub_rn(m, ps[k - K]), Lf);
        if (lane == 0) CT[k] = d;
    }
    for (int i = 0; i < K - 1; ++i) {
        const float pi = ps[i];
        const int bi = start[i + 1];
        for (int j = i + 1 + warp; j < K; j += kS2Warps) {
            const double d = range_error(tile, bi, start[j + 1], pi, __fsub_rn(ps[j], pi), Lf);
            if (lane == 0) M[pair_index(i, j, K)] = d;
        }
    }
    __syncthreads();

    // totals and the first minimal pair in the order (i, j)
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
    if (tid == 0) {
        for (int w = 1; w < kS2Warps; ++w) {
            const double ov = red_val[w];
            const int oi = red_idx[w];
            if (oi != 0x7fffffff && (best_idx == 0x7fffffff || ov < best || (ov == best && oi < best_idx))) {
                best = ov; best_idx = oi;
            }
        }
        int i = 0, base = 0;
        while (best_idx >= base + (K - 1 - i)) { base += K - 1 - i; ++i; }
        const int j = i + 1 + (best_idx - base);
        a.idx1_out[row] = i;
        a.idx2_out[row] = j;
        a.p1_out[row] = ps[i];
        a.p2_out[row] = ps[j];
        if (a.err_out) a.err_out[row] = (float)best;
    }
    if (a.sse_pairs) {
        float* dst = a.sse_pairs + row * K * K;
        for (int t = tid; t < K * K; t += kS2Threads) {
            const int i = t / K, j = t - i * K;
            dst[t] = (i < j) ? (float)M[pair_index(i, j, K)] : 0.0f;
        }
    }
}

cudaError_t launch_search2(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                           int64_t max_n, int bits, const float* ratios, int K, const float* m,
                           float* p1_out, float* p2_out, float* err_out, int32_t* idx1_out,
                           int32_t* idx2_out, float* sse_pairs, void* workspace,
                           cudaStream_t stream) {
    cudaError_t e = cudaMemsetAsync(workspace, 0, 256, stream);          // status word
    if (e != cudaSuccess) return e;
    Search2Args a;
    a.x = x;
    a.rows = Rows{row_offsets, C, n, n > 0 ? 1.0 / (double)n : 0.0};
    a.m = m;
    a.ratios = ratios;
    a.K = K;
    a.levels = (1 << (bits - 1)) - 1;
    a.cap = (int)((max_n + 3) / 4 * 4);
    a.p1_out = p1_out;
    a.p2_out = p2_out;
    a.err_out = err_out;
    a.idx1_out = idx1_out;
    a.idx2_out = idx2_out;
    a.sse_pairs = sse_pairs;
    a.status = static_cast<int*>(workspace);
    size_t off[7];
    const size_t smem = search2_smem(a.cap, K, off);
    if (smem > 48 * 1024) {
        e = cudaFuncSetAttribute(search2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem);
        if (e != cudaSuccess) return e;
    }
    search2_kernel<<<(unsigned)C, kS2Threads, smem, stream>>>(a);
    return cudaGetLastError();
}

// ------------------------------------------------------------- quantize / dequantize, 3 regions
// Constants of the three regions of one row.
struct Params3 {
    float z[3], s[3], inv[3];
};
__device__ __forceinline__ Params3 make_params3(float m, float p1, float p2, float Lf) {
    Params3 P;
    P.z[0] = 0.0f; P.z[1] = p1; P.z[2] = p2;
    const float d[3] = {p1, __fsub_rn(p2, p1), __fsub_rn(m, p2)};
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        if (d[r] > 0.0f) { P.s[r] = __fdiv_rn(d[r], Lf); P.inv[r] = __fdiv_rn(Lf, d[r]); }
        else             { P.s[r] = 0.0f;                P.inv[r] = 0.0f; }
    }
    return P;
}

constexpr int kQ2Threads = 256;
constexpr int kQ2PerThread = 16;      // consecutive values per thread: four region bytes

// Row state of a thread that walks consecutive values.
struct Row3 {
    int64_t row = -1, end = 0;
    float m = 0.0f;
    Params3 P;
    __device__ __forceinline__ void seek(const Rows& rows, const float* m_arr, const float* p1,
                                         const float* p2, float Lf, int64_t i) {
        if (row >= 0 && i < end) return;
        row = (row < 0) ? rows.row_of(i) : row + 1;
        while (rows.begin(row + 1) <= i) ++row;              // skips empty rows
        end = rows.begin(row + 1);
        m = __ldg(m_arr + row);
        P = make_params3(m, __ldg(p1 + row), __ldg(p2 + row), Lf);
    }
};

template <bool PACKED, bool WANT_FAKE>
__global__ void __launch_bounds__(kQ2Threads)
quantize2_kernel(const float* __restrict__ x, Rows rows, int64_t total, int bits,
                 const float* __restrict__ m_arr, const float* __restrict__ p1_arr,
                 const float* __restrict__ p2_arr, uint8_t* __restrict__ codes,
                 uint8_t* __restrict__ region2, float* __restrict__ fake) {
    const int64_t i0 = ((int64_t)blockIdx.x * kQ2Threads + threadIdx.x) * kQ2PerThread;
    if (i0 >= total) return;
    const float Lf = (float)((1 << (bits - 1)) - 1);
    const int cnt = (int)min((int64_t)kQ2PerThread, total - i0);
    Row3 rs;
    uint32_t code[kQ2PerThread], reg[kQ2PerThread];
#pragma unroll
    for (int t = 0; t < kQ2PerThread; ++t) {
        code[t] = reg[t] = 0;
        if (t < cnt) {
            rs.seek(rows, m_arr, p1_arr, p2_arr, Lf, i0 + t);
            const float xi = x[i0 + t];
            float y = 0.0f;
            if (rs.m > 0.0f) {
                const float a = fminf(fabsf(xi), rs.m);
                const int r = (a > rs.P.z[1]) + (a > rs.P.z[2]);
                const float z = r == 0 ? 0.0f : (r == 1 ? rs.P.z[1] : rs.P.z[2]);
                const float inv = r == 0 ? rs.P.inv[0] : (r == 1 ? rs.P.inv[1] : rs.P.inv[2]);
                const float s = r == 0 ? rs.P.s[0] : (r == 1 ? rs.P.s[1] : rs.P.s[2]);
                const float rr = __fadd_rn(__fmul_rn(__fsub_rn(a, z), inv), kMagic2);
                const float q = fminf(__fsub_rn(rr, kMagic2), Lf);
                const float v = __fadd_rn(__fmul_rn(q, s), z);
                const int neg = xi < 0.0f;
                code[t] = (uint32_t)((neg << (bits - 1)) | (int)q);
                reg[t] = (uint32_t)r;
                y = neg ? -v : v;
            }
            if (WANT_FAKE) fake[i0 + t] = y;
        }
    }
    // i0 is a multiple of 16: region bytes i0/4 .. i0/4 + 3, code bytes i0 .. (or i0/2 ..)
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
                   const float* __restrict__ p1_arr, const float* __restrict__ p2_arr,
                   float* __restrict__ y) {
    const int64_t i0 = ((int64_t)blockIdx.x * kQ2Threads + threadIdx.x) * kQ2PerThread;
    if (i0 >= total) return;
    const float Lf = (float)((1 << (bits - 1)) - 1);
    const int qmask = (1 << (bits - 1)) - 1;
    const int cnt = (int)min((int64_t)kQ2PerThread, total - i0);
    Row3 rs;
#pragma unroll
    for (int t = 0; t < kQ2PerThread; ++t) {
        if (t < cnt) {
            rs.seek(rows, m_arr, p1_arr, p2_arr, Lf, i0 + t);
            const int64_t i = i0 + t;
            const int code = PACKED ? ((codes[i >> 1] >> ((i & 1) * 4)) & 0xF) : codes[i];
            int r = (region2[i >> 2] >> ((i & 3) * 2)) & 3;
            r = min(r, 2);
            const float s = r == 0 ? rs.P.s[0] : (r == 1 ? rs.P.s[1] : rs.P.s[2]);
            const float z = r == 0 ? 0.0f : (r == 1 ? rs.P.z[1] : rs.P.z[2]);
            float v = __fadd_rn(__fmul_rn((float)(code & qmask), s), z);
            int neg = (code >> (bits - 1)) & 1;
            if (!(rs.m > 0.0f)) { v = 0.0f; neg = 0; }
            y[i] = neg ? -v : v;
        }
    }
}

cudaError_t launch_quantize2(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                             int64_t total, int bits, const float* m, const float* p1,
                             const float* p2, uint8_t* codes, uint8_t* region2, float* fake,
                             int layout, cudaStream_t stream) {
    if (total == 0) return cudaSuccess;
    Rows rows{row_offsets, C, n, n > 0 ? 1.0 / (double)n : 0.0};
    const bool packed = (layout == 1 && bits <= 4);
    const int64_t per_cta = (int64_t)kQ2Threads * kQ2PerThread;
    const unsigned grid = (unsigned)((total + per_cta - 1) / per_cta);
    if (packed) {
        if (fake) quantize2_kernel<true, true><<<grid, kQ2Threads, 0, stream>>>(x, rows, total, bits, m, p1, p2, codes, region2, fake);
        else      quantize2_kernel<true, false><<<grid, kQ2Threads, 0, stream>>>(x, rows, total, bits, m, p1, p2, codes, region2, fake);
    } else {
        if (fake) quantize2_kernel<false, true><<<grid, kQ2Threads, 0, stream>>>(x, rows, total, bits, m, p1, p2, codes, region2, fake);
        else      quantize2_kernel<false, false><<<grid, kQ2Threads, 0, stream>>>(x, rows, total, bits, m, p1, p2, codes, region2, fake);
    }
    return cudaGetLastError();
}

cudaError_t launch_dequantize2(const uint8_t* codes, const uint8_t* region2,
                               const int64_t* row_offsets, int64_t C, int64_t n, int64_t total,
                               int bits, const float* m, const float* p1, const float* p2,
                               float* y, int layout, cudaStream_t stream) {
    if (total == 0) return cudaSuccess;
    Rows rows{row_offsets, C, n, n > 0 ? 1.0 / (double)n : 0.0};
    const bool packed = (layout == 1 && bits <= 4);
    const int64_t per_cta = (int64_t)kQ2Threads * kQ2PerThread;
    const unsigned grid = (unsigned)((total + per_cta - 1) / per_cta);
    if (packed) dequantize2_kernel<true><<<grid, kQ2Threads, 0, stream>>>(codes, region2, rows, total, bits, m, p1, p2, y);
    else        dequantize2_kernel<false><<<grid, kQ2Threads, 0, stream>>>(codes, region2, rows, total, bits, m, p1, p2, y);
    return cudaGetLastError();
}

}  // namespace pwlq
