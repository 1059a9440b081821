// Breakpoint search: for every row and each of K candidate breakpoints p_k = m * ratio_k,
// SSE_k = sum_i (pw(x_i; b, m, p_k) - x_i)^2 with the quantizer of Eq. 3, then the first minimal
// k (grid form of Eq. 6).
//
// One CTA per (row, tile of at most kSearchTile values).  The tile's magnitudes are staged once
// in shared memory; every lane owns one candidate and walks the tile with 128-bit shared-memory
// broadcasts, so HBM is read once per value and no per-candidate cross-lane reduction exists.
// Sums run in binary32 over at most 256 terms per accumulator and are then carried in binary64,
// always in the same order.
#include "pwlq_common.cuh"
#include "pwlq_kernels.h"

namespace pwlq {

constexpr int kSThreads = 256;
constexpr int kSWarps = kSThreads / 32;
constexpr int kChunkVec = 256;   // float4 vectors per binary32 accumulation run

struct SearchArgs {
    const float* x;
    Rows rows;
    const float* m;
    const float* ratios;
    int K;
    int bits;
    int64_t tiles;
    double* partials;
    float* p_out;
    float* err_out;
    int32_t* idx_out;
    float* sse_all;
    int* status;
};

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

// Squared error of one magnitude under one candidate, operation by operation as in Eq. 1 / Eq. 3.
__device__ __forceinline__ float sq_err_acc(float a, const PieceParams& P, float acc) {
    const bool tail = a > P.p;
    const float z = tail ? P.p : 0.0f;
    const float inv = tail ? P.inv2 : P.inv1;
    const float s = tail ? P.s2 : P.s1;
    const float u = __fsub_rn(a, z);
    const float t = __fmul_rn(u, inv);
    const float q = rintf(t);                       // t <= L (1 + 2^-22): saturation cannot trigger
    float v = __fmul_rn(q, s);
    v = __fadd_rn(v, z);
    const float e = __fsub_rn(v, a);
    return __fmaf_rn(e, e, acc);
}

__global__ void __launch_bounds__(kSThreads)
search_kernel(SearchArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int64_t row = blockIdx.x / a.tiles;
    const int64_t tile = blockIdx.x - row * a.tiles;
    const int64_t beg = a.rows.begin(row), end = a.rows.begin(row + 1);
    const int64_t t_beg = beg + tile * kSearchTile;
    if (t_beg >= end && tile > 0) return;            // this row has fewer tiles than the longest
    const int cnt = (int)min((int64_t)kSearchTile, end - t_beg);
    const float m = a.m[row];
    const bool finite = __float_as_uint(m) < 0x7f800000u;
    if (!finite || !(m > 0.0f) || cnt <= 0) {
        if (!finite && threadIdx.x == 0 && tile == 0) atomicOr(a.status, kStatusNonFinite);
        if (a.tiles == 1) write_degenerate_row(a, row);
        return;                                      // tiles > 1: the combine kernel handles it
    }

    const int K = a.K;
    const int G = (K + 31) / 32;                     // candidate groups of one warp
    const int E = (G >= kSWarps) ? 1 : (kSWarps / G);  // element slices per group
    const int cnt4 = (cnt + 3) >> 2;

    float* tile_s = reinterpret_cast<float*>(smem_raw);                       // [cnt4 * 4]
    double* part = reinterpret_cast<double*>(smem_raw + (size_t)((kSearchTile * 4 + 15) & ~15));
    __shared__ double red_val[kSWarps];
    __shared__ int red_idx[kSWarps];

    for (int i = threadIdx.x; i < cnt4 * 4; i += kSThreads)
        tile_s[i] = (i < cnt) ? fminf(fabsf(a.x[t_beg + i]), m) : 0.0f;   // zero padding: error 0
    __syncthreads();

    const float Lf = (float)((1 << (a.bits - 1)) - 1);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float4* tile4 = reinterpret_cast<const float4*>(tile_s);
    for (int item = warp; item < G * E; item += kSWarps) {
        const int g = item % G, e = item / G;
        const int k = g * 32 + lane;
        const int lo = (int)((int64_t)cnt4 * e / E), hi = (int)((int64_t)cnt4 * (e + 1) / E);
        if (k < K) {
            const PieceParams P = make_params(m, __fmul_rn(m, a.ratios[k]), Lf);
            double dacc = 0.0;
            for (int base = lo; base < hi; base += kChunkVec) {
                const int stop = min(base + kChunkVec, hi);
                float a0 = 0.0f, a1 = 0.0f, a2 = 0.0f, a3 = 0.0f;
#pragma unroll 2
                for (int j = base; j < stop; ++j) {
                    const float4 v = tile4[j];
                    a0 = sq_err_acc(v.x, P, a0);
                    a1 = sq_err_acc(v.y, P, a1);
                    a2 = sq_err_acc(v.z, P, a2);
                    a3 = sq_err_acc(v.w, P, a3);
                }
                dacc += ((double)a0 + (double)a1) + ((double)a2 + (double)a3);
            }
            part[e * K + k] = dacc;
        }
    }
    __syncthreads();

    for (int k = threadIdx.x; k < K; k += kSThreads) {
        double tot = part[k];
        for (int e = 1; e < E; ++e) tot += part[e * K + k];
        if (a.tiles > 1) {
            a.partials[((size_t)row * a.tiles + tile) * K + k] = tot;
        } else {
            part[k] = tot;
            if (a.sse_all) a.sse_all[row * K + k] = (float)tot;
        }
    }
    if (a.tiles > 1) return;
    __syncthreads();
    double best; int idx;
    block_argmin(part, K, red_val, red_idx, best, idx);
    if (threadIdx.x == 0) write_row_result(a, row, m, best, idx);
}

// Combines the tiles of long rows in ascending tile order and takes the argmin.
__global__ void __launch_bounds__(kSThreads)
search_combine_kernel(SearchArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double* sse = reinterpret_cast<double*>(smem_raw);
    __shared__ double red_val[kSWarps];
    __shared__ int red_idx[kSWarps];
    const int64_t row = blockIdx.x;
    const int64_t n_row = a.rows.begin(row + 1) - a.rows.begin(row);
    const float m = a.m[row];
    const bool finite = __float_as_uint(m) < 0x7f800000u;
    if (!finite || !(m > 0.0f) || n_row <= 0) { write_degenerate_row(a, row); return; }
    const int64_t nt = (n_row + kSearchTile - 1) / kSearchTile;
    const int K = a.K;
    for (int k = threadIdx.x; k < K; k += kSThreads) {
        const double* src = a.partials + (size_t)row * a.tiles * K + k;
        double tot = 0.0;
        for (int64_t t = 0; t < nt; ++t) tot += src[(size_t)t * K];
        sse[k] = tot;
        if (a.sse_all) a.sse_all[row * K + k] = (float)tot;
    }
    __syncthreads();
    double best; int idx;
    block_argmin(sse, K, red_val, red_idx, best, idx);
    if (threadIdx.x == 0) write_row_result(a, row, m, best, idx);
}

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

SearchPlan plan_search(int64_t C, int64_t max_n, int K) {
    SearchPlan p;
    p.tiles = (max_n + kSearchTile - 1) / kSearchTile;
    if (p.tiles < 1) p.tiles = 1;
    p.off_m = 256;
    p.off_partials = align_up(p.off_m + sizeof(float) * (size_t)C, 256);
    p.bytes = p.off_partials;
    if (p.tiles > 1) p.bytes += sizeof(double) * (size_t)C * (size_t)p.tiles * (size_t)K;
    p.bytes = align_up(p.bytes, 256);
    return p;
}

static size_t search_smem_bytes(int K) {
    const int G = (K + 31) / 32;
    const int E = (G >= kSWarps) ? 1 : (kSWarps / G);
    return (size_t)((kSearchTile * 4 + 15) & ~15) + sizeof(double) * (size_t)E * (size_t)K;
}

cudaError_t launch_search(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                          int64_t total, int bits, const float* ratios, int K, const float* m,
                          float* p_out, float* err_out, int32_t* idx_out, float* sse_all,
                          void* workspace, const SearchPlan& plan, cudaStream_t stream) {
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    cudaError_t e = cudaMemsetAsync(ws, 0, 256, stream);          // status word
    if (e != cudaSuccess) return e;
    if (!m) {
        float* m_ws = reinterpret_cast<float*>(ws + plan.off_m);
        e = launch_absmax(x, row_offsets, C, n, total, m_ws, stream);
        if (e != cudaSuccess) return e;
        m = m_ws;
    }
    SearchArgs a;
    a.x = x;
    a.rows = Rows{row_offsets, C, n};
    a.m = m;
    a.ratios = ratios;
    a.K = K;
    a.bits = bits;
    a.tiles = plan.tiles;
    a.partials = reinterpret_cast<double*>(ws + plan.off_partials);
    a.p_out = p_out;
    a.err_out = err_out;
    a.idx_out = idx_out;
    a.sse_all = sse_all;
    a.status = reinterpret_cast<int*>(ws);

    const size_t smem = search_smem_bytes(K);
    if (smem > 48 * 1024) {          // above the default limit: opt in (idempotent, per device)
        e = cudaFuncSetAttribute(search_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem);
        if (e != cudaSuccess) return e;
    }
    const int64_t grid = C * plan.tiles;
    search_kernel<<<(unsigned)grid, kSThreads, smem, stream>>>(a);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (plan.tiles > 1) {
        search_combine_kernel<<<(unsigned)C, kSThreads, sizeof(double) * (size_t)K, stream>>>(a);
        e = cudaGetLastError();
    }
    return e;
}

}  // namespace pwlq
