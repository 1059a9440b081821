// Analytic breakpoint selection (Sec. 3.3, Sec. 5.1): the breakpoint that minimises the expected
// error of Eq. 5 under an assumed zero-mean Gaussian or Laplacian density, i.e. the root of the
// stationarity condition Eq. 9 on (0, m/2), or the closed-form approximation of Sec. 5.1.
//
// One streaming pass for the density's scale (sum of squares / of magnitudes per row, binary64,
// fixed order: per-thread strided sums, shuffle tree, shared-memory tree, then the tiles of a
// long row in ascending order), then O(1) work per row.  HBM-bound, 4 bytes per value.
#include <algorithm>

#include "pwlq_common.cuh"
#include "pwlq_kernels.h"

namespace pwlq {

constexpr int kSelThreads = 128;
constexpr int kSelTile = 8192;

// Eq. 9 in units of the density's scale: with t = p / scale and M = m / scale, and F0, f0 the CDF
// and PDF of the unit-scale density,
//     h(t) = 2 M F0(t) - 2 M + t - M (M - 2 t) f0(t),       h < 0 left of the root,
//     h'(t) = 1 + 4 M f0(t) - M (M - 2 t) f0'(t),           f0' = -t f0 (Gaussian), -f0 (Laplacian).
struct Eq9 {
    double M;
    bool laplace;
    __device__ __forceinline__ void eval(double t, double& h, double& dh) const {
        double F0, f0, df0;
        if (laplace) {
            const double e = exp(-t);
            F0 = 1.0 - 0.5 * e;
            f0 = 0.5 * e;
            df0 = -f0;
        } else {
            F0 = 0.5 * erfc(t * -0.70710678118654752);          // -t / sqrt(2)
            f0 = 0.39894228040143268 * exp(-0.5 * t * t);         // 1 / sqrt(2 pi)
            df0 = -t * f0;
        }
        const double w = M * (M - 2.0 * t);
        h = 2.0 * M * (F0 - 1.0) + t - w * f0;
        dh = 1.0 + 4.0 * M * f0 - w * df0;
    }
};

// Root of Eq. 9 on (0, M/2) by Newton's iteration kept inside a shrinking bracket (a step that
// leaves the bracket, or does not at least halve it, is replaced by the bracket's midpoint).
// Returns M/2 when h(M/2) <= 0 (no sign change inside: the row is flatter than the model).
__device__ double eq9_root(double M, bool laplace) {
    const Eq9 g{M, laplace};
    double a = 0.0, b = 0.5 * M, h, dh;
    g.eval(b, h, dh);
    if (!(h > 0.0)) return b;
    double t = 0.5 * b, width = b - a;
    for (int it = 0; it < 200; ++it) {
        g.eval(t, h, dh);
        if (h < 0.0) a = t; else b = t;
        if (h == 0.0) break;
        double next = t - h / dh;
        const double new_width = b - a;
        if (!(next > a && next < b) || 2.0 * new_width > width) next = 0.5 * (a + b);
        width = new_width;
        if (fabs(next - t) <= 4e-16 * t || new_width <= 4e-16 * b) { t = next; break; }
        t = next;
    }
    return t;
}

// model 0: Gaussian closed form p = sigma ln(0.8614 m / sigma + 0.6079) (Sec. 5.1, m and p in units
// of sigma); 1: Gaussian root of Eq. 9; 2: Laplacian root of Eq. 9.  Result in (0, m/2]: m/2 when
// Eq. 9 has no root there, and m/2 * 1e-6 when the closed form's logarithm is not positive.
__device__ double analytic_breakpoint(double m, double scale, int model) {
    if (!(m > 0.0) || !(scale > 0.0)) return 0.0;
    const double M = m / scale;
    const double t = (model == 0) ? log(0.8614 * M + 0.6079) : eq9_root(M, model == 2);
    double p = t * scale;
    if (!(p > 0.0)) p = 0.5 * m * 1e-6;
    if (p > 0.5 * m) p = 0.5 * m;
    return p;
}

__device__ __forceinline__ void finish_row(int64_t row, int64_t n_row, double s2, double s1,
                                           const float* __restrict__ m, int model,
                                           float* __restrict__ p_out, float* __restrict__ scale_out) {
    double scale = 0.0;
    if (n_row > 0) scale = (model == 2) ? s1 / (double)n_row : sqrt(s2 / (double)n_row);
    if (scale_out) scale_out[row] = (float)scale;
    p_out[row] = (float)analytic_breakpoint((double)m[row], scale, model);
}

// One CTA per (row, tile): sums of x^2 and |x| over the tile.  The breakpoint itself is left to
// select_finish_kernel, one thread per row: a Newton iteration in binary64 run by one thread of a
// CTA while the other 127 wait took ten times as long as the sums.
__global__ void __launch_bounds__(kSelThreads)
moments_kernel(const float* __restrict__ x, Rows rows, int64_t tiles, double* __restrict__ partial) {
    __shared__ double red[2][kSelThreads / 32];
    const int64_t row = blockIdx.x / tiles, tile = blockIdx.x - row * tiles;
    const int64_t beg = rows.begin(row), end = rows.begin(row + 1);
    const int64_t t_beg = beg + tile * kSelTile;
    const int64_t t_end = min(t_beg + kSelTile, end);
    double s2 = 0.0, s1 = 0.0;
    for (int64_t i = t_beg + threadIdx.x; i < t_end; i += kSelThreads) {
        const double v = (double)x[i];
        s2 += v * v;
        s1 += fabs(v);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        s2 += __shfl_xor_sync(0xffffffffu, s2, o);
        s1 += __shfl_xor_sync(0xffffffffu, s1, o);
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { red[0][warp] = s2; red[1][warp] = s1; }
    __syncthreads();
    if (threadIdx.x == 0) {
        s2 = red[0][0]; s1 = red[1][0];
        for (int w = 1; w < kSelThreads / 32; ++w) { s2 += red[0][w]; s1 += red[1][w]; }
        partial[2 * blockIdx.x] = s2;
        partial[2 * blockIdx.x + 1] = s1;
    }
}

// The tiles' sums of every row in ascending order, then the breakpoint.
__global__ void select_finish_kernel(Rows rows, int64_t tiles, const double* __restrict__ partial,
                                     const float* __restrict__ m, int model,
                                     float* __restrict__ p_out, float* __restrict__ scale_out) {
    const int64_t row = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= rows.C) return;
    const int64_t n_row = rows.begin(row + 1) - rows.begin(row);
    const int64_t nt = (n_row + kSelTile - 1) / kSelTile;
    double s2 = 0.0, s1 = 0.0;
    for (int64_t t = 0; t < nt; ++t) {
        s2 += partial[2 * (row * tiles + t)];
        s1 += partial[2 * (row * tiles + t) + 1];
    }
    finish_row(row, n_row, s2, s1, m, model, p_out, scale_out);
}

size_t select_workspace_bytes(int64_t C, int64_t max_n) {
    const int64_t tiles = (max_n + kSelTile - 1) / kSelTile;
    return (size_t)(16 * C * tiles + 255) / 256 * 256;
}

cudaError_t launch_select_analytic(const float* x, const int64_t* row_offsets, int64_t C,
                                   int64_t n, int64_t max_n, const float* m, int model,
                                   float* p_out, float* scale_out, void* workspace,
                                   cudaStream_t stream) {
    Rows rows{row_offsets, C, n, n > 0 ? 1.0 / (double)n : 0.0, 0};
    const int64_t tiles = std::max<int64_t>(1, (max_n + kSelTile - 1) / kSelTile);
    double* partial = static_cast<double*>(workspace);
    moments_kernel<<<(unsigned)(C * tiles), kSelThreads, 0, stream>>>(x, rows, tiles, partial);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    select_finish_kernel<<<(unsigned)((C + 127) / 128), 128, 0, stream>>>(rows, tiles, partial, m,
                                                                          model, p_out, scale_out);
    return cudaGetLastError();
}

}  // namespace pwlq
