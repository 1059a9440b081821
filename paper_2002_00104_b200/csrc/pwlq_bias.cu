// Bias correction (Sec. 5.1, "Bias Correction") and dense (b+1)-bit storage (Sec. 4: b bits per
// value plus one region bit).
//
// Bias correction: quantization shifts the mean and the variance of a row; the correction is
// folded into one scale xi and one offset beta per row,
//     xi   = sqrt( sum (x - mean x)^2 / sum (y - mean y)^2 ),   beta = mean x - xi * mean y,
// with y = pw(x) the quantizer's delivered value, so that xi * y + beta has the mean and the
// centred norm of x.  One streaming pass: sums of (x - x0), (y - y0) and their squares in binary64
// around a pivot (the row's first value and its quantized value), which keeps constant rows exact
// and the variance formula well conditioned; fixed summation order.
#include <algorithm>

#include "pwlq_common.cuh"
#include "pwlq_kernels.h"

namespace pwlq {

constexpr int kBcThreads = 128;
constexpr int kBcTile = 8192;

// Delivered value of the quantizer (Eq. 3) for one input.
__device__ __forceinline__ float fake_value(float x, float m, const PieceParams& P, float Lf) {
    if (!(m > 0.0f)) return 0.0f;
    int q, tail;
    float v;
    quantize_mag(fminf(fabsf(x), m), P, Lf, q, tail, v);
    return x < 0.0f ? -v : v;
}

__device__ __forceinline__ void finish_bias_row(int64_t row, int64_t n_row, double x0, double y0,
                                                const double s[4], float* __restrict__ xi_out,
                                                float* __restrict__ beta_out) {
    double xi = 1.0, beta = 0.0;
    if (n_row > 0) {
        const double n = (double)n_row;
        const double mx = x0 + s[0] / n, my = y0 + s[1] / n;
        const double vx = s[2] - s[0] * s[0] / n, vy = s[3] - s[1] * s[1] / n;
        if (vx > 0.0 && vy > 0.0) xi = sqrt(vx / vy);
        beta = mx - xi * my;
    }
    xi_out[row] = (float)xi;
    beta_out[row] = (float)beta;
}

// One CTA per (row, tile): sums of (x - x0), (y - y0), (x - x0)^2, (y - y0)^2 over the tile.
__global__ void __launch_bounds__(kBcThreads)
bias_moments_kernel(const float* __restrict__ x, Rows rows, int64_t tiles, int bits,
                    const float* __restrict__ m_arr, const float* __restrict__ p_arr,
                    double* __restrict__ partial, float* __restrict__ xi_out,
                    float* __restrict__ beta_out) {
    __shared__ double red[4][kBcThreads / 32];
    const int64_t row = blockIdx.x / tiles, tile = blockIdx.x - row * tiles;
    const int64_t beg = rows.begin(row), end = rows.begin(row + 1);
    const int64_t t_beg = beg + tile * kBcTile;
    const int64_t t_end = min(t_beg + kBcTile, end);
    const float Lf = (float)((1 << (bits - 1)) - 1);
    const float m = m_arr[row];
    const PieceParams P = make_params(m, p_arr[row], Lf);
    double x0 = 0.0, y0 = 0.0;
    if (end > beg) {
        const float xf = __ldg(x + beg);
        x0 = (double)xf;
        y0 = (double)fake_value(xf, m, P, Lf);
    }
    double s[4] = {0.0, 0.0, 0.0, 0.0};
    for (int64_t i = t_beg + threadIdx.x; i < t_end; i += kBcThreads) {
        const float xf = x[i];
        const double dx = (double)xf - x0;
        const double dy = (double)fake_value(xf, m, P, Lf) - y0;
        s[0] += dx; s[1] += dy; s[2] += dx * dx; s[3] += dy * dy;
    }
#pragma unroll
    for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s[k] += __shfl_xor_sync(0xffffffffu, s[k], o);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0)
        for (int k = 0; k < 4; ++k) red[k][warp] = s[k];
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int k = 0; k < 4; ++k) {
            s[k] = red[k][0];
            for (int w = 1; w < kBcThreads / 32; ++w) s[k] += red[k][w];
        }
        if (tiles == 1) {
            finish_bias_row(row, end - beg, x0, y0, s, xi_out, beta_out);
        } else {
            for (int k = 0; k < 4; ++k) partial[4 * blockIdx.x + k] = s[k];
        }
    }
}

// Long rows: the tiles' sums in ascending order, then xi and beta.
__global__ void bias_finish_kernel(const float* __restrict__ x, Rows rows, int64_t tiles, int bits,
                                   const float* __restrict__ m_arr,
                                   const float* __restrict__ p_arr,
                                   const double* __restrict__ partial, float* __restrict__ xi_out,
                                   float* __restrict__ beta_out) {
    const int64_t row = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= rows.C) return;
    const int64_t beg = rows.begin(row), end = rows.begin(row + 1);
    const int64_t nt = (end - beg + kBcTile - 1) / kBcTile;
    const float Lf = (float)((1 << (bits - 1)) - 1);
    double x0 = 0.0, y0 = 0.0;
    if (end > beg) {
        const float m = m_arr[row];
        const PieceParams P = make_params(m, p_arr[row], Lf);
        const float xf = x[beg];
        x0 = (double)xf;
        y0 = (double)fake_value(xf, m, P, Lf);
    }
    double s[4] = {0.0, 0.0, 0.0, 0.0};
    for (int64_t t = 0; t < nt; ++t)
        for (int k = 0; k < 4; ++k) s[k] += partial[4 * (row * tiles + t) + k];
    finish_bias_row(row, end - beg, x0, y0, s, xi_out, beta_out);
}

size_t bias_workspace_bytes(int64_t C, int64_t max_n) {
    const int64_t tiles = (max_n + kBcTile - 1) / kBcTile;
    return tiles > 1 ? (size_t)(32 * C * tiles + 255) / 256 * 256 : 256;
}

cudaError_t launch_bias_correction(const float* x, const int64_t* row_offsets, int64_t C,
                                   int64_t n, int64_t max_n, int bits, const float* m,
                                   const float* p, float* xi_out, float* beta_out, void* workspace,
                                   cudaStream_t stream) {
    Rows rows{row_offsets, C, n, n > 0 ? 1.0 / (double)n : 0.0, 0};
    const int64_t tiles = std::max<int64_t>(1, (max_n + kBcTile - 1) / kBcTile);
    double* partial = static_cast<double*>(workspace);
    bias_moments_kernel<<<(unsigned)(C * tiles), kBcThreads, 0, stream>>>(
        x, rows, tiles, bits, m, p, partial, xi_out, beta_out);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || tiles == 1) return e;
    bias_finish_kernel<<<(unsigned)((C + 127) / 128), 128, 0, stream>>>(
        x, rows, tiles, bits, m, p, partial, xi_out, beta_out);
    return cudaGetLastError();
}

// ---------------------------------------------------------------- dequantize with the correction
// y' = xi * y + beta with y the value pwlq_dequantize delivers (one multiply, one add): the
// dequantize kernel with the two per-row constants added to its row maps.
cudaError_t launch_dequantize_bc(const uint8_t* codes, const uint8_t* mask,
                                 const int64_t* row_offsets, int64_t C, int64_t n, int64_t total,
                                 int bits, const float* m, const float* p, const float* xi,
                                 const float* beta, float* y, int layout, cudaStream_t stream) {
    return launch_dequantize(codes, mask, row_offsets, C, n, total, bits, m, nullptr, p, y, layout,
                             stream, 0, xi, beta);
}

// ------------------------------------------------------------------------- dense bit stream
// Value i occupies bits [i (b+1), (i+1) (b+1)) of a little-endian bit stream, field =
// code | region << b.  Eight values make b + 1 whole bytes, so a thread that owns eight values
// owns whole bytes of the stream.
constexpr int kPkThreads = 256;

__global__ void __launch_bounds__(kPkThreads)
pack_dense_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ mask,
                  int64_t total, int bits, uint8_t* __restrict__ out) {
    const int64_t g = (int64_t)blockIdx.x * kPkThreads + threadIdx.x;
    const int64_t i0 = g * 8;
    if (i0 >= total) return;
    const int cnt = (int)min((int64_t)8, total - i0);
    const int w = bits + 1;
    const uint32_t cmask = (1u << bits) - 1u;
    const uint32_t mb = mask[i0 >> 3];
    unsigned long long lo = 0;
    uint32_t hi = 0;                                  // bits 64.. of the 8 (b+1)-bit fields (b = 8)
    for (int t = 0; t < cnt; ++t) {
        const unsigned long long field = (codes[i0 + t] & cmask) | (((mb >> t) & 1u) << bits);
        const int sh = t * w;
        lo |= field << sh;
        if (sh + w > 64) hi |= (uint32_t)(field >> (64 - sh));
    }
    const int nbytes = (cnt * w + 7) / 8;
    uint8_t* dst = out + g * w;
    for (int b = 0; b < nbytes; ++b)
        dst[b] = (uint8_t)(b < 8 ? (lo >> (8 * b)) : (hi >> (8 * (b - 8))));
}

__global__ void __launch_bounds__(kPkThreads)
unpack_dense_kernel(const uint8_t* __restrict__ in, int64_t total, int bits,
                    uint8_t* __restrict__ codes, uint8_t* __restrict__ mask) {
    const int64_t g = (int64_t)blockIdx.x * kPkThreads + threadIdx.x;
    const int64_t i0 = g * 8;
    if (i0 >= total) return;
    const int cnt = (int)min((int64_t)8, total - i0);
    const int w = bits + 1;
    const uint32_t cmask = (1u << bits) - 1u;
    const int nbytes = (cnt * w + 7) / 8;
    const uint8_t* src = in + g * w;
    unsigned long long lo = 0;
    uint32_t hi = 0;
    for (int b = 0; b < nbytes; ++b) {
        if (b < 8) lo |= (unsigned long long)src[b] << (8 * b);
        else hi |= (uint32_t)src[b] << (8 * (b - 8));
    }
    uint32_t mb = 0;
    for (int t = 0; t < cnt; ++t) {
        const int sh = t * w;
        unsigned long long field = lo >> sh;
        if (sh + w > 64) field |= (unsigned long long)hi << (64 - sh);
        codes[i0 + t] = (uint8_t)((uint32_t)field & cmask);
        mb |= (uint32_t)((field >> bits) & 1ull) << t;
    }
    mask[i0 >> 3] = (uint8_t)mb;
}

// Whole groups of 32 values with aligned buffers: a thread reads its 32 codes and 32 region bits
// as two 128-bit words and one 32-bit word and writes b + 1 whole 32-bit words of the stream
// (every shift is a compile-time constant).
template <int BITS>
__global__ void __launch_bounds__(kPkThreads)
pack_dense32_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ mask,
                    int64_t groups32, uint8_t* __restrict__ out) {
    constexpr int W = BITS + 1;
    const int64_t g = (int64_t)blockIdx.x * kPkThreads + threadIdx.x;
    if (g >= groups32) return;
    const uint4 c0 = __ldcs(reinterpret_cast<const uint4*>(codes) + 2 * g);
    const uint4 c1 = __ldcs(reinterpret_cast<const uint4*>(codes) + 2 * g + 1);
    const uint32_t mb = __ldcs(reinterpret_cast<const uint32_t*>(mask) + g);
    const uint32_t cw[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
    uint32_t ow[W + 1];
#pragma unroll
    for (int j = 0; j <= W; ++j) ow[j] = 0u;
#pragma unroll
    for (int t = 0; t < 32; ++t) {
        const uint32_t field = ((cw[t >> 2] >> (8 * (t & 3))) & ((1u << BITS) - 1u)) |
                               (((mb >> t) & 1u) << BITS);
        const int word = (t * W) >> 5, sh = (t * W) & 31;
        ow[word] |= field << sh;
        if (sh + W > 32) ow[word + 1] |= field >> (32 - sh);
    }
    uint32_t* dst = reinterpret_cast<uint32_t*>(out) + g * W;
#pragma unroll
    for (int j = 0; j < W; ++j) __stcs(dst + j, ow[j]);
}

template <int BITS>
__global__ void __launch_bounds__(kPkThreads)
unpack_dense32_kernel(const uint8_t* __restrict__ in, int64_t groups32,
                      uint8_t* __restrict__ codes, uint8_t* __restrict__ mask) {
    constexpr int W = BITS + 1;
    const int64_t g = (int64_t)blockIdx.x * kPkThreads + threadIdx.x;
    if (g >= groups32) return;
    const uint32_t* src = reinterpret_cast<const uint32_t*>(in) + g * W;
    uint32_t iw[W + 1];
#pragma unroll
    for (int j = 0; j < W; ++j) iw[j] = __ldcs(src + j);
    iw[W] = 0u;
    uint32_t cw[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u}, mb = 0u;
#pragma unroll
    for (int t = 0; t < 32; ++t) {
        const int word = (t * W) >> 5, sh = (t * W) & 31;
        uint32_t field = iw[word] >> sh;
        if (sh + W > 32) field |= iw[word + 1] << (32 - sh);
        cw[t >> 2] |= (field & ((1u << BITS) - 1u)) << (8 * (t & 3));
        mb |= ((field >> BITS) & 1u) << t;
    }
    __stcs(reinterpret_cast<uint4*>(codes) + 2 * g, make_uint4(cw[0], cw[1], cw[2], cw[3]));
    __stcs(reinterpret_cast<uint4*>(codes) + 2 * g + 1, make_uint4(cw[4], cw[5], cw[6], cw[7]));
    __stcs(reinterpret_cast<uint32_t*>(mask) + g, mb);
}

static inline bool pk_aligned(const void* p, size_t a) {
    return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0;
}

cudaError_t launch_pack_dense(const uint8_t* codes, const uint8_t* mask, int64_t total, int bits,
                              uint8_t* out, cudaStream_t stream) {
    if (total == 0) return cudaSuccess;
    // whole groups of 32 values through the word-wise kernel, the rest (and everything, when a
    // buffer is not aligned) through the byte-wise one
    int64_t done = 0;
    if (pk_aligned(codes, 16) && pk_aligned(mask, 4) && pk_aligned(out, 4) && total >= 32) {
        const int64_t g32 = total / 32;
        const unsigned grid = (unsigned)((g32 + kPkThreads - 1) / kPkThreads);
        switch (bits) {
#define PWLQ_PACK_CASE(B) case B: pack_dense32_kernel<B><<<grid, kPkThreads, 0, stream>>>(codes, mask, g32, out); break;
            PWLQ_PACK_CASE(2) PWLQ_PACK_CASE(3) PWLQ_PACK_CASE(4) PWLQ_PACK_CASE(5)
            PWLQ_PACK_CASE(6) PWLQ_PACK_CASE(7) PWLQ_PACK_CASE(8)
#undef PWLQ_PACK_CASE
            default: return cudaErrorInvalidValue;
        }
        done = g32 * 32;
    }
    if (done < total) {
        const int64_t groups = (total - done + 7) / 8;
        pack_dense_kernel<<<(unsigned)((groups + kPkThreads - 1) / kPkThreads), kPkThreads, 0, stream>>>(
            codes + done, mask + done / 8, total - done, bits, out + done / 8 * (bits + 1));
    }
    return cudaGetLastError();
}

cudaError_t launch_unpack_dense(const uint8_t* in, int64_t total, int bits, uint8_t* codes,
                                uint8_t* mask, cudaStream_t stream) {
    if (total == 0) return cudaSuccess;
    int64_t done = 0;
    if (pk_aligned(codes, 16) && pk_aligned(mask, 4) && pk_aligned(in, 4) && total >= 32) {
        const int64_t g32 = total / 32;
        const unsigned grid = (unsigned)((g32 + kPkThreads - 1) / kPkThreads);
        switch (bits) {
#define PWLQ_UNPACK_CASE(B) case B: unpack_dense32_kernel<B><<<grid, kPkThreads, 0, stream>>>(in, g32, codes, mask); break;
            PWLQ_UNPACK_CASE(2) PWLQ_UNPACK_CASE(3) PWLQ_UNPACK_CASE(4) PWLQ_UNPACK_CASE(5)
            PWLQ_UNPACK_CASE(6) PWLQ_UNPACK_CASE(7) PWLQ_UNPACK_CASE(8)
#undef PWLQ_UNPACK_CASE
            default: return cudaErrorInvalidValue;
        }
        done = g32 * 32;
    }
    if (done < total) {
        const int64_t groups = (total - done + 7) / 8;
        unpack_dense_kernel<<<(unsigned)((groups + kPkThreads - 1) / kPkThreads), kPkThreads, 0, stream>>>(
            in + done / 8 * (bits + 1), total - done, bits, codes + done, mask + done / 8);
    }
    return cudaGetLastError();
}

}  // namespace pwlq
