// Quantizer of Eq. 3 (integer code + region bit, Sec. 4) and its inverse (Eq. 1, first line).
//
// Both are single streaming passes bound by HBM.  A thread owns 8 consecutive values: two
// 128-bit loads of x, then one 64-bit store of byte codes (or one 32-bit store of nibble-packed
// codes) and one region-mask byte, so that a warp writes contiguous 256 / 128 / 32-byte runs.
// The per-row constants are recomputed only when the thread crosses into another row.
#include "pwlq_common.cuh"
#include "pwlq_kernels.h"

namespace pwlq {

constexpr int kQThreads = 256;

struct RowState {
    int64_t row = -1, beg = 0, end = 0;
    float m = 0.0f;
    PieceParams P;

    __device__ __forceinline__ void seek(const Rows& rows, const float* __restrict__ m_arr,
                                         const float* __restrict__ p_arr, float Lf, int64_t i) {
        if (i >= beg && i < end) return;
        if (row >= 0 && i == end && !rows.offsets) { ++row; }     // dense: next row follows
        else row = rows.row_of(i);
        beg = rows.begin(row);
        end = rows.begin(row + 1);
        m = m_arr[row];
        P = make_params(m, p_arr[row], Lf);
    }
};

template <bool PACKED>
__global__ void __launch_bounds__(kQThreads)
quantize_kernel(const float* __restrict__ x, Rows rows, int64_t total, int bits,
                const float* __restrict__ m_arr, const float* __restrict__ p_arr,
                uint8_t* __restrict__ codes, uint8_t* __restrict__ mask, float* __restrict__ fake,
                int vec_in, int vec_fake, int vec_codes) {
    const int64_t i0 = ((int64_t)blockIdx.x * kQThreads + threadIdx.x) * 8;
    if (i0 >= total) return;
    const float Lf = (float)((1 << (bits - 1)) - 1);
    const int cnt = (int)min((int64_t)8, total - i0);

    float xv[8];
    if (vec_in && cnt == 8) {
        const float4 a = __ldcs(reinterpret_cast<const float4*>(x + i0));
        const float4 b = __ldcs(reinterpret_cast<const float4*>(x + i0 + 4));
        xv[0] = a.x; xv[1] = a.y; xv[2] = a.z; xv[3] = a.w;
        xv[4] = b.x; xv[5] = b.y; xv[6] = b.z; xv[7] = b.w;
    } else {
#pragma unroll
        for (int t = 0; t < 8; ++t) xv[t] = (t < cnt) ? x[i0 + t] : 0.0f;
    }

    RowState rs;
    uint32_t code[8];
    float yv[8];
    uint32_t mbyte = 0;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        code[t] = 0;
        yv[t] = 0.0f;
        if (t < cnt) {
            rs.seek(rows, m_arr, p_arr, Lf, i0 + t);
            if (rs.m > 0.0f) {
                const float xi = xv[t];
                const int neg = xi < 0.0f;
                int q, tail;
                float v;
                quantize_mag(fminf(fabsf(xi), rs.m), rs.P, Lf, q, tail, v);
                code[t] = (uint32_t)((neg << (bits - 1)) | q);
                mbyte |= (uint32_t)tail << t;
                yv[t] = neg ? -v : v;
            }
        }
    }

    mask[i0 >> 3] = (uint8_t)mbyte;
    if (PACKED) {
        const uint32_t w = code[0] | (code[1] << 4) | (code[2] << 8) | (code[3] << 12) |
                           (code[4] << 16) | (code[5] << 20) | (code[6] << 24) | (code[7] << 28);
        uint8_t* dst = codes + (i0 >> 1);
        if (vec_codes && cnt == 8) {
            *reinterpret_cast<uint32_t*>(dst) = w;
        } else {
            const int nb = (cnt + 1) >> 1;
            for (int b = 0; b < nb; ++b) dst[b] = (uint8_t)(w >> (8 * b));
        }
    } else {
        uint8_t* dst = codes + i0;
        if (vec_codes && cnt == 8) {
            uint2 w;
            w.x = code[0] | (code[1] << 8) | (code[2] << 16) | (code[3] << 24);
            w.y = code[4] | (code[5] << 8) | (code[6] << 16) | (code[7] << 24);
            *reinterpret_cast<uint2*>(dst) = w;
        } else {
            for (int t = 0; t < cnt; ++t) dst[t] = (uint8_t)code[t];
        }
    }
    if (fake) {
        if (vec_fake && cnt == 8) {
            __stcs(reinterpret_cast<float4*>(fake + i0), make_float4(yv[0], yv[1], yv[2], yv[3]));
            __stcs(reinterpret_cast<float4*>(fake + i0 + 4), make_float4(yv[4], yv[5], yv[6], yv[7]));
        } else {
            for (int t = 0; t < cnt; ++t) fake[i0 + t] = yv[t];
        }
    }
}

template <bool PACKED>
__global__ void __launch_bounds__(kQThreads)
dequantize_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ mask, Rows rows,
                  int64_t total, int bits, const float* __restrict__ m_arr,
                  const float* __restrict__ p_arr, float* __restrict__ y, int vec_codes,
                  int vec_out) {
    const int64_t i0 = ((int64_t)blockIdx.x * kQThreads + threadIdx.x) * 8;
    if (i0 >= total) return;
    const float Lf = (float)((1 << (bits - 1)) - 1);
    const int qmask = (1 << (bits - 1)) - 1;
    const int cnt = (int)min((int64_t)8, total - i0);

    uint32_t code[8];
    if (PACKED) {
        const uint8_t* src = codes + (i0 >> 1);
        uint32_t w = 0;
        if (vec_codes && cnt == 8) {
            w = __ldcs(reinterpret_cast<const unsigned int*>(src));
        } else {
            const int nb = (cnt + 1) >> 1;
            for (int b = 0; b < nb; ++b) w |= (uint32_t)src[b] << (8 * b);
        }
#pragma unroll
        for (int t = 0; t < 8; ++t) code[t] = (w >> (4 * t)) & 0xFu;
    } else {
        const uint8_t* src = codes + i0;
        if (vec_codes && cnt == 8) {
            const uint2 w = __ldcs(reinterpret_cast<const uint2*>(src));
#pragma unroll
            for (int t = 0; t < 4; ++t) { code[t] = (w.x >> (8 * t)) & 0xFFu; code[4 + t] = (w.y >> (8 * t)) & 0xFFu; }
        } else {
#pragma unroll
            for (int t = 0; t < 8; ++t) code[t] = (t < cnt) ? src[t] : 0u;
        }
    }
    const uint32_t mbyte = mask[i0 >> 3];

    RowState rs;
    float yv[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        yv[t] = 0.0f;
        if (t < cnt) {
            rs.seek(rows, m_arr, p_arr, Lf, i0 + t);
            if (rs.m > 0.0f) {
                const int tail = (mbyte >> t) & 1;
                const int neg = (code[t] >> (bits - 1)) & 1;
                const float q = (float)(code[t] & qmask);
                const float s = tail ? rs.P.s2 : rs.P.s1;
                const float z = tail ? rs.P.p : 0.0f;
                float v = __fmul_rn(q, s);
                v = __fadd_rn(v, z);
                yv[t] = neg ? -v : v;
            }
        }
    }
    if (vec_out && cnt == 8) {
        __stcs(reinterpret_cast<float4*>(y + i0), make_float4(yv[0], yv[1], yv[2], yv[3]));
        __stcs(reinterpret_cast<float4*>(y + i0 + 4), make_float4(yv[4], yv[5], yv[6], yv[7]));
    } else {
        for (int t = 0; t < cnt; ++t) y[i0 + t] = yv[t];
    }
}

static inline bool aligned(const void* p, size_t a) {
    return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0;
}

cudaError_t launch_quantize(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                            int64_t total, int bits, const float* m, const float* p,
                            uint8_t* codes, uint8_t* mask, float* fake, int layout,
                            cudaStream_t stream) {
    if (total == 0) return cudaSuccess;
    Rows rows{row_offsets, C, n};
    const bool packed = (layout == 1 && bits <= 4);
    const int64_t threads = (total + 7) / 8;
    const unsigned grid = (unsigned)((threads + kQThreads - 1) / kQThreads);
    const int vec_in = aligned(x, 16), vec_fake = fake ? aligned(fake, 16) : 0;
    if (packed)
        quantize_kernel<true><<<grid, kQThreads, 0, stream>>>(x, rows, total, bits, m, p, codes,
                                                              mask, fake, vec_in, vec_fake,
                                                              aligned(codes, 4));
    else
        quantize_kernel<false><<<grid, kQThreads, 0, stream>>>(x, rows, total, bits, m, p, codes,
                                                               mask, fake, vec_in, vec_fake,
                                                               aligned(codes, 8));
    return cudaGetLastError();
}

cudaError_t launch_dequantize(const uint8_t* codes, const uint8_t* mask,
                              const int64_t* row_offsets, int64_t C, int64_t n, int64_t total,
                              int bits, const float* m, const float* p, float* y, int layout,
                              cudaStream_t stream) {
    if (total == 0) return cudaSuccess;
    Rows rows{row_offsets, C, n};
    const bool packed = (layout == 1 && bits <= 4);
    const int64_t threads = (total + 7) / 8;
    const unsigned grid = (unsigned)((threads + kQThreads - 1) / kQThreads);
    if (packed)
        dequantize_kernel<true><<<grid, kQThreads, 0, stream>>>(codes, mask, rows, total, bits, m,
                                                                p, y, aligned(codes, 4),
                                                                aligned(y, 16));
    else
        dequantize_kernel<false><<<grid, kQThreads, 0, stream>>>(codes, mask, rows, total, bits,
                                                                 m, p, y, aligned(codes, 8),
                                                                 aligned(y, 16));
    return cudaGetLastError();
}

}  // namespace pwlq
