// Quantizer of Eq. 3 (integer code + region bit, Sec. 4) and its inverse (Eq. 1, first line).
//
// Both are single streaming passes bound by HBM.  A thread owns 8 consecutive values: two
// 128-bit loads of x, then one 64-bit store of byte codes (or one 32-bit store of nibble-packed
// codes) and one region-mask byte, so that a warp writes contiguous 256 / 128 / 32-byte runs.
// CTAs are persistent and walk spans of 8192 values; the rows that overlap a span are staged in
// shared memory with their constants (four divisions per row, done once per span), so a thread's
// row lookups and constant fetches stay on chip, and the next span's loads are already in flight
// while the current one is staged and computed.
#include <mutex>

#include "pwlq_common.cuh"
#include "pwlq_kernels.h"
#include "pwlq_pipeline.cuh"

namespace pwlq {

constexpr int kQThreads = 256;
constexpr int kQChunk = kQThreads * 8;           // values one pass of the CTA covers
constexpr int kQChunks = 4;                      // passes per span
constexpr int kQSpan = kQChunk * kQChunks;       // values per span (one staged row table)
constexpr int kQStages = 2;                      // spans in flight per CTA (quantize)

static __device__ int g_quantize_timeout;        // set when a bounded wait expired

// Ragged rows: the rows overlapping the CTA's current span, with their constants.
typedef SpanTable<true> QuantSmem;

// The row a thread is currently in: constants in registers, refreshed when it crosses a boundary.
struct RowState {
    int64_t beg = 0, end = 0;
    float m = 0.0f;
    PieceParams P;

    __device__ __forceinline__ void seek(const QuantSmem& S, const Rows& rows,
                                         const float* __restrict__ m_arr,
                                         const float* __restrict__ p_arr, float Lf, int64_t i) {
        if (i >= beg && i < end) return;
        if (!rows.offsets) {                       // dense: arithmetic, constants from L1 / L2
            const int64_t row = rows.dense_row(i);
            beg = row * rows.n;
            end = beg + rows.n;
            m = __ldg(m_arr + row);
            P = make_params(m, __ldg(p_arr + row), Lf);
            return;
        }
        const int loc = S.find(i);
        if (loc >= 0) {
            beg = S.off[loc];
            end = S.off[loc + 1];
            m = S.m[loc];
            P = S.P[loc];
        } else {                                   // beyond the staged rows (very many tiny rows)
            const int64_t row = rows.row_of(i);
            beg = rows.begin(row);
            end = rows.begin(row + 1);
            m = m_arr[row];
            P = make_params(m, p_arr[row], Lf);
        }
    }
};

struct QuantizeSmem {
    BulkRing<kQStages, kQSpan * 4> ring;
    QuantSmem rows;
};

// Bytes of span `span` if it can be fetched by a bulk copy (aligned base, whole 16-byte units).
__device__ __forceinline__ unsigned q_bulk_bytes(int64_t span, int64_t total, int vec_in) {
    const int64_t beg = span * kQSpan;
    const int64_t cnt = min((int64_t)kQSpan, total - beg);
    return (vec_in && (cnt & 3) == 0) ? (unsigned)(cnt * 4) : 0u;
}

// Persistent CTAs: each walks spans blockIdx.x, blockIdx.x + gridDim.x, ...; the values of the
// next three spans are already on their way into a ring of shared-memory slots (bulk
// asynchronous copies) while the rows of the current span are staged and its values quantized.
template <bool PACKED, bool WANT_FAKE, bool RAGGED>
__global__ void __launch_bounds__(kQThreads)
quantize_kernel(const float* __restrict__ x, Rows rows, int64_t total, int bits,
                const float* __restrict__ m_arr, const float* __restrict__ p_arr,
                uint8_t* __restrict__ codes, uint8_t* __restrict__ mask, float* __restrict__ fake,
                int vec_in, int vec_fake, int vec_codes) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    QuantizeSmem& Q = *reinterpret_cast<QuantizeSmem*>(smem_raw);
    QuantSmem& S = Q.rows;
    __shared__ int s_abort;
    const float Lf = (float)((1 << (bits - 1)) - 1);
    const int Li = (1 << (bits - 1)) - 1;
    const uint32_t sign_unit = 1u << (bits - 1);      // value of the sign bit inside a code
    const int sign_shift = 32 - bits;                 // moves bit 31 onto the code's sign bit
    const int64_t nspans = (total + kQSpan - 1) / kQSpan;
    // The CTA's spans: ragged rows -> a block of consecutive spans (the next span's first row is
    // then the row this span ends in, so its table can be requested without a search); dense rows
    // -> every gridDim.x-th span.
    const int64_t first = RAGGED ? nspans * blockIdx.x / gridDim.x : blockIdx.x;
    const int64_t stride = RAGGED ? 1 : gridDim.x;
    const int64_t last = RAGGED ? nspans * (blockIdx.x + 1) / gridDim.x : nspans;   // exclusive
    if (threadIdx.x == 0) s_abort = 0;
    Q.ring.init();
    for (int it = 0; it < kQStages; ++it) {
        const int64_t span = first + (int64_t)it * stride;
        if (span < last) Q.ring.issue(it, x + span * kQSpan, q_bulk_bytes(span, total, vec_in));
    }
    int64_t row0 = 0;                               // first staged row of the current span
    RowFetch nf;
    if (RAGGED && first < last) {
        row0 = warp_row_of(rows, first * kQSpan);   // every warp finds the same row
        S.fetch(rows, m_arr, p_arr, row0, nf);
        S.commit(nf, min((first + 1) * kQSpan, total), Lf);
        __syncthreads();
    }
    RowState rs;                                    // survives from span to span
    int64_t it = 0;
    for (int64_t span = first; span < last; span += stride, ++it) {
        const int64_t span_beg = span * kQSpan;
        const int64_t span_end = min(span_beg + kQSpan, total);
        // ragged rows: request the next span's table now, write it when this span is done
        int64_t next_row0 = 0;
        const bool has_next = RAGGED && span + 1 < last;
        if (has_next) {
            const int l = S.find(span_end);
            next_row0 = (l >= 0) ? row0 + l : warp_row_of(rows, span_end);
            S.fetch(rows, m_arr, p_arr, next_row0, nf);
        }
        float* xs = reinterpret_cast<float*>(Q.ring.slot(it));
        if (q_bulk_bytes(span, total, vec_in) != 0) {
            if (!Q.ring.wait(it, (unsigned)(it / kQStages))) s_abort = 1;   // never expected
        } else {                                       // unaligned base or ragged tail: plain loads
            for (int i = threadIdx.x; i < (int)(span_end - span_beg); i += kQThreads)
                xs[i] = x[span_beg + i];
            __syncthreads();
        }
#pragma unroll
        for (int c = 0; c < kQChunks; ++c) {
            const int li = c * kQChunk + (int)threadIdx.x * 8;
            const int64_t i0 = span_beg + li;
            const int cnt = (int)max((int64_t)0, min((int64_t)8, total - i0));
            if (cnt == 0) continue;
            const float4 xa = *reinterpret_cast<const float4*>(xs + li);
            const float4 xb = *reinterpret_cast<const float4*>(xs + li + 4);
            const float xv[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
            uint32_t code[8];
            float yv[8];
            uint32_t mbyte = 0;
            rs.seek(S, rows, m_arr, p_arr, Lf, i0);
            if (cnt == 8 && i0 + 8 <= rs.end) {
                // all eight values in one row: the sequence of quantize_mag with the per-row
                // tests hoisted, the level taken from the mantissa of t + 1.5 * 2^23, and the sign
                // flag (x < 0, false for -0.0) read off the sign bit of x + 0.0
                // Codes are packed and region bits gathered on the fly (no per-value branch).
                const float m = rs.m;
                const PieceParams P = rs.P;
                uint32_t w0 = 0, w1 = 0, mb = 0;       // packed codes (w1: upper four, byte layout)
                if (m > 0.0f) {
#pragma unroll
                    for (int t = 0; t < 8; ++t) {
                        const float xi = xv[t];
                        const float a = fminf(fabsf(xi), m);
                        const bool tail = a > P.p;
                        const float z = tail ? P.p : 0.0f;
                        const float inv = tail ? P.inv2 : P.inv1;
                        const float r = __fadd_rn(__fmul_rn(__fsub_rn(a, z), inv), 12582912.0f);
                        const uint32_t q = (uint32_t)min(__float_as_int(r) - 0x4B400000, Li);
                        const uint32_t xs0 = __float_as_uint(__fadd_rn(xi, 0.0f));   // sign bit = (x < 0)
                        const uint32_t code = ((xs0 >> sign_shift) & sign_unit) | q;
                        if (PACKED) w0 += code << (4 * t);
                        else if (t < 4) w0 += code << (8 * t);
                        else w1 += code << (8 * (t - 4));
                        mb += tail ? (1u << t) : 0u;
                        if (WANT_FAKE) {
                            const float s = tail ? P.s2 : P.s1;
                            const float qf = fminf(__fsub_rn(r, 12582912.0f), Lf);
                            const float v = __fadd_rn(__fmul_rn(qf, s), z);
                            yv[t] = __uint_as_float(__float_as_uint(v) | (xs0 & 0x80000000u));
                        }
                    }
                } else if (WANT_FAKE) {
#pragma unroll
                    for (int t = 0; t < 8; ++t) yv[t] = 0.0f;
                }
                mask[i0 >> 3] = (uint8_t)mb;
                if (PACKED) {
                    uint8_t* dst = codes + (i0 >> 1);
                    if (vec_codes) *reinterpret_cast<uint32_t*>(dst) = w0;
                    else for (int b = 0; b < 4; ++b) dst[b] = (uint8_t)(w0 >> (8 * b));
                } else {
                    uint8_t* dst = codes + i0;
                    if (vec_codes) *reinterpret_cast<uint2*>(dst) = make_uint2(w0, w1);
                    else for (int b = 0; b < 8; ++b) dst[b] = (uint8_t)((b < 4 ? w0 : w1) >> (8 * (b & 3)));
                }
                if (WANT_FAKE) {
                    if (vec_fake) {
                        __stcs(reinterpret_cast<float4*>(fake + i0), make_float4(yv[0], yv[1], yv[2], yv[3]));
                        __stcs(reinterpret_cast<float4*>(fake + i0 + 4), make_float4(yv[4], yv[5], yv[6], yv[7]));
                    } else {
                        for (int t = 0; t < 8; ++t) fake[i0 + t] = yv[t];
                    }
                }
                continue;
            } else {
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    code[t] = 0;
                    yv[t] = 0.0f;
                    if (t < cnt) {
                        rs.seek(S, rows, m_arr, p_arr, Lf, i0 + t);
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
            }
            mask[i0 >> 3] = (uint8_t)mbyte;
            if (PACKED) {
                const uint32_t w = code[0] | (code[1] << 4) | (code[2] << 8) | (code[3] << 12) |
                                   (code[4] << 16) | (code[5] << 20) | (code[6] << 24) |
                                   (code[7] << 28);
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
            if (WANT_FAKE) {
                if (vec_fake && cnt == 8) {
                    __stcs(reinterpret_cast<float4*>(fake + i0), make_float4(yv[0], yv[1], yv[2], yv[3]));
                    __stcs(reinterpret_cast<float4*>(fake + i0 + 4), make_float4(yv[4], yv[5], yv[6], yv[7]));
                } else {
                    for (int t = 0; t < cnt; ++t) fake[i0 + t] = yv[t];
                }
            }
        }
        __syncthreads();                            // slot and row table are free again
        if (s_abort) {                               // a wait ran out: report and leave
            if (threadIdx.x == 0) atomicExch(&g_quantize_timeout, 1);
            return;
        }
        if (has_next) {
            S.commit(nf, min(span_end + kQSpan, total), Lf);
            row0 = next_row0;
            rs.beg = rs.end = 0;                     // staged constants are per span
        }
        const int64_t ahead = span + (int64_t)kQStages * stride;
        if (ahead < last)
            Q.ring.issue(it + kQStages, x + ahead * kQSpan, q_bulk_bytes(ahead, total, vec_in));
        if (RAGGED) __syncthreads();                // the next table is published
    }
}

// One span's worth of a thread's codes and region bits, requested ahead of use.
template <bool PACKED>
struct CodeRegs {
    uint32_t w0[kQChunks], w1[kQChunks], mb[kQChunks];
    __device__ __forceinline__ void load(const uint8_t* __restrict__ codes,
                                         const uint8_t* __restrict__ mask, int64_t span_beg,
                                         int64_t total, int vec_codes) {
#pragma unroll
        for (int c = 0; c < kQChunks; ++c) {
            const int64_t i0 = span_beg + (int64_t)c * kQChunk + (int64_t)threadIdx.x * 8;
            const int cnt = (int)max((int64_t)0, min((int64_t)8, total - i0));
            w0[c] = w1[c] = mb[c] = 0;
            if (cnt == 0) continue;
            if (PACKED) {
                const uint8_t* src = codes + (i0 >> 1);
                if (vec_codes && cnt == 8) {
                    w0[c] = __ldcs(reinterpret_cast<const unsigned int*>(src));
                } else {
                    const int nb = (cnt + 1) >> 1;
                    for (int b = 0; b < nb; ++b) w0[c] |= (uint32_t)src[b] << (8 * b);
                }
            } else {
                const uint8_t* src = codes + i0;
                if (vec_codes && cnt == 8) {
                    const uint2 w = __ldcs(reinterpret_cast<const uint2*>(src));
                    w0[c] = w.x; w1[c] = w.y;
                } else {
                    for (int t = 0; t < cnt; ++t) {
                        if (t < 4) w0[c] |= (uint32_t)src[t] << (8 * t);
                        else       w1[c] |= (uint32_t)src[t] << (8 * (t - 4));
                    }
                }
            }
            mb[c] = mask[i0 >> 3];
        }
    }
    __device__ __forceinline__ uint32_t code(int c, int t) const {
        if (PACKED) return (w0[c] >> (4 * t)) & 0xFu;
        return ((t < 4 ? w0[c] : w1[c]) >> (8 * (t & 3))) & 0xFFu;
    }
};

template <bool PACKED, bool RAGGED>
__global__ void __launch_bounds__(kQThreads)
dequantize_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ mask, Rows rows,
                  int64_t total, int bits, const float* __restrict__ m_arr,
                  const float* __restrict__ p_arr, float* __restrict__ y, int vec_codes,
                  int vec_out) {
    __shared__ QuantSmem S;
    const float Lf = (float)((1 << (bits - 1)) - 1);
    const int qmask = (1 << (bits - 1)) - 1;
    const int sign_shift = 32 - bits;                 // moves a code's sign bit to bit 31
    const int64_t nspans = (total + kQSpan - 1) / kQSpan;
    // the CTA's spans: consecutive for ragged rows (chained row tables), strided for dense rows
    const int64_t first = RAGGED ? nspans * blockIdx.x / gridDim.x : blockIdx.x;
    const int64_t stride = RAGGED ? 1 : gridDim.x;
    const int64_t last = RAGGED ? nspans * (blockIdx.x + 1) / gridDim.x : nspans;   // exclusive
    CodeRegs<PACKED> cur, nxt;
    RowState rs;                                    // survives from span to span
    cur.load(codes, mask, first * kQSpan, total, vec_codes);
    int64_t row0 = 0;                               // first staged row of the current span
    RowFetch nf;
    if (RAGGED && first < last) {
        row0 = warp_row_of(rows, first * kQSpan);
        S.fetch(rows, m_arr, p_arr, row0, nf);
        S.commit(nf, min((first + 1) * kQSpan, total), Lf);
        __syncthreads();
    }
    for (int64_t span = first; span < last; span += stride) {
        const int64_t span_beg = span * kQSpan;
        const int64_t span_end = min(span_beg + kQSpan, total);
        if (span + stride < last) nxt.load(codes, mask, (span + stride) * kQSpan, total, vec_codes);
        int64_t next_row0 = 0;
        const bool has_next = RAGGED && span + 1 < last;
        if (has_next) {
            const int l = S.find(span_end);
            next_row0 = (l >= 0) ? row0 + l : warp_row_of(rows, span_end);
            S.fetch(rows, m_arr, p_arr, next_row0, nf);
        }
#pragma unroll
        for (int c = 0; c < kQChunks; ++c) {
            const int64_t i0 = span_beg + (int64_t)c * kQChunk + (int64_t)threadIdx.x * 8;
            const int cnt = (int)max((int64_t)0, min((int64_t)8, total - i0));
            if (cnt == 0) continue;
            float yv[8];
            rs.seek(S, rows, m_arr, p_arr, Lf, i0);
            if (cnt == 8 && i0 + 8 <= rs.end) {
                // all eight values in one row; the level becomes a float through the mantissa of
                // 1.5 * 2^23 (exact for q < 2^22) instead of an integer conversion
                const PieceParams P = rs.P;
#pragma unroll
                for (int t = 0; t < 8; ++t) yv[t] = 0.0f;
                if (rs.m > 0.0f) {                     // one test per chunk; no branch per value
                    const uint32_t mb = cur.mb[c];
#pragma unroll
                    for (int t = 0; t < 8; ++t) {
                        const uint32_t code = cur.code(c, t);
                        const bool tail = (mb & (1u << t)) != 0;
                        const float q = __fsub_rn(__uint_as_float(0x4B400000u | (code & (uint32_t)qmask)),
                                                  12582912.0f);
                        const float v = __fadd_rn(__fmul_rn(q, tail ? P.s2 : P.s1), tail ? P.p : 0.0f);
                        // the code's sign bit moved to bit 31
                        yv[t] = __uint_as_float(__float_as_uint(v) | ((code << sign_shift) & 0x80000000u));
                    }
                }
            } else {
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    yv[t] = 0.0f;
                    if (t < cnt) {
                        rs.seek(S, rows, m_arr, p_arr, Lf, i0 + t);
                        if (rs.m > 0.0f) {
                            const uint32_t code = cur.code(c, t);
                            const int tail = (cur.mb[c] >> t) & 1;
                            const int neg = (code >> (bits - 1)) & 1;
                            const float q = (float)(code & qmask);
                            const float s = tail ? rs.P.s2 : rs.P.s1;
                            const float z = tail ? rs.P.p : 0.0f;
                            float v = __fmul_rn(q, s);
                            v = __fadd_rn(v, z);
                            yv[t] = neg ? -v : v;
                        }
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
        if (RAGGED) {
            __syncthreads();                        // the row table is no longer read
            if (has_next) {
                S.commit(nf, min(span_end + kQSpan, total), Lf);
                row0 = next_row0;
                rs.beg = rs.end = 0;
            }
            __syncthreads();                        // the next table is published
        }
        cur = nxt;
    }
}

static inline bool aligned(const void* p, size_t a) {
    return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0;
}

// CTAs that fit the device at once: the persistent grid.  Looked up once per (kernel, device);
// the first lookup also opts the kernel in to its dynamic shared memory size.
static unsigned persistent_grid(const void* kernel, int threads, size_t smem, int64_t nspans) {
    struct Entry { const void* kernel; int dev; int ctas; };
    static Entry table[64];
    static int used = 0;
    static std::mutex mu;
    int dev = 0;
    cudaGetDevice(&dev);
    int ctas = 0;
    {
        std::lock_guard<std::mutex> lock(mu);
        for (int i = 0; i < used; ++i)
            if (table[i].kernel == kernel && table[i].dev == dev) ctas = table[i].ctas;
        if (ctas == 0) {
            if (smem > 0)
                cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            int sms = 0, per_sm = 0;
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, smem);
            ctas = (sms > 0 && per_sm > 0) ? sms * per_sm : 148;
            if (used < 64) table[used++] = Entry{kernel, dev, ctas};
        }
    }
    return (unsigned)(nspans < ctas ? nspans : ctas);
}

int quantize_timeout_flag() {
    int v = 0;
    cudaMemcpyFromSymbol(&v, g_quantize_timeout, sizeof(int));
    return v;
}

cudaError_t launch_quantize(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                            int64_t total, int bits, const float* m, const float* p,
                            uint8_t* codes, uint8_t* mask, float* fake, int layout,
                            cudaStream_t stream) {
    if (total == 0) return cudaSuccess;
    Rows rows{row_offsets, C, n, n > 0 ? 1.0 / (double)n : 0.0};
    const bool packed = (layout == 1 && bits <= 4);
    const int64_t nspans = (total + kQSpan - 1) / kQSpan;
    const int vec_in = aligned(x, 16), vec_fake = fake ? aligned(fake, 16) : 0;
    const size_t smem = sizeof(QuantizeSmem);
    const int vec_codes = packed ? aligned(codes, 4) : aligned(codes, 8);
#define PWLQ_LAUNCH_QUANTIZE(PK, FK, RG)                                                          \
    quantize_kernel<PK, FK, RG><<<persistent_grid((const void*)quantize_kernel<PK, FK, RG>,       \
                                                  kQThreads, smem, nspans),                       \
                                  kQThreads, smem, stream>>>(x, rows, total, bits, m, p, codes,   \
                                                             mask, fake, vec_in, vec_fake,        \
                                                             vec_codes)
#define PWLQ_LAUNCH_QUANTIZE_RG(PK, FK) \
    do { if (row_offsets) PWLQ_LAUNCH_QUANTIZE(PK, FK, true); else PWLQ_LAUNCH_QUANTIZE(PK, FK, false); } while (0)
    if (packed) { if (fake) PWLQ_LAUNCH_QUANTIZE_RG(true, true); else PWLQ_LAUNCH_QUANTIZE_RG(true, false); }
    else        { if (fake) PWLQ_LAUNCH_QUANTIZE_RG(false, true); else PWLQ_LAUNCH_QUANTIZE_RG(false, false); }
#undef PWLQ_LAUNCH_QUANTIZE_RG
#undef PWLQ_LAUNCH_QUANTIZE
    return cudaGetLastError();
}

cudaError_t launch_dequantize(const uint8_t* codes, const uint8_t* mask,
                              const int64_t* row_offsets, int64_t C, int64_t n, int64_t total,
                              int bits, const float* m, const float* p, float* y, int layout,
                              cudaStream_t stream) {
    if (total == 0) return cudaSuccess;
    Rows rows{row_offsets, C, n, n > 0 ? 1.0 / (double)n : 0.0};
    const bool packed = (layout == 1 && bits <= 4);
    const int64_t nspans = (total + kQSpan - 1) / kQSpan;
#define PWLQ_LAUNCH_DEQUANTIZE(PK, RG)                                                            \
    dequantize_kernel<PK, RG><<<persistent_grid((const void*)dequantize_kernel<PK, RG>, kQThreads, \
                                                0, nspans),                                       \
                                kQThreads, 0, stream>>>(codes, mask, rows, total, bits, m, p, y,   \
                                                        aligned(codes, PK ? 4 : 8), aligned(y, 16))
    if (packed) { if (row_offsets) PWLQ_LAUNCH_DEQUANTIZE(true, true); else PWLQ_LAUNCH_DEQUANTIZE(true, false); }
    else        { if (row_offsets) PWLQ_LAUNCH_DEQUANTIZE(false, true); else PWLQ_LAUNCH_DEQUANTIZE(false, false); }
#undef PWLQ_LAUNCH_DEQUANTIZE
    return cudaGetLastError();
}

}  // namespace pwlq
