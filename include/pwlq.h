/*
 * pwlq.h -- C ABI of the PWLQ hot path for NVIDIA B200 (sm_100a).
 *
 * The library implements the data-parallel part of post-training piecewise
 * linear quantization (arXiv 2002.00104): the range m of every row (Sec. 3.2),
 * an empirical breakpoint search that evaluates the b-bit piecewise quantizer
 * pw(r; b, m, p) of Eq. 3 for K candidate breakpoints p and keeps the one with
 * the smallest squared error (the grid counterpart of Eq. 6), the quantizer
 * itself (integer code + region bit, Sec. 4) and its inverse (Eq. 1, first line).
 *
 * Rows.  A tensor is viewed as C rows ("channels": per-output-channel weights,
 * or one row for a per-layer tensor, Sec. 5).  The dense calls take a row-major
 * [C, n] array; the *_ragged calls take rows of different lengths stored back
 * to back, described by row_offsets[C + 1] (ascending flat element offsets,
 * row_offsets[0] = 0, row_offsets[C] = total).  Flat index i = position in
 * that storage.
 *
 * Arithmetic.  All values are IEEE binary32.  With L = 2^(bits-1) - 1, for a row
 * with range m and breakpoint p:
 *     s1 = p / L, inv1 = L / p, d = m - p, s2 = d / L, inv2 = L / d
 *     (a piece whose range is not positive gets s = inv = 0),
 *     a = min(|x|, m); tail = a > p; (z, s, inv) = tail ? (p, s2, inv2) : (0, s1, inv1);
 *     q = min(rint((a - z) * inv), L)   (round half to even);  v = (q * s) + z,
 * one rounding per operation, no fused multiply-add.  code = (x < 0) << (bits-1) | q,
 * region = tail, y = (x < 0) ? -v : v.  Rows with m == 0 give code 0, region 0, y = +0.
 * Quantize and dequantize follow this sequence exactly; the search may fuse
 * operations (its sums agree with the sequence above to about 1e-6 relative).
 *
 * Pointers.  Unless a parameter says "host", every pointer is a DEVICE pointer
 * owned by the caller, valid on the device that is current at the call; fp32 and
 * int32 arrays need 4-byte alignment, int64 and workspace 8 / 256 bytes.  The
 * library allocates no device memory (the *_host call included: it works in
 * caller-provided device scratch).  What it keeps per device, for the life of
 * the process: the occupancy figures of its kernels (looked up at a kernel's first
 * launch), two streams and a few events of pwlq_encode_host (created at its first
 * call), the device address of the built-in scratch of pwlq_search_noalloc, and
 * the two expiry flags that pwlq_device_status reads and clears.  The tables are
 * guarded by mutexes; calls may come from several host threads.
 *
 * Execution.  Every call only enqueues work on `stream` (a cudaStream_t passed
 * as void*, NULL = default stream) and returns; results are valid after the
 * stream is synchronised.  Argument errors are reported by the return value
 * with nothing enqueued.  Conditions found on the device (a non-finite range)
 * are OR-ed into a 32-bit status word as bit (1 << code): the first 4 bytes of
 * the search workspace, cleared by the call itself.
 */
#ifndef PWLQ_H_
#define PWLQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    PWLQ_OK = 0,
    PWLQ_ERR_INVALID_ARG = 1, /* null pointer, bits outside [2,8], C/n/K < 1, misaligned pointer */
    PWLQ_ERR_UNSUPPORTED = 2, /* K or a size above the documented limit                       */
    PWLQ_ERR_WORKSPACE = 3,   /* workspace missing or smaller than the *_workspace_bytes value  */
    PWLQ_ERR_CUDA = 4,        /* a CUDA runtime call failed (launch configuration, stream, ...) */
    PWLQ_ERR_NONFINITE = 5,   /* device status, bit 1 << 5: a row's range is Inf or NaN          */
    PWLQ_ERR_TIMEOUT = 6      /* device status, bit 1 << 6: a bounded wait expired               */
};

enum {
    PWLQ_CODES_U8 = 0,    /* one byte per value: low `bits` bits = sign << (bits-1) | q          */
    PWLQ_CODES_PACKED = 1 /* bits <= 4: two values per byte, flat element 2j in the low nibble,
                             (total+1)/2 bytes; bits > 4: same as PWLQ_CODES_U8                  */
};

#define PWLQ_MAX_K 4096 /* largest number of candidate breakpoints per search */

/* Range of Sec. 3.2: m_out[c] = max_i |x[c, i]| (0 for an empty or all-zero row).  Exact
 * (order-free integer maximum of the magnitude bits).  x: [C, n].  m_out: [C]. */
int pwlq_absmax(const float* x, int64_t C, int64_t n, float* m_out, void* stream);
/* Same for ragged rows.  total = row_offsets[C] (known to the host). */
int pwlq_absmax_ragged(const float* x, const int64_t* row_offsets, int64_t C, int64_t total,
                       float* m_out, void* stream);

/* Bytes of device workspace pwlq_search needs for C rows of at most n values and K candidates
 * (for the ragged call pass n = the longest row).  Returns 0 for invalid arguments. */
size_t pwlq_search_workspace_bytes(int64_t C, int64_t n, int K);

/* Breakpoint search, the grid form of Eq. 6 on the empirical error of Eq. 3.  For every row c
 * and candidate k: p_k = m[c] * ratios[k] (one multiply), SSE[c,k] = sum_i (v_i - a_i)^2 over the
 * row; idx_out[c] = smallest k attaining the minimum, p_out[c] = p_idx, err_out[c] = SSE[c,idx].
 *   bits      b of the b-bit scheme, 2..8 (Sec. 3.2 requires b >= 2)
 *   ratios    [K] candidate p/m in (0, 1], ascending; K in [1, PWLQ_MAX_K]
 *   m         [C] ranges, or NULL: computed by the call (as pwlq_absmax) into the workspace
 *   p_out, err_out, idx_out   [C] each; err_out may be NULL
 *   sse_all   [C*K] row-major, or NULL
 *   workspace at least pwlq_search_workspace_bytes(...), 256-byte aligned; its first 4 bytes
 *             receive the device status (0, or 1 << PWLQ_ERR_NONFINITE) after the stream has run
 * Rows with m == 0: idx 0, p 0, err 0.  Rows with a non-finite m: idx 0, p = err = 0, status set.
 * Sums are formed in a fixed order: results are bit-reproducible from run to run. */
int pwlq_search(const float* x, int64_t C, int64_t n, int bits, const float* ratios, int K,
                const float* m, float* p_out, float* err_out, int32_t* idx_out, float* sse_all,
                void* workspace, size_t workspace_bytes, void* stream);
/* Same for ragged rows; max_n = longest row, total = row_offsets[C] (both known to the host). */
int pwlq_search_ragged(const float* x, const int64_t* row_offsets, int64_t C, int64_t total,
                       int64_t max_n, int bits, const float* ratios, int K, const float* m,
                       float* p_out, float* err_out, int32_t* idx_out, float* sse_all,
                       void* workspace, size_t workspace_bytes, void* stream);

/* The search of a row that is cut into pieces -- one tensor quantized per layer (Sec. 5:
 * activations) whose elements are spread over several GPUs, or fed in several calls.  The squared
 * error of Eq. 3 is a sum over values, so every piece contributes its own per-candidate sums under
 * the row's common range; the pieces' sums are added in a fixed order and the first minimum is
 * taken (grid form of Eq. 6), exactly as pwlq_search does for the tiles of a long row.
 *
 * pwlq_search_partial: x is this piece, [C, n] (n values of each of the C rows); m [C] is the
 * range of the WHOLE row (e.g. the maximum over the pieces' pwlq_absmax results), required; lo is
 * NULL for the signed scheme or [C] lower bounds of one-sided ranges [lo, m] as in
 * pwlq_search_unsigned.  sums_out [C, K] receives the binary64 sums of this piece, 8-byte aligned.
 * workspace as for pwlq_search (pwlq_search_workspace_bytes(C, n, K); status word in its first
 * 4 bytes).  No p, error or index is produced.
 * pwlq_search_finish: sums is [parts, C, K] (the pieces' sums_out stacked in a fixed order, e.g. by
 * rank); for every row the parts are added in ascending order in binary64, then idx_out = first
 * minimum, p_out = m * ratios[idx] ((m - lo) * ratios[idx] for one-sided ranges), err_out (may be
 * NULL) = the minimum, sse_all ([C, K] or NULL) = the totals in binary32.  status_out (4 bytes,
 * may be NULL) receives the status word (non-finite range).  All pointers are device pointers. */
int pwlq_search_partial(const float* x, int64_t C, int64_t n, int bits, const float* ratios,
                        int K, const float* m, const float* lo, double* sums_out, void* workspace,
                        size_t workspace_bytes, void* stream);
int pwlq_search_finish(const double* sums, int parts, int64_t C, int K, const float* m,
                       const float* lo, const float* ratios, float* p_out, float* err_out,
                       int32_t* idx_out, float* sse_all, int32_t* status_out, void* stream);

/* Quantizer of Eq. 3 with the chosen (m[c], p[c]) of each row, 0 < p <= m.
 *   codes        PWLQ_CODES_U8: total bytes; PWLQ_CODES_PACKED and bits <= 4: (total+1)/2 bytes
 *   region_mask  (total+7)/8 bytes; value i is bit (i & 7) of byte (i >> 3); 1 = tail region
 *                (the one extra bit per value of Sec. 4); unused bits of the last byte are 0
 *   fake_out     [total] reconstructed values y, or NULL
 * Every output byte is written (no pre-clearing needed). */
int pwlq_quantize(const float* x, int64_t C, int64_t n, int bits, const float* m, const float* p,
                  uint8_t* codes, uint8_t* region_mask, float* fake_out, int code_layout,
                  void* stream);
int pwlq_quantize_ragged(const float* x, const int64_t* row_offsets, int64_t C, int64_t total,
                         int bits, const float* m, const float* p, uint8_t* codes,
                         uint8_t* region_mask, float* fake_out, int code_layout, void* stream);

/* Inverse map, Eq. 1 first line: y = +-(q * s_region + z_region), z in {0, p} (Eq. 3, Sec. 4).
 * Bit-identical to the fake_out of pwlq_quantize for the same (m, p). */
int pwlq_dequantize(const uint8_t* codes, const uint8_t* region_mask, int64_t C, int64_t n,
                    int bits, const float* m, const float* p, float* y, int code_layout,
                    void* stream);
int pwlq_dequantize_ragged(const uint8_t* codes, const uint8_t* region_mask,
                           const int64_t* row_offsets, int64_t C, int64_t total, int bits,
                           const float* m, const float* p, float* y, int code_layout,
                           void* stream);

/* Row maps built once per layout.  The three streaming calls above (abs-max, quantize,
 * dequantize) work on spans of 4096 consecutive values and must know, for every span, which rows
 * overlap it (Sec. 5: weights are quantized per output channel, so a network's weights are many
 * short rows).  That description depends on the row layout only -- not on the values, m or p --
 * and without help every call rebuilds it inside the kernel.  A caller that runs several calls over
 * one layout builds it once:
 *   pwlq_rowmap_bytes(total)   size of the map buffer (0 if total is out of range)
 *   pwlq_rowmap_build          fills `rowmap` (device memory of the caller, 16-byte aligned,
 *                              rowmap_bytes >= pwlq_rowmap_bytes(total), else PWLQ_ERR_WORKSPACE)
 *                              for ragged rows (row_offsets != NULL; n ignored) or for dense rows
 *                              of n values (row_offsets == NULL, total = C * n)
 *   pwlq_*_mapped              the same operation and bit-identical results as pwlq_absmax /
 *                              pwlq_quantize / pwlq_dequantize (and their _ragged forms), given the
 *                              maps of this very layout.  The maps are only read: any number of
 *                              calls, on any streams, may share them once the build has finished.
 * Maps built for another layout (other C, total or n) are detected on the device: the call then
 * writes nothing and pwlq_device_status() reports 1 << PWLQ_ERR_INVALID_ARG.  Offsets that were
 * changed after the build while C and total stayed the same are not detected. */
size_t pwlq_rowmap_bytes(int64_t total);
int pwlq_rowmap_build(const int64_t* row_offsets, int64_t C, int64_t n, int64_t total,
                      void* rowmap, size_t rowmap_bytes, void* stream);
int pwlq_absmax_mapped(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                       int64_t total, const void* rowmap, float* m_out, void* stream);
int pwlq_quantize_mapped(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                         int64_t total, const void* rowmap, int bits, const float* m,
                         const float* p, uint8_t* codes, uint8_t* region_mask, float* fake_out,
                         int code_layout, void* stream);
int pwlq_dequantize_mapped(const uint8_t* codes, const uint8_t* region_mask,
                           const int64_t* row_offsets, int64_t C, int64_t n, int64_t total,
                           const void* rowmap, int bits, const float* m, const float* p, float* y,
                           int code_layout, void* stream);

/* One-sided ranges: unsigned tensors such as ReLU activations, or any asymmetric range [m1, m2]
 * (Sec. 3.2, footnote to the range; Eq. 1 with z = r_l and the unsigned integer domain
 * {0, ..., 2^b - 1} for one-sided distributions).  The paper does not spell the piecewise form
 * out; this library takes the range [lo, hi] of a row, shifts it to [0, m], m = hi - lo, with the
 * dense end at the lower bound, and splits it at one breakpoint p into the center [0, p] and the
 * tail (p, m].  No sign is stored, so each piece keeps all 2^b levels, s = Delta / (2^b - 1):
 *   a = min(max(x - lo, 0), m)           (one binary32 subtraction, then the clamp of Eq. 1)
 *   tail = a > p;  q, v as in pwlq_quantize with L = 2^b - 1;  delivered value y = v + lo.
 * The stored code is the level q (b bits); code and region-mask layouts are those of
 * pwlq_quantize.  The squared error of the search is (v - a)^2, i.e. taken in the shifted domain
 * (for lo = 0 the error of the delivered value).  A constant row (hi <= lo) gets code 0, y = lo,
 * index 0, p = 0 and error 0.  On non-negative data with lo = 0 the result equals the signed
 * scheme at b + 1 bits with the sign bit dropped.
 *
 * pwlq_minmax: lo_out[c] = min_i x[c, i], hi_out[c] = max_i x[c, i] (device, [C] each, distinct
 * buffers); an empty row gets 0, 0; zeros are written as +0.  The other calls take lo and hi
 * (device, [C], both required) where their signed counterparts take m; p, workspace, layouts,
 * asynchrony, ownership and error behaviour are the same (workspace size:
 * pwlq_search_workspace_bytes). */
int pwlq_minmax(const float* x, int64_t C, int64_t n, float* lo_out, float* hi_out, void* stream);
int pwlq_minmax_ragged(const float* x, const int64_t* row_offsets, int64_t C, int64_t total,
                       float* lo_out, float* hi_out, void* stream);
int pwlq_search_unsigned(const float* x, int64_t C, int64_t n, int bits, const float* ratios,
                         int K, const float* lo, const float* hi, float* p_out, float* err_out,
                         int32_t* idx_out, float* sse_all, void* workspace,
                         size_t workspace_bytes, void* stream);
int pwlq_search_unsigned_ragged(const float* x, const int64_t* row_offsets, int64_t C,
                                int64_t total, int64_t max_n, int bits, const float* ratios,
                                int K, const float* lo, const float* hi, float* p_out,
                                float* err_out, int32_t* idx_out, float* sse_all, void* workspace,
                                size_t workspace_bytes, void* stream);
int pwlq_quantize_unsigned(const float* x, int64_t C, int64_t n, int bits, const float* lo,
                           const float* hi, const float* p, uint8_t* codes,
                           uint8_t* region_mask, float* fake_out, int code_layout, void* stream);
int pwlq_quantize_unsigned_ragged(const float* x, const int64_t* row_offsets, int64_t C,
                                  int64_t total, int bits, const float* lo, const float* hi,
                                  const float* p, uint8_t* codes, uint8_t* region_mask,
                                  float* fake_out, int code_layout, void* stream);
int pwlq_dequantize_unsigned(const uint8_t* codes, const uint8_t* region_mask, int64_t C,
                             int64_t n, int bits, const float* lo, const float* hi,
                             const float* p, float* y, int code_layout, void* stream);
int pwlq_dequantize_unsigned_ragged(const uint8_t* codes, const uint8_t* region_mask,
                                    const int64_t* row_offsets, int64_t C, int64_t total,
                                    int bits, const float* lo, const float* hi, const float* p,
                                    float* y, int code_layout, void* stream);

/* Two breakpoints (Sec. 5.1, "Multiple Breakpoints": more non-overlapping regions, found by
 * minimising the same error over an enlarged search space).  The paper gives no formulas beyond
 * that; this library extends Eq. 3 in the obvious way: breakpoints 0 < p1 < p2 <= m split [0, m]
 * into R1 = [0, p1], R2 = (p1, p2], R3 = (p2, m]; inside every region (and sign) Eq. 1 is applied
 * with b-1 bits on the range [z, z + Delta], z = 0, p1, p2 and Delta = p1, p2 - p1, m - p2, with
 * the arithmetic of pwlq_quantize.  The code is the sign-magnitude code of pwlq_quantize; the region
 * index r in {0, 1, 2} takes two bits per value: bits 2 (i & 3), 2 (i & 3) + 1 of byte i >> 2 of
 * region2 (ceil(total / 4) bytes), i the flat index.  With p2 = m the scheme is pwlq_quantize's.
 *
 * pwlq_search2: for every row, all pairs i < j of the K candidate ratios (ascending, K in
 * [2, PWLQ_MAX_K2]), p1 = m * ratios[i], p2 = m * ratios[j]; squared error summed as in
 * pwlq_search; the first minimal pair in the order (i, j) wins.  Rows of more than 8192 values are
 * cut into tiles whose terms are added in ascending tile order (reproducible).  m (device, [C]) is
 * required.
 *   p1_out, p2_out, idx1_out, idx2_out   device, [C]; err_out device [C] or NULL
 *   sse_pairs   device, [C, K, K] or NULL; entry (i, j) is written with the sum for i < j, 0 otherwise
 *   workspace   device, 256-byte aligned, pwlq_search2_workspace_bytes(...) bytes; its first word
 *               is a status word as in pwlq_search (bit 1 << PWLQ_ERR_INVALID_ARG: the ratios do
 *               not ascend, results of the launch are zeros)
 * A row with m = 0 or no values gets indices (0, 1), p1 = p2 = 0, error 0.
 * pwlq_quantize2 / pwlq_dequantize2 (and the three-breakpoint forms below): breakpoints
 * p1 <= p2 (<= p3) <= m per row; any alignment of the buffers is accepted, the streaming kernels
 * run when x, codes, fake_out and y are 16-byte and region2 4-byte aligned.  A row with m <= 0
 * gets codes 0, region 0 and values +0.
 * Asynchrony, ownership and error behaviour as for the one-breakpoint calls. */
#define PWLQ_MAX_K2 64
size_t pwlq_search2_workspace_bytes(int64_t C, int64_t max_n, int K);
int pwlq_search2(const float* x, int64_t C, int64_t n, int bits, const float* ratios, int K,
                 const float* m, float* p1_out, float* p2_out, float* err_out, int32_t* idx1_out,
                 int32_t* idx2_out, float* sse_pairs, void* workspace, size_t workspace_bytes,
                 void* stream);
int pwlq_search2_ragged(const float* x, const int64_t* row_offsets, int64_t C, int64_t total,
                        int64_t max_n, int bits, const float* ratios, int K, const float* m,
                        float* p1_out, float* p2_out, float* err_out, int32_t* idx1_out,
                        int32_t* idx2_out, float* sse_pairs, void* workspace,
                        size_t workspace_bytes, void* stream);
int pwlq_quantize2(const float* x, int64_t C, int64_t n, int bits, const float* m,
                   const float* p1, const float* p2, uint8_t* codes, uint8_t* region2,
                   float* fake_out, int code_layout, void* stream);
int pwlq_quantize2_ragged(const float* x, const int64_t* row_offsets, int64_t C, int64_t total,
                          int bits, const float* m, const float* p1, const float* p2,
                          uint8_t* codes, uint8_t* region2, float* fake_out, int code_layout,
                          void* stream);
int pwlq_dequantize2(const uint8_t* codes, const uint8_t* region2, int64_t C, int64_t n,
                     int bits, const float* m, const float* p1, const float* p2, float* y,
                     int code_layout, void* stream);
int pwlq_dequantize2_ragged(const uint8_t* codes, const uint8_t* region2,
                            const int64_t* row_offsets, int64_t C, int64_t total, int bits,
                            const float* m, const float* p1, const float* p2, float* y,
                            int code_layout, void* stream);

/* Three breakpoints (Sec. 5.1 "Multiple Breakpoints"; Table 1 of the paper compares one, two and
 * three).  The same reading with one more region: 0 < p1 < p2 < p3 <= m, regions [0, p1],
 * (p1, p2], (p2, p3], (p3, m], each quantized by Eq. 1 with b-1 bits and offset z = its lower
 * end; the region index 0..3 fills the two bits per value of region2.  With p3 = m the scheme is
 * the two-breakpoint one.
 *
 * pwlq_search3: all triples i < j < k of the K candidate ratios (ascending, K in [3, PWLQ_MAX_K2]);
 * the first minimal triple in the order (i, j, k) wins.  The error of a triple is the sum of its
 * four regions' errors, which share their terms with the pair search: the cost is that of
 * pwlq_search2 plus O(K^2) per row, not K^3 / 6 evaluations.
 *   p_out, idx_out   device, [C, 3] (the three breakpoints / grid indices of a row side by side)
 *   err_out          device [C] or NULL
 *   sse_triples      device, [C, K, K, K] or NULL; entry (i, j, k) holds the sum for i < j < k,
 *                    0 otherwise (meant for small K: K^3 floats per row)
 *   workspace        as for pwlq_search2 (pwlq_search2_workspace_bytes)
 * A row with m = 0 or no values gets indices (0, 1, 2), p = 0, error 0.
 * pwlq_quantize3 / pwlq_dequantize3 take the breakpoints as one [C, 3] array p. */
int pwlq_search3(const float* x, int64_t C, int64_t n, int bits, const float* ratios, int K,
                 const float* m, float* p_out, float* err_out, int32_t* idx_out,
                 float* sse_triples, void* workspace, size_t workspace_bytes, void* stream);
int pwlq_search3_ragged(const float* x, const int64_t* row_offsets, int64_t C, int64_t total,
                        int64_t max_n, int bits, const float* ratios, int K, const float* m,
                        float* p_out, float* err_out, int32_t* idx_out, float* sse_triples,
                        void* workspace, size_t workspace_bytes, void* stream);
int pwlq_quantize3(const float* x, int64_t C, int64_t n, int bits, const float* m, const float* p,
                   uint8_t* codes, uint8_t* region2, float* fake_out, int code_layout,
                   void* stream);
int pwlq_quantize3_ragged(const float* x, const int64_t* row_offsets, int64_t C, int64_t total,
                          int bits, const float* m, const float* p, uint8_t* codes,
                          uint8_t* region2, float* fake_out, int code_layout, void* stream);
int pwlq_dequantize3(const uint8_t* codes, const uint8_t* region2, int64_t C, int64_t n,
                     int bits, const float* m, const float* p, float* y, int code_layout,
                     void* stream);
int pwlq_dequantize3_ragged(const uint8_t* codes, const uint8_t* region2,
                            const int64_t* row_offsets, int64_t C, int64_t total, int bits,
                            const float* m, const float* p, float* y, int code_layout,
                            void* stream);

/* Bias correction (Sec. 5.1, "Bias Correction"): quantization shifts the mean and the variance of
 * a row; the paper compensates this by folding correction terms into the scale and the offset and
 * prints no formula.  This library computes, per row, with y = the value pwlq_quantize delivers,
 *     xi   = sqrt( sum (x - mean x)^2 / sum (y - mean y)^2 )      (1 when either sum is 0)
 *     beta = mean x - xi * mean y
 * in binary64, delivered in binary32, so that xi * y + beta has the mean and the centred norm of
 * x.  An empty row gets xi = 1, beta = 0.
 *   xi_out, beta_out   device, [C]
 *   workspace          device, 256-byte aligned, pwlq_bias_workspace_bytes(C, longest row) bytes
 * pwlq_dequantize_bc is pwlq_dequantize followed by y' = xi * y + beta in binary32 (one multiply,
 * one add).  Asynchrony, ownership and error behaviour as for the other calls. */
size_t pwlq_bias_workspace_bytes(int64_t C, int64_t max_n);
int pwlq_bias_correction(const float* x, int64_t C, int64_t n, int bits, const float* m,
                         const float* p, float* xi_out, float* beta_out, void* workspace,
                         size_t workspace_bytes, void* stream);
int pwlq_bias_correction_ragged(const float* x, const int64_t* row_offsets, int64_t C,
                                int64_t total, int64_t max_n, int bits, const float* m,
                                const float* p, float* xi_out, float* beta_out, void* workspace,
                                size_t workspace_bytes, void* stream);
int pwlq_dequantize_bc(const uint8_t* codes, const uint8_t* region_mask, int64_t C, int64_t n,
                       int bits, const float* m, const float* p, const float* xi,
                       const float* beta, float* y, int code_layout, void* stream);
int pwlq_dequantize_bc_ragged(const uint8_t* codes, const uint8_t* region_mask,
                              const int64_t* row_offsets, int64_t C, int64_t total, int bits,
                              const float* m, const float* p, const float* xi, const float* beta,
                              float* y, int code_layout, void* stream);

/* Dense storage (Sec. 4: b bits per value plus one bit for the region): code and region bit of
 * value i as one (b+1)-bit field, field = code | region << b, in bits [i (b+1), (i+1) (b+1)) of a
 * little-endian bit stream (bit k of the stream is bit k & 7 of byte k >> 3);
 * pwlq_dense_bytes(total, bits) = ceil(total (b+1) / 8) bytes.  pwlq_pack_dense reads codes in the
 * PWLQ_CODES_U8 layout and the region mask of pwlq_quantize; pwlq_unpack_dense restores both.
 * All pointers are device pointers owned by the caller. */
size_t pwlq_dense_bytes(int64_t total, int bits);
int pwlq_pack_dense(const uint8_t* codes_u8, const uint8_t* region_mask, int64_t total, int bits,
                    uint8_t* stream_out, void* stream);
int pwlq_unpack_dense(const uint8_t* stream_in, int64_t total, int bits, uint8_t* codes_u8,
                      uint8_t* region_mask, void* stream);

/* Analytic breakpoint selection, the paper's own way of choosing p (Sec. 3.3, Sec. 5.1): assume a
 * zero-mean density for each row, fit its scale, and take the breakpoint that minimises the
 * expected error of Eq. 5 -- the root of Eq. 9 on (0, m/2) -- or the closed form of Sec. 5.1.
 * O(n) per row instead of O(n K); the result can be fed to pwlq_quantize directly.
 *   model      PWLQ_MODEL_GAUSS_APPROX   p = sigma ln(0.8614 m / sigma + 0.6079)  (Sec. 5.1, m and p
 *                                        in units of sigma)
 *              PWLQ_MODEL_GAUSS_ROOT     Gaussian, root of Eq. 9 (bracketed Newton iteration, binary64)
 *              PWLQ_MODEL_LAPLACE        Laplacian, root of Eq. 9
 *   scale fit  sigma = sqrt(mean x^2) (Gaussian), b = mean |x| (Laplacian), binary64 sums in a
 *              fixed order
 *   m          [C] ranges (pwlq_absmax);  p_out [C], 0 < p <= m/2 (m/2 when Eq. 9 has no root
 *              inside, 0 for an all-zero row);  scale_out [C] or NULL
 *   workspace  pwlq_select_workspace_bytes(C, longest row) bytes, 256-byte aligned */
enum { PWLQ_MODEL_GAUSS_APPROX = 0, PWLQ_MODEL_GAUSS_ROOT = 1, PWLQ_MODEL_LAPLACE = 2 };
size_t pwlq_select_workspace_bytes(int64_t C, int64_t n);
int pwlq_select_analytic(const float* x, int64_t C, int64_t n, const float* m, int model,
                         float* p_out, float* scale_out, void* workspace, size_t workspace_bytes,
                         void* stream);
int pwlq_select_analytic_ragged(const float* x, const int64_t* row_offsets, int64_t C,
                                int64_t total, int64_t max_n, const float* m, int model,
                                float* p_out, float* scale_out, void* workspace,
                                size_t workspace_bytes, void* stream);

/* Whole path from HOST buffers: copies x (and row_offsets, ratios) to the device, runs abs-max,
 * search, quantize and dequantize there, and copies m, p, err, idx, codes and region_mask back.
 * All *_host pointers are host memory (pinned memory makes the copies asynchronous); NULL
 * row_offsets_host means dense [C, n] with n = total / C.  dev_scratch is device memory of at
 * least pwlq_encode_host_scratch_bytes(...) bytes, 256-byte aligned.  The call returns after
 * enqueueing; the host outputs are valid once `stream` is synchronised.  The dequantized tensor
 * stays in dev_scratch (offset reported through y_dev_out when non-NULL).
 * Rows are independent, so large tensors are cut into up to eight runs of whole rows whose input
 * copy, kernels and output copies overlap: the copies run on two internal streams (created once
 * per device, the only resources this library ever creates) chained to `stream` by events; work
 * queued on `stream` before the call is finished before any of it starts, and `stream` ends the
 * call.  The results are those of the four device calls run one after another.
 * The search's status word (a non-finite range) of the whole call sits in dev_scratch at byte
 * offset pwlq_encode_host_status_offset(...): copy its 4 bytes back after synchronising. */
size_t pwlq_encode_host_scratch_bytes(int64_t C, int64_t total, int64_t max_n, int K);
size_t pwlq_encode_host_status_offset(int64_t C, int64_t total, int64_t max_n, int K);
int pwlq_encode_host(const float* x_host, const int64_t* row_offsets_host, int64_t C,
                     int64_t total, int64_t max_n, int bits, const float* ratios_host, int K,
                     float* m_host, float* p_host, float* err_host, int32_t* idx_host,
                     uint8_t* codes_host, uint8_t* region_mask_host, int code_layout,
                     void* dev_scratch, size_t dev_scratch_bytes, float** y_dev_out,
                     void* stream);
/* The same for one-sided ranges (pwlq_minmax, pwlq_search_unsigned, pwlq_quantize_unsigned,
 * pwlq_dequantize_unsigned): lo_host / hi_host [C] receive the rows' lower and upper bounds;
 * everything else as in pwlq_encode_host (same scratch size). */
int pwlq_encode_host_unsigned(const float* x_host, const int64_t* row_offsets_host, int64_t C,
                              int64_t total, int64_t max_n, int bits, const float* ratios_host,
                              int K, float* lo_host, float* hi_host, float* p_host,
                              float* err_host, int32_t* idx_host, uint8_t* codes_host,
                              uint8_t* region_mask_host, int code_layout, void* dev_scratch,
                              size_t dev_scratch_bytes, float** y_dev_out, void* stream);

/* No counterpart in the paper: a packaging variant of pwlq_search for callers that cannot
 * allocate device memory -- for example a plugin inside an application whose own memory pool
 * already holds the whole device (cudaMalloc fails or is against the host's rules), a
 * latency-critical loop that must avoid cudaMalloc's device-wide synchronisation, or a component
 * that is only ever handed input and output buffers.  It computes exactly what pwlq_search
 * computes for a dense [C, n] tensor (same kernels, bit-identical results), but its workspace is
 * a fixed array of PWLQ_NOALLOC_SCRATCH_BYTES in device global memory that belongs to the library
 * image; every GPU on which the library is used carries that array until the process exits.
 *   - The call allocates nothing and calls no allocating routine; the caller passes only inputs
 *     and outputs.  status_out (device, 4 bytes, may be NULL) receives the device status word.
 *   - Problems whose workspace need, pwlq_search_workspace_bytes(C, n, K), exceeds
 *     PWLQ_NOALLOC_SCRATCH_BYTES are rejected with PWLQ_ERR_UNSUPPORTED and nothing is enqueued.
 *   - The first call on each device looks up the array's device address (with that device
 *     current).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array.  Each call rewrites everything it later reads,
 *     so leftovers of earlier calls are harmless, but two calls that can overlap on the GPU
 *     (different streams, no ordering between them) race on it: order them. */
#define PWLQ_NOALLOC_SCRATCH_BYTES (4 << 20)
int pwlq_search_noalloc(const float* x, int64_t C, int64_t n, int bits, const float* ratios,
                        int K, const float* m, float* p_out, float* err_out, int32_t* idx_out,
                        float* sse_all, int32_t* status_out, void* stream);
size_t pwlq_search_noalloc_max_bytes(void);

/* The streaming kernels (abs-max, quantize, dequantize) hand their data over through shared-memory
 * barriers that they await with a bounded number of polls; a wait that runs out makes the kernel
 * stop early and sets a flag on the current device.  This call reads the flags (it synchronises
 * with the device) and returns 0, or 1 << PWLQ_ERR_TIMEOUT if a wait has expired on the current
 * device since the previous call of pwlq_device_status, OR-ed with 1 << PWLQ_ERR_INVALID_ARG if a
 * *_mapped call was given row maps of another layout -- the outputs of the streaming calls made
 * in between are then not valid -- or 1 << PWLQ_ERR_CUDA if the flags could not be read.  Reading
 * clears the flags: call it after synchronising the work it is meant to vouch for. */
int pwlq_device_status(void);

/* Text for a status value (static storage). */
const char* pwlq_status_string(int status);
/* Library version, "major.minor". */
const char* pwlq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* PWLQ_H_ */
