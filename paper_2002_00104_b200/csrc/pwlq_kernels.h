// Host-side launchers of the PWLQ kernels (internal to the library).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace pwlq {

// Values of one row that a search CTA stages in shared memory at a time; longer rows are cut
// into tiles whose partial sums are combined in a fixed order by a second kernel.
constexpr int kSearchTile = 8192;

// shift (here and below): for a slice of a longer list of ragged rows -- row_offsets points at the
// slice's first offset, the data pointers were advanced by `shift` values, `total` counts the
// slice's values; every offset read is reduced by `shift`.  0 for whole tensors.
// rowmap (here and in launch_quantize / launch_dequantize): nullptr, or row maps of this layout
// built by launch_rowmap_build, which spare the kernel's producer warps the map building.
cudaError_t launch_absmax(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                          int64_t total, float* m_out, cudaStream_t stream, int64_t shift = 0,
                          const void* rowmap = nullptr);

// Row maps of a layout (ragged rows, or dense rows of n values), built once into `rowmap`
// (rowmap_bytes(total) bytes, 16-byte aligned) for any number of streaming calls.
size_t rowmap_bytes(int64_t total);
cudaError_t launch_rowmap_build(const int64_t* row_offsets, int64_t C, int64_t n, int64_t total,
                                void* rowmap, cudaStream_t stream);

// Per-row minimum and maximum (the range [m1, m2] of a one-sided / asymmetric tensor).
cudaError_t launch_minmax(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                          int64_t total, float* lo_out, float* hi_out, cudaStream_t stream,
                          int64_t shift = 0);

struct SearchPlan {
    int64_t max_n;         // longest row
    int64_t tiles;         // tiles per row (by the longest row)
    int64_t tile;          // values per tile when a row has several (<= kSearchTile)
    size_t off_m;          // workspace offset of the internally computed ranges [C] floats
    size_t off_partials;   // workspace offset of the partial sums [C * tiles * K] doubles (tiles > 1)
    size_t off_sums;       // workspace offset of the combined sums [C * K] doubles (tiles > 1)
    size_t bytes;          // total workspace bytes
};
SearchPlan plan_search(int64_t C, int64_t max_n, int K);

cudaError_t launch_search(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                          int64_t total, int bits, const float* ratios, int K, const float* m,
                          const float* lo, float* p_out, float* err_out, int32_t* idx_out, float* sse_all,
                          void* workspace, const SearchPlan& plan, cudaStream_t stream,
                          int64_t shift = 0, bool clear_status = true, double* sums64 = nullptr);
// sums64 != nullptr: only the binary64 per-candidate sums [C][K] are delivered (p_out, err_out,
// idx_out, sse_all are not touched and may be null).  launch_search_finish adds `parts` such sets
// ([parts][C][K]) in ascending order and takes the first minimum of every row.
cudaError_t launch_search_finish(const double* sums, int parts, int64_t C, int K, const float* m,
                                 const float* lo, const float* ratios, float* p_out, float* err_out,
                                 int32_t* idx_out, float* sse_all, int* status,
                                 cudaStream_t stream);

// lo == nullptr: signed scheme with m = abs-max; lo != nullptr: one-sided ranges [lo, m] (m = upper
// bounds), unsigned b-bit levels.  The same convention holds for launch_dequantize and
// launch_search.  launch_dequantize with xi and beta (signed scheme only) delivers the
// bias-corrected values xi[row] * y + beta[row].
cudaError_t launch_quantize(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                            int64_t total, int bits, const float* m, const float* lo,
                            const float* p, uint8_t* codes, uint8_t* mask, float* fake, int layout,
                            cudaStream_t stream, int64_t shift = 0, const void* rowmap = nullptr);

cudaError_t launch_dequantize(const uint8_t* codes, const uint8_t* mask,
                              const int64_t* row_offsets, int64_t C, int64_t n, int64_t total,
                              int bits, const float* m, const float* lo, const float* p, float* y,
                              int layout, cudaStream_t stream, int64_t shift = 0,
                              const float* xi = nullptr, const float* beta = nullptr,
                              const void* rowmap = nullptr);

// Two or three breakpoints (three or four regions): search over all pairs (nbp = 2) or triples
// (nbp = 3) of a grid of K <= kSearch2MaxK ascending ratios; rows longer than kSearchTile values
// are cut into tiles whose terms a second kernel adds in a fixed order (workspace:
// search2_workspace_bytes).  Breakpoint t of row c is delivered to p_out[t][c * out_stride] (and
// its grid index to idx_out[t][...]).  sse_out: [C, K, K] (pairs) or [C, K, K, K] (triples) or
// nullptr.  Quantize / dequantize with a two-bit region index; p3 == nullptr: two breakpoints;
// breakpoint arrays are read with stride p_stride.
constexpr int kSearch2MaxK = 64;
size_t search2_workspace_bytes(int64_t C, int64_t max_n, int K);
cudaError_t launch_search2(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                           int64_t max_n, int bits, const float* ratios, int K, const float* m,
                           int nbp, float* const* p_out, int32_t* const* idx_out, int out_stride,
                           float* err_out, float* sse_out, void* workspace, cudaStream_t stream);
cudaError_t launch_quantize2(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                             int64_t total, int bits, const float* m, const float* p1,
                             const float* p2, const float* p3, int p_stride, uint8_t* codes,
                             uint8_t* region2, float* fake, int layout, cudaStream_t stream);
cudaError_t launch_dequantize2(const uint8_t* codes, const uint8_t* region2,
                               const int64_t* row_offsets, int64_t C, int64_t n, int64_t total,
                               int bits, const float* m, const float* p1, const float* p2,
                               const float* p3, int p_stride, float* y, int layout,
                               cudaStream_t stream);

// The element-wise forms (any alignment; what the two above fall back to).
cudaError_t launch_quantize2_plain(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                             int64_t total, int bits, const float* m, const float* p1,
                             const float* p2, const float* p3, int p_stride, uint8_t* codes,
                             uint8_t* region2, float* fake, int layout, cudaStream_t stream);
cudaError_t launch_dequantize2_plain(const uint8_t* codes, const uint8_t* region2,
                               const int64_t* row_offsets, int64_t C, int64_t n, int64_t total,
                               int bits, const float* m, const float* p1, const float* p2,
                               const float* p3, int p_stride, float* y, int layout,
                               cudaStream_t stream);

// Bias correction: folded scale xi and offset beta per row; dequantize that applies them; dense
// (b+1)-bit storage of code and region bit.
size_t bias_workspace_bytes(int64_t C, int64_t max_n);
cudaError_t launch_bias_correction(const float* x, const int64_t* row_offsets, int64_t C,
                                   int64_t n, int64_t max_n, int bits, const float* m,
                                   const float* p, float* xi_out, float* beta_out, void* workspace,
                                   cudaStream_t stream);
cudaError_t launch_dequantize_bc(const uint8_t* codes, const uint8_t* mask,
                                 const int64_t* row_offsets, int64_t C, int64_t n, int64_t total,
                                 int bits, const float* m, const float* p, const float* xi,
                                 const float* beta, float* y, int layout, cudaStream_t stream);
cudaError_t launch_pack_dense(const uint8_t* codes, const uint8_t* mask, int64_t total, int bits,
                              uint8_t* out, cudaStream_t stream);
cudaError_t launch_unpack_dense(const uint8_t* in, int64_t total, int bits, uint8_t* codes,
                                uint8_t* mask, cudaStream_t stream);

size_t select_workspace_bytes(int64_t C, int64_t max_n);
cudaError_t launch_select_analytic(const float* x, const int64_t* row_offsets, int64_t C,
                                   int64_t n, int64_t max_n, const float* m, int model,
                                   float* p_out, float* scale_out, void* workspace,
                                   cudaStream_t stream);

// Conditions the kernel family met on the current device since the last call of the same
// function, which also clears them (reads a device flag: synchronises with the device): bit 0, a
// bounded wait expired; bit 1, a call was given row maps of another layout.  -1 when the flag
// could not be read.
int take_absmax_timeout_flag();
int take_quantize_timeout_flag();
// Runs a bounded wait that is certain to expire after `polls` polls (self-test of the reporting).
cudaError_t launch_expire_wait(int polls, cudaStream_t stream);

}  // namespace pwlq
