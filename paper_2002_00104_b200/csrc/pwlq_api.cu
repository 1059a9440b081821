// C ABI of the PWLQ library: argument checks and kernel launches, nothing else.
#include <algorithm>
#include <mutex>

#include "../../include/pwlq.h"
#include "pwlq_kernels.h"

namespace {

inline bool misaligned(const void* p, size_t a) {
    return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0;
}
inline cudaStream_t as_stream(void* s) { return static_cast<cudaStream_t>(s); }
inline int from_cuda(cudaError_t e) { return e == cudaSuccess ? PWLQ_OK : PWLQ_ERR_CUDA; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Largest flat size: the streaming kernels index 8 values per thread with a 32-bit grid.
constexpr int64_t kMaxTotal = (int64_t)1 << 40;

int check_rows(int64_t C, int64_t n_or_total) {
    if (C < 1 || n_or_total < 1) return PWLQ_ERR_INVALID_ARG;
    if (C > ((int64_t)1 << 31) - 1) return PWLQ_ERR_UNSUPPORTED;
    return PWLQ_OK;
}

int absmax_impl(const float* x, const int64_t* ro, int64_t C, int64_t n, int64_t total,
                float* m_out, void* stream, const void* rowmap = nullptr) {
    if (!x || !m_out || misaligned(x, 4) || misaligned(m_out, 4) || misaligned(ro, 8) ||
        misaligned(rowmap, 16))
        return PWLQ_ERR_INVALID_ARG;
    if (total > kMaxTotal) return PWLQ_ERR_UNSUPPORTED;
    return from_cuda(pwlq::launch_absmax(x, ro, C, n, total, m_out, as_stream(stream), 0, rowmap));
}

// Arguments of the *_mapped entry points that describe the layout: ragged rows (row_offsets, n
// ignored) or dense rows of n values with total = C * n.
int check_layout(const int64_t* ro, int64_t C, int64_t& n, int64_t total, const void* rowmap) {
    if (int rc = check_rows(C, total)) return rc;
    if (!rowmap) return PWLQ_ERR_INVALID_ARG;
    if (ro) { n = 0; return PWLQ_OK; }
    if (n < 1 || C * n != total) return PWLQ_ERR_INVALID_ARG;
    return PWLQ_OK;
}

int minmax_impl(const float* x, const int64_t* ro, int64_t C, int64_t n, int64_t total,
                float* lo_out, float* hi_out, void* stream) {
    if (!x || !lo_out || !hi_out || lo_out == hi_out || misaligned(x, 4) ||
        misaligned(lo_out, 4) || misaligned(hi_out, 4) || misaligned(ro, 8))
        return PWLQ_ERR_INVALID_ARG;
    if (total > kMaxTotal) return PWLQ_ERR_UNSUPPORTED;
    return from_cuda(pwlq::launch_minmax(x, ro, C, n, total, lo_out, hi_out, as_stream(stream)));
}

// lo == nullptr: signed scheme (m = abs-max, may be null: computed internally);
// lo != nullptr: one-sided ranges [lo, m], both required.
int search_impl(const float* x, const int64_t* ro, int64_t C, int64_t n, int64_t total,
                int64_t max_n, int bits, const float* ratios, int K, const float* m,
                const float* lo, float* p_out,
                float* err_out, int32_t* idx_out, float* sse_all, void* ws, size_t ws_bytes,
                void* stream) {
    if (!x || !ratios || !p_out || !idx_out || bits < 2 || bits > 8 || K < 1 || max_n < 1 ||
        (lo && !m))
        return PWLQ_ERR_INVALID_ARG;
    if (misaligned(x, 4) || misaligned(ratios, 4) || misaligned(m, 4) || misaligned(lo, 4) ||
        misaligned(p_out, 4) ||
        misaligned(err_out, 4) || misaligned(idx_out, 4) || misaligned(sse_all, 4) ||
        misaligned(ro, 8))
        return PWLQ_ERR_INVALID_ARG;
    if (K > PWLQ_MAX_K || total > kMaxTotal) return PWLQ_ERR_UNSUPPORTED;
    const pwlq::SearchPlan plan = pwlq::plan_search(C, max_n, K);
    if (C * plan.tiles > ((int64_t)1 << 31) - 1 || C * ((K + 31) / 32) > ((int64_t)1 << 31) - 1)
        return PWLQ_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < plan.bytes) return PWLQ_ERR_WORKSPACE;
    if (misaligned(ws, 256)) return PWLQ_ERR_INVALID_ARG;
    return from_cuda(pwlq::launch_search(x, ro, C, n, total, bits, ratios, K, m, lo, p_out,
                                         err_out, idx_out, sse_all, ws, plan, as_stream(stream)));
}

int quantize_impl(const float* x, const int64_t* ro, int64_t C, int64_t n, int64_t total,
                  int bits, const float* m, const float* lo, const float* p, uint8_t* codes,
                  uint8_t* mask, float* fake, int layout, void* stream,
                  const void* rowmap = nullptr) {
    if (!x || !m || !p || !codes || !mask || bits < 2 || bits > 8 || misaligned(rowmap, 16) ||
        (layout != PWLQ_CODES_U8 && layout != PWLQ_CODES_PACKED))
        return PWLQ_ERR_INVALID_ARG;
    if (misaligned(x, 4) || misaligned(m, 4) || misaligned(lo, 4) || misaligned(p, 4) ||
        misaligned(fake, 4) || misaligned(ro, 8))
        return PWLQ_ERR_INVALID_ARG;
    if (total > kMaxTotal) return PWLQ_ERR_UNSUPPORTED;
    return from_cuda(pwlq::launch_quantize(x, ro, C, n, total, bits, m, lo, p, codes, mask, fake,
                                           layout, as_stream(stream), 0, rowmap));
}

int dequantize_impl(const uint8_t* codes, const uint8_t* mask, const int64_t* ro, int64_t C,
                    int64_t n, int64_t total, int bits, const float* m, const float* lo,
                    const float* p, float* y, int layout, void* stream,
                    const void* rowmap = nullptr) {
    if (!codes || !mask || !m || !p || !y || bits < 2 || bits > 8 || misaligned(rowmap, 16) ||
        (layout != PWLQ_CODES_U8 && layout != PWLQ_CODES_PACKED))
        return PWLQ_ERR_INVALID_ARG;
    if (misaligned(m, 4) || misaligned(lo, 4) || misaligned(p, 4) || misaligned(y, 4) ||
        misaligned(ro, 8))
        return PWLQ_ERR_INVALID_ARG;
    if (total > kMaxTotal) return PWLQ_ERR_UNSUPPORTED;
    return from_cuda(pwlq::launch_dequantize(codes, mask, ro, C, n, total, bits, m, lo, p, y,
                                             layout, as_stream(stream), 0, nullptr, nullptr,
                                             rowmap));
}

inline size_t code_bytes(int64_t total, int bits, int layout) {
    return (layout == PWLQ_CODES_PACKED && bits <= 4) ? (size_t)((total + 1) / 2) : (size_t)total;
}

// Layout of the device scratch of pwlq_encode_host (every block 256-byte aligned).
struct HostPlan {
    size_t x, ro, ratios, m, lo, p, err, idx, codes, mask, y, ws, bytes;
    pwlq::SearchPlan sp;
};
HostPlan plan_host(int64_t C, int64_t total, int64_t max_n, int K) {
    HostPlan h;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes, 256); return r; };
    h.x = take(sizeof(float) * (size_t)total);
    h.ro = take(sizeof(int64_t) * (size_t)(C + 1));
    h.ratios = take(sizeof(float) * (size_t)K);
    h.m = take(sizeof(float) * (size_t)C);
    h.lo = take(sizeof(float) * (size_t)C);            // lower bounds (one-sided form only)
    h.p = take(sizeof(float) * (size_t)C);
    h.err = take(sizeof(float) * (size_t)C);
    h.idx = take(sizeof(int32_t) * (size_t)C);
    h.codes = take((size_t)total);
    h.mask = take((size_t)((total + 7) / 8));
    h.y = take(sizeof(float) * (size_t)total);
    h.sp = pwlq::plan_search(C, max_n, K);
    h.ws = take(h.sp.bytes);
    h.bytes = o;
    return h;
}

// ---- pipelining of pwlq_encode_host
constexpr int kHostChunks = 8;
constexpr int64_t kHostChunkMin = 1 << 20;     // values: below this a run is not worth its launches

// Internal streams and events of the host-buffer entry point, created once per device.
struct HostPipe {
    std::mutex mu;
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t start = nullptr, finished = nullptr;
    cudaEvent_t in_done[kHostChunks] = {}, out_ready[kHostChunks] = {};
    bool ready = false;
};
HostPipe* host_pipe() {
    static HostPipe pipes[64];
    static std::mutex create_mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    HostPipe& p = pipes[dev];
    std::lock_guard<std::mutex> lock(create_mu);
    if (!p.ready) {
        bool ok = cudaStreamCreateWithFlags(&p.copy_in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&p.copy_out, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&p.finished, cudaEventDisableTiming) == cudaSuccess;
        for (int k = 0; ok && k < kHostChunks; ++k)
            ok = cudaEventCreateWithFlags(&p.in_done[k], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&p.out_ready[k], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) return nullptr;
        p.ready = true;
    }
    return &p;
}

// Cuts rows [0, C) into at most kHostChunks runs of about equal size whose first flat index is a
// multiple of 8; row_b[0 .. runs] receives the run boundaries.  Returns the number of runs.
int split_rows(const int64_t* ro, int64_t C, int64_t n, int64_t total, int64_t* row_b) {
    auto flat = [&](int64_t c) { return ro ? ro[c] : c * n; };
    int runs = 0;
    row_b[0] = 0;
    const int want = (int)std::min<int64_t>(kHostChunks, std::max<int64_t>(1, total / kHostChunkMin));
    for (int k = 1; k < want; ++k) {
        const int64_t target = total / want * k;
        int64_t lo = row_b[runs], hi = C;               // first row with flat(row) >= target
        while (lo < hi) {
            const int64_t mid = (lo + hi) / 2;
            if (flat(mid) < target) lo = mid + 1; else hi = mid;
        }
        int64_t r = lo;
        for (int step = 0; r < C && (flat(r) & 7) != 0 && step < 4096; ++step) ++r;
        if (r >= C || (flat(r) & 7) != 0 || r <= row_b[runs]) continue;
        row_b[++runs] = r;
    }
    row_b[++runs] = C;
    return runs;
}

}  // namespace

extern "C" {

int pwlq_absmax(const float* x, int64_t C, int64_t n, float* m_out, void* stream) {
    if (int rc = check_rows(C, n)) return rc;
    return absmax_impl(x, nullptr, C, n, C * n, m_out, stream);
}

int pwlq_absmax_ragged(const float* x, const int64_t* row_offsets, int64_t C, int64_t total,
                       float* m_out, void* stream) {
    if (int rc = check_rows(C, total)) return rc;
    if (!row_offsets) return PWLQ_ERR_INVALID_ARG;
    return absmax_impl(x, row_offsets, C, 0, total, m_out, stream);
}

size_t pwlq_search_workspace_bytes(int64_t C, int64_t n, int K) {
    if (C < 1 || n < 1 || K < 1 || K > PWLQ_MAX_K) return 0;
    return pwlq::plan_search(C, n, K).bytes;
}

int pwlq_search(const float* x, int64_t C, int64_t n, int bits, const float* ratios, int K,
                const float* m, float* p_out, float* err_out, int32_t* idx_out, float* sse_all,
                void* workspace, size_t workspace_bytes, void* stream) {
    if (int rc = check_rows(C, n)) return rc;
    return search_impl(x, nullptr, C, n, C * n, n, bits, ratios, K, m, nullptr, p_out, err_out,
                       idx_out, sse_all, workspace, workspace_bytes, stream);
}

int pwlq_search_ragged(const float* x, const int64_t* row_offsets, int64_t C, int64_t total,
                       int64_t max_n, int bits, const float* ratios, int K, const float* m,
                       float* p_out, float* err_out, int32_t* idx_out, float* sse_all,
                       void* workspace, size_t workspace_bytes, void* stream) {
    if (int rc = check_rows(C, total)) return rc;
    if (!row_offsets || max_n > total) return PWLQ_ERR_INVALID_ARG;
    return search_impl(x, row_offsets, C, 0, total, max_n, bits, ratios, K, m, nullptr, p_out,
                       err_out, idx_out, sse_all, workspace, workspace_bytes, stream);
}

int pwlq_search_partial(const float* x, int64_t C, int64_t n, int bits, const float* ratios,
                        int K, const float* m, const float* lo, double* sums_out, void* workspace,
                        size_t workspace_bytes, void* stream) {
    if (int rc = check_rows(C, n)) return rc;
    if (!x || !ratios || !m || !sums_out || bits < 2 || bits > 8 || K < 1)
        return PWLQ_ERR_INVALID_ARG;
    if (misaligned(x, 4) || misaligned(ratios, 4) || misaligned(m, 4) || misaligned(lo, 4) ||
        misaligned(sums_out, 8))
        return PWLQ_ERR_INVALID_ARG;
    if (K > PWLQ_MAX_K || C * n > kMaxTotal) return PWLQ_ERR_UNSUPPORTED;
    const pwlq::SearchPlan plan = pwlq::plan_search(C, n, K);
    if (C * plan.tiles > ((int64_t)1 << 31) - 1 || C * ((K + 31) / 32) > ((int64_t)1 << 31) - 1)
        return PWLQ_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < plan.bytes) return PWLQ_ERR_WORKSPACE;
    if (misaligned(workspace, 256)) return PWLQ_ERR_INVALID_ARG;
    return from_cuda(pwlq::launch_search(x, nullptr, C, n, C * n, bits, ratios, K, m, lo, nullptr,
                                         nullptr, nullptr, nullptr, workspace, plan,
                                         as_stream(stream), 0, true, sums_out));
}

int pwlq_search_finish(const double* sums, int parts, int64_t C, int K, const float* m,
                       const float* lo, const float* ratios, float* p_out, float* err_out,
                       int32_t* idx_out, float* sse_all, int32_t* status_out, void* stream) {
    if (!sums || !m || !ratios || !p_out || !idx_out || parts < 1 || C < 1 || K < 1)
        return PWLQ_ERR_INVALID_ARG;
    if (misaligned(sums, 8) || misaligned(m, 4) || misaligned(lo, 4) || misaligned(ratios, 4) ||
        misaligned(p_out, 4) || misaligned(err_out, 4) || misaligned(idx_out, 4) ||
        misaligned(sse_all, 4) || misaligned(status_out, 4))
        return PWLQ_ERR_INVALID_ARG;
    if (K > PWLQ_MAX_K || C > ((int64_t)1 << 31) - 1) return PWLQ_ERR_UNSUPPORTED;
    return from_cuda(pwlq::launch_search_finish(sums, parts, C, K, m, lo, ratios, p_out, err_out,
                                                idx_out, sse_all, status_out, as_stream(stream)));
}

int pwlq_quantize(const float* x, int64_t C, int64_t n, int bits, const float* m, const float* p,
                  uint8_t* codes, uint8_t* region_mask, float* fake_out, int code_layout,
                  void* stream) {
    if (int rc = check_rows(C, n)) return rc;
    return quantize_impl(x, nullptr, C, n, C * n, bits, m, nullptr, p, codes, region_mask,
                         fake_out, code_layout, stream);
}

int pwlq_quantize_ragged(const float* x, const int64_t* row_offsets, int64_t C, int64_t total,
                         int bits, const float* m, const float* p, uint8_t* codes,
                         uint8_t* region_mask, float* fake_out, int code_layout, void* stream) {
    if (int rc = check_rows(C, total)) return rc;
    if (!row_offsets) return PWLQ_ERR_INVALID_ARG;
    return quantize_impl(x, row_offsets, C, 0, total, bits, m, nullptr, p, codes, region_mask,
                         fake_out, code_layout, stream);
}

int pwlq_dequantize(const uint8_t* codes, const uint8_t* region_mask, int64_t C, int64_t n,
                    int bits, const float* m, const float* p, float* y, int code_layout,
                    void* stream) {
    if (int rc = check_rows(C, n)) return rc;
    return dequantize_impl(codes, region_mask, nullptr, C, n, C * n, bits, m, nullptr, p, y,
                           code_layout, stream);
}

int pwlq_dequantize_ragged(const uint8_t* codes, const uint8_t* region_mask,
                           const int64_t* row_offsets, int64_t C, int64_t total, int bits,
                           const float* m, const float* p, float* y, int code_layout,
                           void* stream) {
    if (int rc = check_rows(C, total)) return rc;
    if (!row_offsets) return PWLQ_ERR_INVALID_ARG;
    return dequantize_impl(codes, region_mask, row_offsets, C, 0, total, bits, m, nullptr, p, y,
                           code_layout, stream);
}

size_t pwlq_rowmap_bytes(int64_t total) {
    if (total < 1 || total > kMaxTotal) return 0;
    return pwlq::rowmap_bytes(total);
}

int pwlq_rowmap_build(const int64_t* row_offsets, int64_t C, int64_t n, int64_t total,
                      void* rowmap, size_t rowmap_bytes, void* stream) {
    if (int rc = check_layout(row_offsets, C, n, total, rowmap)) return rc;
    if (misaligned(rowmap, 16) || misaligned(row_offsets, 8)) return PWLQ_ERR_INVALID_ARG;
    if (total > kMaxTotal) return PWLQ_ERR_UNSUPPORTED;
    if (rowmap_bytes < pwlq::rowmap_bytes(total)) return PWLQ_ERR_WORKSPACE;
    return from_cuda(pwlq::launch_rowmap_build(row_offsets, C, n, total, rowmap, as_stream(stream)));
}

int pwlq_absmax_mapped(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                       int64_t total, const void* rowmap, float* m_out, void* stream) {
    if (int rc = check_layout(row_offsets, C, n, total, rowmap)) return rc;
    return absmax_impl(x, row_offsets, C, n, total, m_out, stream, rowmap);
}

int pwlq_quantize_mapped(const float* x, const int64_t* row_offsets, int64_t C, int64_t n,
                         int64_t total, const void* rowmap, int bits, const float* m,
                         const float* p, uint8_t* codes, uint8_t* region_mask, float* fake_out,
                         int code_layout, void* stream) {
    if (int rc = check_layout(row_offsets, C, n, total, rowmap)) return rc;
    return quantize_impl(x, row_offsets, C, n, total, bits, m, nullptr, p, codes, region_mask,
                         fake_out, code_layout, stream, rowmap);
}

int pwlq_dequantize_mapped(const uint8_t* codes, const uint8_t* region_mask,
                           const int64_t* row_offsets, int64_t C, int64_t n, int64_t total,
                           const void* rowmap, int bits, const float* m, const float* p, float* y,
                           int code_layout, void* stream) {
    if (int rc = check_layout(row_offsets, C, n, total, rowmap)) return rc;
    return dequantize_impl(codes, region_mask, row_offsets, C, n, total, bits, m, nullptr, p, y,
                           code_layout, stream, rowmap);
}

int pwlq_minmax(const float* x, int64_t C, int64_t n, float* lo_out, float* hi_out,
                void* stream) {
    if (int rc = check_rows(C, n)) return rc;
    return minmax_impl(x, nullptr, C, n, C * n, lo_out, hi_out, stream);
}

int pwlq_minmax_ragged(const float* x, const int64_t* row_offsets, int64_t C, int64_t total,
                       float* lo_out, float* hi_out, void* stream) {
    if (int rc = check_rows(C, total)) return rc;
    if (!row_offsets) return PWLQ_ERR_INVALID_ARG;
    return minmax_impl(x, row_offsets, C, 0, total, lo_out, hi_out, stream);
}

int pwlq_search_unsigned(const float* x, int64_t C, int64_t n, int bits, const float* ratios,
                         int K, const float* lo, const float* hi, float* p_out, float* err_out,
                         int32_t* idx_out, float* sse_all, void* workspace,
                         size_t workspace_bytes, void* stream) {
    if (int rc = check_rows(C, n)) return rc;
    if (!lo || !hi) return PWLQ_ERR_INVALID_ARG;
    return search_impl(x, nullptr, C, n, C * n, n, bits, ratios, K, hi, lo, p_out, err_out,
                       idx_out, sse_all, workspace, workspace_bytes, stream);
}

int pwlq_search_unsigned_ragged(const float* x, const int64_t* row_offsets, int64_t C,
                                int64_t total, int64_t max_n, int bits, const float* ratios,
                                int K, const float* lo, const float* hi, float* p_out,
                                float* err_out, int32_t* idx_out, float* sse_all, void* workspace,
                                size_t workspace_bytes, void* stream) {
    if (int rc = check_rows(C, total)) return rc;
    if (!row_offsets || max_n > total || !lo || !hi) return PWLQ_ERR_INVALID_ARG;
    return search_impl(x, row_offsets, C, 0, total, max_n, bits, ratios, K, hi, lo, p_out,
                       err_out, idx_out, sse_all, workspace, workspace_bytes, stream);
}

int pwlq_quantize_unsigned(const float* x, int64_t C, int64_t n, int bits, const float* lo,
                           const float* hi, const float* p, uint8_t* codes,
                           uint8_t* region_mask, float* fake_out, int code_layout, void* stream) {
    if (int rc = check_rows(C, n)) return rc;
    if (!lo) return PWLQ_ERR_INVALID_ARG;
    return quantize_impl(x, nullptr, C, n, C * n, bits, hi, lo, p, codes, region_mask, fake_out,
                         code_layout, stream);
}

int pwlq_quantize_unsigned_ragged(const float* x, const int64_t* row_offsets, int64_t C,
                                  int64_t total, int bits, const float* lo, const float* hi,
                                  const float* p, uint8_t* codes, uint8_t* region_mask,
                                  float* fake_out, int code_layout, void* stream) {
    if (int rc = check_rows(C, total)) return rc;
    if (!row_offsets || !lo) return PWLQ_ERR_INVALID_ARG;
    return quantize_impl(x, row_offsets, C, 0, total, bits, hi, lo, p, codes, region_mask,
                         fake_out, code_layout, stream);
}

int pwlq_dequantize_unsigned(const uint8_t* codes, const uint8_t* region_mask, int64_t C,
                             int64_t n, int bits, const float* lo, const float* hi,
                             const float* p, float* y, int code_layout, void* stream) {
    if (int rc = check_rows(C, n)) return rc;
    if (!lo) return PWLQ_ERR_INVALID_ARG;
    return dequantize_impl(codes, region_mask, nullptr, C, n, C * n, bits, hi, lo, p, y,
                           code_layout, stream);
}

int pwlq_dequantize_unsigned_ragged(const uint8_t* codes, const uint8_t* region_mask,
                                    const int64_t* row_offsets, int64_t C, int64_t total,
                                    int bits, const float* lo, const float* hi, const float* p,
                                    float* y, int code_layout, void* stream) {
    if (int rc = check_rows(C, total)) return rc;
    if (!row_offsets || !lo) return PWLQ_ERR_INVALID_ARG;
    return dequantize_impl(codes, region_mask, row_offsets, C, 0, total, bits, hi, lo, p, y,
                           code_layout, stream);
}

size_t pwlq_search2_workspace_bytes(int64_t C, int64_t max_n, int K) {
    if (C < 1 || max_n < 1 || K < 2 || K > PWLQ_MAX_K2) return 0;
    return pwlq::search2_workspace_bytes(C, max_n, K);
}

// nbp = 2: p_out / idx_out are {p1, p2} / {idx1, idx2} arrays of [C]; nbp = 3: one [C, 3] array each.
static int search23_impl(const float* x, const int64_t* ro, int64_t C, int64_t n, int64_t total,
                         int64_t max_n, int bits, const float* ratios, int K, const float* m,
                         int nbp, float* const* p_out, int32_t* const* idx_out, int out_stride,
                         float* err_out, float* sse_out, void* ws, size_t ws_bytes, void* stream) {
    if (!x || !ratios || !m || bits < 2 || bits > 8 || K < nbp || max_n < 1)
        return PWLQ_ERR_INVALID_ARG;
    for (int t = 0; t < nbp; ++t)
        if (!p_out[t] || !idx_out[t] || misaligned(p_out[t], 4) || misaligned(idx_out[t], 4))
            return PWLQ_ERR_INVALID_ARG;
    if (misaligned(x, 4) || misaligned(ratios, 4) || misaligned(m, 4) || misaligned(err_out, 4) ||
        misaligned(sse_out, 4) || misaligned(ro, 8))
        return PWLQ_ERR_INVALID_ARG;
    if (K > PWLQ_MAX_K2 || total > kMaxTotal) return PWLQ_ERR_UNSUPPORTED;
    const int64_t tiles = (max_n + pwlq::kSearchTile - 1) / pwlq::kSearchTile;
    if (C * tiles > ((int64_t)1 << 31) - 1) return PWLQ_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < pwlq::search2_workspace_bytes(C, max_n, K)) return PWLQ_ERR_WORKSPACE;
    if (misaligned(ws, 256)) return PWLQ_ERR_INVALID_ARG;
    return from_cuda(pwlq::launch_search2(x, ro, C, n, max_n, bits, ratios, K, m, nbp, p_out,
                                          idx_out, out_stride, err_out, sse_out, ws,
                                          as_stream(stream)));
}

int pwlq_search2(const float* x, int64_t C, int64_t n, int bits, const float* ratios, int K,
                 const float* m, float* p1_out, float* p2_out, float* err_out, int32_t* idx1_out,
                 int32_t* idx2_out, float* sse_pairs, void* workspace, size_t workspace_bytes,
                 void* stream) {
    if (int rc = check_rows(C, n)) return rc;
    float* const p[3] = {p1_out, p2_out, nullptr};
    int32_t* const idx[3] = {idx1_out, idx2_out, nullptr};
    return search23_impl(x, nullptr, C, n, C * n, n, bits, ratios, K, m, 2, p, idx, 1, err_out,
                         sse_pairs, workspace, workspace_bytes, stream);
}

int pwlq_search2_ragged(const float* x, const int64_t* row_offsets, int64_t C, int64_t total,
                        int64_t max_n, int bits, const float* ratios, int K, const float* m,
                        float* p1_out, float* p2_out, float* err_out, int32_t* idx1_out,
                        int32_t* idx2_out, float* sse_pairs, void* workspace,
                        size_t workspace_bytes, void* stream) {
    if (int rc = check_rows(C, total)) return rc;
    if (!row_offsets || max_n > total) return PWLQ_ERR_INVALID_ARG;
    float* const p[3] = {p1_out, p2_out, nullptr};
    int32_t* const idx[3] = {idx1_out, idx2_out, nullptr};
    return search23_impl(x, row_offsets, C, 0, total, max_n, bits, ratios, K, m, 2, p, idx, 1,
                         err_out, sse_pairs, workspace, workspace_bytes, stream);
}

int pwlq_search3(const float* x, int64_t C, int64_t n, int bits, const float* ratios, int K,
                 const float* m, float* p_out, float* err_out, int32_t* idx_out,
                 float* sse_triples, void* workspace, size_t workspace_bytes, void* stream) {
    if (int rc = check_rows(C, n)) return rc;
    if (!p_out || !idx_out) return PWLQ_ERR_INVALID_ARG;
    float* const p[3] = {p_out, p_out + 1, p_out + 2};
    int32_t* const idx[3] = {idx_out, idx_out + 1, idx_out + 2};
    return search23_impl(x, nullptr, C, n, C * n, n, bits, ratios, K, m, 3, p, idx, 3, err_out,
                         sse_triples, workspace, workspace_bytes, stream);
}

int pwlq_search3_ragged(const float* x, const int64_t* row_offsets, int64_t C, int64_t total,
                        int64_t max_n, int bits, const float* ratios, int K, const float* m,
                        float* p_out, float* err_out, int32_t* idx_out, float* sse_triples,
                        void* workspace, size_t workspace_bytes, void* stream) {
    if (int rc = check_rows(C, total)) return rc;
    if (!row_offsets || max_n > total || !p_out || !idx_out) return PWLQ_ERR_INVALID_ARG;
    float* const p[3] = {p_out, p_out + 1, p_out + 2};
    int32_t* const idx[3] = {idx_out, idx_out + 1, idx_out + 2};
    return search23_impl(x, row_offsets, C, 0, total, max_n, bits, ratios, K, m, 3, p, idx, 3,
                         err_out, sse_triples, workspace, workspace_bytes, stream);
}

// p3 == nullptr: two breakpoints in separate arrays (stride 1); otherwise p1 = p, p2 = p + 1,
// p3 = p + 2 of one [C, 3] array (stride 3).
static int quantize23_impl(const float* x, const int64_t* ro, int64_t C, int64_t n, int64_t total,
                           int bits, const float* m, const float* p1, const float* p2,
                           const float* p3, int p_stride, uint8_t* codes, uint8_t* region2,
                           float* fake, int layout, void* stream) {
    if (!x || !m || !p1 || !p2 || !codes || !region2 || bits < 2 || bits > 8 ||
        (layout != PWLQ_CODES_U8 && layout != PWLQ_CODES_PACKED))
        return PWLQ_ERR_INVALID_ARG;
    if (misaligned(x, 4) || misaligned(m, 4) || misaligned(p1, 4) || misaligned(p2, 4) ||
        misaligned(fake, 4) || misaligned(ro, 8))
        return PWLQ_ERR_INVALID_ARG;
    if (total > kMaxTotal) return PWLQ_ERR_UNSUPPORTED;
    return from_cuda(pwlq::launch_quantize2(x, ro, C, n, total, bits, m, p1, p2, p3, p_stride,
                                            codes, region2, fake, layout, as_stream(stream)));
}

int pwlq_quantize2(const float* x, int64_t C, int64_t n, int bits, const float* m,
                   const float* p1, const float* p2, uint8_t* codes, uint8_t* region2,
                   float* fake_out, int code_layout, void* stream) {
    if (int rc = check_rows(C, n)) return rc;
    return quantize23_impl(x, nullptr, C, n, C * n, bits, m, p1, p2, nullptr, 1, codes, region2,
                           fake_out, code_layout, stream);
}

int pwlq_quantize2_ragged(const float* x, const int64_t* row_offsets, int64_t C, int64_t total,
                          int bits, const float* m, const float* p1, const float* p2,
                          uint8_t* codes, uint8_t* region2, float* fake_out, int code_layout,
                          void* stream) {
    if (int rc = check_rows(C, total)) return rc;
    if (!row_offsets) return PWLQ_ERR_INVALID_ARG;
    return quantize23_impl(x, row_offsets, C, 0, total, bits, m, p1, p2, nullptr, 1, codes,
                           region2, fake_out, code_layout, stream);
}

int pwlq_quantize3(const float* x, int64_t C, int64_t n, int bits, const float* m, const float* p,
                   uint8_t* codes, uint8_t* region2, float* fake_out, int code_layout,
                   void* stream) {
    if (int rc = check_rows(C, n)) return rc;
    if (!p) return PWLQ_ERR_INVALID_ARG;
    return quantize23_impl(x, nullptr, C, n, C * n, bits, m, p, p + 1, p + 2, 3, codes, region2,
                           fake_out, code_layout, stream);
}

int pwlq_quantize3_ragged(const float* x, const int64_t* row_offsets, int64_t C, int64_t total,
                          int bits, const float* m, const float* p, uint8_t* codes,
                          uint8_t* region2, float* fake_out, int code_layout, void* stream) {
    if (int rc = check_rows(C, total)) return rc;
    if (!row_offsets || !p) return PWLQ_ERR_INVALID_ARG;
    return quantize23_impl(x, row_offsets, C, 0, total, bits, m, p, p + 1, p + 2, 3, codes,
                           region2, fake_out, code_layout, stream);
}

static int dequantize23_impl(const uint8_t* codes, const uint8_t* region2, const int64_t* ro,
                             int64_t C, int64_t n, int64_t total, int bits, const float* m,
                             const float* p1, const float* p2, const float* p3, int p_stride,
                             float* y, int layout, void* stream) {
    if (!codes || !region2 || !m || !p1 || !p2 || !y || bits < 2 || bits > 8 ||
        (layout != PWLQ_CODES_U8 && layout != PWLQ_CODES_PACKED))
        return PWLQ_ERR_INVALID_ARG;
    if (misaligned(m, 4) || misaligned(p1, 4) || misaligned(p2, 4) || misaligned(y, 4) ||
        misaligned(ro, 8))
        return PWLQ_ERR_INVALID_ARG;
    if (total > kMaxTotal) return PWLQ_ERR_UNSUPPORTED;
    return from_cuda(pwlq::launch_dequantize2(codes, region2, ro, C, n, total, bits, m, p1, p2, p3,
                                              p_stride, y, layout, as_stream(stream)));
}

int pwlq_dequantize2(const uint8_t* codes, const uint8_t* region2, int64_t C, int64_t n,
                     int bits, const float* m, const float* p1, const float* p2, float* y,
                     int code_layout, void* stream) {
    if (int rc = check_rows(C, n)) return rc;
    return dequantize23_impl(codes, region2, nullptr, C, n, C * n, bits, m, p1, p2, nullptr, 1, y,
                             code_layout, stream);
}

int pwlq_dequantize2_ragged(const uint8_t* codes, const uint8_t* region2,
                            const int64_t* row_offsets, int64_t C, int64_t total, int bits,
                            const float* m, const float* p1, const float* p2, float* y,
                            int code_layout, void* stream) {
    if (int rc = check_rows(C, total)) return rc;
    if (!row_offsets) return PWLQ_ERR_INVALID_ARG;
    return dequantize23_impl(codes, region2, row_offsets, C, 0, total, bits, m, p1, p2, nullptr, 1,
                             y, code_layout, stream);
}

int pwlq_dequantize3(const uint8_t* codes, const uint8_t* region2, int64_t C, int64_t n,
                     int bits, const float* m, const float* p, float* y, int code_layout,
                     void* stream) {
    if (int rc = check_rows(C, n)) return rc;
    if (!p) return PWLQ_ERR_INVALID_ARG;
    return dequantize23_impl(codes, region2, nullptr, C, n, C * n, bits, m, p, p + 1, p + 2, 3, y,
                             code_layout, stream);
}

int pwlq_dequantize3_ragged(const uint8_t* codes, const uint8_t* region2,
                            const int64_t* row_offsets, int64_t C, int64_t total, int bits,
                            const float* m, const float* p, float* y, int code_layout,
                            void* stream) {
    if (int rc = check_rows(C, total)) return rc;
    if (!row_offsets || !p) return PWLQ_ERR_INVALID_ARG;
    return dequantize23_impl(codes, region2, row_offsets, C, 0, total, bits, m, p, p + 1, p + 2, 3,
                             y, code_layout, stream);
}

size_t pwlq_bias_workspace_bytes(int64_t C, int64_t max_n) {
    if (C < 1 || max_n < 1) return 0;
    return pwlq::bias_workspace_bytes(C, max_n);
}

static int bias_impl(const float* x, const int64_t* ro, int64_t C, int64_t n, int64_t total,
                     int64_t max_n, int bits, const float* m, const float* p, float* xi_out,
                     float* beta_out, void* ws, size_t ws_bytes, void* stream) {
    if (!x || !m || !p || !xi_out || !beta_out || bits < 2 || bits > 8 || max_n < 1)
        return PWLQ_ERR_INVALID_ARG;
    if (misaligned(x, 4) || misaligned(m, 4) || misaligned(p, 4) || misaligned(xi_out, 4) ||
        misaligned(beta_out, 4) || misaligned(ro, 8))
        return PWLQ_ERR_INVALID_ARG;
    if (total > kMaxTotal) return PWLQ_ERR_UNSUPPORTED;
    const int64_t tiles = (max_n + 8191) / 8192;
    if (C * tiles > ((int64_t)1 << 31) - 1) return PWLQ_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < pwlq::bias_workspace_bytes(C, max_n)) return PWLQ_ERR_WORKSPACE;
    if (misaligned(ws, 256)) return PWLQ_ERR_INVALID_ARG;
    return from_cuda(pwlq::launch_bias_correction(x, ro, C, n, max_n, bits, m, p, xi_out, beta_out,
                                                  ws, as_stream(stream)));
}

int pwlq_bias_correction(const float* x, int64_t C, int64_t n, int bits, const float* m,
                         const float* p, float* xi_out, float* beta_out, void* workspace,
                         size_t workspace_bytes, void* stream) {
    if (int rc = check_rows(C, n)) return rc;
    return bias_impl(x, nullptr, C, n, C * n, n, bits, m, p, xi_out, beta_out, workspace,
                     workspace_bytes, stream);
}

int pwlq_bias_correction_ragged(const float* x, const int64_t* row_offsets, int64_t C,
                                int64_t total, int64_t max_n, int bits, const float* m,
                                const float* p, float* xi_out, float* beta_out, void* workspace,
                                size_t workspace_bytes, void* stream) {
    if (int rc = check_rows(C, total)) return rc;
    if (!row_offsets || max_n > total) return PWLQ_ERR_INVALID_ARG;
    return bias_impl(x, row_offsets, C, 0, total, max_n, bits, m, p, xi_out, beta_out, workspace,
                     workspace_bytes, stream);
}

static int dequantize_bc_impl(const uint8_t* codes, const uint8_t* mask, const int64_t* ro,
                              int64_t C, int64_t n, int64_t total, int bits, const float* m,
                              const float* p, const float* xi, const float* beta, float* y,
                              int layout, void* stream) {
    if (!codes || !mask || !m || !p || !xi || !beta || !y || bits < 2 || bits > 8 ||
        (layout != PWLQ_CODES_U8 && layout != PWLQ_CODES_PACKED))
        return PWLQ_ERR_INVALID_ARG;
    if (misaligned(m, 4) || misaligned(p, 4) || misaligned(xi, 4) || misaligned(beta, 4) ||
        misaligned(y, 4) || misaligned(ro, 8))
        return PWLQ_ERR_INVALID_ARG;
    if (total > kMaxTotal) return PWLQ_ERR_UNSUPPORTED;
    return from_cuda(pwlq::launch_dequantize_bc(codes, mask, ro, C, n, total, bits, m, p, xi, beta,
                                                y, layout, as_stream(stream)));
}

int pwlq_dequantize_bc(const uint8_t* codes, const uint8_t* region_mask, int64_t C, int64_t n,
                       int bits, const float* m, const float* p, const float* xi,
                       const float* beta, float* y, int code_layout, void* stream) {
    if (int rc = check_rows(C, n)) return rc;
    return dequantize_bc_impl(codes, region_mask, nullptr, C, n, C * n, bits, m, p, xi, beta, y,
                              code_layout, stream);
}

int pwlq_dequantize_bc_ragged(const uint8_t* codes, const uint8_t* region_mask,
                              const int64_t* row_offsets, int64_t C, int64_t total, int bits,
                              const float* m, const float* p, const float* xi, const float* beta,
                              float* y, int code_layout, void* stream) {
    if (int rc = check_rows(C, total)) return rc;
    if (!row_offsets) return PWLQ_ERR_INVALID_ARG;
    return dequantize_bc_impl(codes, region_mask, row_offsets, C, 0, total, bits, m, p, xi, beta,
                              y, code_layout, stream);
}

size_t pwlq_dense_bytes(int64_t total, int bits) {
    if (total < 0 || bits < 2 || bits > 8) return 0;
    return (size_t)((total * (bits + 1) + 7) / 8);
}

int pwlq_pack_dense(const uint8_t* codes_u8, const uint8_t* region_mask, int64_t total, int bits,
                    uint8_t* stream_out, void* stream) {
    if (!codes_u8 || !region_mask || !stream_out || total < 1 || bits < 2 || bits > 8)
        return PWLQ_ERR_INVALID_ARG;
    if (total > kMaxTotal) return PWLQ_ERR_UNSUPPORTED;
    return from_cuda(pwlq::launch_pack_dense(codes_u8, region_mask, total, bits, stream_out,
                                             as_stream(stream)));
}

int pwlq_unpack_dense(const uint8_t* stream_in, int64_t total, int bits, uint8_t* codes_u8,
                      uint8_t* region_mask, void* stream) {
    if (!codes_u8 || !region_mask || !stream_in || total < 1 || bits < 2 || bits > 8)
        return PWLQ_ERR_INVALID_ARG;
    if (total > kMaxTotal) return PWLQ_ERR_UNSUPPORTED;
    return from_cuda(pwlq::launch_unpack_dense(stream_in, total, bits, codes_u8, region_mask,
                                               as_stream(stream)));
}

size_t pwlq_encode_host_scratch_bytes(int64_t C, int64_t total, int64_t max_n, int K) {
    if (C < 1 || total < 1 || max_n < 1 || K < 1 || K > PWLQ_MAX_K) return 0;
    return plan_host(C, total, max_n, K).bytes;
}

size_t pwlq_encode_host_status_offset(int64_t C, int64_t total, int64_t max_n, int K) {
    if (C < 1 || total < 1 || max_n < 1 || K < 1 || K > PWLQ_MAX_K) return 0;
    return plan_host(C, total, max_n, K).ws;
}

// lo_host == nullptr: signed scheme, m_host receives the abs-max values; otherwise one-sided ranges,
// lo_host / m_host receive the rows' lower / upper bounds.
static int encode_host_impl(const float* x_host, const int64_t* row_offsets_host, int64_t C,
                            int64_t total, int64_t max_n, int bits, const float* ratios_host,
                            int K, float* lo_host, float* m_host, float* p_host, float* err_host,
                            int32_t* idx_host, uint8_t* codes_host, uint8_t* region_mask_host,
                            int code_layout, void* dev_scratch, size_t dev_scratch_bytes,
                            float** y_dev_out, void* stream) {
    if (int rc = check_rows(C, total)) return rc;
    if (!x_host || !ratios_host || !m_host || !p_host || !idx_host || !codes_host ||
        !region_mask_host || bits < 2 || bits > 8 || K < 1 || max_n < 1 || max_n > total ||
        (code_layout != PWLQ_CODES_U8 && code_layout != PWLQ_CODES_PACKED))
        return PWLQ_ERR_INVALID_ARG;
    if (K > PWLQ_MAX_K || total > kMaxTotal) return PWLQ_ERR_UNSUPPORTED;
    int64_t n = 0;
    if (!row_offsets_host) {
        if (total % C != 0 || max_n != total / C) return PWLQ_ERR_INVALID_ARG;
        n = total / C;
    }
    const HostPlan h = plan_host(C, total, max_n, K);
    if (!dev_scratch || dev_scratch_bytes < h.bytes) return PWLQ_ERR_WORKSPACE;
    if (misaligned(dev_scratch, 256)) return PWLQ_ERR_INVALID_ARG;
    unsigned char* d = static_cast<unsigned char*>(dev_scratch);
    cudaStream_t st = as_stream(stream);
    float* dx = reinterpret_cast<float*>(d + h.x);
    int64_t* dro = row_offsets_host ? reinterpret_cast<int64_t*>(d + h.ro) : nullptr;
    float* dr = reinterpret_cast<float*>(d + h.ratios);
    float* dm = reinterpret_cast<float*>(d + h.m);
    float* dlo = lo_host ? reinterpret_cast<float*>(d + h.lo) : nullptr;
    float* dp = reinterpret_cast<float*>(d + h.p);
    float* de = reinterpret_cast<float*>(d + h.err);
    int32_t* di = reinterpret_cast<int32_t*>(d + h.idx);
    uint8_t* dc = d + h.codes;
    uint8_t* dk = d + h.mask;
    float* dy = reinterpret_cast<float*>(d + h.y);

    // The rows are independent, so the tensor is cut into up to kHostChunks runs of whole rows
    // and the three phases of a run -- copy in, compute, copy out -- overlap with those of its
    // neighbours: the input copies queue on one internal stream, the kernels on the caller's
    // stream, the output copies on a second internal stream, chained by events.  A run starts
    // at a multiple of 8 values so that its slices of every buffer are vector- and byte-aligned.
    int64_t row_b[kHostChunks + 1];
    const int nchunks = split_rows(row_offsets_host, C, n, total, row_b);
    auto flat = [&](int64_t c) { return row_offsets_host ? row_offsets_host[c] : c * n; };
    HostPipe* hp = host_pipe();
    if (!hp) return PWLQ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(hp->mu);

    cudaError_t e;
#define PWLQ_TRY(call) do { e = (call); if (e != cudaSuccess) return PWLQ_ERR_CUDA; } while (0)
    PWLQ_TRY(cudaEventRecord(hp->start, st));
    PWLQ_TRY(cudaStreamWaitEvent(hp->copy_in, hp->start, 0));
    PWLQ_TRY(cudaStreamWaitEvent(hp->copy_out, hp->start, 0));
    if (dro)
        PWLQ_TRY(cudaMemcpyAsync(dro, row_offsets_host, sizeof(int64_t) * (size_t)(C + 1),
                                 cudaMemcpyHostToDevice, hp->copy_in));
    PWLQ_TRY(cudaMemcpyAsync(dr, ratios_host, sizeof(float) * (size_t)K, cudaMemcpyHostToDevice,
                             hp->copy_in));
    const bool packed = (code_layout == PWLQ_CODES_PACKED && bits <= 4);
    for (int k = 0; k < nchunks; ++k) {
        const int64_t c0 = row_b[k], c1 = row_b[k + 1], f0 = flat(c0), f1 = flat(c1);
        const int64_t Ck = c1 - c0, tk = f1 - f0;
        const int64_t* rok = dro ? dro + c0 : nullptr;
        PWLQ_TRY(cudaMemcpyAsync(dx + f0, x_host + f0, sizeof(float) * (size_t)tk,
                                 cudaMemcpyHostToDevice, hp->copy_in));
        PWLQ_TRY(cudaEventRecord(hp->in_done[k], hp->copy_in));
        PWLQ_TRY(cudaStreamWaitEvent(st, hp->in_done[k], 0));
        uint8_t* dck = dc + (packed ? f0 / 2 : f0);
        uint8_t* dkk = dk + f0 / 8;
        if (tk > 0) {
            float* lok = dlo ? dlo + c0 : nullptr;
            if (dlo) PWLQ_TRY(pwlq::launch_minmax(dx + f0, rok, Ck, n, tk, lok, dm + c0, st, f0));
            else     PWLQ_TRY(pwlq::launch_absmax(dx + f0, rok, Ck, n, tk, dm + c0, st, f0));
            PWLQ_TRY(pwlq::launch_search(dx + f0, rok, Ck, n, tk, bits, dr, K, dm + c0, lok,
                                         dp + c0, de + c0, di + c0, nullptr, d + h.ws, h.sp, st, f0,
                                         k == 0));
            PWLQ_TRY(pwlq::launch_quantize(dx + f0, rok, Ck, n, tk, bits, dm + c0, lok, dp + c0,
                                           dck, dkk, nullptr, code_layout, st, f0));
            PWLQ_TRY(pwlq::launch_dequantize(dck, dkk, rok, Ck, n, tk, bits, dm + c0, lok,
                                             dp + c0, dy + f0, code_layout, st, f0));
        }
        PWLQ_TRY(cudaEventRecord(hp->out_ready[k], st));
        PWLQ_TRY(cudaStreamWaitEvent(hp->copy_out, hp->out_ready[k], 0));
        const size_t cbk = code_bytes(f1, bits, code_layout) - code_bytes(f0, bits, code_layout);
        const size_t mbk = (size_t)((f1 + 7) / 8 - f0 / 8);
        if (tk > 0) {
            PWLQ_TRY(cudaMemcpyAsync(codes_host + (dck - dc), dck, cbk, cudaMemcpyDeviceToHost,
                                     hp->copy_out));
            PWLQ_TRY(cudaMemcpyAsync(region_mask_host + f0 / 8, dkk, mbk, cudaMemcpyDeviceToHost,
                                     hp->copy_out));
        }
    }
    PWLQ_TRY(cudaMemcpyAsync(m_host, dm, sizeof(float) * (size_t)C, cudaMemcpyDeviceToHost,
                             hp->copy_out));
    if (lo_host)
        PWLQ_TRY(cudaMemcpyAsync(lo_host, dlo, sizeof(float) * (size_t)C, cudaMemcpyDeviceToHost,
                                 hp->copy_out));
    PWLQ_TRY(cudaMemcpyAsync(p_host, dp, sizeof(float) * (size_t)C, cudaMemcpyDeviceToHost,
                             hp->copy_out));
    if (err_host)
        PWLQ_TRY(cudaMemcpyAsync(err_host, de, sizeof(float) * (size_t)C, cudaMemcpyDeviceToHost,
                                 hp->copy_out));
    PWLQ_TRY(cudaMemcpyAsync(idx_host, di, sizeof(int32_t) * (size_t)C, cudaMemcpyDeviceToHost,
                             hp->copy_out));
    PWLQ_TRY(cudaEventRecord(hp->finished, hp->copy_out));
    PWLQ_TRY(cudaStreamWaitEvent(st, hp->finished, 0));    // the caller's stream ends the call
#undef PWLQ_TRY
    if (y_dev_out) *y_dev_out = dy;
    return PWLQ_OK;
}

int pwlq_encode_host(const float* x_host, const int64_t* row_offsets_host, int64_t C,
                     int64_t total, int64_t max_n, int bits, const float* ratios_host, int K,
                     float* m_host, float* p_host, float* err_host, int32_t* idx_host,
                     uint8_t* codes_host, uint8_t* region_mask_host, int code_layout,
                     void* dev_scratch, size_t dev_scratch_bytes, float** y_dev_out,
                     void* stream) {
    return encode_host_impl(x_host, row_offsets_host, C, total, max_n, bits, ratios_host, K,
                            nullptr, m_host, p_host, err_host, idx_host, codes_host,
                            region_mask_host, code_layout, dev_scratch, dev_scratch_bytes,
                            y_dev_out, stream);
}

int pwlq_encode_host_unsigned(const float* x_host, const int64_t* row_offsets_host, int64_t C,
                              int64_t total, int64_t max_n, int bits, const float* ratios_host,
                              int K, float* lo_host, float* hi_host, float* p_host,
                              float* err_host, int32_t* idx_host, uint8_t* codes_host,
                              uint8_t* region_mask_host, int code_layout, void* dev_scratch,
                              size_t dev_scratch_bytes, float** y_dev_out, void* stream) {
    if (!lo_host) return PWLQ_ERR_INVALID_ARG;
    return encode_host_impl(x_host, row_offsets_host, C, total, max_n, bits, ratios_host, K,
                            lo_host, hi_host, p_host, err_host, idx_host, codes_host,
                            region_mask_host, code_layout, dev_scratch, dev_scratch_bytes,
                            y_dev_out, stream);
}

size_t pwlq_select_workspace_bytes(int64_t C, int64_t n) {
    if (C < 1 || n < 1) return 0;
    return pwlq::select_workspace_bytes(C, n);
}

static int select_impl(const float* x, const int64_t* ro, int64_t C, int64_t n, int64_t total,
                       int64_t max_n, const float* m, int model, float* p_out, float* scale_out,
                       void* ws, size_t ws_bytes, void* stream) {
    if (!x || !m || !p_out || model < PWLQ_MODEL_GAUSS_APPROX || model > PWLQ_MODEL_LAPLACE ||
        max_n < 1 || max_n > total)
        return PWLQ_ERR_INVALID_ARG;
    if (misaligned(x, 4) || misaligned(m, 4) || misaligned(p_out, 4) || misaligned(scale_out, 4) ||
        misaligned(ro, 8))
        return PWLQ_ERR_INVALID_ARG;
    const int64_t tiles = (max_n + 8191) / 8192;
    if (total > kMaxTotal || C * tiles > ((int64_t)1 << 31) - 1) return PWLQ_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < pwlq::select_workspace_bytes(C, max_n)) return PWLQ_ERR_WORKSPACE;
    if (misaligned(ws, 256)) return PWLQ_ERR_INVALID_ARG;
    return from_cuda(pwlq::launch_select_analytic(x, ro, C, n, max_n, m, model, p_out, scale_out,
                                                  ws, as_stream(stream)));
}

int pwlq_select_analytic(const float* x, int64_t C, int64_t n, const float* m, int model,
                         float* p_out, float* scale_out, void* workspace, size_t workspace_bytes,
                         void* stream) {
    if (int rc = check_rows(C, n)) return rc;
    return select_impl(x, nullptr, C, n, C * n, n, m, model, p_out, scale_out, workspace,
                       workspace_bytes, stream);
}

int pwlq_select_analytic_ragged(const float* x, const int64_t* row_offsets, int64_t C,
                                int64_t total, int64_t max_n, const float* m, int model,
                                float* p_out, float* scale_out, void* workspace,
                                size_t workspace_bytes, void* stream) {
    if (int rc = check_rows(C, total)) return rc;
    if (!row_offsets) return PWLQ_ERR_INVALID_ARG;
    return select_impl(x, row_offsets, C, 0, total, max_n, m, model, p_out, scale_out, workspace,
                       workspace_bytes, stream);
}

int pwlq_device_status(void) {
    const int a = pwlq::take_absmax_timeout_flag(), q = pwlq::take_quantize_timeout_flag();
    if (a < 0 || q < 0) return 1 << PWLQ_ERR_CUDA;
    return (((a | q) & 1) ? (1 << PWLQ_ERR_TIMEOUT) : 0) |
           (((a | q) & 2) ? (1 << PWLQ_ERR_INVALID_ARG) : 0);
}

// Not part of the public interface (include/pwlq.h does not declare it): lets the test suite see
// a bounded device wait run out.  A one-warp kernel waits `polls` times (1 .. 1024) on a barrier
// nobody arrives on, sets the flag pwlq_device_status() reports, and returns.
int pwlq_selftest_expire_wait(int polls, void* stream) {
    if (polls < 1 || polls > 1024) return PWLQ_ERR_INVALID_ARG;
    return from_cuda(pwlq::launch_expire_wait(polls, as_stream(stream)));
}

const char* pwlq_status_string(int status) {
    switch (status) {
        case PWLQ_OK: return "ok";
        case PWLQ_ERR_INVALID_ARG: return "invalid argument";
        case PWLQ_ERR_UNSUPPORTED: return "size or K above the supported limit";
        case PWLQ_ERR_WORKSPACE: return "workspace missing or too small";
        case PWLQ_ERR_CUDA: return "CUDA runtime error";
        case PWLQ_ERR_NONFINITE: return "a row's range is not finite";
        case PWLQ_ERR_TIMEOUT: return "a bounded device wait expired";
        default: return "unknown status";
    }
}

const char* pwlq_version(void) { return "0.1"; }

}  // extern "C"
