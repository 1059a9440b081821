/*
 * PWLQ CPU oracle -- TEST INFRASTRUCTURE, not part of the product path.
 *
 * A plain, single-threaded, deliberately slow restatement of the piecewise
 * linear quantizer (Eq. 3) built on the uniform quantizer (Eq. 1), the
 * empirical squared quantization error (the error eps_pw = pw(r) - r defined
 * under Eq. 3), and the argmin over breakpoints (Eq. 6) restricted to a
 * user-supplied grid of K candidate ratios p/m.
 *
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg may
 * call this file.  It shares no code with the CUDA path.
 *
 * Arithmetic: every per-element quantity is IEEE binary32, one rounding per
 * operation, no fused multiply-add (compile with -ffp-contract=off); the
 * integer code is decided in binary32 so that it means the same thing on the
 * CPU and on the GPU.  Sums of squared errors are accumulated in binary64 in
 * ascending element order.
 *
 * Pinned by tests/test_oracle_*.py: a hand-worked dyadic example (Eq. 1, 3),
 * the half-step error bound implied by Eq. 2, the p = m and p = m/2 special
 * cases, an independent binary64 true-division brute force on <= 64 elements,
 * and the closed forms Eq. 5, Eq. 9, Eq. 10 and Lemma 2 on Gaussian and
 * Laplacian samples.
 *
 * Readings of the paper taken here (each listed with its reason in the
 * project's design notes):
 *   - clamp(r; rl, ru) = min(max(r, rl), ru)       (Eq. 1 prints the bounds swapped)
 *   - rounding is round-half-to-even               (Eq. 1 leaves the tie rule open)
 *   - s = Delta / (2^(b-1) - 1) inside every piece ((b-1)-bit pieces, Sec. 3.2)
 *   - the center region is closed: tail iff |r| > p (R1 = [-p, p])
 *   - (r - z) / s is evaluated as (|r| - z) * fl(L / Delta)
 *   - the stored integer is sign-magnitude: sign bit, then the (b-1)-bit level
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>

#define ORACLE_OK 0
#define ORACLE_ERR_ARG 1
#define ORACLE_ERR_NONFINITE 5

typedef struct {
    float Lf;   /* largest level of a (b-1)-bit piece, 2^(b-1) - 1 (Eq. 1: N - 1) */
    float s1;   /* step of the center pieces, p / L                               */
    float inv1; /* L / p                                                          */
    float s2;   /* step of the tail pieces, (m - p) / L                           */
    float inv2; /* L / (m - p)                                                    */
} pw_params;

/* Eq. 1, last line: s = Delta / (N - 1) with N = 2^(b-1) per piece (Sec. 3.2);
 * Delta = p for the center (range [0, p]) and m - p for the tail (range [p, m]).
 * An empty piece (Delta <= 0) gets step 0. */
static pw_params make_params(float m, float p, int bits)
{
    pw_params P;
    float d;
    P.Lf = (float)((1 << (bits - 1)) - 1);
    if (p > 0.0f) { P.s1 = p / P.Lf; P.inv1 = P.Lf / p; }
    else          { P.s1 = 0.0f;     P.inv1 = 0.0f; }
    d = m - p;
    if (d > 0.0f) { P.s2 = d / P.Lf; P.inv2 = P.Lf / d; }
    else          { P.s2 = 0.0f;     P.inv2 = 0.0f; }
    return P;
}

/* Eq. 3 applied to one value: returns the reconstructed magnitude v and writes
 * the level q, the region (1 = tail) and the clamped magnitude a. */
static float pw_elem(float x, float m, float p, const pw_params *P,
                     int *q_out, int *region_out, float *a_out)
{
    float a = fminf(fabsf(x), m);          /* clamp(|r|; 0, m), Eq. 1           */
    int tail = (a > p);                    /* R2 = (p, m], Sec. 3.2             */
    float z = tail ? p : 0.0f;             /* offsets 0 and p, Eq. 3            */
    float inv = tail ? P->inv2 : P->inv1;
    float s = tail ? P->s2 : P->s1;
    float u = a - z;
    float t = u * inv;                     /* (clamp - z) / s                   */
    float q = fminf(rintf(t), P->Lf);      /* round half to even, saturate      */
    float v = q * s;                       /* s * r_q ...                       */
    v = v + z;                             /* ... + z, Eq. 1 first line         */
    *q_out = (int)q;
    *region_out = tail;
    *a_out = a;
    return v;
}

static int64_t row_begin(const int64_t *row_offsets, int64_t n, int64_t c)
{
    return row_offsets ? row_offsets[c] : c * n;
}

/* Range [-m, m] of Sec. 3.2: m_c = max_i |x_{c,i}| for every row. */
int pwlq_oracle_absmax(const float *x, const int64_t *row_offsets, int64_t C, int64_t n,
                       float *m_out)
{
    int64_t c, i;
    if (!x || !m_out || C < 1) return ORACLE_ERR_ARG;
    for (c = 0; c < C; ++c) {
        int64_t b = row_begin(row_offsets, n, c), e = row_begin(row_offsets, n, c + 1);
        float m = 0.0f;
        for (i = b; i < e; ++i) {
            float a = fabsf(x[i]);
            if (!(a <= 3.402823466e+38f)) return ORACLE_ERR_NONFINITE;
            if (a > m) m = a;
        }
        m_out[c] = m;
    }
    return ORACLE_OK;
}

/* Empirical counterpart of Eq. 6 on a grid: for every row and every candidate
 * p_k = m * ratios[k], SSE_k = sum_i (pw(x_i) - x_i)^2; pick the first minimal k.
 * sse_f32 / sse_f64 (either may be NULL) receive all C*K sums. */
int pwlq_oracle_search(const float *x, const int64_t *row_offsets, int64_t C, int64_t n,
                       int bits, const float *ratios, int K, const float *m_in,
                       float *p_out, float *err_out, int32_t *idx_out,
                       float *sse_f32, double *sse_f64)
{
    int64_t c, i;
    int k;
    if (!x || !ratios || C < 1 || K < 1 || bits < 2 || bits > 8) return ORACLE_ERR_ARG;
    for (c = 0; c < C; ++c) {
        int64_t b = row_begin(row_offsets, n, c), e = row_begin(row_offsets, n, c + 1);
        float m = 0.0f;
        double best = 0.0;
        int best_k = 0;
        if (m_in) m = m_in[c];
        else for (i = b; i < e; ++i) {
            float a = fabsf(x[i]);
            if (!(a <= 3.402823466e+38f)) return ORACLE_ERR_NONFINITE;
            if (a > m) m = a;
        }
        if (!(m <= 3.402823466e+38f)) return ORACLE_ERR_NONFINITE;
        for (k = 0; k < K; ++k) {
            double sse = 0.0;
            if (m > 0.0f) {
                float p = m * ratios[k];
                pw_params P = make_params(m, p, bits);
                for (i = b; i < e; ++i) {
                    int q, r; float a;
                    float v = pw_elem(x[i], m, p, &P, &q, &r, &a);
                    double d = (double)v - (double)a;   /* eps_pw up to sign(r) */
                    sse += d * d;
                }
            }
            if (sse_f32) sse_f32[c * (int64_t)K + k] = (float)sse;
            if (sse_f64) sse_f64[c * (int64_t)K + k] = sse;
            if (k == 0 || sse < best) { best = sse; best_k = k; }
        }
        if (idx_out) idx_out[c] = best_k;
        if (p_out)   p_out[c] = (m > 0.0f) ? m * ratios[best_k] : 0.0f;
        if (err_out) err_out[c] = (float)best;
    }
    return ORACLE_OK;
}

/* Eq. 3 with the chosen (m, p) of each row: b-bit sign-magnitude code, region
 * bit (Sec. 4: one extra bit per value), optional reconstructed value.
 * layout 0: one byte per code.  layout 1: for bits <= 4 two codes per byte,
 * flat element 2j in the low nibble; for bits > 4 identical to layout 0.
 * region_mask: bit (i & 7) of byte (i >> 3), i the flat element index. */
int pwlq_oracle_quantize(const float *x, const int64_t *row_offsets, int64_t C, int64_t n,
                         int bits, const float *m_in, const float *p_in,
                         uint8_t *codes, uint8_t *region_mask, float *fake_out, int layout)
{
    int64_t c, i, total;
    int packed = (layout == 1 && bits <= 4);
    if (!x || !m_in || !p_in || C < 1 || bits < 2 || bits > 8) return ORACLE_ERR_ARG;
    total = row_begin(row_offsets, n, C);
    if (codes)       for (i = 0; i < (packed ? (total + 1) / 2 : total); ++i) codes[i] = 0;
    if (region_mask) for (i = 0; i < (total + 7) / 8; ++i) region_mask[i] = 0;
    for (c = 0; c < C; ++c) {
        int64_t b = row_begin(row_offsets, n, c), e = row_begin(row_offsets, n, c + 1);
        float m = m_in[c], p = p_in[c];
        pw_params P = make_params(m, p, bits);
        for (i = b; i < e; ++i) {
            int q = 0, r = 0, neg = 0, code;
            float a, v = 0.0f, y;
            if (m > 0.0f) {
                neg = (x[i] < 0.0f);
                v = pw_elem(x[i], m, p, &P, &q, &r, &a);
            }
            code = (neg << (bits - 1)) | q;
            y = neg ? -v : v;                       /* sign(r) * uni(|r|; ...) */
            if (codes) {
                if (packed) codes[i >> 1] |= (uint8_t)(code << ((i & 1) * 4));
                else        codes[i] = (uint8_t)code;
            }
            if (region_mask && r) region_mask[i >> 3] |= (uint8_t)(1u << (i & 7));
            if (fake_out) fake_out[i] = y;
        }
    }
    return ORACLE_OK;
}

/* Eq. 1 first line, r_hat = s * r_q + z, with (s, z) of the stored region. */
int pwlq_oracle_dequantize(const uint8_t *codes, const uint8_t *region_mask,
                           const int64_t *row_offsets, int64_t C, int64_t n, int bits,
                           const float *m_in, const float *p_in, float *y, int layout)
{
    int64_t c, i;
    int packed = (layout == 1 && bits <= 4);
    int qmask = (1 << (bits - 1)) - 1;
    if (!codes || !region_mask || !m_in || !p_in || !y || C < 1 || bits < 2 || bits > 8)
        return ORACLE_ERR_ARG;
    for (c = 0; c < C; ++c) {
        int64_t b = row_begin(row_offsets, n, c), e = row_begin(row_offsets, n, c + 1);
        float m = m_in[c], p = p_in[c];
        pw_params P = make_params(m, p, bits);
        for (i = b; i < e; ++i) {
            int code = packed ? ((codes[i >> 1] >> ((i & 1) * 4)) & 0xF) : codes[i];
            int r = (region_mask[i >> 3] >> (i & 7)) & 1;
            int neg = (code >> (bits - 1)) & 1;
            float q = (float)(code & qmask);
            float s = r ? P.s2 : P.s1;
            float z = r ? p : 0.0f;
            float v = q * s;
            v = v + z;
            if (!(m > 0.0f)) { v = 0.0f; neg = 0; }
            y[i] = neg ? -v : v;
        }
    }
    return ORACLE_OK;
}

/* One value, for hand-checkable tests: returns code, region, q and y. */
void pwlq_oracle_elem(float x, float m, float p, int bits,
                      int *code_out, int *region_out, int *q_out, float *y_out)
{
    pw_params P = make_params(m, p, bits);
    int q = 0, r = 0, neg = 0;
    float a, v = 0.0f;
    if (m > 0.0f) { neg = (x < 0.0f); v = pw_elem(x, m, p, &P, &q, &r, &a); }
    *code_out = (neg << (bits - 1)) | q;
    *region_out = r;
    *q_out = q;
    *y_out = neg ? -v : v;
}

/* The five per-(row, candidate) constants, for tests of Eq. 1's step. */
void pwlq_oracle_params(float m, float p, int bits, float *out5)
{
    pw_params P = make_params(m, p, bits);
    out5[0] = P.Lf; out5[1] = P.s1; out5[2] = P.inv1; out5[3] = P.s2; out5[4] = P.inv2;
}

/* ------------------------------------------------------------------------------------------
 * Analytic breakpoint selection (Sec. 3.3 and Sec. 5.1): instead of searching a grid, assume a
 * zero-mean Gaussian or Laplacian density for the row and take the breakpoint that minimises the
 * expected error of Eq. 5, i.e. the root of the stationarity condition Eq. 9 on (0, m/2), or the
 * closed-form approximation of Sec. 5.1.  All in binary64.
 *
 *   model 0: Gaussian, p = sigma * ln(0.8614 m / sigma + 0.6079)    (Sec. 5.1, read with m and p
 *            in units of sigma: the printed form p / m = ln(0.8614 m + 0.6079) exceeds 1)
 *   model 1: Gaussian, root of Eq. 9
 *   model 2: Laplacian, root of Eq. 9
 * Scale estimates (the paper does not say how the density is fitted; these are the maximum
 * likelihood fits of the zero-mean models): sigma = sqrt(mean x^2), Laplace b = mean |x|.
 * The result is clamped to (0, m/2] (the domain of Eq. 6); if Eq. 9 has no sign change there
 * (a row that is flatter than the model allows), p = m/2. */
static double model_cdf(int model, double scale, double p)
{
    if (model == 2) return 1.0 - 0.5 * exp(-p / scale);              /* Laplace, p >= 0 */
    return 0.5 * erfc(-p / (scale * 1.4142135623730951));            /* Gaussian */
}
static double model_pdf(int model, double scale, double p)
{
    if (model == 2) return 0.5 / scale * exp(-p / scale);
    return exp(-0.5 * (p / scale) * (p / scale)) / (scale * 2.5066282746310002);
}
/* Eq. 9 written as g(p) = 2 m F(p) - [2 m - p + m (m - 2 p) f(p)]; g < 0 left of the root. */
static double eq9_residual(int model, double scale, double m, double p)
{
    return 2.0 * m * model_cdf(model, scale, p)
           - (2.0 * m - p + m * (m - 2.0 * p) * model_pdf(model, scale, p));
}

double pwlq_oracle_analytic_p(double m, double scale, int model)
{
    double lo, hi, p;
    int it;
    if (!(m > 0.0) || !(scale > 0.0)) return 0.0;
    if (model == 0) {
        p = scale * log(0.8614 * (m / scale) + 0.6079);
    } else {
        lo = 0.0; hi = 0.5 * m;
        if (!(eq9_residual(model, scale, m, hi) > 0.0)) return 0.5 * m;
        for (it = 0; it < 80; ++it) {
            double mid = 0.5 * (lo + hi);
            if (eq9_residual(model, scale, m, mid) < 0.0) lo = mid; else hi = mid;
        }
        p = 0.5 * (lo + hi);
    }
    if (!(p > 0.0)) p = 0.5 * m * 1e-6;     /* the approximation's logarithm can go negative */
    if (p > 0.5 * m) p = 0.5 * m;
    return p;
}

int pwlq_oracle_select_analytic(const float *x, const int64_t *row_offsets, int64_t C, int64_t n,
                                const float *m_in, int model, float *p_out, double *scale_out)
{
    int64_t c, i;
    if (!x || !m_in || !p_out || C < 1 || model < 0 || model > 2) return ORACLE_ERR_ARG;
    for (c = 0; c < C; ++c) {
        int64_t b = row_begin(row_offsets, n, c), e = row_begin(row_offsets, n, c + 1);
        double s2 = 0.0, s1 = 0.0, scale = 0.0;
        for (i = b; i < e; ++i) {
            double v = (double)x[i];
            s2 += v * v;
            s1 += fabs(v);
        }
        if (e > b) scale = (model == 2) ? s1 / (double)(e - b) : sqrt(s2 / (double)(e - b));
        if (scale_out) scale_out[c] = scale;
        p_out[c] = (float)pwlq_oracle_analytic_p((double)m_in[c], scale, model);
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------
 * One-sided ranges (unsigned tensors such as ReLU activations; asymmetric ranges [m1, m2]).
 *
 * Sec. 3.2 (footnote to the range) says the scheme extends to asymmetric ranges [m1, m2], and
 * Eq. 1 takes the offset z = r_l and the unsigned integer domain {0, ..., 2^b - 1} for one-sided
 * distributions.  The paper does not spell the piecewise form out; the reading taken here:
 *   - a row's range [lo, hi] is shifted to [0, m] with m = hi - lo (binary32), its dense end
 *     being the lower bound (as for ReLU outputs, lo = 0);
 *   - one breakpoint p splits [0, m] into the center [0, p] and the tail (p, m];
 *   - no sign is stored, so each of the two pieces keeps the whole b-bit level set:
 *     N = 2^b levels, s = Delta / (2^b - 1) (Eq. 1 with N = 2^b);
 *   - a = min(max(x - lo, 0), m) (one binary32 subtraction, then the clamp of Eq. 1), after which
 *     the steps are those of the positive half of Eq. 3; the delivered value is y = v + lo;
 *   - the squared error is taken in the shifted domain, (v - a)^2, which for lo = 0 is the
 *     error of the delivered value itself;
 *   - a constant row (m = 0) gets code 0 everywhere and y = lo.
 * The stored integer is the b-bit level q; the region bit is kept separately as before.
 * With x >= 0 and lo = 0 this is exactly the positive half of the signed scheme at b + 1 bits
 * (same L = 2^b - 1), which is what the tests pin it to.
 */
static pw_params make_params_u(float m, float p, int bits)
{
    return make_params(m, p, bits + 1);          /* L = 2^b - 1 */
}

static float shifted_mag(float x, float lo, float m)
{
    float a = x - lo;
    a = fmaxf(a, 0.0f);
    return fminf(a, m);
}

/* Per-row minimum and maximum (the range [m1, m2]); an empty row gets lo = hi = 0. */
int pwlq_oracle_minmax(const float *x, const int64_t *row_offsets, int64_t C, int64_t n,
                       float *lo_out, float *hi_out)
{
    int64_t c, i;
    if (!x || !lo_out || !hi_out || C < 1) return ORACLE_ERR_ARG;
    for (c = 0; c < C; ++c) {
        int64_t b = row_begin(row_offsets, n, c), e = row_begin(row_offsets, n, c + 1);
        float lo = 0.0f, hi = 0.0f;
        for (i = b; i < e; ++i) {
            if (!(fabsf(x[i]) <= 3.402823466e+38f)) return ORACLE_ERR_NONFINITE;
            if (i == b || x[i] < lo) lo = x[i];
            if (i == b || x[i] > hi) hi = x[i];
        }
        lo_out[c] = lo;
        hi_out[c] = hi;
    }
    return ORACLE_OK;
}

/* Grid search of the breakpoint for one-sided ranges: p_k = m * ratios[k], m = hi - lo. */
int pwlq_oracle_search_u(const float *x, const int64_t *row_offsets, int64_t C, int64_t n,
                         int bits, const float *ratios, int K, const float *lo_in,
                         const float *hi_in, float *p_out, float *err_out, int32_t *idx_out,
                         float *sse_f32, double *sse_f64)
{
    int64_t c, i;
    int k;
    if (!x || !ratios || !lo_in || !hi_in || C < 1 || K < 1 || bits < 2 || bits > 8)
        return ORACLE_ERR_ARG;
    for (c = 0; c < C; ++c) {
        int64_t b = row_begin(row_offsets, n, c), e = row_begin(row_offsets, n, c + 1);
        float lo = lo_in[c];
        float m = hi_in[c] - lo;
        double best = 0.0;
        int best_k = 0;
        if (!(fabsf(m) <= 3.402823466e+38f) || !(fabsf(lo) <= 3.402823466e+38f))
            return ORACLE_ERR_NONFINITE;
        for (k = 0; k < K; ++k) {
            double sse = 0.0;
            if (m > 0.0f) {
                float p = m * ratios[k];
                pw_params P = make_params_u(m, p, bits);
                for (i = b; i < e; ++i) {
                    int q, r; float a;
                    float v = pw_elem(shifted_mag(x[i], lo, m), m, p, &P, &q, &r, &a);
                    double d = (double)v - (double)a;
                    sse += d * d;
                }
            }
            if (sse_f32) sse_f32[c * (int64_t)K + k] = (float)sse;
            if (sse_f64) sse_f64[c * (int64_t)K + k] = sse;
            if (k == 0 || sse < best) { best = sse; best_k = k; }
        }
        if (idx_out) idx_out[c] = best_k;
        if (p_out)   p_out[c] = (m > 0.0f) ? m * ratios[best_k] : 0.0f;
        if (err_out) err_out[c] = (float)best;
    }
    return ORACLE_OK;
}

/* One-sided quantizer: b-bit level (no sign), region bit, optional delivered value v + lo.
 * Code and mask layouts as in pwlq_oracle_quantize. */
int pwlq_oracle_quantize_u(const float *x, const int64_t *row_offsets, int64_t C, int64_t n,
                           int bits, const float *lo_in, const float *hi_in, const float *p_in,
                           uint8_t *codes, uint8_t *region_mask, float *fake_out, int layout)
{
    int64_t c, i, total;
    int packed = (layout == 1 && bits <= 4);
    if (!x || !lo_in || !hi_in || !p_in || C < 1 || bits < 2 || bits > 8) return ORACLE_ERR_ARG;
    total = row_begin(row_offsets, n, C);
    if (codes)       for (i = 0; i < (packed ? (total + 1) / 2 : total); ++i) codes[i] = 0;
    if (region_mask) for (i = 0; i < (total + 7) / 8; ++i) region_mask[i] = 0;
    for (c = 0; c < C; ++c) {
        int64_t b = row_begin(row_offsets, n, c), e = row_begin(row_offsets, n, c + 1);
        float lo = lo_in[c], p = p_in[c];
        float m = hi_in[c] - lo;
        pw_params P = make_params_u(m, p, bits);
        for (i = b; i < e; ++i) {
            int q = 0, r = 0;
            float a, v = 0.0f;
            if (m > 0.0f) v = pw_elem(shifted_mag(x[i], lo, m), m, p, &P, &q, &r, &a);
            if (codes) {
                if (packed) codes[i >> 1] |= (uint8_t)(q << ((i & 1) * 4));
                else        codes[i] = (uint8_t)q;
            }
            if (region_mask && r) region_mask[i >> 3] |= (uint8_t)(1u << (i & 7));
            if (fake_out) fake_out[i] = v + lo;
        }
    }
    return ORACLE_OK;
}

/* Inverse of the one-sided quantizer: y = (s * q + z) + lo with (s, z) of the stored region. */
int pwlq_oracle_dequantize_u(const uint8_t *codes, const uint8_t *region_mask,
                             const int64_t *row_offsets, int64_t C, int64_t n, int bits,
                             const float *lo_in, const float *hi_in, const float *p_in, float *y,
                             int layout)
{
    int64_t c, i;
    int packed = (layout == 1 && bits <= 4);
    int qmask = (1 << bits) - 1;
    if (!codes || !region_mask || !lo_in || !hi_in || !p_in || !y || C < 1 || bits < 2 || bits > 8)
        return ORACLE_ERR_ARG;
    for (c = 0; c < C; ++c) {
        int64_t b = row_begin(row_offsets, n, c), e = row_begin(row_offsets, n, c + 1);
        float lo = lo_in[c], p = p_in[c];
        float m = hi_in[c] - lo;
        pw_params P = make_params_u(m, p, bits);
        for (i = b; i < e; ++i) {
            int code = packed ? ((codes[i >> 1] >> ((i & 1) * 4)) & 0xF) : codes[i];
            int r = (region_mask[i >> 3] >> (i & 7)) & 1;
            float q = (float)(code & qmask);
            float s = r ? P.s2 : P.s1;
            float z = r ? p : 0.0f;
            float v = q * s;
            v = v + z;
            if (!(m > 0.0f)) v = 0.0f;
            y[i] = v + lo;
        }
    }
    return ORACLE_OK;
}

/* One value of the one-sided quantizer, for hand-checkable tests. */
void pwlq_oracle_elem_u(float x, float lo, float hi, float p, int bits,
                        int *code_out, int *region_out, float *y_out)
{
    float m = hi - lo;
    pw_params P = make_params_u(m, p, bits);
    int q = 0, r = 0;
    float a, v = 0.0f;
    if (m > 0.0f) v = pw_elem(shifted_mag(x, lo, m), m, p, &P, &q, &r, &a);
    *code_out = q;
    *region_out = r;
    *y_out = v + lo;
}

/* ------------------------------------------------------------------------------------------
 * Two breakpoints (Sec. 5.1, "Multiple Breakpoints"): the paper says only that more breakpoints
 * give more non-overlapping regions, each quantized uniformly, and that they are found by
 * minimising the same error in an enlarged search space.  Reading taken here: breakpoints
 * 0 < p1 < p2 <= m split [0, m] into R1 = [0, p1], R2 = (p1, p2], R3 = (p2, m]; inside every
 * region (and sign) Eq. 1 is applied with b-1 bits, range [z, z + Delta] and offset z equal to
 * the region's lower end (z = 0, p1, p2; Delta = p1, p2 - p1, m - p2), exactly as Eq. 3 does for
 * its two regions.  The stored integer is the sign-magnitude code of Eq. 3; the region index
 * (0, 1, 2) takes two bits per value: bits 2 (i & 3) and 2 (i & 3) + 1 of byte i >> 2.
 * The search minimises the empirical squared error over all pairs i < j of the K candidate ratios,
 * p1 = m * ratios[i], p2 = m * ratios[j]; the first minimal pair in the order (i, j) wins.
 * With p2 = m the scheme is the one-breakpoint scheme with p = p1, which is what the tests pin
 * it to first.
 */
typedef struct { float z[3], s[3], inv[3], Lf; } pw2_params;

static pw2_params make_params2(float m, float p1, float p2, int bits)
{
    pw2_params P;
    float d[3];
    int r;
    P.Lf = (float)((1 << (bits - 1)) - 1);
    P.z[0] = 0.0f; P.z[1] = p1; P.z[2] = p2;
    d[0] = p1; d[1] = p2 - p1; d[2] = m - p2;
    for (r = 0; r < 3; ++r) {
        if (d[r] > 0.0f) { P.s[r] = d[r] / P.Lf; P.inv[r] = P.Lf / d[r]; }
        else             { P.s[r] = 0.0f;        P.inv[r] = 0.0f; }
    }
    return P;
}

static float pw2_elem(float x, float m, float p1, float p2, const pw2_params *P,
                      int *q_out, int *region_out, float *a_out)
{
    float a = fminf(fabsf(x), m);
    int r = (a > p1) + (a > p2);
    float u = a - P->z[r];
    float t = u * P->inv[r];
    float q = fminf(rintf(t), P->Lf);
    float v = q * P->s[r];
    v = v + P->z[r];
    *q_out = (int)q;
    *region_out = r;
    *a_out = a;
    return v;
}

/* sse_f32 / sse_f64 (either may be NULL): [C, K, K], entry (i, j) valid for i < j, others 0. */
int pwlq_oracle_search2(const float *x, const int64_t *row_offsets, int64_t C, int64_t n,
                        int bits, const float *ratios, int K, const float *m_in,
                        float *p1_out, float *p2_out, float *err_out, int32_t *idx1_out,
                        int32_t *idx2_out, float *sse_f32, double *sse_f64)
{
    int64_t c, e, b, t;
    int i, j;
    if (!x || !ratios || !m_in || C < 1 || K < 2 || bits < 2 || bits > 8) return ORACLE_ERR_ARG;
    for (c = 0; c < C; ++c) {
        float m = m_in[c];
        double best = 0.0;
        int bi = 0, bj = 1, first = 1;
        b = row_begin(row_offsets, n, c);
        e = row_begin(row_offsets, n, c + 1);
        if (!(m <= 3.402823466e+38f)) return ORACLE_ERR_NONFINITE;
        for (i = 0; i < K; ++i) for (j = 0; j < K; ++j) {
            double sse = 0.0;
            if (i < j && m > 0.0f) {
                float p1 = m * ratios[i], p2 = m * ratios[j];
                pw2_params P = make_params2(m, p1, p2, bits);
                for (t = b; t < e; ++t) {
                    int q, r; float a;
                    float v = pw2_elem(x[t], m, p1, p2, &P, &q, &r, &a);
                    double d = (double)v - (double)a;
                    sse += d * d;
                }
            }
            if (sse_f32) sse_f32[(c * (int64_t)K + i) * K + j] = (float)sse;
            if (sse_f64) sse_f64[(c * (int64_t)K + i) * K + j] = sse;
            if (i < j && (first || sse < best)) { best = sse; bi = i; bj = j; first = 0; }
        }
        if (idx1_out) idx1_out[c] = bi;
        if (idx2_out) idx2_out[c] = bj;
        if (p1_out) p1_out[c] = (m > 0.0f) ? m * ratios[bi] : 0.0f;
        if (p2_out) p2_out[c] = (m > 0.0f) ? m * ratios[bj] : 0.0f;
        if (err_out) err_out[c] = (float)best;
    }
    return ORACLE_OK;
}

int pwlq_oracle_quantize2(const float *x, const int64_t *row_offsets, int64_t C, int64_t n,
                          int bits, const float *m_in, const float *p1_in, const float *p2_in,
                          uint8_t *codes, uint8_t *region2, float *fake_out, int layout)
{
    int64_t c, i, total;
    int packed = (layout == 1 && bits <= 4);
    if (!x || !m_in || !p1_in || !p2_in || C < 1 || bits < 2 || bits > 8) return ORACLE_ERR_ARG;
    total = row_begin(row_offsets, n, C);
    if (codes)   for (i = 0; i < (packed ? (total + 1) / 2 : total); ++i) codes[i] = 0;
    if (region2) for (i = 0; i < (total + 3) / 4; ++i) region2[i] = 0;
    for (c = 0; c < C; ++c) {
        int64_t b = row_begin(row_offsets, n, c), e = row_begin(row_offsets, n, c + 1);
        float m = m_in[c], p1 = p1_in[c], p2 = p2_in[c];
        pw2_params P = make_params2(m, p1, p2, bits);
        for (i = b; i < e; ++i) {
            int q = 0, r = 0, neg = 0, code;
            float a, v = 0.0f;
            if (m > 0.0f) {
                neg = (x[i] < 0.0f);
                v = pw2_elem(x[i], m, p1, p2, &P, &q, &r, &a);
            }
            code = (neg << (bits - 1)) | q;
            if (codes) {
                if (packed) codes[i >> 1] |= (uint8_t)(code << ((i & 1) * 4));
                else        codes[i] = (uint8_t)code;
            }
            if (region2) region2[i >> 2] |= (uint8_t)(r << ((i & 3) * 2));
            if (fake_out) fake_out[i] = neg ? -v : v;
        }
    }
    return ORACLE_OK;
}

int pwlq_oracle_dequantize2(const uint8_t *codes, const uint8_t *region2,
                            const int64_t *row_offsets, int64_t C, int64_t n, int bits,
                            const float *m_in, const float *p1_in, const float *p2_in, float *y,
                            int layout)
{
    int64_t c, i;
    int packed = (layout == 1 && bits <= 4);
    int qmask = (1 << (bits - 1)) - 1;
    if (!codes || !region2 || !m_in || !p1_in || !p2_in || !y || C < 1 || bits < 2 || bits > 8)
        return ORACLE_ERR_ARG;
    for (c = 0; c < C; ++c) {
        int64_t b = row_begin(row_offsets, n, c), e = row_begin(row_offsets, n, c + 1);
        float m = m_in[c];
        pw2_params P = make_params2(m, p1_in[c], p2_in[c], bits);
        for (i = b; i < e; ++i) {
            int code = packed ? ((codes[i >> 1] >> ((i & 1) * 4)) & 0xF) : codes[i];
            int r = (region2[i >> 2] >> ((i & 3) * 2)) & 3;
            int neg = (code >> (bits - 1)) & 1;
            float q = (float)(code & qmask);
            float v;
            if (r > 2) r = 2;
            v = q * P.s[r];
            v = v + P.z[r];
            if (!(m > 0.0f)) { v = 0.0f; neg = 0; }
            y[i] = neg ? -v : v;
        }
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------
 * Three breakpoints (Sec. 5.1, "Multiple Breakpoints"; Table 1 of the paper lists one, two and
 * three).  The reading is the two-breakpoint one with one more region: 0 < p1 < p2 < p3 <= m,
 * R1 = [0, p1], R2 = (p1, p2], R3 = (p2, p3], R4 = (p3, m]; inside every region (and sign) Eq. 1
 * with b-1 bits, range [z, z + Delta], offset z = the region's lower end.  Sign-magnitude code as
 * before; the region index (0..3) fills the two bits per value of the region stream.  The search
 * takes all triples i < j < k of the K candidate ratios; the first minimal triple in the order
 * (i, j, k) wins.  With p3 = m the scheme is the two-breakpoint scheme, which is what the tests
 * pin it to first.
 */
typedef struct { float z[4], s[4], inv[4], Lf; } pw3_params;

static pw3_params make_params3(float m, float p1, float p2, float p3, int bits)
{
    pw3_params P;
    float d[4];
    int r;
    P.Lf = (float)((1 << (bits - 1)) - 1);
    P.z[0] = 0.0f; P.z[1] = p1; P.z[2] = p2; P.z[3] = p3;
    d[0] = p1; d[1] = p2 - p1; d[2] = p3 - p2; d[3] = m - p3;
    for (r = 0; r < 4; ++r) {
        if (d[r] > 0.0f) { P.s[r] = d[r] / P.Lf; P.inv[r] = P.Lf / d[r]; }
        else             { P.s[r] = 0.0f;        P.inv[r] = 0.0f; }
    }
    return P;
}

static float pw3_elem(float x, float m, const pw3_params *P, int *q_out, int *region_out,
                      float *a_out)
{
    float a = fminf(fabsf(x), m);
    int r = (a > P->z[1]) + (a > P->z[2]) + (a > P->z[3]);
    float u = a - P->z[r];
    float t = u * P->inv[r];
    float q = fminf(rintf(t), P->Lf);
    float v = q * P->s[r];
    v = v + P->z[r];
    *q_out = (int)q;
    *region_out = r;
    *a_out = a;
    return v;
}

/* sse_f64 (may be NULL): [C, K, K, K], entry (i, j, k) valid for i < j < k, others 0. */
int pwlq_oracle_search3(const float *x, const int64_t *row_offsets, int64_t C, int64_t n,
                        int bits, const float *ratios, int K, const float *m_in,
                        float *p_out /* [C, 3] */, float *err_out, int32_t *idx_out /* [C, 3] */,
                        double *sse_f64)
{
    int64_t c, e, b, t;
    int i, j, k;
    if (!x || !ratios || !m_in || C < 1 || K < 3 || bits < 2 || bits > 8) return ORACLE_ERR_ARG;
    for (c = 0; c < C; ++c) {
        float m = m_in[c];
        double best = 0.0;
        int bi = 0, bj = 1, bk = 2, first = 1;
        b = row_begin(row_offsets, n, c);
        e = row_begin(row_offsets, n, c + 1);
        if (!(m <= 3.402823466e+38f)) return ORACLE_ERR_NONFINITE;
        for (i = 0; i < K; ++i) for (j = 0; j < K; ++j) for (k = 0; k < K; ++k) {
            double sse = 0.0;
            int valid = (i < j && j < k);
            if (valid && m > 0.0f) {
                pw3_params P = make_params3(m, m * ratios[i], m * ratios[j], m * ratios[k], bits);
                for (t = b; t < e; ++t) {
                    int q, r; float a;
                    float v = pw3_elem(x[t], m, &P, &q, &r, &a);
                    double d = (double)v - (double)a;
                    sse += d * d;
                }
            }
            if (sse_f64) sse_f64[((c * (int64_t)K + i) * K + j) * K + k] = sse;
            if (valid && (first || sse < best)) { best = sse; bi = i; bj = j; bk = k; first = 0; }
        }
        if (idx_out) { idx_out[3 * c] = bi; idx_out[3 * c + 1] = bj; idx_out[3 * c + 2] = bk; }
        if (p_out) {
            p_out[3 * c]     = (m > 0.0f) ? m * ratios[bi] : 0.0f;
            p_out[3 * c + 1] = (m > 0.0f) ? m * ratios[bj] : 0.0f;
            p_out[3 * c + 2] = (m > 0.0f) ? m * ratios[bk] : 0.0f;
        }
        if (err_out) err_out[c] = (float)best;
    }
    return ORACLE_OK;
}

/* p_in: [C, 3] breakpoints p1 <= p2 <= p3 <= m of every row. */
int pwlq_oracle_quantize3(const float *x, const int64_t *row_offsets, int64_t C, int64_t n,
                          int bits, const float *m_in, const float *p_in, uint8_t *codes,
                          uint8_t *region2, float *fake_out, int layout)
{
    int64_t c, i, total;
    int packed = (layout == 1 && bits <= 4);
    if (!x || !m_in || !p_in || C < 1 || bits < 2 || bits > 8) return ORACLE_ERR_ARG;
    total = row_begin(row_offsets, n, C);
    if (codes)   for (i = 0; i < (packed ? (total + 1) / 2 : total); ++i) codes[i] = 0;
    if (region2) for (i = 0; i < (total + 3) / 4; ++i) region2[i] = 0;
    for (c = 0; c < C; ++c) {
        int64_t b = row_begin(row_offsets, n, c), e = row_begin(row_offsets, n, c + 1);
        float m = m_in[c];
        pw3_params P = make_params3(m, p_in[3 * c], p_in[3 * c + 1], p_in[3 * c + 2], bits);
        for (i = b; i < e; ++i) {
            int q = 0, r = 0, neg = 0, code;
            float a, v = 0.0f;
            if (m > 0.0f) {
                neg = (x[i] < 0.0f);
                v = pw3_elem(x[i], m, &P, &q, &r, &a);
            }
            code = (neg << (bits - 1)) | q;
            if (codes) {
                if (packed) codes[i >> 1] |= (uint8_t)(code << ((i & 1) * 4));
                else        codes[i] = (uint8_t)code;
            }
            if (region2) region2[i >> 2] |= (uint8_t)(r << ((i & 3) * 2));
            if (fake_out) fake_out[i] = neg ? -v : v;
        }
    }
    return ORACLE_OK;
}

int pwlq_oracle_dequantize3(const uint8_t *codes, const uint8_t *region2,
                            const int64_t *row_offsets, int64_t C, int64_t n, int bits,
                            const float *m_in, const float *p_in, float *y, int layout)
{
    int64_t c, i;
    int packed = (layout == 1 && bits <= 4);
    int qmask = (1 << (bits - 1)) - 1;
    if (!codes || !region2 || !m_in || !p_in || !y || C < 1 || bits < 2 || bits > 8)
        return ORACLE_ERR_ARG;
    for (c = 0; c < C; ++c) {
        int64_t b = row_begin(row_offsets, n, c), e = row_begin(row_offsets, n, c + 1);
        float m = m_in[c];
        pw3_params P = make_params3(m, p_in[3 * c], p_in[3 * c + 1], p_in[3 * c + 2], bits);
        for (i = b; i < e; ++i) {
            int code = packed ? ((codes[i >> 1] >> ((i & 1) * 4)) & 0xF) : codes[i];
            int r = (region2[i >> 2] >> ((i & 3) * 2)) & 3;
            int neg = (code >> (bits - 1)) & 1;
            float q = (float)(code & qmask);
            float v = q * P.s[r];
            v = v + P.z[r];
            if (!(m > 0.0f)) { v = 0.0f; neg = 0; }
            y[i] = neg ? -v : v;
        }
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------
 * Bias correction (Sec. 5.1, "Bias Correction"): quantization shifts the mean and the variance of
 * a row; the paper compensates this by folding correction terms into the scale and the offset,
 * citing earlier work, and prints no formula.  Reading taken here: with y_i = pw(x_i) the
 * delivered value of the quantizer for row c,
 *     xi_c   = sqrt( sum_i (x_i - mean x)^2 / sum_i (y_i - mean y)^2 )     (1 if a sum is 0)
 *     beta_c = mean x - xi_c * mean y
 * and the corrected value is y'_i = xi_c * y_i + beta_c, so that the corrected row has exactly
 * the mean and the centred norm of the original row.  Means and sums in binary64 (two passes);
 * xi and beta are delivered in binary32 and applied as one binary32 multiply and one add.
 * An empty row gets xi = 1, beta = 0.
 */
int pwlq_oracle_bias_correction(const float *x, const int64_t *row_offsets, int64_t C, int64_t n,
                                int bits, const float *m_in, const float *p_in, float *xi_out,
                                float *beta_out)
{
    int64_t c, i;
    if (!x || !m_in || !p_in || !xi_out || !beta_out || C < 1 || bits < 2 || bits > 8)
        return ORACLE_ERR_ARG;
    for (c = 0; c < C; ++c) {
        int64_t b = row_begin(row_offsets, n, c), e = row_begin(row_offsets, n, c + 1);
        float m = m_in[c], p = p_in[c];
        pw_params P = make_params(m, p, bits);
        double sx = 0.0, sy = 0.0, vx = 0.0, vy = 0.0, mx, my, xi = 1.0;
        if (e <= b) { xi_out[c] = 1.0f; beta_out[c] = 0.0f; continue; }
        for (i = b; i < e; ++i) {
            int q, r; float a, v = 0.0f;
            if (m > 0.0f) v = pw_elem(x[i], m, p, &P, &q, &r, &a);
            sx += (double)x[i];
            sy += (double)((m > 0.0f && x[i] < 0.0f) ? -v : v);
        }
        mx = sx / (double)(e - b);
        my = sy / (double)(e - b);
        for (i = b; i < e; ++i) {
            int q, r; float a, v = 0.0f;
            double y;
            if (m > 0.0f) v = pw_elem(x[i], m, p, &P, &q, &r, &a);
            y = (double)((m > 0.0f && x[i] < 0.0f) ? -v : v);
            vx += ((double)x[i] - mx) * ((double)x[i] - mx);
            vy += (y - my) * (y - my);
        }
        if (vx > 0.0 && vy > 0.0) xi = sqrt(vx / vy);
        xi_out[c] = (float)xi;
        beta_out[c] = (float)(mx - xi * my);
    }
    return ORACLE_OK;
}

/* Dequantize with the folded correction: y' = xi * y + beta (binary32, two roundings). */
int pwlq_oracle_dequantize_bc(const uint8_t *codes, const uint8_t *region_mask,
                              const int64_t *row_offsets, int64_t C, int64_t n, int bits,
                              const float *m_in, const float *p_in, const float *xi_in,
                              const float *beta_in, float *y, int layout)
{
    int64_t c, i;
    int rc = pwlq_oracle_dequantize(codes, region_mask, row_offsets, C, n, bits, m_in, p_in, y,
                                    layout);
    if (rc != ORACLE_OK) return rc;
    if (!xi_in || !beta_in) return ORACLE_ERR_ARG;
    for (c = 0; c < C; ++c) {
        int64_t b = row_begin(row_offsets, n, c), e = row_begin(row_offsets, n, c + 1);
        for (i = b; i < e; ++i) {
            float t = xi_in[c] * y[i];
            y[i] = t + beta_in[c];
        }
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------
 * Dense storage: Sec. 4 counts b bits per value plus one bit for the region.  Here the two are
 * stored together as a (b+1)-bit field, field = code | region << b, value i occupying bits
 * [i (b+1), (i+1) (b+1)) of a little-endian bit stream (bit k of the stream is bit k & 7 of byte
 * k >> 3).  ceil(total (b+1) / 8) bytes.
 */
int pwlq_oracle_pack_dense(const uint8_t *codes_u8, const uint8_t *region_mask, int64_t total,
                           int bits, uint8_t *stream)
{
    int64_t i, nbytes = (total * (bits + 1) + 7) / 8;
    int k;
    if (!codes_u8 || !region_mask || !stream || bits < 2 || bits > 8 || total < 0)
        return ORACLE_ERR_ARG;
    for (i = 0; i < nbytes; ++i) stream[i] = 0;
    for (i = 0; i < total; ++i) {
        int r = (region_mask[i >> 3] >> (i & 7)) & 1;
        int field = (codes_u8[i] & ((1 << bits) - 1)) | (r << bits);
        for (k = 0; k <= bits; ++k) {
            int64_t pos = i * (bits + 1) + k;
            if ((field >> k) & 1) stream[pos >> 3] |= (uint8_t)(1u << (pos & 7));
        }
    }
    return ORACLE_OK;
}

int pwlq_oracle_unpack_dense(const uint8_t *stream, int64_t total, int bits, uint8_t *codes_u8,
                             uint8_t *region_mask)
{
    int64_t i;
    int k;
    if (!codes_u8 || !region_mask || !stream || bits < 2 || bits > 8 || total < 0)
        return ORACLE_ERR_ARG;
    for (i = 0; i < (total + 7) / 8; ++i) region_mask[i] = 0;
    for (i = 0; i < total; ++i) {
        int field = 0;
        for (k = 0; k <= bits; ++k) {
            int64_t pos = i * (bits + 1) + k;
            field |= ((stream[pos >> 3] >> (pos & 7)) & 1) << k;
        }
        codes_u8[i] = (uint8_t)(field & ((1 << bits) - 1));
        if (field >> bits) region_mask[i >> 3] |= (uint8_t)(1u << (i & 7));
    }
    return ORACLE_OK;
}
