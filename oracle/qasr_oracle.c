/*
 * CPU oracle for the integer-only inference path of Q-ASR (arXiv 2103.16827).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition of what the
 * GPU library must compute.  It shares no code, header, table or constant with
 * the CUDA sources, is never linked into the product library, and is only ever
 * called from the tests, from the smoke check and from the benchmark's CPU
 * baseline leg.
 *
 * Every function is the textbook definition written as nested loops with 64-bit
 * intermediates; the only parallelism is an OpenMP loop over independent
 * (batch, output-channel) rows.  No blocking, no SIMD intrinsics, no reordering.
 *
 * Passages followed:
 *   - Sec. 2.1, Eq. 1: uniform symmetric quantisation, q in [-2^(b-1), 2^(b-1)-1],
 *     and the dequantiser DQ(q, S) = S*q.
 *   - Sec. 2.2: integer convolution on (q_W, q_x) by linearity, ReLU on integers,
 *     BatchNorm folded into the preceding convolution (so a layer is
 *     integer conv + int32 bias).
 *   - The paper does not print the requantisation step.  The reading used here is
 *     the dyadic one of the integer-only works it cites: an int32 accumulator is
 *     multiplied by an integer multiplier, shifted right with round-half-up, and
 *     clamped to int8:  sat8( floor( (acc*mult + 2^(shift-1)) / 2^shift ) ).
 *   - Residual branches sit at different scales; each int8 term is rescaled by
 *     its own dyadic number (rounded on its own), the rescaled terms are summed,
 *     then ReLU, then the clamp to int8.
 *
 * Pins (see tests/test_oracle_*.py): exact rational arithmetic for the rounding
 * shift, float64 library convolution for the integer convolution (all values
 * are far below 2^53 so float64 is exact), shifted-copy and identity cases,
 * saturation boundaries, BN-fold equivalence, 1-LSB bound against float
 * rescaling.
 *
 * qo_glu: parity unpinned (the paper gives no coefficients for its polynomial
 * non-linearities; only the closeness of the gate to a true sigmoid is tested).
 */
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define QO_OK 0
#define QO_ERR_ARG (-1)
#define QO_ERR_OVERFLOW (-2)
#define QO_ERR_NOMEM (-3)

int qo_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* RS(v, c) = floor((v + 2^(c-1)) / 2^c): add half, then floor division.
 * Floor division is written out so that nothing depends on how the compiler
 * shifts negative numbers. Ties go toward +infinity. Requires 1 <= c <= 62. */
int64_t qo_rs(int64_t v, int c) {
    int64_t d = (int64_t)1 << c;
    int64_t n = v + (d >> 1);
    int64_t q = n / d; /* C division truncates toward zero */
    if ((n % d) != 0 && n < 0) q -= 1;
    return q;
}

/* clamp to the b = 8 integer grid of Eq. 1: [-128, 127] */
int64_t qo_sat8(int64_t v) {
    if (v > 127) return 127;
    if (v < -128) return -128;
    return v;
}

static int out_len(int T, int K, int stride, int dilation) {
    (void)K; (void)dilation; /* "same" padding: pad = dilation*(K-1)/2 on both sides */
    return (T - 1) / stride + 1;
}

/*
 * Integer 1-D convolution (cross-correlation, no kernel flip), zero padding
 * pad = dilation*(K-1)/2 on both sides, K odd.
 *
 *   depthwise == 0:  acc[b,o,t] = bias[o] + sum_{i<C_in} sum_{k<K} w[o,i,k] * x[b,i,t*stride + k*dilation - pad]
 *                    w is [C_out][C_in][K]   (K == 1 is the pointwise 1x1 conv)
 *   depthwise != 0:  C_out == C_in, acc[b,c,t] = bias[c] + sum_k w[c,k] * x[b,c,t*stride + k*dilation - pad]
 *                    w is [C][K]
 *
 * x is [B][C_in][T] int8, acc is [B][C_out][T_out] int32, T_out = (T-1)/stride + 1.
 * bias may be NULL.  Sums are carried in int64 and checked to fit int32.
 */
int qo_conv1d(const int8_t* x, int B, int C_in, int T,
              const int8_t* w, int C_out, int K, int stride, int dilation, int depthwise,
              const int32_t* bias, int32_t* acc) {
    if (!x || !w || !acc || B <= 0 || C_in <= 0 || C_out <= 0 || T <= 0) return QO_ERR_ARG;
    if (K <= 0 || (K % 2) == 0 || stride <= 0 || dilation <= 0) return QO_ERR_ARG;
    if (depthwise && C_in != C_out) return QO_ERR_ARG;
    const int pad = dilation * (K - 1) / 2;
    const int T_out = out_len(T, K, stride, dilation);
    int status = QO_OK;

#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b) {
        for (int o = 0; o < C_out; ++o) {
            int64_t* row = (int64_t*)malloc((size_t)T_out * sizeof(int64_t));
            if (!row) {
#pragma omp atomic write
                status = QO_ERR_NOMEM;
                continue;
            }
            const int64_t b0 = bias ? (int64_t)bias[o] : 0;
            for (int t = 0; t < T_out; ++t) row[t] = b0;
            const int i_lo = depthwise ? o : 0;
            const int i_hi = depthwise ? o + 1 : C_in;
            for (int i = i_lo; i < i_hi; ++i) {
                const int8_t* xr = x + ((size_t)b * C_in + i) * T;
                const int8_t* wr = depthwise ? w + (size_t)o * K
                                             : w + ((size_t)o * C_in + i) * K;
                for (int k = 0; k < K; ++k) {
                    const int64_t wk = wr[k];
                    const int off = k * dilation - pad;
                    for (int t = 0; t < T_out; ++t) {
                        const int ti = t * stride + off;
                        if (ti >= 0 && ti < T) row[t] += wk * (int64_t)xr[ti];
                    }
                }
            }
            int32_t* ar = acc + ((size_t)b * C_out + o) * T_out;
            for (int t = 0; t < T_out; ++t) {
                if (row[t] > INT32_MAX || row[t] < INT32_MIN) {
#pragma omp atomic write
                    status = QO_ERR_OVERFLOW;
                    ar[t] = 0;
                } else {
                    ar[t] = (int32_t)row[t];
                }
            }
            free(row);
        }
    }
    return status;
}

/* y[b,c,t] = sat8( relu?( RS(acc[b,c,t] * mult[c], shift[c]) ) ), per-channel mult/shift */
int qo_requant(const int32_t* acc, int B, int C, int T,
               const int32_t* mult, const uint8_t* shift, int relu, int8_t* y) {
    if (!acc || !mult || !shift || !y || B <= 0 || C <= 0 || T <= 0) return QO_ERR_ARG;
    for (int c = 0; c < C; ++c)
        if (shift[c] < 1 || shift[c] > 62 || mult[c] < 0) return QO_ERR_ARG;
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b) {
        for (int c = 0; c < C; ++c) {
            const size_t base = ((size_t)b * C + c) * T;
            for (int t = 0; t < T; ++t) {
                int64_t v = qo_rs((int64_t)acc[base + t] * (int64_t)mult[c], shift[c]);
                if (relu && v < 0) v = 0;
                y[base + t] = (int8_t)qo_sat8(v);
            }
        }
    }
    return QO_OK;
}

/* y[i] = sat8( relu?( sum_j RS(term_j[i] * mult[j], shift[j]) ) ), per-term mult/shift,
 * every term rounded on its own before the sum. n = number of elements. */
int qo_residual_add(int n_terms, const int8_t* const* terms, const int32_t* mult,
                    const uint8_t* shift, size_t n, int relu, int8_t* y) {
    if (n_terms <= 0 || !terms || !mult || !shift || !y) return QO_ERR_ARG;
    for (int j = 0; j < n_terms; ++j)
        if (!terms[j] || shift[j] < 1 || shift[j] > 62 || mult[j] < 0) return QO_ERR_ARG;
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < n; ++i) {
        int64_t s = 0;
        for (int j = 0; j < n_terms; ++j)
            s += qo_rs((int64_t)terms[j][i] * (int64_t)mult[j], shift[j]);
        if (relu && s < 0) s = 0;
        y[i] = (int8_t)qo_sat8(s);
    }
    return QO_OK;
}

/* DQ of Eq. 1's inverse on the last layer: out = float(acc) * scale[c], one fp32 multiply */
int qo_dequant(const int32_t* acc, int B, int C, int T, const float* scale, float* out) {
    if (!acc || !scale || !out || B <= 0 || C <= 0 || T <= 0) return QO_ERR_ARG;
    for (int b = 0; b < B; ++b)
        for (int c = 0; c < C; ++c) {
            const size_t base = ((size_t)b * C + c) * T;
            for (int t = 0; t < T; ++t) {
                volatile float a = (float)acc[base + t]; /* keep the int->float rounding separate */
                out[base + t] = a * scale[c];
            }
        }
    return QO_OK;
}

/* Integer gate for the GLU of the Conformer convolution module.  The paper says
 * the non-linearities are replaced by 2nd-order polynomials but prints no
 * coefficients, so this function is the library's own definition (parity with
 * the paper unpinned): a piecewise-quadratic sigmoid on the integer grid.
 *   u = min(|q|, q_c);  p = q_c - u;  g = 2*q_c^2 - p^2
 *   sig_int(q) = q >= 0 ? g : 2*q_c^2 - g        (in [0, 2*q_c^2], approx 2*q_c^2 * sigmoid)
 *   y = sat8( RS( a * sig_int(q) * mult[c], shift[c] ) )
 * a and q are the two int8 halves [B][C][T] of the expansion output. */
int qo_glu(const int8_t* a, const int8_t* q, int B, int C, int T, int q_c,
           const int32_t* mult, const uint8_t* shift, int8_t* y) {
    if (!a || !q || !mult || !shift || !y || B <= 0 || C <= 0 || T <= 0 || q_c <= 0 || q_c > 128)
        return QO_ERR_ARG;
    for (int c = 0; c < C; ++c)
        if (shift[c] < 1 || shift[c] > 62 || mult[c] < 0) return QO_ERR_ARG;
    for (int b = 0; b < B; ++b)
        for (int c = 0; c < C; ++c) {
            const size_t base = ((size_t)b * C + c) * T;
            for (int t = 0; t < T; ++t) {
                int64_t qq = q[base + t];
                int64_t u = qq < 0 ? -qq : qq;
                if (u > q_c) u = q_c;
                int64_t p = q_c - u;
                int64_t full = 2 * (int64_t)q_c * q_c;
                int64_t g = full - p * p;
                int64_t sig = qq >= 0 ? g : full - g;
                int64_t v = qo_rs((int64_t)a[base + t] * sig * (int64_t)mult[c], shift[c]);
                y[base + t] = (int8_t)qo_sat8(v);
            }
        }
    return QO_OK;
}
