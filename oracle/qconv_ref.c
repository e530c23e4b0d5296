/*
 * qconv_ref.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, CPU statement of what the quantized convolution path of
 * "Quantizing Convolutional Neural Networks for Low-Power High-Throughput
 * Inference Engines" (Settle et al., 2018) computes, restricted to the integer
 * special case of the paper's data type: beta is an n-bit signed integer and the
 * scale alpha is a power of two, alpha = 2^e.
 *
 * Everything here is nested loops with 64-bit accumulation, in the order the
 * paper states the steps.  There is no tiling, no fusion and no reordering.  It
 * shares no code, header, table or helper with the CUDA library; only tests, the
 * smoke check and the CPU-baseline timing leg of the benchmark may call it.
 *
 * Pinned (see tests/test_oracle_*.py): round_shift against exact rational
 * arithmetic; the convolution against an independent im2col + int64 matrix
 * product and against a float64 library convolution; saturation bounds, the
 * shift-0 identity and the "equals the float convolution when representable"
 * invariant; scale exponents against brute force; the histogram against
 * numpy.histogram on dyadic data; sums against math.fsum.
 *
 * Build: gcc -O2 -fopenmp -ffp-contract=off -fPIC -shared qconv_ref.c -o libqconv_oracle.so -lm
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---------------------------------------------------------------------------
 * Rounding of acc / 2^s to an integer (Section 3: after dividing by the scale
 * the value is rounded to the target beta; the paper does not name the mode, so
 * all four candidates are stated here; mode 0 is the default reading because
 * the paper presents the type as an extension of IEEE 754).
 *   mode 0: nearest, ties to even     mode 1: nearest, ties away from zero
 *   mode 2: nearest, ties toward +inf mode 3: floor
 * s = 0 returns acc unchanged.
 * ------------------------------------------------------------------------- */
int64_t oracle_round_shift(int64_t acc, int s, int mode)
{
    if (s <= 0) return acc;
    /* floor quotient and non-negative remainder: acc = q * 2^s + rem, 0 <= rem < 2^s */
    int64_t two_s = (int64_t)1 << s;
    int64_t q = acc / two_s;
    int64_t rem = acc - q * two_s;
    if (rem < 0) { rem += two_s; q -= 1; }
    int64_t half = two_s / 2;
    switch (mode) {
    case 0:
        if (rem > half) q += 1;
        else if (rem == half && (q % 2 != 0)) q += 1;
        break;
    case 1:
        if (rem > half) q += 1;
        else if (rem == half && acc > 0) q += 1; /* tie: away from zero; for acc<0 floor already is away */
        break;
    case 2:
        if (rem >= half) q += 1;
        break;
    case 3:
    default:
        break;
    }
    return q;
}

/* Saturation bounds of an n-bit signed integer beta.  Eq. 5 with p = n-1 gives
 * beta_max = 2^(n-1) - 1; the symmetric clamp to [-beta_max, beta_max] is the
 * epsilon = 0 requirement stated after Eq. 9.  symmetric = 0 admits -2^(n-1). */
static void sat_bounds(int n, int symmetric, int64_t *lo, int64_t *hi)
{
    *hi = ((int64_t)1 << (n - 1)) - 1;
    *lo = symmetric ? -*hi : -((int64_t)1 << (n - 1));
}

static int64_t weight_at(const int8_t *w, int layout, int K, int R, int S, int Cg,
                         int k, int r, int s, int c)
{
    /* layout 0: [K][R][S][Cg]   layout 1: [R][S][Cg][K] */
    if (layout == 0) return w[(((size_t)k * R + r) * S + s) * Cg + c];
    return w[(((size_t)r * S + s) * Cg + c) * K + k];
}

/* One output value, all steps in the paper's order:
 *   1. sum of products beta_x * beta_w (Eq. 6), taps outside the image are 0
 *   2. + bias (bias folded into the convolution, Section 3 preprocessing; bias
 *      held at the input-times-weight scale)
 *   3. + residual << t (Eq. 10 with alpha_res / alpha_acc = 2^t >= 1)
 *   4. ReLU on the wide value (threshold is chosen after the ReLU, Section 3)
 *   5. multiply by alpha_x alpha_w / alpha_z = 2^-s and round
 *   6. clamp to [-beta_max, beta_max]
 * Returns the wide value after step 4 in *wide, the clamped value as result. */
static int64_t one_output(const int8_t *x, const int8_t *w, const int32_t *bias,
                          const int32_t *shift, const int8_t *res, const int32_t *res_lshift,
                          int H, int W, int C, int K, int R, int S,
                          int stride_h, int stride_w, int pad_h, int pad_w, int groups,
                          int n_out, int symmetric, int relu, int rounding, int weight_layout,
                          int P, int Q, int n, int p, int q, int k, int64_t *wide)
{
    int Cg = C / groups;
    int Kg = K / groups;
    int grp = k / Kg;
    int64_t acc = 0;
    for (int r = 0; r < R; ++r) {
        int h = p * stride_h - pad_h + r;
        if (h < 0 || h >= H) continue;
        for (int s = 0; s < S; ++s) {
            int wq = q * stride_w - pad_w + s;
            if (wq < 0 || wq >= W) continue;
            const int8_t *xp = x + (((size_t)n * H + h) * W + wq) * C + (size_t)grp * Cg;
            for (int c = 0; c < Cg; ++c)
                acc += (int64_t)xp[c] * weight_at(w, weight_layout, K, R, S, Cg, k, r, s, c);
        }
    }
    if (bias) acc += (int64_t)bias[k];
    if (res) {
        int64_t rv = res[(((size_t)n * P + p) * Q + q) * K + k];
        acc += rv * ((int64_t)1 << res_lshift[k]);
    }
    if (relu && acc < 0) acc = 0;
    *wide = acc;
    int64_t v = oracle_round_shift(acc, shift ? shift[k] : 0, rounding);
    int64_t lo, hi;
    sat_bounds(n_out, symmetric, &lo, &hi);
    if (v < lo) v = lo;
    if (v > hi) v = hi;
    return v;
}

static void store_output(void *y, int out_mode, size_t idx, int64_t v, int64_t wide,
                         const int32_t *acc_exp, int k)
{
    if (out_mode == 0) {
        ((int8_t *)y)[idx] = (int8_t)v;
    } else if (out_mode == 1) {
        ((int32_t *)y)[idx] = (int32_t)wide;
    } else {
        /* beta -> float: multiply by the scale (Section 3).  The integer is first
         * converted to binary32 (round to nearest even), then scaled exactly. */
        float f = (float)wide;
        ((float *)y)[idx] = ldexpf(f, acc_exp ? acc_exp[k] : 0);
    }
}

/* Full layer.  x: int8 [N][H][W][C]; y: [N][P][Q][out_c_pitch] with the K
 * channels of this layer at channel offset out_c_offset (concat written in
 * place, Section 3); res: int8 [N][P][Q][K] or NULL.
 * out_mode 0: int8 after steps 1-6; 1: int32 wide value after step 4;
 * 2: float32 = wide value * 2^acc_exp[k]. */
void oracle_qconv(const int8_t *x, const int8_t *w, const int32_t *bias, const int32_t *shift,
                  const int8_t *res, const int32_t *res_lshift, const int32_t *acc_exp, void *y,
                  int N, int H, int W, int C, int K, int R, int S,
                  int stride_h, int stride_w, int pad_h, int pad_w, int groups,
                  int n_out, int symmetric, int relu, int rounding, int out_mode,
                  int out_c_offset, int out_c_pitch, int weight_layout)
{
    int P = (H + 2 * pad_h - R) / stride_h + 1;
    int Q = (W + 2 * pad_w - S) / stride_w + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int p = 0; p < P; ++p)
            for (int q = 0; q < Q; ++q)
                for (int k = 0; k < K; ++k) {
                    int64_t wide;
                    int64_t v = one_output(x, w, bias, shift, res, res_lshift, H, W, C, K, R, S,
                                           stride_h, stride_w, pad_h, pad_w, groups, n_out,
                                           symmetric, relu, rounding, weight_layout, P, Q,
                                           n, p, q, k, &wide);
                    size_t idx = (((size_t)n * P + p) * Q + q) * out_c_pitch + out_c_offset + k;
                    store_output(y, out_mode, idx, v, wide, acc_exp, k);
                }
}

/* The same computation for a list of output coordinates only (n, p, q, k per
 * point); out has one entry per point, densely packed, typed by out_mode.
 * Used to check full-size layers on sampled outputs. */
void oracle_qconv_points(const int8_t *x, const int8_t *w, const int32_t *bias,
                         const int32_t *shift, const int8_t *res, const int32_t *res_lshift,
                         const int32_t *acc_exp, void *out, const int32_t *points, size_t npoints,
                         int N, int H, int W, int C, int K, int R, int S,
                         int stride_h, int stride_w, int pad_h, int pad_w, int groups,
                         int n_out, int symmetric, int relu, int rounding, int out_mode,
                         int weight_layout)
{
    (void)N;
    int P = (H + 2 * pad_h - R) / stride_h + 1;
    int Q = (W + 2 * pad_w - S) / stride_w + 1;
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < npoints; ++i) {
        int n = points[4 * i], p = points[4 * i + 1], q = points[4 * i + 2], k = points[4 * i + 3];
        int64_t wide;
        int64_t v = one_output(x, w, bias, shift, res, res_lshift, H, W, C, K, R, S,
                               stride_h, stride_w, pad_h, pad_w, groups, n_out, symmetric, relu,
                               rounding, weight_layout, P, Q, n, p, q, k, &wide);
        store_output(out, out_mode, i, v, wide, acc_exp, k);
    }
}

/* ---------------------------------------------------------------------------
 * Scale exponent: alpha = 2^e with the smallest integer e such that the
 * threshold gamma = alpha * beta_max (relation stated before Eq. 5) does not
 * clip the measured gamma:  e = min { e : beta_max * 2^e >= gamma }.
 * gamma = 0 (or not finite / negative) gives e = 0.
 * ------------------------------------------------------------------------- */
int oracle_scale_exponent(float gamma, int n)
{
    if (!(gamma > 0.0f) || isinf(gamma)) return 0;
    double g = (double)gamma;
    double bmax = (double)(((int64_t)1 << (n - 1)) - 1);
    int e = 0;
    while (ldexp(bmax, e) < g) e += 1;          /* exact: powers of two times a small integer */
    while (ldexp(bmax, e - 1) >= g) e -= 1;
    return e;
}

/* float -> beta (Section 3): clamp to [-gamma', gamma'] with gamma' = beta_max * 2^e,
 * divide by the scale, round to nearest even, clamp to +-beta_max.
 * NaN maps to 0; +-Inf clamp to +-beta_max. */
static int8_t quantize_one(float v, int e, int n)
{
    float bmax = (float)(((int32_t)1 << (n - 1)) - 1);
    float gam = ldexpf(bmax, e);
    if (isnan(v)) return 0;
    if (v > gam) v = gam;
    if (v < -gam) v = -gam;
    float scaled = ldexpf(v, -e);
    float r = nearbyintf(scaled);               /* default rounding mode: nearest even */
    if (r > bmax) r = bmax;
    if (r < -bmax) r = -bmax;
    return (int8_t)r;
}

void oracle_quantize_f32(const float *x, size_t count, int e, int n, int8_t *y)
{
    for (size_t i = 0; i < count; ++i) y[i] = quantize_one(x[i], e, n);
}

/* Weights: threshold = max |w| per output channel (Section 3), or over the whole
 * tensor when per_channel = 0.  w is [K][R][S][Cg] (layout 0) or [R][S][Cg][K]
 * (layout 1); wq has the same layout; e_w receives K exponents. */
void oracle_quantize_weights(const float *w, int K, int R, int S, int Cg, int layout,
                             int per_channel, int n, int8_t *wq, int32_t *e_w)
{
    size_t per_k = (size_t)R * S * Cg;
    float gmax_all = 0.0f;
    for (int k = 0; k < K; ++k) {
        float g = 0.0f;
        for (size_t j = 0; j < per_k; ++j) {
            size_t idx = layout == 0 ? (size_t)k * per_k + j : j * (size_t)K + k;
            float a = fabsf(w[idx]);
            if (isfinite(a) && a > g) g = a;
        }
        if (g > gmax_all) gmax_all = g;
        e_w[k] = oracle_scale_exponent(g, n);
    }
    if (!per_channel) {
        int e = oracle_scale_exponent(gmax_all, n);
        for (int k = 0; k < K; ++k) e_w[k] = e;
    }
    for (int k = 0; k < K; ++k)
        for (size_t j = 0; j < per_k; ++j) {
            size_t idx = layout == 0 ? (size_t)k * per_k + j : j * (size_t)K + k;
            wq[idx] = quantize_one(w[idx], e_w[k], n);
        }
}

/* Bias at the input-times-weight scale (Section 3 lets the bias threshold be a
 * function of the input and weight thresholds): round-to-nearest-even of
 * b / 2^(e_x + e_w[k]), saturated to int32. */
void oracle_quantize_bias(const float *b, int K, int e_x, const int32_t *e_w, int32_t *bq)
{
    for (int k = 0; k < K; ++k) {
        double v = ldexp((double)b[k], -(e_x + e_w[k]));
        double r = nearbyint(v);
        if (isnan(r)) r = 0.0;
        if (r > 2147483647.0) r = 2147483647.0;
        if (r < -2147483648.0) r = -2147483648.0;
        bq[k] = (int32_t)r;
    }
}

/* ---------------------------------------------------------------------------
 * Calibration statistics over one batch of float activations (Algorithm 1 opens
 * with hist(abs(x)); Section 3 names the maximum as the default threshold).
 * range_hi <= 0: the histogram range is [0, max|x|].  Non-finite values are
 * counted apart and excluded.  Bin index is a single fp32 product truncated:
 * bin = min(nbins-1, (int)(|x| * inv_w)), inv_w = (float)nbins / hi in fp32;
 * hi = 0 puts every finite value in bin 0.
 * ------------------------------------------------------------------------- */
void oracle_calib_stats(const float *x, size_t count, int nbins, float range_hi,
                        float *maxabs_out, uint64_t *hist, uint64_t *finite_out,
                        uint64_t *nonfinite_out, double *sum_out, double *sumsq_out)
{
    float maxabs = 0.0f;
    uint64_t finite = 0, nonfinite = 0;
    double sum = 0.0, sumsq = 0.0;
    for (size_t i = 0; i < count; ++i) {
        float v = x[i];
        if (!isfinite(v)) { nonfinite += 1; continue; }
        finite += 1;
        float a = fabsf(v);
        if (a > maxabs) maxabs = a;
        sum += (double)v;
        sumsq += (double)v * (double)v;
    }
    float hi = range_hi > 0.0f ? range_hi : maxabs;
    for (int b = 0; b < nbins; ++b) hist[b] = 0;
    float inv_w = hi > 0.0f ? (float)nbins / hi : 0.0f;
    for (size_t i = 0; i < count; ++i) {
        float v = x[i];
        if (!isfinite(v)) continue;
        float t = fabsf(v) * inv_w;
        int b = t >= (float)nbins ? nbins - 1 : (int)t;
        if (b > nbins - 1) b = nbins - 1;
        hist[b] += 1;
    }
    *maxabs_out = maxabs;
    *finite_out = finite;
    *nonfinite_out = nonfinite;
    *sum_out = sum;
    *sumsq_out = sumsq;
}

/* int8 max-pool, NHWC; taps outside the image are ignored.  Max commutes with
 * the monotone requantization, so pooling acts on the int8 codes. */
void oracle_maxpool_i8(const int8_t *x, int8_t *y, int N, int H, int W, int C,
                       int R, int S, int stride, int pad)
{
    int P = (H + 2 * pad - R) / stride + 1;
    int Q = (W + 2 * pad - S) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int p = 0; p < P; ++p)
            for (int q = 0; q < Q; ++q)
                for (int c = 0; c < C; ++c) {
                    int m = -128;
                    for (int r = 0; r < R; ++r) {
                        int h = p * stride - pad + r;
                        if (h < 0 || h >= H) continue;
                        for (int s = 0; s < S; ++s) {
                            int wq = q * stride - pad + s;
                            if (wq < 0 || wq >= W) continue;
                            int v = x[(((size_t)n * H + h) * W + wq) * C + c];
                            if (v > m) m = v;
                        }
                    }
                    y[(((size_t)n * P + p) * Q + q) * C + c] = (int8_t)m;
                }
}

/* Eltwise addition with per-input scales (Eq. 10): z = alpha_z * sum_i (alpha_xi / alpha_z) beta_xi
 * with alpha_xi <= alpha_z.  With power-of-two scales the sum is formed exactly at the finest input
 * scale -- wide = sum_i beta_xi * 2^lshift[i], lshift[i] = e_i - min_j e_j -- then ReLU (optional, on
 * the wide value), division by 2^rshift = alpha_z / alpha_min with rounding, and the symmetric clamp. */
void oracle_eltwise_add(const int8_t *const *inputs, int n_inputs, const int32_t *lshift, int rshift,
                        int relu, int rounding, int n_out, int symmetric, size_t count, int8_t *y)
{
    int64_t lo, hi;
    sat_bounds(n_out, symmetric, &lo, &hi);
    for (size_t j = 0; j < count; ++j) {
        int64_t wide = 0;
        for (int i = 0; i < n_inputs; ++i)
            wide += (int64_t)inputs[i][j] * ((int64_t)1 << lshift[i]);
        if (relu && wide < 0) wide = 0;
        int64_t v = oracle_round_shift(wide, rshift, rounding);
        if (v < lo) v = lo;
        if (v > hi) v = hi;
        y[j] = (int8_t)v;
    }
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
