/*
 * CPU oracle for low-bit floating-point quantized layers.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against.  It shares no code, table or constant with
 * the CUDA path, and nothing in the product imports it: only the tests, the
 * smoke check and the benchmark's CPU-baseline leg call it.
 *
 * What it follows (paper = "Low-Bitwidth Floating Point Quantization for
 * Efficient High-Quality Diffusion Models"):
 *   - number format           Sec. IV-B, the format equation
 *                             f = (-1)^s 2^(p-b) (1 + d_1/2 + ... + d_m/2^m)
 *   - clipping value c        Sec. IV-B, c = (2 - 2^-m) 2^(2^e - b - 1)
 *   - round to nearest        Sec. IV-B, X_fp = clamp(s_i round(X'/s_i); -c, c)
 *   - per-element step s_i    Sec. IV-B, the two-case equation for s_i
 *   - learned rounding        Sec. V-B, W_q = clamp(s (floor(W/s) + sigma(alpha)); -c, c)
 *                             with sigma(alpha) hardened to 0 or 1 at inference;
 *                             the soft form and its derivative for the learning step
 *   - the quantized layer     Sec. V-B (Y = W A), Sec. VI-A (conv and linear
 *                             weights and activations are quantized, everything
 *                             else stays FP32)
 *
 * Readings taken where the paper is silent (all listed in the design notes):
 *   - the input is first divided by the scale as  t = x * (1.0f / scale)  in
 *     FP32 (one IEEE division per channel/tensor, one IEEE multiply per
 *     element); everything after that is exact in double;
 *   - ties of round() go to the even multiple of the step;
 *   - floor() in learned rounding acts on the signed value (toward -inf) and the
 *     step is the one of the input's own binade;
 *   - a zero result is always the code 0 (plus zero); NaN maps to code 0;
 *   - FPQ_SAT_NATIVE lowers c to the largest finite value of the OCP FP8 type
 *     with the same (e, m) (E4M3: top mantissa pattern of the top exponent is
 *     not used; E5M2: the top exponent is not used).
 *
 * Code layout of one value: bit (e+m) sign, bits [m, e+m) exponent field p,
 * bits [0, m) mantissa d.  4-bit codes are packed two per byte, even index in
 * the low nibble.  Rounding bits: 1 bit per weight, LSB first along K, every
 * row padded to a whole byte.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define SAT_PAPER 0
#define SAT_NATIVE 1

typedef struct {
    int32_t e, m, B, sat;
} ofmt;

/* ---- format ------------------------------------------------------------ */

/* Value of the magnitude part of a code (sign bit ignored). Format equation;
 * exponent field 0 holds the subnormals d * 2^(1-B-m) (the "otherwise" branch
 * of the step equation). */
static double mag_value(int mcode, ofmt f)
{
    int p = (mcode >> f.m) & ((1 << f.e) - 1);
    int d = mcode & ((1 << f.m) - 1);
    if (p == 0)
        return ldexp((double)d, 1 - f.B - f.m);
    return ldexp(1.0 + ldexp((double)d, -f.m), p - f.B);
}

double fpq_o_decode(int code, int e, int m, int B)
{
    ofmt f = {e, m, B, SAT_PAPER};
    double v = mag_value(code & ((1 << (e + m)) - 1), f);
    return ((code >> (e + m)) & 1) ? -v : v;
}

/* Clipping value c. */
double fpq_o_cmax(int e, int m, int B, int sat)
{
    int top = (1 << e) - 1;
    if (sat == SAT_NATIVE && e == 4 && m == 3)
        return ldexp(2.0 - 2.0 * ldexp(1.0, -m), top - B);
    if (sat == SAT_NATIVE && e == 5 && m == 2)
        return ldexp(2.0 - ldexp(1.0, -m), top - 1 - B);
    return ldexp(2.0 - ldexp(1.0, -m), top - B);
}

/* Step of the grid around the (clipped) value a. */
static double step_of(double a, ofmt f)
{
    if (a == 0.0)
        return ldexp(1.0, 1 - f.B - f.m);
    int ex;
    (void)frexp(fabs(a), &ex); /* |a| = frac * 2^ex, frac in [0.5, 1) */
    int fl = ex - 1;           /* floor(log2 |a|), exact */
    if (fl + f.B < 1)
        return ldexp(1.0, 1 - f.B - f.m);
    return ldexp(1.0, fl - f.m);
}

/* Code of a value that lies on the grid: search the decoded magnitudes. */
static int encode_exact(double q, ofmt f)
{
    if (q == 0.0)
        return 0;
    double aq = fabs(q);
    int ncodes = 1 << (f.e + f.m);
    for (int c = 0; c < ncodes; ++c)
        if (mag_value(c, f) == aq)
            return c | ((q < 0.0) ? (1 << (f.e + f.m)) : 0);
    return -1; /* not on the grid: a bug in the caller */
}

/* One element, value domain: the grid value q (in units of the scale) that the
 * scaled input t = x * (1.0f / scale) is rounded to.  h < 0: round to nearest
 * (ties to even); h = 0 / 1: learned rounding with the hardened decision h.
 * *nan is set (and 0 returned) when the scaled input is NaN. */
static double quantize_value(float x, float scale, ofmt f, int h, int *nan)
{
    volatile float r = 1.0f / scale;
    volatile float t = x * r;
    if (t != t) {
        if (nan)
            *nan = 1;
        return 0.0;
    }
    double c = fpq_o_cmax(f.e, f.m, f.B, f.sat);
    double a = (double)t;
    if (a > c)
        a = c;
    if (a < -c)
        a = -c;
    double s = step_of(a, f);
    double k;
    if (h < 0)
        k = nearbyint(a / s); /* default rounding mode: ties to even */
    else
        k = floor(a / s) + (double)h;
    double q = k * s;
    if (q > c)
        q = c;
    if (q < -c)
        q = -c;
    return q;
}

/* One element: the code of that grid value. */
int fpq_o_quantize_one(float x, float scale, int e, int m, int B, int sat, int h, int *nan)
{
    ofmt f = {e, m, B, sat};
    int isnan = 0;
    double q = quantize_value(x, scale, f, h, &isnan);
    if (isnan) {
        if (nan)
            *nan = 1;
        return 0;
    }
    return encode_exact(q, f);
}

static void put_code(uint8_t *codes, int64_t row_bytes, int64_t n, int64_t k, int bits, int code)
{
    if (bits == 8) {
        codes[n * row_bytes + k] = (uint8_t)code;
    } else {
        uint8_t *p = &codes[n * row_bytes + k / 2];
        if (k & 1)
            *p = (uint8_t)((*p & 0x0F) | (code << 4));
        else
            *p = (uint8_t)((*p & 0xF0) | (code & 0x0F));
    }
}

static int get_code(const uint8_t *codes, int64_t row_bytes, int64_t n, int64_t k, int bits)
{
    if (bits == 8)
        return codes[n * row_bytes + k];
    uint8_t b = codes[n * row_bytes + k / 2];
    return (k & 1) ? (b >> 4) : (b & 0x0F);
}

static int code_bits(int e, int m) { return (1 + e + m <= 4) ? 4 : 8; }

/* Weights [N][K], one scale per row.  rounding_bits may be NULL (round to
 * nearest).  codes: [N][K] bytes or [N][ceil(K/2)] packed nibbles.
 * Returns the number of NaN inputs seen. */
int64_t fpq_o_quantize_weight(const float *w, int64_t N, int64_t K, const float *scale, int e, int m,
                              int B, int sat, const uint8_t *rounding_bits, uint8_t *codes)
{
    int bits = code_bits(e, m);
    int64_t row_bytes = (bits == 8) ? K : (K + 1) / 2;
    int64_t rb_row = (K + 7) / 8;
    int64_t nans = 0;
    memset(codes, 0, (size_t)(N * row_bytes));
#pragma omp parallel for reduction(+ : nans) schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t k = 0; k < K; ++k) {
            int h = -1;
            if (rounding_bits)
                h = (rounding_bits[n * rb_row + k / 8] >> (k % 8)) & 1;
            int nan = 0;
            int code = fpq_o_quantize_one(w[n * K + k], scale[n], e, m, B, sat, h, &nan);
            nans += nan;
            put_code(codes, row_bytes, n, k, bits, code);
        }
    }
    return nans;
}

/* Activations: n elements, one scale, round to nearest.  One code per byte,
 * or two per byte for 4-bit formats (even index in the low nibble). */
int64_t fpq_o_quantize_act(const float *x, int64_t n, float scale, int e, int m, int B, int sat,
                           uint8_t *codes)
{
    int bits = code_bits(e, m);
    int64_t nans = 0;
    if (bits == 8) {
#pragma omp parallel for reduction(+ : nans) schedule(static)
        for (int64_t i = 0; i < n; ++i) {
            int nan = 0;
            codes[i] = (uint8_t)fpq_o_quantize_one(x[i], scale, e, m, B, sat, -1, &nan);
            nans += nan;
        }
    } else {
        memset(codes, 0, (size_t)((n + 1) / 2));
        for (int64_t i = 0; i < n; ++i) {
            int nan = 0;
            int code = fpq_o_quantize_one(x[i], scale, e, m, B, sat, -1, &nan);
            nans += nan;
            put_code(codes, 0, 0, i, 4, code);
        }
    }
    return nans;
}

/* ---- the quantized layer ------------------------------------------------ */

static double *decode_all(const uint8_t *codes, int64_t rows, int64_t cols, int e, int m, int B)
{
    int bits = code_bits(e, m);
    int64_t row_bytes = (bits == 8) ? cols : (cols + 1) / 2;
    double *v = (double *)malloc(sizeof(double) * (size_t)(rows * cols));
    if (!v)
        return NULL;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c)
            v[r * cols + c] = fpq_o_decode(get_code(codes, row_bytes, r, c, bits), e, m, B);
    return v;
}

/*
 * Linear layer on codes: y[i][n] = xs * ws[n] * sum_k dec(xc[i][k]) dec(wc[n][k]) + bias[n],
 * summed in double in index order.  absum[i][n] = |xs ws[n]| sum_k |dec dec| is
 * the scale of the acceptance tolerance.  If idx != NULL only the nidx flat
 * output positions idx[j] = i*N + n are computed, into y[j] / absum[j].
 */
int fpq_o_linear(const uint8_t *xc, const uint8_t *wc, const float *w_scale, float x_scale, int ex,
                 int mx, int Bx, int ew, int mw, int Bw, const float *bias, int64_t M, int64_t N,
                 int64_t K, const int64_t *idx, int64_t nidx, double *y, double *absum)
{
    double *xv = decode_all(xc, M, K, ex, mx, Bx);
    double *wv = decode_all(wc, N, K, ew, mw, Bw);
    if (!xv || !wv) {
        free(xv);
        free(wv);
        return -1;
    }
    int64_t total = idx ? nidx : M * N;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < total; ++j) {
        int64_t flat = idx ? idx[j] : j;
        int64_t i = flat / N, n = flat % N;
        double acc = 0.0, aacc = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            double p = xv[i * K + k] * wv[n * K + k];
            acc += p;
            aacc += fabs(p);
        }
        double g = (double)x_scale * (double)w_scale[n];
        y[j] = g * acc + (bias ? (double)bias[n] : 0.0);
        if (absum)
            absum[j] = fabs(g) * aacc;
    }
    free(xv);
    free(wv);
    return 0;
}

/*
 * 2-D convolution (cross-correlation, zero padding) on codes.
 *   xc: [B][C][H][W] one code per byte (activations are 8-bit formats)
 *   wc: [Co][C*R*S] codes in [C][R][S] order (bytes, or packed nibbles per row)
 *   y : [B][Co][Ho][Wo],  Ho = (H + 2 pad - R)/stride + 1, same for Wo.
 * idx, if not NULL, lists flat positions in y to compute.
 */
int fpq_o_conv2d(const uint8_t *xc, const uint8_t *wc, const float *w_scale, float x_scale, int ex,
                 int mx, int Bx, int ew, int mw, int Bw, const float *bias, int64_t Bn, int64_t C,
                 int64_t H, int64_t W, int64_t Co, int64_t R, int64_t S, int64_t pad, int64_t stride,
                 const int64_t *idx, int64_t nidx, double *y, double *absum)
{
    int64_t Ho = (H + 2 * pad - R) / stride + 1;
    int64_t Wo = (W + 2 * pad - S) / stride + 1;
    int64_t K = C * R * S;
    double *xv = decode_all(xc, Bn * C, H * W, ex, mx, Bx);
    double *wv = decode_all(wc, Co, K, ew, mw, Bw);
    if (!xv || !wv) {
        free(xv);
        free(wv);
        return -1;
    }
    int64_t total = idx ? nidx : Bn * Co * Ho * Wo;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < total; ++j) {
        int64_t flat = idx ? idx[j] : j;
        int64_t ox = flat % Wo;
        int64_t oy = (flat / Wo) % Ho;
        int64_t n = (flat / (Wo * Ho)) % Co;
        int64_t b = flat / (Wo * Ho * Co);
        double acc = 0.0, aacc = 0.0;
        for (int64_t c = 0; c < C; ++c)
            for (int64_t r = 0; r < R; ++r)
                for (int64_t s = 0; s < S; ++s) {
                    int64_t iy = oy * stride - pad + r;
                    int64_t ix = ox * stride - pad + s;
                    if (iy < 0 || iy >= H || ix < 0 || ix >= W)
                        continue; /* zero padding */
                    double p = xv[((b * C + c) * H + iy) * W + ix] * wv[n * K + (c * R + r) * S + s];
                    acc += p;
                    aacc += fabs(p);
                }
        double g = (double)x_scale * (double)w_scale[n];
        y[j] = g * acc + (bias ? (double)bias[n] : 0.0);
        if (absum)
            absum[j] = fabs(g) * aacc;
    }
    free(xv);
    free(wv);
    return 0;
}

/* ---- encoding and bias search (Sec. V-A, Algorithm 1) ---------------------
 *
 * For every encoding candidate i (exponent bits, mantissa bits; the integer
 * bias B_i only fixes the unit) and every clipping candidate c_j, the tensor is
 * quantized with the format whose largest value is c_j and compared with the
 * full-precision data:
 *     scale_ij = (float)c_j / (float)c(F_i)      (FP32 division; this is the
 *                real-valued bias of the clipping equation, b = B_i - log2 scale_ij)
 *     xq       = scale_ij * q(x * (1.0f / scale_ij))   round to nearest, in double
 *     mse_ij   = (1/n) sum (x - xq)^2                   in double, index order
 * mse is written as [n_enc][n_clip].  The encodings use the paper's clipping
 * value (all exponent fields finite).  Returns the number of NaN inputs. */
int64_t fpq_o_search_mse(const float *x, int64_t n, const int32_t *enc /* [n_enc][3]: e, m, B */, int n_enc,
                         const float *clip, int n_clip, double *mse)
{
    int64_t nans = 0;
#pragma omp parallel for collapse(2) schedule(dynamic) reduction(+ : nans)
    for (int i = 0; i < n_enc; ++i) {
        for (int j = 0; j < n_clip; ++j) {
            ofmt f = {enc[3 * i], enc[3 * i + 1], enc[3 * i + 2], SAT_PAPER};
            volatile float cf = (float)fpq_o_cmax(f.e, f.m, f.B, f.sat);
            volatile float scale = clip[j] / cf;
            double sum = 0.0;
            for (int64_t k = 0; k < n; ++k) {
                int isnan = 0;
                double q = quantize_value(x[k], scale, f, -1, &isnan);
                nans += isnan;
                double err = (double)x[k] - (double)scale * q;
                sum += err * err;
            }
            mse[(int64_t)i * n_clip + j] = n > 0 ? sum / (double)n : 0.0;
        }
    }
    return nans;
}

/* ---- rounding learning (Sec. V-B) ------------------------------------------ */

/* Soft-rounded weights of Sec. V-B, the learned-rounding equation before hardening:
 *     a      = clamp(w * (1.0f / scale); -c, c)           (FP32 scaling as everywhere above)
 *     pre    = s(a) * (floor(a / s(a)) + sigma(alpha))    sigma(alpha) = 1 / (1 + exp(-alpha))
 *     wq     = scale * clamp(pre; -c, c)                  back in the weight's own units
 * and its derivative with respect to alpha,
 *     dwq    = scale * s(a) * sigma (1 - sigma)           where pre lies in [-c, c], else 0
 * (floor is piecewise constant; a clamp passes the gradient inside its range and
 * blocks it outside).  Everything after the FP32 scaling is double.  A NaN weight
 * gives wq = dwq = 0.  wq, dwq: [N][K] doubles. */
int64_t fpq_o_soft_weight(const float *w, int64_t N, int64_t K, const float *scale, int e, int m, int B,
                          int sat, const float *alpha, double *wq, double *dwq)
{
    ofmt f = {e, m, B, sat};
    double c = fpq_o_cmax(e, m, B, sat);
    int64_t nans = 0;
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t k = 0; k < K; ++k) {
            int64_t i = n * K + k;
            volatile float r = 1.0f / scale[n];
            volatile float t = w[i] * r;
            if (t != t) {
                wq[i] = 0.0;
                dwq[i] = 0.0;
                ++nans;
                continue;
            }
            double a = (double)t;
            if (a > c)
                a = c;
            if (a < -c)
                a = -c;
            double s = step_of(a, f);
            double sig = 1.0 / (1.0 + exp(-(double)alpha[i]));
            double pre = s * (floor(a / s) + sig);
            double q = pre;
            if (q > c)
                q = c;
            if (q < -c)
                q = -c;
            wq[i] = (double)scale[n] * q;
            dwq[i] = (pre >= -c && pre <= c) ? (double)scale[n] * s * sig * (1.0 - sig) : 0.0;
        }
    }
    return nans;
}
