// Element-wise quantizer kernels: weight encode, activation quantize, and the
// two layout-changing activation quantizers that feed the contraction.
#include "fpq_common.cuh"
#include "fpq_kernels.h"

namespace fpq {

// ---------------------------------------------------------------------------------
// Activation quantize, flat: 16 elements per thread, 4 x 128-bit loads, one
// 128-bit store.  HBM-bound: 5 bytes per element.
// ---------------------------------------------------------------------------------
// MODE selects the conversion: 0 the general rounding arithmetic (any format), 1 E4M3, 2 OCP E5M2 and
// 3 E2M1 with the hardware converts (round to nearest even, saturating at the type's largest finite value:
// the same function of t, -0 and NaN mapped to code 0 afterwards).
constexpr int Q_GENERAL = 0, Q_E4M3 = 1, Q_E5M2 = 2, Q_E2M1 = 3;

// Eight E2M1 codes (bias 1, grid 0 .. 6) from eight scaled floats, element j in nibble j.
__device__ __forceinline__ uint32_t e2m1x8_from_scaled(const float (&t)[8], bool& nan)
{
    uint32_t v = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        uint32_t b;
        asm("{\n\t.reg .b8 q;\n\t"
            "cvt.rn.satfinite.e2m1x2.f32 q, %1, %2;\n\t"
            "cvt.u32.u8 %0, q;\n\t}"
            : "=r"(b)
            : "f"(t[2 * j + 1]), "f"(t[2 * j]));
        v |= b << (8 * j);
        nan |= (t[2 * j] != t[2 * j]) | (t[2 * j + 1] != t[2 * j + 1]);
    }
    // a NaN converts to the largest magnitude: those nibbles are cleared; -0 becomes +0
#pragma unroll
    for (int j = 0; j < 8; ++j)
        if (t[j] != t[j])
            v &= ~(0xfu << (4 * j));
    const uint32_t mag = v & 0x77777777u;
    const uint32_t nonzero = (mag + 0x77777777u) & 0x88888888u;
    return mag | (v & nonzero);
}

// ---- the general rounding arithmetic, four elements at a time ---------------------------------------
// The magic-number addition of quantize_rne_bits with everything that depends on the format alone taken
// out of the loop and as much as possible on the floating-point pipe.  With E the power of two at or below
// max(|a|, smallest normal of the format), C = E * 1.5 * 2^(23-m) is 1.5 * 2^23 steps of the element's
// binade, the FP32 sum |a| + C is a whole number of steps (rounded as the add's rounding mode says) and
// (bits(E) >> sh) + (bits(sum) - bits(C)) - c2 is the code.  These forms assume finite inputs: the caller
// looks for NaN and infinity once per thread item and falls back on the element-wise functions.
struct WordConsts {
    float cmax, lo, kmul;
    uint32_t c2, code_max, mag4, sign4, pow_m;
    int sh, sign_down, sign_shift;
};
__device__ __forceinline__ WordConsts word_consts(const QFormat& f)
{
    WordConsts c;
    c.cmax = __uint_as_float(f.cmax_bits);
    c.lo = __uint_as_float((uint32_t)(128 - f.B) << 23);
    c.kmul = __uint_as_float(((uint32_t)(127 + 23 - f.m) << 23) | 0x400000u);
    c.c2 = (uint32_t)(128 - f.B) << f.m;
    c.code_max = (uint32_t)f.code_max;
    c.sign4 = 0x01010101u << f.sign_shift;
    c.mag4 = c.sign4 - 0x01010101u;
    c.pow_m = 1u << f.m;
    c.sh = 23 - f.m;
    c.sign_down = 7 - f.sign_shift;
    c.sign_shift = f.sign_shift;
    return c;
}

// the sign bits of four floats at bit `sign_shift` of the four bytes of a word
__device__ __forceinline__ uint32_t signs4(uint32_t u0, uint32_t u1, uint32_t u2, uint32_t u3, const WordConsts& c)
{
    const uint32_t t01 = __byte_perm(u0, u1, 0x0073), t23 = __byte_perm(u2, u3, 0x0073);
    return (__byte_perm(t01, t23, 0x5410) & 0x80808080u) >> c.sign_down;
}

// Round to nearest even: four byte codes in one word (sign included; a zero magnitude has no sign).  The clipping
// value is the largest code's value, so no code can come out above it.
__device__ __forceinline__ uint32_t rne_word(float t0, float t1, float t2, float t3, const WordConsts& c)
{
    const float t[4] = {t0, t1, t2, t3};
    uint32_t w = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float a = fminf(fabsf(t[j]), c.cmax);
        const uint32_t ebits = __float_as_uint(fmaxf(a, c.lo)) & 0x7f800000u;
        const float C = __fmul_rn(__uint_as_float(ebits), c.kmul);
        const uint32_t k = __float_as_uint(__fadd_rn(a, C)) - __float_as_uint(C);
        w |= ((ebits >> c.sh) + k - c.c2) << (8 * j);
    }
    const uint32_t nonzero = ((w & c.mag4) + c.mag4) & c.sign4;
    return w | (signs4(__float_as_uint(t0), __float_as_uint(t1), __float_as_uint(t2), __float_as_uint(t3), c) & nonzero);
}

// Signed floor plus the learned decision h (Sec. V-B): the sum a + C rounded toward minus infinity is
// floor(a / step) steps above C for either sign of a (a minus zero counts as zero), h is added to that whole
// number and the magnitude is encoded.  One step above a binade's lower edge toward zero lies in the finer
// binade below (k < 2^m in a normal binade): there the code is one less than the plain sum.
__device__ __forceinline__ uint32_t floor_word(float t0, float t1, float t2, float t3, uint32_t h4, const WordConsts& c)
{
    const float t[4] = {t0, t1, t2, t3};
    uint32_t w = 0, sg = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float a = fminf(fabsf(t[j]), c.cmax);
        const uint32_t ebits = __float_as_uint(fmaxf(a, c.lo)) & 0x7f800000u;
        const float C = __fmul_rn(__uint_as_float(ebits), c.kmul);
        const int k = (int)(__float_as_uint(__fadd_rd(copysignf(a, t[j]), C)) - __float_as_uint(C)) + (int)((h4 >> j) & 1u);
        const uint32_t kmag = (uint32_t)abs(k);
        const uint32_t base = (ebits >> c.sh) - c.c2;          // (exponent field - 1 of the binade) << m
        const uint32_t code = min(base + kmag - ((kmag < c.pow_m && base >= c.pow_m) ? 1u : 0u), c.code_max);
        w |= code << (8 * j);
        sg |= (k < 0 ? 1u : 0u) << (8 * j);
    }
    const uint32_t nonzero = ((w & c.mag4) + c.mag4) & c.sign4;
    return w | ((sg << c.sign_shift) & nonzero);
}

// 0 if all sixteen values are finite (anything else otherwise): x * 0 is 0 for a finite x and NaN for the rest
__device__ __forceinline__ float nonfinite_probe(const float (&t)[16])
{
    float acc = 0.0f;
#pragma unroll
    for (int j = 0; j < 16; ++j)
        acc = fmaf(t[j], 0.0f, acc);
    return acc;
}

// four byte codes of a 4-bit format -> 16 bits of nibbles
__device__ __forceinline__ uint32_t nibbles_of(uint32_t w)
{
    const uint32_t x = (w | (w >> 4)) & 0x00ff00ffu;
    return (x | (x >> 8)) & 0xffffu;
}

// 16 scaled values -> their codes: four words of bytes, or two words of nibbles for 4-bit formats
template <int MODE>
__device__ __forceinline__ void encode16_rne(const float (&t)[16], const QFormat& f, uint32_t (&out)[4], bool& nan)
{
    if constexpr (MODE == Q_E2M1) {
        const float lo[8] = {t[0], t[1], t[2], t[3], t[4], t[5], t[6], t[7]};
        const float hi[8] = {t[8], t[9], t[10], t[11], t[12], t[13], t[14], t[15]};
        out[0] = e2m1x8_from_scaled(lo, nan);
        out[1] = e2m1x8_from_scaled(hi, nan);
    } else {
        const WordConsts c = word_consts(f);
        const bool slow = MODE == Q_GENERAL && nonfinite_probe(t) != 0.0f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (MODE == Q_E4M3)
                out[j] = e4m3x4_from_scaled(t[4 * j], t[4 * j + 1], t[4 * j + 2], t[4 * j + 3], nan);
            else if (MODE == Q_E5M2)
                out[j] = e5m2x4_from_scaled(t[4 * j], t[4 * j + 1], t[4 * j + 2], t[4 * j + 3], nan);
            else if (!slow)
                out[j] = rne_word(t[4 * j], t[4 * j + 1], t[4 * j + 2], t[4 * j + 3], c);
            else
                out[j] = quantize_rne_bits(t[4 * j], f, nan) | (quantize_rne_bits(t[4 * j + 1], f, nan) << 8) |
                         (quantize_rne_bits(t[4 * j + 2], f, nan) << 16) | (quantize_rne_bits(t[4 * j + 3], f, nan) << 24);
        }
        if (f.four_bit) {
            out[0] = nibbles_of(out[0]) | (nibbles_of(out[1]) << 16);
            out[1] = nibbles_of(out[2]) | (nibbles_of(out[3]) << 16);
        }
    }
}

template <int MODE>
__global__ void __launch_bounds__(256) quantize_act_kernel(const float* __restrict__ x, int64_t n, float rinv,
                                                           QFormat f, uint8_t* __restrict__ codes, int* status)
{
    bool nan = false;
    int64_t nvec = n / 16;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < nvec; v += stride) {
        const float4* px = reinterpret_cast<const float4*>(x) + v * 4;
        float4 a[4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
            a[j] = __ldg(px + j);
        float t[16];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            t[4 * j] = __fmul_rn(a[j].x, rinv);
            t[4 * j + 1] = __fmul_rn(a[j].y, rinv);
            t[4 * j + 2] = __fmul_rn(a[j].z, rinv);
            t[4 * j + 3] = __fmul_rn(a[j].w, rinv);
        }
        uint32_t out[4];
        encode16_rne<MODE>(t, f, out, nan);
        if (!f.four_bit)
            reinterpret_cast<uint4*>(codes)[v] = make_uint4(out[0], out[1], out[2], out[3]);
        else
            reinterpret_cast<uint2*>(codes)[v] = make_uint2(out[0], out[1]);
    }
    // tail (fewer than 16 elements): one thread, in order, so nibbles never race
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        for (int64_t i = nvec * 16; i < n; ++i) {
            uint32_t c = quantize_rne_bits(__fmul_rn(x[i], rinv), f, nan);
            if (!f.four_bit) {
                codes[i] = (uint8_t)c;
            } else if (i & 1) {
                codes[i >> 1] = (uint8_t)(codes[i >> 1] | (c << 4));
            } else {
                codes[i >> 1] = (uint8_t)c;
            }
        }
    }
    if (nan)
        flag_status(status, FPQ_ERR_NAN_INPUT);
}

// Unaligned input: one output byte per thread (two elements for 4-bit codes).
__global__ void __launch_bounds__(256) quantize_act_scalar_kernel(const float* __restrict__ x, int64_t n, float rinv,
                                                                  QFormat f, uint8_t* __restrict__ codes, int* status)
{
    bool nan = false;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    int64_t per = f.four_bit ? 2 : 1;
    int64_t nout = (n + per - 1) / per;
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < nout; o += stride) {
        uint32_t c = quantize_rne_bits(__fmul_rn(x[o * per], rinv), f, nan);
        if (f.four_bit && o * 2 + 1 < n)
            c |= quantize_rne_bits(__fmul_rn(x[o * 2 + 1], rinv), f, nan) << 4;
        codes[o] = (uint8_t)c;
    }
    if (nan)
        flag_status(status, FPQ_ERR_NAN_INPUT);
}

// ---------------------------------------------------------------------------------
// Weight encode: one thread per group of 8 weights of a row (one rounding byte).
// ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) quantize_weight_kernel(const float* __restrict__ w, int64_t N, int64_t K,
                                                              const float* __restrict__ scale, QFormat f,
                                                              const uint8_t* __restrict__ rbits,
                                                              uint8_t* __restrict__ codes, int* status)
{
    bool nan = false;
    int64_t groups = (K + 7) / 8;
    int64_t total = N * groups;
    int64_t row_bytes = f.four_bit ? (K + 1) / 2 : K;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += stride) {
        int64_t n = t / groups, g = t % groups;
        float rinv = __fdiv_rn(1.0f, __ldg(scale + n));
        int hb = rbits ? (int)__ldg(rbits + n * groups + g) : 0;
        const float* pw = w + n * K + g * 8;
        int cnt = (int)min((int64_t)8, K - g * 8);
        uint32_t c[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            c[j] = 0;
            if (j < cnt) {
                int h = rbits ? ((hb >> j) & 1) : -1;
                c[j] = quantize_bits(__fmul_rn(__ldg(pw + j), rinv), f, h, nan);
            }
        }
        if (!f.four_bit) {
            uint8_t* po = codes + n * row_bytes + g * 8;
            for (int j = 0; j < cnt; ++j)
                po[j] = (uint8_t)c[j];
        } else {
            uint8_t* po = codes + n * row_bytes + g * 4;
            for (int j = 0; j < (cnt + 1) / 2; ++j)
                po[j] = (uint8_t)(c[2 * j] | (c[2 * j + 1] << 4));
        }
    }
    if (nan)
        flag_status(status, FPQ_ERR_NAN_INPUT);
}

// The same for rows whose length is a multiple of 16 (aligned buffers): one thread per 16 weights of a row (two
// rounding bytes), 4 x 128-bit loads, one 128-bit (64-bit for 4-bit codes) store.  HBM-bound: 4 bytes in,
// 1 or 0.5 out, 1/8 of rounding decisions per weight.  LEARNED: the rounding decisions are given.
template <int MODE, bool LEARNED>
__global__ void __launch_bounds__(256) quantize_weight_vec_kernel(const float* __restrict__ w, int64_t N, int64_t K,
                                                                  const float* __restrict__ scale, QFormat f,
                                                                  const uint8_t* __restrict__ rbits,
                                                                  uint8_t* __restrict__ codes, int* status)
{
    bool nan = false;
    const int64_t per_row = K / 16;
    const int64_t total = N * per_row;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < total; v += stride) {
        const int64_t n = v / per_row;
        const float rinv = __fdiv_rn(1.0f, __ldg(scale + n));
        const float4* pw = reinterpret_cast<const float4*>(w) + v * 4;
        float4 a[4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
            a[j] = __ldg(pw + j);
        float t[16];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            t[4 * j] = __fmul_rn(a[j].x, rinv);
            t[4 * j + 1] = __fmul_rn(a[j].y, rinv);
            t[4 * j + 2] = __fmul_rn(a[j].z, rinv);
            t[4 * j + 3] = __fmul_rn(a[j].w, rinv);
        }
        uint32_t out[4];
        if (!LEARNED) {
            encode16_rne<MODE>(t, f, out, nan);
        } else {
            // 16 decisions: the row's bytes 2 g and 2 g + 1 (K / 8 is even, so the pair is 2-byte aligned)
            const uint32_t hb = __ldg(reinterpret_cast<const uint16_t*>(rbits) + v);
            const WordConsts c = word_consts(f);
            if (nonfinite_probe(t) == 0.0f) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    out[j] = floor_word(t[4 * j], t[4 * j + 1], t[4 * j + 2], t[4 * j + 3], hb >> (4 * j), c);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    out[j] = 0;
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        out[j] |= quantize_bits(t[4 * j + q], f, (int)((hb >> (4 * j + q)) & 1u), nan) << (8 * q);
                }
            }
            if (f.four_bit) {
                out[0] = nibbles_of(out[0]) | (nibbles_of(out[1]) << 16);
                out[1] = nibbles_of(out[2]) | (nibbles_of(out[3]) << 16);
            }
        }
        if (!f.four_bit)
            reinterpret_cast<uint4*>(codes)[v] = make_uint4(out[0], out[1], out[2], out[3]);
        else
            reinterpret_cast<uint2*>(codes)[v] = make_uint2(out[0], out[1]);
    }
    if (nan)
        flag_status(status, FPQ_ERR_NAN_INPUT);
}

// ---------------------------------------------------------------------------------
// Row-major activations [M][K] FP32 -> codes [M][Kp] (Kp = K rounded up to 16, pad = 0),
// the A operand of the linear contraction.  16 elements per thread.
// ---------------------------------------------------------------------------------
// TWICE: every row is written two times side by side, [M][2 Kp] (Kp a multiple of 128), for weights that
// are the sum of two E4M3 terms: the reduction then runs over (x | x) against (first terms | second terms).
template <bool TWICE, bool E5>
__global__ void __launch_bounds__(256) quantize_rows_e4m3_kernel(const float* __restrict__ x, int64_t M, int64_t K,
                                                                 int64_t Kp, float rinv, uint8_t* __restrict__ codes,
                                                                 int* status)
{
    asm volatile("griddepcontrol.launch_dependents;");
    bool nan = false;
    int64_t vec_per_row = Kp / 16;
    int64_t total = M * vec_per_row;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const bool aligned = (K % 4) == 0;
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < total; v += stride) {
        int64_t row = v / vec_per_row, k0 = (v % vec_per_row) * 16;
        const float* px = x + row * K + k0;
        uint32_t out[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
            int64_t k = k0 + 4 * j;
            if (aligned && k + 4 <= K) {
                float4 q = __ldg(reinterpret_cast<const float4*>(px + 4 * j));
                a0 = q.x; a1 = q.y; a2 = q.z; a3 = q.w;
            } else {
                if (k + 0 < K) a0 = __ldg(px + 4 * j + 0);
                if (k + 1 < K) a1 = __ldg(px + 4 * j + 1);
                if (k + 2 < K) a2 = __ldg(px + 4 * j + 2);
                if (k + 3 < K) a3 = __ldg(px + 4 * j + 3);
            }
            out[j] = fp8x4_from_scaled<E5>(__fmul_rn(a0, rinv), __fmul_rn(a1, rinv), __fmul_rn(a2, rinv),
                                           __fmul_rn(a3, rinv), nan);
        }
        if (TWICE) {
            int64_t o = row * 2 * vec_per_row + v % vec_per_row;
            reinterpret_cast<uint4*>(codes)[o] = make_uint4(out[0], out[1], out[2], out[3]);
            reinterpret_cast<uint4*>(codes)[o + vec_per_row] = make_uint4(out[0], out[1], out[2], out[3]);
        } else {
            reinterpret_cast<uint4*>(codes)[v] = make_uint4(out[0], out[1], out[2], out[3]);
        }
    }
    if (nan)
        flag_status(status, FPQ_ERR_NAN_INPUT);
}

// ---------------------------------------------------------------------------------
// NCHW FP32 -> channels-last codes with a zero frame: [B][H+2p][W+2p][row] (channel padding
// and frame = code 0), the A operand of the implicit-GEMM convolution.  The kernel fills the
// channels [c_off, c_off + Cp) of every pixel row (Cp = C rounded up to 16, or further for the
// first of two concatenated tensors); row = Cp and c_off = 0 for a single input tensor.  A block transposes 128 channels x 32 pixels through
// shared memory: loads are coalesced along pixels (16 in flight per thread), stores
// are whole 128-byte channel rows.  The blocks also share out the frame pixels.
// ---------------------------------------------------------------------------------
template <bool E5>
__global__ void __launch_bounds__(256) quantize_nchw_to_nhwc_e4m3_kernel(const float* __restrict__ x, int C, int H,
                                                                         int W, int pad, int Cp, int row, int c_off,
                                                                         float rinv, uint8_t* __restrict__ codes,
                                                                         int* status)
{
    __shared__ __align__(16) uint8_t tile[32][128 + 16];
    // the contraction queued behind this kernel may start its set-up (it waits for this grid
    // to finish before it reads the codes)
    asm volatile("griddepcontrol.launch_dependents;");
    bool nan = false;
    const int HW = H * W, Wp = W + 2 * pad, Hp = H + 2 * pad;
    const int b = blockIdx.z;
    const int c0 = blockIdx.y * 128;
    const int p0 = blockIdx.x * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 pixels x 8 channel groups of 16
    const float* xb = x + (int64_t)b * C * HW;
    uint8_t* ob = codes + (int64_t)b * Hp * Wp * row + c_off;
    const int p = p0 + tx;
    {
        const int cl = ty * 16;
        float a[16];
        const float* px = xb + (int64_t)(c0 + cl) * HW + p;
        if (c0 + 128 <= C && p0 + 32 <= HW) {            // interior tile: no predicates
#pragma unroll
            for (int q = 0; q < 16; ++q)
                a[q] = __ldg(px + (int64_t)q * HW);
        } else {
#pragma unroll
            for (int q = 0; q < 16; ++q)
                a[q] = (c0 + cl + q < C && p < HW) ? __ldg(px + (int64_t)q * HW) : 0.f;
        }
        uint4 v;
        v.x = fp8x4_from_scaled<E5>(__fmul_rn(a[0], rinv), __fmul_rn(a[1], rinv), __fmul_rn(a[2], rinv), __fmul_rn(a[3], rinv), nan);
        v.y = fp8x4_from_scaled<E5>(__fmul_rn(a[4], rinv), __fmul_rn(a[5], rinv), __fmul_rn(a[6], rinv), __fmul_rn(a[7], rinv), nan);
        v.z = fp8x4_from_scaled<E5>(__fmul_rn(a[8], rinv), __fmul_rn(a[9], rinv), __fmul_rn(a[10], rinv), __fmul_rn(a[11], rinv), nan);
        v.w = fp8x4_from_scaled<E5>(__fmul_rn(a[12], rinv), __fmul_rn(a[13], rinv), __fmul_rn(a[14], rinv), __fmul_rn(a[15], rinv), nan);
        *reinterpret_cast<uint4*>(&tile[tx][cl]) = v;
    }
    __syncthreads();
    {
        // 32 pixels x 8 chunks of 16 channels: 8 consecutive threads write one pixel's row
        const int pl = threadIdx.x >> 3, ch = (threadIdx.x & 7) * 16;
        const int pp = p0 + pl, c = c0 + ch;
        if (pp < HW && c < Cp) {
            const int yy = pp / W, xx = pp - yy * W;
            const uint4 v = *reinterpret_cast<const uint4*>(&tile[pl][ch]);
            *reinterpret_cast<uint4*>(ob + ((int64_t)(yy + pad) * Wp + (xx + pad)) * row + c) = v;
        }
    }
    // frame pixels of this image, shared out over the blocks of the image's pixel axis
    if (pad > 0) {
        const int nframe = Hp * Wp - HW;
        const int chunks = (min(Cp - c0, 128)) / 16;
        const int total = nframe * chunks;
        for (int t = blockIdx.x * 256 + threadIdx.x; t < total; t += gridDim.x * 256) {
            const int j = t / chunks, ch = (t - j * chunks) * 16;
            int yp, xp;
            const int top = pad * Wp;
            if (j < top) {
                yp = j / Wp; xp = j - yp * Wp;
            } else if (j < 2 * top) {
                const int k = j - top;
                yp = H + pad + k / Wp; xp = k % Wp;
            } else {
                const int k = j - 2 * top;             // 2*pad frame pixels per interior row
                yp = pad + k / (2 * pad);
                const int e = k % (2 * pad);
                xp = (e < pad) ? e : W + e;
            }
            *reinterpret_cast<uint4*>(ob + ((int64_t)yp * Wp + xp) * row + c0 + ch) = make_uint4(0, 0, 0, 0);
        }
    }
    if (nan)
        flag_status(status, FPQ_ERR_NAN_INPUT);
}

// ---------------------------------------------------------------------------------
// Contraction-ready weight copy: [N][C][R][S] codes -> [N][R*S][Cp] codes, zero padded.
// One thread per output byte.  For an input made of two concatenated tensors (C1 > 0) the
// channels from C1 on start at position C1p (C1 rounded up to 128), so that each tensor's
// channels fill whole 128-wide chunks of the reduction.
// ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) prepare_weight_kernel(const uint8_t* __restrict__ codes, int N, int C, int RS,
                                                             int Cp, int in_four_bit, int use_table, CodeTable table,
                                                             int two_term, CodeTable table2, int C1, int C1p,
                                                             uint8_t* __restrict__ prepared)
{
    // two_term: a row holds the channels twice, [first terms | second terms], Cp / 2 positions each
    __shared__ uint8_t s_tab[256], s_tab2[256];
    s_tab[threadIdx.x] = table.t[threadIdx.x];
    s_tab2[threadIdx.x] = table2.t[threadIdx.x];
    __syncthreads();
    const int four_bit = in_four_bit && !use_table;      // layout of the prepared copy
    int64_t row_out = four_bit ? (int64_t)RS * Cp / 2 : (int64_t)RS * Cp;
    int64_t total = (int64_t)N * row_out;
    int64_t K = (int64_t)C * RS;
    int64_t row_in = in_four_bit ? (K + 1) / 2 : K;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += stride) {
        int64_t n = o / row_out, within = o % row_out;
        uint32_t outb = 0;
        int per = four_bit ? 2 : 1;
        for (int q = 0; q < per; ++q) {
            int64_t e = within * per + q;       // element index in [RS][Cp]
            int tap = (int)(e / Cp), c = (int)(e % Cp);
            uint32_t code = 0;
            bool second = false;
            if (two_term && c >= Cp / 2) {
                second = true;
                c -= Cp / 2;
            }
            bool real = c < C;
            if (C1 > 0) {
                real = c < C1 || (c >= C1p && c - C1p + C1 < C);
                if (c >= C1p)
                    c = c - C1p + C1;
            }
            if (real) {
                int64_t k = (int64_t)c * RS + tap;   // source order [C][R][S]
                if (in_four_bit) {
                    uint8_t bsrc = __ldg(codes + n * row_in + (k >> 1));
                    code = (k & 1) ? (bsrc >> 4) : (bsrc & 0xf);
                } else {
                    code = __ldg(codes + n * row_in + k);
                }
                if (use_table)
                    code = second ? s_tab2[code] : s_tab[code];
            }
            outb |= code << (4 * q * four_bit);
        }
        prepared[o] = (uint8_t)outb;
    }
}

// ---- launchers ----------------------------------------------------------------------
static int grid_for(int64_t work_items, int threads)
{
    int64_t blocks = (work_items + threads - 1) / threads;
    const int64_t cap = 148 * 16;
    if (blocks > cap)
        blocks = cap;
    if (blocks < 1)
        blocks = 1;
    return (int)blocks;
}

// which conversion a format's round-to-nearest encode may use
static int rne_mode(const QFormat& f)
{
    if (f.native_e4m3)
        return Q_E4M3;
    if (f.e == 5 && f.m == 2 && f.B == 15 && f.code_max == 0x7B)
        return Q_E5M2;
    if (f.e == 2 && f.m == 1 && f.B == 1)
        return Q_E2M1;
    return Q_GENERAL;
}

cudaError_t launch_quantize_act(const float* x, int64_t n, float scale, const QFormat& f, uint8_t* codes,
                                cudaStream_t st)
{
    if (n == 0)
        return cudaSuccess;
    float rinv = 1.0f / scale;
    bool aligned = ((uintptr_t)x % 16 == 0) && ((uintptr_t)codes % 16 == 0);
    const int grid = grid_for(n / 16 + 1, 256);
    if (!aligned) {
        quantize_act_scalar_kernel<<<grid_for(n, 256), 256, 0, st>>>(x, n, rinv, f, codes, status_word());
    } else {
        switch (rne_mode(f)) {
        case Q_E4M3: quantize_act_kernel<Q_E4M3><<<grid, 256, 0, st>>>(x, n, rinv, f, codes, status_word()); break;
        case Q_E5M2: quantize_act_kernel<Q_E5M2><<<grid, 256, 0, st>>>(x, n, rinv, f, codes, status_word()); break;
        case Q_E2M1: quantize_act_kernel<Q_E2M1><<<grid, 256, 0, st>>>(x, n, rinv, f, codes, status_word()); break;
        default: quantize_act_kernel<Q_GENERAL><<<grid, 256, 0, st>>>(x, n, rinv, f, codes, status_word()); break;
        }
    }
    return cudaGetLastError();
}

cudaError_t launch_quantize_weight(const float* w, int64_t N, int64_t K, const float* scale, const QFormat& f,
                                   const uint8_t* rbits, uint8_t* codes, cudaStream_t st)
{
    if (N == 0 || K == 0)
        return cudaSuccess;
    const bool vec = K % 16 == 0 && (uintptr_t)w % 16 == 0 && (uintptr_t)codes % 16 == 0 && (uintptr_t)rbits % 2 == 0;
    if (vec) {
        const int grid = grid_for(N * (K / 16), 256);
        if (rbits) {
            quantize_weight_vec_kernel<Q_GENERAL, true><<<grid, 256, 0, st>>>(w, N, K, scale, f, rbits, codes, status_word());
        } else {
            switch (rne_mode(f)) {
            case Q_E4M3: quantize_weight_vec_kernel<Q_E4M3, false><<<grid, 256, 0, st>>>(w, N, K, scale, f, rbits, codes, status_word()); break;
            case Q_E5M2: quantize_weight_vec_kernel<Q_E5M2, false><<<grid, 256, 0, st>>>(w, N, K, scale, f, rbits, codes, status_word()); break;
            case Q_E2M1: quantize_weight_vec_kernel<Q_E2M1, false><<<grid, 256, 0, st>>>(w, N, K, scale, f, rbits, codes, status_word()); break;
            default: quantize_weight_vec_kernel<Q_GENERAL, false><<<grid, 256, 0, st>>>(w, N, K, scale, f, rbits, codes, status_word()); break;
            }
        }
        return cudaGetLastError();
    }
    int64_t total = N * ((K + 7) / 8);
    quantize_weight_kernel<<<grid_for(total, 256), 256, 0, st>>>(w, N, K, scale, f, rbits, codes, status_word());
    return cudaGetLastError();
}

cudaError_t launch_quantize_rows_e4m3(const float* x, int64_t M, int64_t K, int64_t Kp, float scale, uint8_t* codes,
                                      cudaStream_t st, int e5m2)
{
    int64_t total = M * (Kp / 16);
    if (e5m2)
        quantize_rows_e4m3_kernel<false, true><<<grid_for(total, 256), 256, 0, st>>>(x, M, K, Kp, 1.0f / scale, codes,
                                                                                    status_word());
    else
        quantize_rows_e4m3_kernel<false, false><<<grid_for(total, 256), 256, 0, st>>>(x, M, K, Kp, 1.0f / scale, codes,
                                                                                     status_word());
    return cudaGetLastError();
}

cudaError_t launch_quantize_rows_e4m3_twice(const float* x, int64_t M, int64_t K, int64_t Kp, float scale, uint8_t* codes,
                                            cudaStream_t st, int e5m2)
{
    int64_t total = M * (Kp / 16);
    if (e5m2)
        quantize_rows_e4m3_kernel<true, true><<<grid_for(total, 256), 256, 0, st>>>(x, M, K, Kp, 1.0f / scale, codes,
                                                                                   status_word());
    else
        quantize_rows_e4m3_kernel<true, false><<<grid_for(total, 256), 256, 0, st>>>(x, M, K, Kp, 1.0f / scale, codes,
                                                                                    status_word());
    return cudaGetLastError();
}

cudaError_t launch_quantize_nchw_to_nhwc_e4m3(const float* x, int B, int C, int H, int W, int pad, int Cp, int row,
                                              int c_off, float scale, uint8_t* codes, cudaStream_t st, int e5m2)
{
    dim3 grid((H * W + 31) / 32, (Cp + 127) / 128, B);
    if (e5m2)
        quantize_nchw_to_nhwc_e4m3_kernel<true><<<grid, 256, 0, st>>>(x, C, H, W, pad, Cp, row, c_off, 1.0f / scale, codes,
                                                                      status_word());
    else
        quantize_nchw_to_nhwc_e4m3_kernel<false><<<grid, 256, 0, st>>>(x, C, H, W, pad, Cp, row, c_off, 1.0f / scale, codes,
                                                                       status_word());
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------
// Activations in a format the tensor cores have no type for, whose every value is one value or the sum of two
// values of a tensor-core type (tables: code of the format -> code of each term; the same classification as for
// weights): quantize with the general arithmetic, look the terms up, and write them as operand codes.  TERMS = 2:
// every row (pixel) holds [first terms | second terms], Kp (Cp) positions each, and the contraction runs over
// twice the padded reduction length against the weights repeated.
// ---------------------------------------------------------------------------------
// 16 scaled values -> 16 codes of any format, one per byte (4-bit formats too), four per word
__device__ __forceinline__ void codes16_bytes(const float (&t)[16], const QFormat& f, uint32_t (&w)[4], bool& nan)
{
    if (nonfinite_probe(t) == 0.0f) {
        const WordConsts c = word_consts(f);
#pragma unroll
        for (int j = 0; j < 4; ++j)
            w[j] = rne_word(t[4 * j], t[4 * j + 1], t[4 * j + 2], t[4 * j + 3], c);
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            w[j] = quantize_rne_bits(t[4 * j], f, nan) | (quantize_rne_bits(t[4 * j + 1], f, nan) << 8) |
                   (quantize_rne_bits(t[4 * j + 2], f, nan) << 16) | (quantize_rne_bits(t[4 * j + 3], f, nan) << 24);
    }
}

// the same four positions of a table-mapped word
__device__ __forceinline__ uint32_t map4(uint32_t w, const uint8_t* tab)
{
    return (uint32_t)tab[w & 0xffu] | ((uint32_t)tab[(w >> 8) & 0xffu] << 8) | ((uint32_t)tab[(w >> 16) & 0xffu] << 16) |
           ((uint32_t)tab[w >> 24] << 24);
}

template <int TERMS>
__global__ void __launch_bounds__(256) quantize_rows_terms_kernel(const float* __restrict__ x, int64_t M, int64_t K,
                                                                  int64_t Kp, float rinv, QFormat f, CodeTable tab1,
                                                                  CodeTable tab2, uint8_t* __restrict__ codes, int* status)
{
    __shared__ uint8_t s1[256], s2[256];
    s1[threadIdx.x] = tab1.t[threadIdx.x];
    s2[threadIdx.x] = tab2.t[threadIdx.x];
    __syncthreads();
    asm volatile("griddepcontrol.launch_dependents;");
    bool nan = false;
    const int64_t vec_per_row = Kp / 16;
    const int64_t total = M * vec_per_row;
    const bool aligned = (K % 4) == 0;
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < total; v += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = v / vec_per_row, k0 = (v - row * vec_per_row) * 16;
        const float* px = x + row * K + k0;
        float t[16];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
            const int64_t k = k0 + 4 * j;
            if (aligned && k + 4 <= K) {
                const float4 q = __ldg(reinterpret_cast<const float4*>(px + 4 * j));
                a0 = q.x; a1 = q.y; a2 = q.z; a3 = q.w;
            } else {
                if (k + 0 < K) a0 = __ldg(px + 4 * j + 0);
                if (k + 1 < K) a1 = __ldg(px + 4 * j + 1);
                if (k + 2 < K) a2 = __ldg(px + 4 * j + 2);
                if (k + 3 < K) a3 = __ldg(px + 4 * j + 3);
            }
            t[4 * j] = __fmul_rn(a0, rinv);
            t[4 * j + 1] = __fmul_rn(a1, rinv);
            t[4 * j + 2] = __fmul_rn(a2, rinv);
            t[4 * j + 3] = __fmul_rn(a3, rinv);
        }
        // (positions past K hold 0.0: code 0, and every table maps code 0 to 0)
        uint32_t w[4], o1[4], o2[4];
        codes16_bytes(t, f, w, nan);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            o1[j] = map4(w[j], s1);
            o2[j] = TERMS == 2 ? map4(w[j], s2) : 0u;
        }
        uint4* dst = reinterpret_cast<uint4*>(codes + row * (TERMS * Kp) + k0);
        dst[0] = make_uint4(o1[0], o1[1], o1[2], o1[3]);
        if (TERMS == 2)
            dst[Kp / 16] = make_uint4(o2[0], o2[1], o2[2], o2[3]);
    }
    if (nan)
        flag_status(status, FPQ_ERR_NAN_INPUT);
}

// NCHW FP32 -> zero-framed channels-last term codes [B][Hp][Wp][TERMS * Cp] (as quantize_nchw_to_nhwc_e4m3_kernel,
// with the conversion above)
template <int TERMS>
__global__ void __launch_bounds__(256) quantize_nchw_to_nhwc_terms_kernel(const float* __restrict__ x, int C, int H, int W,
                                                                          int pad, int Cp, float rinv, QFormat f,
                                                                          CodeTable tab1, CodeTable tab2,
                                                                          uint8_t* __restrict__ codes, int* status)
{
    __shared__ __align__(16) uint8_t tile[2][32][128 + 16];
    __shared__ uint8_t s1[256], s2[256];
    s1[threadIdx.x] = tab1.t[threadIdx.x];
    s2[threadIdx.x] = tab2.t[threadIdx.x];
    __syncthreads();
    asm volatile("griddepcontrol.launch_dependents;");
    bool nan = false;
    const int HW = H * W, Wp = W + 2 * pad, Hp = H + 2 * pad;
    const int row = TERMS * Cp;
    const int b = blockIdx.z;
    const int c0 = blockIdx.y * 128;
    const int p0 = blockIdx.x * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 pixels x 8 channel groups of 16
    const float* xb = x + (int64_t)b * C * HW;
    uint8_t* ob = codes + (int64_t)b * Hp * Wp * row;
    const int p = p0 + tx;
    {
        const int cl = ty * 16;
        float t[16];
#pragma unroll
        for (int q = 0; q < 16; ++q)
            t[q] = (c0 + cl + q < C && p < HW) ? __fmul_rn(__ldg(xb + (int64_t)(c0 + cl + q) * HW + p), rinv) : 0.f;
        uint32_t w[4], o1[4], o2[4];
        codes16_bytes(t, f, w, nan);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            o1[j] = map4(w[j], s1);
            o2[j] = TERMS == 2 ? map4(w[j], s2) : 0u;
        }
        *reinterpret_cast<uint4*>(&tile[0][tx][cl]) = make_uint4(o1[0], o1[1], o1[2], o1[3]);
        if (TERMS == 2)
            *reinterpret_cast<uint4*>(&tile[1][tx][cl]) = make_uint4(o2[0], o2[1], o2[2], o2[3]);
    }
    __syncthreads();
    {
        // 32 pixels x 8 chunks of 16 channels: 8 consecutive threads write one pixel's row
        const int pl = threadIdx.x >> 3, ch = (threadIdx.x & 7) * 16;
        const int pp = p0 + pl, c = c0 + ch;
        if (pp < HW && c < Cp) {
            const int yy = pp / W, xx = pp - yy * W;
            uint8_t* dst = ob + ((int64_t)(yy + pad) * Wp + (xx + pad)) * row + c;
            *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(&tile[0][pl][ch]);
            if (TERMS == 2)
                *reinterpret_cast<uint4*>(dst + Cp) = *reinterpret_cast<const uint4*>(&tile[1][pl][ch]);
        }
    }
    // frame pixels of this image, shared out over the blocks of the image's pixel axis
    if (pad > 0) {
        const int nframe = Hp * Wp - HW;
        const int chunks = (min(Cp - c0, 128)) / 16;
        const int total = nframe * chunks;
        for (int t = blockIdx.x * 256 + threadIdx.x; t < total; t += gridDim.x * 256) {
            const int j = t / chunks, ch = (t - j * chunks) * 16;
            int yp, xp;
            const int top = pad * Wp;
            if (j < top) {
                yp = j / Wp; xp = j - yp * Wp;
            } else if (j < 2 * top) {
                const int k = j - top;
                yp = H + pad + k / Wp; xp = k % Wp;
            } else {
                const int k = j - 2 * top;             // 2*pad frame pixels per interior row
                yp = pad + k / (2 * pad);
                const int e = k % (2 * pad);
                xp = (e < pad) ? e : W + e;
            }
            uint8_t* dst = ob + ((int64_t)yp * Wp + xp) * row + c0 + ch;
            *reinterpret_cast<uint4*>(dst) = make_uint4(0, 0, 0, 0);
            if (TERMS == 2)
                *reinterpret_cast<uint4*>(dst + Cp) = make_uint4(0, 0, 0, 0);
        }
    }
    if (nan)
        flag_status(status, FPQ_ERR_NAN_INPUT);
}

// Prepared weights [rows][row_bytes] -> [rows][2 * row_bytes] with every row written twice side by side (the
// weights' side of a contraction over [first terms | second terms] of the activations).  16 bytes per thread.
__global__ void __launch_bounds__(256) repeat_rows_kernel(const uint4* __restrict__ src, int64_t rows, int64_t vec_per_row,
                                                          uint4* __restrict__ dst)
{
    const int64_t total = rows * vec_per_row;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / vec_per_row, c = i - r * vec_per_row;
        const uint4 v = __ldg(src + i);
        dst[r * 2 * vec_per_row + c] = v;
        dst[r * 2 * vec_per_row + vec_per_row + c] = v;
    }
}

cudaError_t launch_quantize_rows_terms(const float* x, int64_t M, int64_t K, int64_t Kp, float scale, const QFormat& f,
                                       const CodeTable& t1, const CodeTable* t2, uint8_t* codes, cudaStream_t st)
{
    const int grid = grid_for(M * (Kp / 16), 256);
    if (t2)
        quantize_rows_terms_kernel<2><<<grid, 256, 0, st>>>(x, M, K, Kp, 1.0f / scale, f, t1, *t2, codes, status_word());
    else
        quantize_rows_terms_kernel<1><<<grid, 256, 0, st>>>(x, M, K, Kp, 1.0f / scale, f, t1, t1, codes, status_word());
    return cudaGetLastError();
}

cudaError_t launch_quantize_nchw_to_nhwc_terms(const float* x, int B, int C, int H, int W, int pad, int Cp, float scale,
                                               const QFormat& f, const CodeTable& t1, const CodeTable* t2, uint8_t* codes,
                                               cudaStream_t st)
{
    dim3 grid((H * W + 31) / 32, (Cp + 127) / 128, B);
    if (t2)
        quantize_nchw_to_nhwc_terms_kernel<2><<<grid, 256, 0, st>>>(x, C, H, W, pad, Cp, 1.0f / scale, f, t1, *t2, codes,
                                                                     status_word());
    else
        quantize_nchw_to_nhwc_terms_kernel<1><<<grid, 256, 0, st>>>(x, C, H, W, pad, Cp, 1.0f / scale, f, t1, t1, codes,
                                                                     status_word());
    return cudaGetLastError();
}

cudaError_t launch_repeat_rows(const void* src, int64_t rows, int64_t row_bytes, void* dst, cudaStream_t st)
{
    const int64_t vec = row_bytes / 16;
    repeat_rows_kernel<<<grid_for(rows * vec, 256), 256, 0, st>>>((const uint4*)src, rows, vec, (uint4*)dst);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------
// Zero census of a code tensor (the sparsity measurement): how many of the n values are the
// code 0.  16 bytes per thread and step, one atomic per block.  *count must be 0 at the start.
// ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) zero_census_kernel(const uint8_t* __restrict__ codes, int64_t n, int four_bit,
                                                          unsigned long long* __restrict__ count)
{
    const int64_t nbytes = four_bit ? n / 2 : n;              // whole bytes; an odd 4-bit tail is handled below
    const int64_t head = min(nbytes, (int64_t)((16 - ((uintptr_t)codes & 15)) & 15));
    const int64_t nvec = (nbytes - head) / 16;
    const uint4* v4 = reinterpret_cast<const uint4*>(codes + head);
    unsigned zeros = 0;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x, stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t v = tid; v < nvec; v += stride) {
        const uint4 q = __ldg(v4 + v);
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (four_bit) {
                // a nibble is zero iff none of its four bits is set
                uint32_t t = w[k] | (w[k] >> 1);
                t |= t >> 2;
                zeros += 8 - __popc(t & 0x11111111u);
            } else {
                uint32_t t = w[k] | (w[k] >> 4);
                t |= t >> 2;
                t |= t >> 1;
                zeros += 4 - __popc(t & 0x01010101u);
            }
        }
    }
    // bytes before the first and after the last aligned 16-byte group
    for (int64_t i = tid; i < nbytes - nvec * 16; i += stride) {
        const uint8_t c = codes[i < head ? i : i + nvec * 16];
        zeros += four_bit ? ((c & 0xf) == 0) + ((c >> 4) == 0) : (c == 0);
    }
    if (four_bit && (n & 1) && tid == 0)
        zeros += (codes[nbytes] & 0xf) == 0;                   // last value sits alone in a low nibble
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        zeros += __shfl_xor_sync(0xffffffffu, zeros, o);
    __shared__ unsigned s_z[8];
    if ((threadIdx.x & 31) == 0)
        s_z[threadIdx.x >> 5] = zeros;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long t = 0;
        for (int w = 0; w < 8; ++w)
            t += s_z[w];
        if (t)
            atomicAdd(count, t);
    }
}

cudaError_t launch_zero_census(const uint8_t* codes, int64_t n, int four_bit, unsigned long long* count, cudaStream_t st)
{
    cudaError_t e = cudaMemsetAsync(count, 0, sizeof(unsigned long long), st);
    if (e != cudaSuccess || n == 0)
        return e;
    const int64_t nbytes = four_bit ? (n + 1) / 2 : n;
    zero_census_kernel<<<grid_for(nbytes / 16 + 1, 256), 256, 0, st>>>(codes, n, four_bit, count);
    return cudaGetLastError();
}

cudaError_t launch_prepare_weight(const uint8_t* codes, int N, int C, int RS, int Cp, int four_bit, int C1, int C1p,
                                  const CodeTable* table, const CodeTable* table2, uint8_t* prepared, cudaStream_t st)
{
    int64_t total = (int64_t)N * RS * Cp / ((four_bit && !table) ? 2 : 1);
    CodeTable tab = {}, tab2 = {};
    if (table)
        tab = *table;
    if (table2)
        tab2 = *table2;
    prepare_weight_kernel<<<grid_for(total, 256), 256, 0, st>>>(codes, N, C, RS, Cp, four_bit, table ? 1 : 0, tab,
                                                                table2 ? 1 : 0, tab2, C1, C1p, prepared);
    return cudaGetLastError();
}

// ---- self-test of the bounded wait every pipeline role uses ---------------------------------------
__global__ void __launch_bounds__(32) bounded_wait_selftest_kernel(long long limit, int* status)
{
    __shared__ __align__(8) unsigned long long bar;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        fence_barrier_init();
    }
    __syncwarp();
    // phase 0 of a fresh barrier never completes without an arrival
    if (!mbar_wait(b, 0, limit) && threadIdx.x == 0)
        flag_status(status, FPQ_ERR_TIMEOUT);
}

cudaError_t launch_bounded_wait_selftest(long long limit, int* status, cudaStream_t st)
{
    bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(limit, status);
    return cudaGetLastError();
}

}  // namespace fpq
