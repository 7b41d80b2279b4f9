// extern "C" entry points: argument checks, format resolution, dispatch.
#include <math.h>
#include <cmath>
#include <string.h>

#include <map>
#include <mutex>

#include "fpq_common.cuh"
#include "fpq_kernels.h"

namespace fpq {

__device__ int g_status = 0;

int* status_word()
{
    // one lookup per device: the symbol has a separate instance on each GPU
    static int* ptr[64] = {nullptr};
    static std::mutex mu;                      // host threads may make their first call at the same time
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64)
        return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_status) != cudaSuccess)
            return nullptr;
        ptr[dev] = (int*)p;
    }
    return ptr[dev];
}

float format_cmax(fpq_format f)
{
    int top = (1 << f.exp_bits) - 1;
    if (f.sat_mode == FPQ_SAT_NATIVE && f.exp_bits == 4 && f.man_bits == 3)
        return ldexpf(1.75f, top - f.exp_bias);
    if (f.sat_mode == FPQ_SAT_NATIVE && f.exp_bits == 5 && f.man_bits == 2)
        return ldexpf(1.75f, top - 1 - f.exp_bias);
    return ldexpf(2.0f - ldexpf(1.0f, -f.man_bits), top - f.exp_bias);
}

bool resolve_format(fpq_format f, QFormat* q)
{
    if (f.exp_bits < 1 || f.man_bits < 1 || 1 + f.exp_bits + f.man_bits > 8)
        return false;
    if (f.sat_mode != FPQ_SAT_PAPER && f.sat_mode != FPQ_SAT_NATIVE)
        return false;
    int top = (1 << f.exp_bits) - 1;
    // every grid value must be a normal FP32 number, and so must 1.5 * 2^23 steps of the top binade (the
    // rounding constant of the quantizer kernels)
    if (top - f.exp_bias + 23 - f.man_bits > 126 || 1 - f.exp_bias - f.man_bits < -125)
        return false;
    q->e = f.exp_bits;
    q->m = f.man_bits;
    q->B = f.exp_bias;
    q->sign_shift = f.exp_bits + f.man_bits;
    q->four_bit = (1 + f.exp_bits + f.man_bits <= 4) ? 1 : 0;
    q->code_max = (1 << (f.exp_bits + f.man_bits)) - 1;
    if (f.sat_mode == FPQ_SAT_NATIVE && f.exp_bits == 4 && f.man_bits == 3)
        q->code_max = 0x7E;
    if (f.sat_mode == FPQ_SAT_NATIVE && f.exp_bits == 5 && f.man_bits == 2)
        q->code_max = 0x7B;
    float c = format_cmax(f);
    memcpy(&q->cmax_bits, &c, 4);
    q->native_e4m3 = (f.exp_bits == 4 && f.man_bits == 3 && f.exp_bias == 7 && f.sat_mode == FPQ_SAT_NATIVE) ? 1 : 0;
    return true;
}

static bool is_e4m3_native(fpq_format f)
{
    return f.exp_bits == 4 && f.man_bits == 3 && f.exp_bias == 7 && f.sat_mode == FPQ_SAT_NATIVE;
}

static bool is_e5m2_native(fpq_format f)
{
    return f.exp_bits == 5 && f.man_bits == 2 && f.exp_bias == 15 && f.sat_mode == FPQ_SAT_NATIVE;
}

// activation formats the tensor cores read as they are: E4M3 (bias 7) and the OCP E5M2 (bias 15), both saturating
// at the type's largest finite value
static bool act_native(fpq_format f) { return is_e4m3_native(f) || is_e5m2_native(f); }

static bool is_e2m1(fpq_format f)
{
    return f.exp_bits == 2 && f.man_bits == 1 && f.exp_bias == 1;
}

// Value of one code of format f (format equation of Sec. IV-B), sign included.
static double code_value(int code, fpq_format f)
{
    int em = f.exp_bits + f.man_bits;
    int p = (code >> f.man_bits) & ((1 << f.exp_bits) - 1);
    int d = code & ((1 << f.man_bits) - 1);
    double v = p == 0 ? ldexp((double)d, 1 - f.exp_bias - f.man_bits)
                      : ldexp(1.0 + ldexp((double)d, -f.man_bits), p - f.exp_bias);
    return ((code >> em) & 1) ? -v : v;
}

// Exact re-encode of a weight format into the contraction's E4M3 operand type: true when every value of
// f (that its quantizer can produce) is also a finite value of E4M3 with bias 7; table[code of f] = the
// E4M3 code of the same value (a zero of either sign maps to +0; codes f never produces map to 0).
static bool embeds_in_e4m3(fpq_format f, CodeTable* tab)
{
    QFormat q;
    if (!resolve_format(f, &q))
        return false;
    const fpq_format e4m3 = {4, 3, 7, FPQ_SAT_NATIVE};
    int ncodes = 1 << (1 + f.exp_bits + f.man_bits);
    int mag_mask = (1 << (f.exp_bits + f.man_bits)) - 1;
    for (int c = 0; c < 256; ++c) {
        uint8_t out = 0;
        if (c < ncodes && (c & mag_mask) <= q.code_max) {
            double v = code_value(c, f);
            if (v != 0.0) {
                int found = -1;
                for (int k = 1; k <= 0x7E && found < 0; ++k)
                    if (code_value(k, e4m3) == fabs(v))
                        found = k;
                if (found < 0)
                    return false;
                out = (uint8_t)(found | (v < 0.0 ? 0x80 : 0));
            }
        }
        if (tab)
            tab->t[c] = out;
    }
    return true;
}

// Exact split of a weight format into two E4M3 terms: true when every value v of f is first + second with
// first = the largest E4M3 magnitude not above |v| (sign of v) and second = v - first also a finite E4M3
// value (formats with up to 7 significant bits inside E4M3's exponent range: E3M4, E2M5, the paper's E4M3
// with its code for 480 = 448 + 32).  Tables: code of f -> E4M3 code of each term.
static bool splits_in_two_at(fpq_format f, fpq_format e4m3 /* the container type */, int top_code, int shift,
                             CodeTable* first, CodeTable* second)
{
    QFormat q;
    if (!resolve_format(f, &q))
        return false;
    int ncodes = 1 << (1 + f.exp_bits + f.man_bits);
    int mag_mask = (1 << (f.exp_bits + f.man_bits)) - 1;
    for (int c = 0; c < 256; ++c) {
        uint8_t o1 = 0, o2 = 0;
        if (c < ncodes && (c & mag_mask) <= q.code_max) {
            double v = ldexp(code_value(c, f), shift), a = fabs(v);
            if (a != 0.0) {
                int k1 = 0;                               // magnitudes increase with the code
                for (int k = 1; k <= top_code; ++k)
                    if (code_value(k, e4m3) <= a)
                        k1 = k;
                double rest = a - code_value(k1, e4m3);
                int k2 = rest == 0.0 ? 0 : -1;
                for (int k = 1; k <= top_code && k2 < 0; ++k)
                    if (code_value(k, e4m3) == rest)
                        k2 = k;
                if (k2 < 0)
                    return false;
                uint8_t sign = v < 0.0 ? 0x80 : 0;
                o1 = (uint8_t)(k1 ? (k1 | sign) : 0);
                o2 = (uint8_t)(k2 ? (k2 | sign) : 0);
            }
        }
        if (first)
            first->t[c] = o1;
        if (second)
            second->t[c] = o2;
    }
    return true;
}

// The terms are those of 2^shift * v for the smallest |shift| <= 16 that works (0 first): a format whose bias
// puts it outside E4M3's range (the paper's default E4M3 with bias 8: shift 1) still splits, and the layer
// multiplies the dequantization scale by 2^-shift, which is exact.
static bool splits_in_two(fpq_format f, fpq_format container, int top_code, CodeTable* first, CodeTable* second,
                          int* shift)
{
    for (int m = 0; m <= 16; ++m)
        for (int sgn = 1; sgn >= (m ? -1 : 1); sgn -= 2)
            if (splits_in_two_at(f, container, top_code, sgn * m, first, second)) {
                if (shift)
                    *shift = sgn * m;
                return true;
            }
    return false;
}

static const fpq_format kE4M3Native = {4, 3, 7, FPQ_SAT_NATIVE};
static const fpq_format kE5M2Native = {5, 2, 15, FPQ_SAT_NATIVE};

// How the layer calls run a weight format: read by the tensor cores as it is, re-encoded into one E4M3
// term when the weights are prepared, prepared as two E4M3 terms (twice the reduction length), or on the
// CUDA cores.  Working this out walks all codes of the format, so the answer (a pure function of the four
// format fields) is kept per format; host threads take turns at the table.
enum { W_INVALID = 0, W_NATIVE, W_ONE_TERM, W_TWO_TERM, W_OTHER };
struct WeightClass {
    int kind;
    int shift;             // W_TWO_TERM: the terms are those of 2^shift * value
    int e5m2;              // W_TWO_TERM: the terms are E5M2 (bias 15) codes instead of E4M3 codes
    CodeTable t1, t2;      // W_ONE_TERM: t1; W_TWO_TERM: t1 (first terms), t2 (second terms)
};

static const WeightClass& classify_weight(fpq_format f)
{
    static std::mutex mu;
    static std::map<uint64_t, WeightClass> known;
    static const WeightClass invalid = {};
    if (f.exp_bits < 1 || f.exp_bits > 8 || f.man_bits < 1 || f.man_bits > 8 || f.sat_mode < 0 || f.sat_mode > 1)
        return invalid;
    const uint64_t key = ((uint64_t)(uint8_t)f.exp_bits << 56) | ((uint64_t)(uint8_t)f.man_bits << 48) |
                         ((uint64_t)(uint8_t)f.sat_mode << 40) | (uint64_t)(uint32_t)f.exp_bias;
    std::lock_guard<std::mutex> lock(mu);
    auto it = known.find(key);
    if (it != known.end())
        return it->second;
    WeightClass c = {};
    QFormat q;
    if (!resolve_format(f, &q))
        c.kind = W_INVALID;
    else if (is_e4m3_native(f) || is_e2m1(f) || is_e5m2_native(f))
        c.kind = W_NATIVE;
    else if (embeds_in_e4m3(f, &c.t1))
        c.kind = W_ONE_TERM;
    else if (splits_in_two(f, kE4M3Native, 0x7E, &c.t1, &c.t2, &c.shift))
        c.kind = W_TWO_TERM;
    else if (splits_in_two(f, kE5M2Native, 0x7B, &c.t1, &c.t2, &c.shift))
        c.kind = W_TWO_TERM, c.e5m2 = 1;                  // the paper's E5M2 with all 32 exponent fields finite
    else
        c.kind = W_OTHER;
    return known.emplace(key, c).first->second;
}

static bool weight_native(fpq_format f) { return classify_weight(f).kind == W_NATIVE; }
static bool weight_reencoded(fpq_format f) { return classify_weight(f).kind == W_ONE_TERM; }
static bool weight_two_term(fpq_format f) { return classify_weight(f).kind == W_TWO_TERM; }

// Operand pairs the tensor-core contraction has no type for run on the CUDA cores (fpq_linear and fpq_conv2d
// only; the staged, host-buffer, two-tensor and built-in-scratch forms keep to the tensor-core pairs).
// Activations of a format whose every value is one value (terms = 1) or the sum of two values (terms = 2) of a
// tensor-core type - the classification the weights use: E3M4, E2M5, the paper's all-finite E4M3 as two E4M3
// terms, the small formats inside E4M3 as one - against weights the tensor cores read as they are (or re-encoded):
// fpq_linear and fpq_conv2d quantize with the general arithmetic, write the terms as operand codes
// [first terms | second terms] and run the ordinary contraction over that against the weights repeated.
static bool act_terms_pair(fpq_format fx, fpq_format fw, int* terms)
{
    QFormat q;
    if (!resolve_format(fx, &q) || !resolve_format(fw, &q) || act_native(fx))
        return false;
    const WeightClass& c = classify_weight(fx);
    if (c.kind != W_ONE_TERM && c.kind != W_TWO_TERM)
        return false;
    if (terms)
        *terms = c.kind == W_TWO_TERM ? 2 : 1;
    return weight_native(fw) || weight_reencoded(fw);
}

static bool general_pair(fpq_format fx, fpq_format fw)
{
    QFormat q;
    if (!resolve_format(fx, &q) || !resolve_format(fw, &q))
        return false;
    if (act_terms_pair(fx, fw, nullptr))
        return false;
    return !(act_native(fx) && (weight_native(fw) || weight_reencoded(fw) || weight_two_term(fw)));
}

static bool two_term_pair(fpq_format fx, fpq_format fw)
{
    QFormat q;
    return resolve_format(fx, &q) && resolve_format(fw, &q) && act_native(fx) && weight_two_term(fw);
}

// Format of the codes in the prepared copy: re-encoded weights are E4M3 there.
static QFormat prepared_format(fpq_format fw)
{
    const fpq_format e4m3 = {4, 3, 7, FPQ_SAT_NATIVE};
    QFormat q;
    const WeightClass& wc = classify_weight(fw);
    resolve_format(wc.kind == W_TWO_TERM ? (wc.e5m2 ? kE5M2Native : kE4M3Native) : (wc.kind == W_ONE_TERM ? e4m3 : fw), &q);
    return q;
}

// 2^-shift of a two-term weight format: what the prepared terms have to be multiplied by.
static float two_term_unshift(fpq_format fw) { return ldexpf(1.0f, -classify_weight(fw).shift); }

static int g_path_policy = FPQ_PATH_AUTO;

static bool aligned(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }

// an activation scale must be a positive finite number: 1 / scale is what the kernels multiply by
static bool bad_scale(float s) { return !(s > 0.f) || std::isinf(s); }

static int64_t padded_c(int64_t C) { return round_up(C, 128); }

// Scratch of the term-activation route: the operand codes [units][terms * Cp] (units = rows or framed pixels), then,
// with two terms, the prepared weights with every (output, tap) row written twice side by side.
struct TermsPlan {
    int terms;
    int64_t Cp;
    size_t codes_bytes, w_off, w_row_bytes, bytes;
};
static TermsPlan terms_plan(fpq_format fx, fpq_format fw, int64_t units, int64_t C, int64_t w_rows)
{
    TermsPlan t = {};
    act_terms_pair(fx, fw, &t.terms);
    QFormat q;
    resolve_format(fw, &q);
    t.Cp = padded_c(C);
    t.codes_bytes = (size_t)units * t.terms * t.Cp;
    t.w_row_bytes = (size_t)((q.four_bit && !weight_reencoded(fw)) ? t.Cp / 2 : t.Cp);
    t.w_off = (size_t)round_up((int64_t)t.codes_bytes, 256);
    t.bytes = t.terms == 2 ? t.w_off + (size_t)w_rows * 2 * t.w_row_bytes : t.codes_bytes;
    return t;
}

static fpq_status check_pair(fpq_format fx, fpq_format fw)
{
    QFormat q;
    if (!resolve_format(fx, &q) || !resolve_format(fw, &q))
        return FPQ_ERR_FORMAT;
    if (!act_native(fx))
        return FPQ_ERR_UNSUPPORTED;
    if (!weight_native(fw) && !weight_reencoded(fw))
        return FPQ_ERR_UNSUPPORTED;
    return FPQ_OK;
}

}  // namespace fpq

using namespace fpq;

extern "C" {

float fpq_format_max(fpq_format fmt)
{
    QFormat q;
    if (!resolve_format(fmt, &q))
        return 0.f;
    return format_cmax(fmt);
}

float fpq_scale_from_max(float maxabs, fpq_format fmt)
{
    float c = fpq_format_max(fmt);
    if (c == 0.f)
        return 0.f;
    return maxabs / c;
}

fpq_status fpq_quantize_weight(const float* w, int64_t N, int64_t K, const float* scale, fpq_format fmt,
                               const uint8_t* rounding_bits, uint8_t* codes, void* stream)
{
    QFormat q;
    if (!resolve_format(fmt, &q))
        return FPQ_ERR_FORMAT;
    if (N < 0 || K < 0 || (N > 0 && K > INT64_MAX / 8 / N))
        return FPQ_ERR_SHAPE;
    if (N == 0 || K == 0)
        return FPQ_OK;
    if (!w || !scale || !codes)
        return FPQ_ERR_NULL;
    if (!aligned(w, 4) || !aligned(scale, 4))
        return FPQ_ERR_ALIGN;
    if (!status_word())
        return FPQ_ERR_CUDA;
    return launch_quantize_weight(w, N, K, scale, q, rounding_bits, codes, (cudaStream_t)stream) == cudaSuccess
               ? FPQ_OK
               : FPQ_ERR_CUDA;
}

fpq_status fpq_quantize_act(const float* x, int64_t n, float scale, fpq_format fmt, uint8_t* codes, void* stream)
{
    if (bad_scale(scale))
        return FPQ_ERR_SCALE;
    QFormat q;
    if (!resolve_format(fmt, &q))
        return FPQ_ERR_FORMAT;
    if (n < 0)
        return FPQ_ERR_SHAPE;
    if (n == 0)
        return FPQ_OK;
    if (!x || !codes)
        return FPQ_ERR_NULL;
    if (!aligned(x, 4))
        return FPQ_ERR_ALIGN;
    if (!status_word())
        return FPQ_ERR_CUDA;
    return launch_quantize_act(x, n, scale, q, codes, (cudaStream_t)stream) == cudaSuccess ? FPQ_OK : FPQ_ERR_CUDA;
}

static fpq_status check_desc(const fpq_layer_desc* d)
{
    if (!d)
        return FPQ_ERR_NULL;
    if (d->kind != FPQ_LINEAR && d->kind != FPQ_CONV2D)
        return FPQ_ERR_SHAPE;
    if (d->N < 1 || d->C < 1 || d->R < 1 || d->S < 1)
        return FPQ_ERR_SHAPE;
    if (d->kind == FPQ_LINEAR && (d->R != 1 || d->S != 1))
        return FPQ_ERR_SHAPE;
    if ((int64_t)d->R * d->S > 1024 || (int64_t)d->N * d->R * d->S * padded_c(d->C) > ((int64_t)1 << 40))
        return FPQ_ERR_SHAPE;
    return FPQ_OK;
}

size_t fpq_prepared_size(fpq_format fmt, const fpq_layer_desc* d)
{
    QFormat q;
    if (!resolve_format(fmt, &q) || check_desc(d) != FPQ_OK)
        return 0;
    size_t elems = (size_t)d->N * d->R * d->S * (size_t)padded_c(d->C);
    if (weight_two_term(fmt))
        return 2 * elems;
    return (q.four_bit && !weight_reencoded(fmt)) ? elems / 2 : elems;
}

fpq_status fpq_prepare_weight(const uint8_t* codes, fpq_format fmt, const fpq_layer_desc* d, void* prepared,
                              void* stream)
{
    QFormat q;
    if (!resolve_format(fmt, &q))
        return FPQ_ERR_FORMAT;
    fpq_status s = check_desc(d);
    if (s != FPQ_OK)
        return s;
    if (!codes || !prepared)
        return FPQ_ERR_NULL;
    if (!aligned(prepared, 128))
        return FPQ_ERR_ALIGN;
    const WeightClass& wc = classify_weight(fmt);
    if (wc.kind == W_TWO_TERM)
        return launch_prepare_weight(codes, d->N, d->C, d->R * d->S, 2 * (int)padded_c(d->C), q.four_bit, 0, 0, &wc.t1,
                                     &wc.t2, (uint8_t*)prepared, (cudaStream_t)stream) == cudaSuccess
                   ? FPQ_OK
                   : FPQ_ERR_CUDA;
    const bool re = wc.kind == W_ONE_TERM;
    return launch_prepare_weight(codes, d->N, d->C, d->R * d->S, (int)padded_c(d->C), q.four_bit, 0, 0,
                                 re ? &wc.t1 : nullptr, nullptr, (uint8_t*)prepared, (cudaStream_t)stream) == cudaSuccess
               ? FPQ_OK
               : FPQ_ERR_CUDA;
}

size_t fpq_linear_workspace_size(int64_t M, int64_t N, int64_t K, fpq_format fx, fpq_format fw)
{
    if (general_pair(fx, fw)) {
        if (M < 0 || N < 0 || K < 1 || M > 0x7fffffff || N > 0x7fffffff || K > 0x7fffffff)
            return 0;
        GeneralLayer g = {};
        g.M = M, g.N = N, g.K = K;
        return general_layer_workspace_bytes(g);
    }
    if (two_term_pair(fx, fw))
        return (M < 0 || K < 0 || K > 0x3fffffff) ? 0 : (size_t)(M * 2 * padded_c(K));
    if (act_terms_pair(fx, fw, nullptr))
        return (M < 0 || N < 0 || K < 1 || M > 0x7fffffff || N > 0x7fffffff || K > 0x3fffffff) ? 0
                                                                                              : terms_plan(fx, fw, M, K, N).bytes;
    (void)N;
    if (check_pair(fx, fw) != FPQ_OK || M < 0 || K < 0)
        return 0;
    return (size_t)(M * round_up(K, 16));
}

static fpq_status linear_checks(fpq_format fx, fpq_format fw, int64_t M, int64_t N, int64_t K, const void* workspace,
                                size_t ws_bytes, bool* empty)
{
    fpq_status s = check_pair(fx, fw);
    if (s != FPQ_OK)
        return s;
    if (M < 0 || N < 0 || K < 0 || M > 0x7fffffff || N > 0x7fffffff || K > 0x7fffffff)
        return FPQ_ERR_SHAPE;
    *empty = (M == 0 || N == 0);
    if (*empty)
        return FPQ_OK;
    if (K == 0)
        return FPQ_ERR_SHAPE;
    if (!workspace || ws_bytes < (size_t)(M * round_up(K, 16)))
        return FPQ_ERR_WORKSPACE;
    if (!aligned(workspace, 128))
        return FPQ_ERR_ALIGN;
    return FPQ_OK;
}

fpq_status fpq_linear_quantize_input(const float* x, float x_scale, fpq_format fx, fpq_format fw, int64_t M, int64_t N,
                                     int64_t K, void* workspace, size_t ws_bytes, void* stream)
{
    if (bad_scale(x_scale))
        return FPQ_ERR_SCALE;
    bool empty = false;
    fpq_status s = linear_checks(fx, fw, M, N, K, workspace, ws_bytes, &empty);
    if (s != FPQ_OK || empty)
        return s;
    if (!x)
        return FPQ_ERR_NULL;
    if (!aligned(x, 16))
        return FPQ_ERR_ALIGN;
    if (!status_word())
        return FPQ_ERR_CUDA;
    return launch_quantize_rows_e4m3(x, M, K, round_up(K, 16), x_scale, (uint8_t*)workspace, (cudaStream_t)stream,
                                     is_e5m2_native(fx) ? 1 : 0) == cudaSuccess
               ? FPQ_OK
               : FPQ_ERR_CUDA;
}

static fpq_status linear_contract_impl(const void* workspace, size_t ws_bytes, const void* w_prepared,
                                       const float* w_scale, float x_scale, fpq_format fx, fpq_format fw,
                                       const float* bias, float* y, int64_t M, int64_t N, int64_t K, void* stream,
                                       int after_stage1, const float* x_fused)
{
    if (bad_scale(x_scale))
        return FPQ_ERR_SCALE;
    bool empty = false;
    fpq_status s = linear_checks(fx, fw, M, N, K, workspace, ws_bytes, &empty);
    if (s != FPQ_OK || empty)
        return s;
    if (!w_prepared || !w_scale || !y)
        return FPQ_ERR_NULL;
    if (!aligned(y, 16) || !aligned(w_prepared, 128) || !aligned(w_scale, 4) || (bias && !aligned(bias, 4)))
        return FPQ_ERR_ALIGN;
    if (!status_word())
        return FPQ_ERR_CUDA;
    GemmProblem p{};
    p.conv = 0;
    p.x = x_fused;
    p.C = (int)K;
    p.after_stage1 = after_stage1;
    p.w4 = is_e2m1(fw) ? 1 : 0;
    p.w_e5m2 = is_e5m2_native(fw) ? 1 : 0;
    p.a_e5m2 = is_e5m2_native(fx) ? 1 : 0;
    p.M = M;
    p.N = (int)N;
    p.Cp = (int)padded_c(K);
    p.Ca = (int)round_up(K, 16);
    p.B = p.H = p.W = p.Ho = p.Wo = 1;
    p.R = p.S = 1;
    p.pad = 0;
    p.stride = 1;
    p.a_codes = (const uint8_t*)workspace;
    p.w_prepared = w_prepared;
    p.w_scale = w_scale;
    p.x_scale = x_scale;
    p.bias = bias;
    p.y = y;
    return launch_gemm(p, (cudaStream_t)stream);
}

fpq_status fpq_linear_contract(const void* workspace, size_t ws_bytes, const void* w_prepared, const float* w_scale,
                               float x_scale, fpq_format fx, fpq_format fw, const float* bias, float* y, int64_t M,
                               int64_t N, int64_t K, void* stream)
{
    return linear_contract_impl(workspace, ws_bytes, w_prepared, w_scale, x_scale, fx, fw, bias, y, M, N, K, stream, 0,
                                nullptr);
}

fpq_status fpq_linear(const float* x, const void* w_prepared, const float* w_scale, float x_scale, fpq_format fx,
                      fpq_format fw, const float* bias, float* y, int64_t M, int64_t N, int64_t K, void* workspace,
                      size_t ws_bytes, void* stream)
{
    if (bad_scale(x_scale))
        return FPQ_ERR_SCALE;
    if (general_pair(fx, fw)) {
        if (M < 0 || N < 0 || K < 0 || M > 0x7fffffff || N > 0x7fffffff || K > 0x7fffffff)
            return FPQ_ERR_SHAPE;
        if (M == 0 || N == 0)
            return FPQ_OK;
        if (K == 0)
            return FPQ_ERR_SHAPE;
        GeneralLayer g = {};
        g.M = M, g.N = N, g.K = K, g.C = (int)K, g.R = 1, g.S = 1, g.Cp = (int)padded_c(K);
        resolve_format(fx, &g.fx);
        g.fw = prepared_format(fw);
        g.w_two_term = weight_two_term(fw) ? 1 : 0;
        g.w_mul = g.w_two_term ? two_term_unshift(fw) : 1.0f;
        g.x = x, g.w_prepared = w_prepared, g.w_scale = w_scale, g.x_scale = x_scale, g.bias = bias, g.y = y;
        if (!x || !w_prepared || !w_scale || !y)
            return FPQ_ERR_NULL;
        if (!aligned(x, 16) || !aligned(y, 16) || !aligned(w_prepared, 128) || !aligned(w_scale, 4) ||
            (bias && !aligned(bias, 4)) || !aligned(workspace, 256))
            return FPQ_ERR_ALIGN;
        if (!workspace || ws_bytes < general_layer_workspace_bytes(g))
            return FPQ_ERR_WORKSPACE;
        return launch_general_layer(g, workspace, (cudaStream_t)stream);
    }
    if (act_terms_pair(fx, fw, nullptr)) {
        if (M < 0 || N < 0 || K < 0 || M > 0x7fffffff || N > 0x7fffffff || K > 0x3fffffff)
            return FPQ_ERR_SHAPE;
        if (M == 0 || N == 0)
            return FPQ_OK;
        if (K == 0)
            return FPQ_ERR_SHAPE;
        if (!x || !w_prepared || !w_scale || !y)
            return FPQ_ERR_NULL;
        if (!aligned(x, 16) || !aligned(y, 16) || !aligned(w_prepared, 128) || !aligned(w_scale, 4) ||
            (bias && !aligned(bias, 4)) || !aligned(workspace, 256))
            return FPQ_ERR_ALIGN;
        const TermsPlan t = terms_plan(fx, fw, M, K, N);
        if (!workspace || ws_bytes < t.bytes)
            return FPQ_ERR_WORKSPACE;
        if (!status_word())
            return FPQ_ERR_CUDA;
        const WeightClass& cx = classify_weight(fx);
        const fpq_format term = cx.e5m2 ? kE5M2Native : kE4M3Native;
        QFormat qx;
        resolve_format(fx, &qx);
        cudaStream_t st = (cudaStream_t)stream;
        const void* wp = w_prepared;
        if (t.terms == 2) {
            if (launch_repeat_rows(w_prepared, N, (int64_t)t.w_row_bytes, (uint8_t*)workspace + t.w_off, st) != cudaSuccess)
                return FPQ_ERR_CUDA;
            wp = (const uint8_t*)workspace + t.w_off;
        }
        if (launch_quantize_rows_terms(x, M, K, t.Cp, x_scale, qx, cx.t1, t.terms == 2 ? &cx.t2 : nullptr,
                                       (uint8_t*)workspace, st) != cudaSuccess)
            return FPQ_ERR_CUDA;
        return linear_contract_impl(workspace, ws_bytes, wp, w_scale, x_scale * ldexpf(1.0f, -cx.shift), term, fw, bias, y, M,
                                    N, t.terms * t.Cp, stream, 1, nullptr);
    }
    if (two_term_pair(fx, fw)) {
        // weights prepared as two E4M3 terms: activation codes written twice per row, then the ordinary
        // contraction over twice the (padded) reduction length
        if (K < 0 || K > 0x3fffffff)
            return FPQ_ERR_SHAPE;
        const int64_t K2 = 2 * padded_c(K);
        bool empty = false;
        const fpq_format term = classify_weight(fw).e5m2 ? kE5M2Native : kE4M3Native;
        fpq_status s = linear_checks(fx, term, M, N, K2, workspace, ws_bytes, &empty);
        if (s != FPQ_OK || empty)
            return s;
        if (K == 0)
            return FPQ_ERR_SHAPE;
        if (!x || !w_prepared || !w_scale || !y)
            return FPQ_ERR_NULL;
        if (!aligned(x, 16) || !aligned(y, 16) || !aligned(w_prepared, 128) || !aligned(w_scale, 4) ||
            (bias && !aligned(bias, 4)))
            return FPQ_ERR_ALIGN;
        if (!status_word())
            return FPQ_ERR_CUDA;
        if (launch_quantize_rows_e4m3_twice(x, M, K, K2 / 2, x_scale, (uint8_t*)workspace, (cudaStream_t)stream,
                                            is_e5m2_native(fx) ? 1 : 0) != cudaSuccess)
            return FPQ_ERR_CUDA;
        // (the contraction uses the activation scale only to dequantize: the weights' power of two goes there)
        return linear_contract_impl(workspace, ws_bytes, w_prepared, w_scale, x_scale * two_term_unshift(fw), fx, term, bias,
                                    y, M, N, K2, stream, 1, nullptr);
    }
    bool empty = false;
    fpq_status s = linear_checks(fx, fw, M, N, K, workspace, ws_bytes, &empty);
    if (s != FPQ_OK || empty)
        return s;
    // reject everything the second stage would reject before the first stage runs
    if (!x || !w_prepared || !w_scale || !y)
        return FPQ_ERR_NULL;
    if (!aligned(x, 16) || !aligned(y, 16) || !aligned(w_prepared, 128) || !aligned(w_scale, 4) ||
        (bias && !aligned(bias, 4)))
        return FPQ_ERR_ALIGN;
    // a handful of rows (time-embedding projections): one pass over the weights on the CUDA cores,
    // whatever the route policy says; the workspace is not touched
    if (small_m_linear_applies(M, K) && N <= 0x7fffffff && !is_e5m2_native(fw) && is_e4m3_native(fx)) {
        if (!status_word())
            return FPQ_ERR_CUDA;
        return launch_small_m_linear(x, (int)M, (int)K, w_prepared, is_e2m1(fw) ? 1 : 0, (int)N, w_scale, x_scale, bias, y,
                                     (cudaStream_t)stream);
    }
    // one kernel: the activations are quantized inside the contraction's operand staging
    // (AUTO takes the two-kernel route: measured faster on B200 so far)
    if (g_path_policy == FPQ_PATH_FUSED && is_e4m3_native(fx)) {
        s = linear_contract_impl(workspace, ws_bytes, w_prepared, w_scale, x_scale, fx, fw, bias, y, M, N, K, stream, 0,
                                 x);
        if (s != FPQ_ERR_UNSUPPORTED)
            return s;
    }
    s = fpq_linear_quantize_input(x, x_scale, fx, fw, M, N, K, workspace, ws_bytes, stream);
    if (s != FPQ_OK)
        return s;
    return linear_contract_impl(workspace, ws_bytes, w_prepared, w_scale, x_scale, fx, fw, bias, y, M, N, K, stream, 1,
                                nullptr);
}

static fpq_status conv_shape(int B, int C, int H, int W, int C_out, int R, int S, int pad, int stride, int* Ho,
                             int* Wo)
{
    if (B < 0 || C < 1 || H < 1 || W < 1 || C_out < 0 || R < 1 || S < 1 || pad < 0 || stride < 1)
        return FPQ_ERR_SHAPE;
    if (H + 2 * pad < R || W + 2 * pad < S)
        return FPQ_ERR_SHAPE;
    *Ho = (H + 2 * pad - R) / stride + 1;
    *Wo = (W + 2 * pad - S) / stride + 1;
    if ((int64_t)B * C * H * W > ((int64_t)1 << 40) || (int64_t)B * C_out * *Ho * *Wo > ((int64_t)1 << 40))
        return FPQ_ERR_SHAPE;
    return FPQ_OK;
}

// Geometry of a convolution on the CUDA-core route; false if the shape is out of range.
static bool general_conv(GeneralLayer* g, fpq_format fx, fpq_format fw, int B, int C, int H, int W, int C_out, int R,
                         int S, int pad, int stride)
{
    int Ho, Wo;
    if (conv_shape(B, C, H, W, C_out, R, S, pad, stride, &Ho, &Wo) != FPQ_OK)
        return false;
    int64_t K = (int64_t)C * R * S, M = (int64_t)B * Ho * Wo;
    if (K > 0x7fffffff || M > 0x7fffffff || (K > 0 && M > ((int64_t)1 << 38) / K))
        return false;
    g->conv = 1;
    g->M = M, g->N = C_out, g->K = K;
    g->B = B, g->C = C, g->H = H, g->W = W, g->R = R, g->S = S, g->pad = pad, g->stride = stride, g->Ho = Ho, g->Wo = Wo;
    g->Cp = (int)padded_c(C);
    resolve_format(fx, &g->fx);
    g->fw = prepared_format(fw);
    g->w_two_term = weight_two_term(fw) ? 1 : 0;
    g->w_mul = g->w_two_term ? two_term_unshift(fw) : 1.0f;
    return true;
}

size_t fpq_conv2d_workspace_size(int B, int C, int H, int W, int C_out, int R, int S, int pad, int stride,
                                 fpq_format fx, fpq_format fw)
{
    int Ho, Wo;
    if (general_pair(fx, fw)) {
        GeneralLayer g = {};
        if (!general_conv(&g, fx, fw, B, C, H, W, C_out, R, S, pad, stride))
            return 0;
        return general_layer_workspace_bytes(g);
    }
    if (two_term_pair(fx, fw)) {
        if (conv_shape(B, C, H, W, C_out, R, S, pad, stride, &Ho, &Wo) != FPQ_OK)
            return 0;
        return (size_t)B * (H + 2 * pad) * (W + 2 * pad) * (size_t)(2 * padded_c(C));
    }
    if (act_terms_pair(fx, fw, nullptr)) {
        if (conv_shape(B, C, H, W, C_out, R, S, pad, stride, &Ho, &Wo) != FPQ_OK || C > 0x3fffffff / 2)
            return 0;
        return terms_plan(fx, fw, (int64_t)B * (H + 2 * pad) * (W + 2 * pad), C, (int64_t)C_out * R * S).bytes;
    }
    if (check_pair(fx, fw) != FPQ_OK || conv_shape(B, C, H, W, C_out, R, S, pad, stride, &Ho, &Wo) != FPQ_OK)
        return 0;
    return (size_t)B * (H + 2 * pad) * (W + 2 * pad) * (size_t)round_up(C, 16);
}

static fpq_status conv_checks(fpq_format fx, fpq_format fw, int B, int C, int H, int W, int C_out, int R, int S,
                              int pad, int stride, const void* workspace, size_t ws_bytes, int* Ho, int* Wo,
                              bool* empty)
{
    fpq_status s = check_pair(fx, fw);
    if (s != FPQ_OK)
        return s;
    s = conv_shape(B, C, H, W, C_out, R, S, pad, stride, Ho, Wo);
    if (s != FPQ_OK)
        return s;
    *empty = (B == 0 || C_out == 0);
    if (*empty)
        return FPQ_OK;
    if (B > 65535)
        return FPQ_ERR_SHAPE;
    if (!workspace || ws_bytes < (size_t)B * (H + 2 * pad) * (W + 2 * pad) * (size_t)round_up(C, 16))
        return FPQ_ERR_WORKSPACE;
    if (!aligned(workspace, 128))
        return FPQ_ERR_ALIGN;
    return FPQ_OK;
}

fpq_status fpq_conv2d_quantize_input(const float* x, float x_scale, fpq_format fx, fpq_format fw, int B, int C, int H,
                                     int W, int C_out, int R, int S, int pad, int stride, void* workspace,
                                     size_t ws_bytes, void* stream)
{
    if (bad_scale(x_scale))
        return FPQ_ERR_SCALE;
    int Ho, Wo;
    bool empty = false;
    fpq_status s = conv_checks(fx, fw, B, C, H, W, C_out, R, S, pad, stride, workspace, ws_bytes, &Ho, &Wo, &empty);
    if (s != FPQ_OK || empty)
        return s;
    if (!x)
        return FPQ_ERR_NULL;
    if (!aligned(x, 4))
        return FPQ_ERR_ALIGN;
    if (!status_word())
        return FPQ_ERR_CUDA;
    return launch_quantize_nchw_to_nhwc_e4m3(x, B, C, H, W, pad, (int)round_up(C, 16), (int)round_up(C, 16), 0, x_scale,
                                             (uint8_t*)workspace, (cudaStream_t)stream, is_e5m2_native(fx) ? 1 : 0) == cudaSuccess
               ? FPQ_OK
               : FPQ_ERR_CUDA;
}

static fpq_status conv2d_contract_impl(const void* workspace, size_t ws_bytes, const void* w_prepared,
                                       const float* w_scale, float x_scale, fpq_format fx, fpq_format fw,
                                       const float* bias, float* y, int B, int C, int H, int W, int C_out, int R,
                                       int S, int pad, int stride, void* stream, int after_stage1,
                                       const float* x_fused, bool pair_only = false)
{
    if (bad_scale(x_scale))
        return FPQ_ERR_SCALE;
    int Ho, Wo;
    bool empty = false;
    fpq_status s = conv_checks(fx, fw, B, C, H, W, C_out, R, S, pad, stride, workspace, ws_bytes, &Ho, &Wo, &empty);
    if (s != FPQ_OK || empty)
        return s;
    if (!w_prepared || !w_scale || !y)
        return FPQ_ERR_NULL;
    if (!aligned(y, 4) || !aligned(w_prepared, 128) || !aligned(w_scale, 4) || (bias && !aligned(bias, 4)))
        return FPQ_ERR_ALIGN;
    if (!status_word())
        return FPQ_ERR_CUDA;
    GemmProblem p{};
    p.conv = 1;
    p.x = x_fused;
    p.C = C;
    p.after_stage1 = after_stage1;
    p.w4 = is_e2m1(fw) ? 1 : 0;
    p.w_e5m2 = is_e5m2_native(fw) ? 1 : 0;
    p.a_e5m2 = is_e5m2_native(fx) ? 1 : 0;
    p.M = (int64_t)B * Ho * Wo;
    p.N = C_out;
    p.Cp = (int)padded_c(C);
    p.Ca = (int)round_up(C, 16);
    p.B = B;
    p.H = H;
    p.W = W;
    p.Ho = Ho;
    p.Wo = Wo;
    p.R = R;
    p.S = S;
    p.pad = pad;
    p.stride = stride;
    p.a_codes = (const uint8_t*)workspace;
    p.w_prepared = w_prepared;
    p.w_scale = w_scale;
    p.x_scale = x_scale;
    p.bias = bias;
    p.y = y;
    if (x_fused) {
        // one kernel on CTA pairs where the weights fit in shared memory; else the general fused form
        if (!pair_only || pair_conv_preferred(p)) {
            const fpq_status sp = launch_pair_conv(p, (cudaStream_t)stream);
            if (sp != FPQ_ERR_UNSUPPORTED)
                return sp;
        }
        if (pair_only)
            return FPQ_ERR_UNSUPPORTED;
    } else if (g_path_policy != FPQ_PATH_TWO_KERNELS_NARROW && pair_gemm_preferred(p)) {
        // long reductions with enough tiles: the wide MMAs of a CTA pair
        const fpq_status sp = launch_pair_gemm(p, (cudaStream_t)stream);
        if (sp != FPQ_ERR_UNSUPPORTED)
            return sp;
    }
    return launch_gemm(p, (cudaStream_t)stream);
}

fpq_status fpq_conv2d_contract(const void* workspace, size_t ws_bytes, const void* w_prepared, const float* w_scale,
                               float x_scale, fpq_format fx, fpq_format fw, const float* bias, float* y, int B, int C,
                               int H, int W, int C_out, int R, int S, int pad, int stride, void* stream)
{
    return conv2d_contract_impl(workspace, ws_bytes, w_prepared, w_scale, x_scale, fx, fw, bias, y, B, C, H, W, C_out,
                                R, S, pad, stride, stream, 0, nullptr);
}

fpq_status fpq_conv2d(const float* x, const void* w_prepared, const float* w_scale, float x_scale, fpq_format fx,
                      fpq_format fw, const float* bias, float* y, int B, int C, int H, int W, int C_out, int R, int S,
                      int pad, int stride, void* workspace, size_t ws_bytes, void* stream)
{
    if (bad_scale(x_scale))
        return FPQ_ERR_SCALE;
    if (general_pair(fx, fw)) {
        GeneralLayer g = {};
        if (!general_conv(&g, fx, fw, B, C, H, W, C_out, R, S, pad, stride))
            return FPQ_ERR_SHAPE;
        if (B == 0 || C_out == 0)
            return FPQ_OK;
        g.x = x, g.w_prepared = w_prepared, g.w_scale = w_scale, g.x_scale = x_scale, g.bias = bias, g.y = y;
        if (!x || !w_prepared || !w_scale || !y)
            return FPQ_ERR_NULL;
        if (!aligned(x, 4) || !aligned(y, 4) || !aligned(w_prepared, 128) || !aligned(w_scale, 4) ||
            (bias && !aligned(bias, 4)) || !aligned(workspace, 256))
            return FPQ_ERR_ALIGN;
        if (!workspace || ws_bytes < general_layer_workspace_bytes(g))
            return FPQ_ERR_WORKSPACE;
        return launch_general_layer(g, workspace, (cudaStream_t)stream);
    }
    if (act_terms_pair(fx, fw, nullptr)) {
        // activations as one or two terms of a tensor-core type: term codes in the framed channels-last scratch
        // ([first terms | second terms] per pixel), the weights' rows repeated behind it, then the ordinary
        // convolution over terms * (padded C) channels
        if (C < 1 || C > 0x3fffffff / 2)
            return FPQ_ERR_SHAPE;
        int Ho3, Wo3;
        fpq_status s3 = conv_shape(B, C, H, W, C_out, R, S, pad, stride, &Ho3, &Wo3);
        if (s3 != FPQ_OK)
            return s3;
        if (B == 0 || C_out == 0)
            return FPQ_OK;
        if (B > 65535)
            return FPQ_ERR_SHAPE;
        if (!x || !w_prepared || !w_scale || !y)
            return FPQ_ERR_NULL;
        if (!aligned(x, 4) || !aligned(y, 4) || !aligned(w_prepared, 128) || !aligned(w_scale, 4) ||
            (bias && !aligned(bias, 4)) || !aligned(workspace, 256))
            return FPQ_ERR_ALIGN;
        const TermsPlan t = terms_plan(fx, fw, (int64_t)B * (H + 2 * pad) * (W + 2 * pad), C, (int64_t)C_out * R * S);
        if (!workspace || ws_bytes < t.bytes)
            return FPQ_ERR_WORKSPACE;
        if (!status_word())
            return FPQ_ERR_CUDA;
        const WeightClass& cx = classify_weight(fx);
        const fpq_format term = cx.e5m2 ? kE5M2Native : kE4M3Native;
        QFormat qx;
        resolve_format(fx, &qx);
        cudaStream_t st = (cudaStream_t)stream;
        const void* wp = w_prepared;
        if (t.terms == 2) {
            if (launch_repeat_rows(w_prepared, (int64_t)C_out * R * S, (int64_t)t.w_row_bytes, (uint8_t*)workspace + t.w_off,
                                   st) != cudaSuccess)
                return FPQ_ERR_CUDA;
            wp = (const uint8_t*)workspace + t.w_off;
        }
        if (launch_quantize_nchw_to_nhwc_terms(x, B, C, H, W, pad, (int)t.Cp, x_scale, qx, cx.t1,
                                               t.terms == 2 ? &cx.t2 : nullptr, (uint8_t*)workspace, st) != cudaSuccess)
            return FPQ_ERR_CUDA;
        return conv2d_contract_impl(workspace, ws_bytes, wp, w_scale, x_scale * ldexpf(1.0f, -cx.shift), term, fw, bias, y, B,
                                    (int)(t.terms * t.Cp), H, W, C_out, R, S, pad, stride, stream, 1, nullptr);
    }
    if (two_term_pair(fx, fw)) {
        // weights prepared as two E4M3 terms per tap: the activation codes fill two channel ranges of the
        // framed channels-last scratch, then the ordinary convolution over 2 * (padded C) channels
        if (C < 1 || C > 0x3fffffff / 2)
            return FPQ_ERR_SHAPE;
        const int Cp = (int)padded_c(C), C2 = 2 * Cp;
        int Ho2, Wo2;
        bool empty2 = false;
        const fpq_format term = classify_weight(fw).e5m2 ? kE5M2Native : kE4M3Native;
        fpq_status s2 = conv_checks(fx, term, B, C2, H, W, C_out, R, S, pad, stride, workspace, ws_bytes, &Ho2, &Wo2, &empty2);
        if (s2 != FPQ_OK || empty2)
            return s2;
        if (!x || !w_prepared || !w_scale || !y)
            return FPQ_ERR_NULL;
        if (!aligned(x, 4) || !aligned(y, 4) || !aligned(w_prepared, 128) || !aligned(w_scale, 4) ||
            (bias && !aligned(bias, 4)))
            return FPQ_ERR_ALIGN;
        if (!status_word())
            return FPQ_ERR_CUDA;
        cudaStream_t st = (cudaStream_t)stream;
        const int e5 = is_e5m2_native(fx) ? 1 : 0;
        if (launch_quantize_nchw_to_nhwc_e4m3(x, B, C, H, W, pad, Cp, C2, 0, x_scale, (uint8_t*)workspace, st, e5) !=
                cudaSuccess ||
            launch_quantize_nchw_to_nhwc_e4m3(x, B, C, H, W, pad, Cp, C2, Cp, x_scale, (uint8_t*)workspace, st, e5) !=
                cudaSuccess)
            return FPQ_ERR_CUDA;
        return conv2d_contract_impl(workspace, ws_bytes, w_prepared, w_scale, x_scale * two_term_unshift(fw), fx, term, bias,
                                    y, B, C2, H, W, C_out, R, S, pad, stride, stream, 1, nullptr);
    }
    int Ho, Wo;
    bool empty = false;
    fpq_status s = conv_checks(fx, fw, B, C, H, W, C_out, R, S, pad, stride, workspace, ws_bytes, &Ho, &Wo, &empty);
    if (s != FPQ_OK || empty)
        return s;
    if (!x || !w_prepared || !w_scale || !y)
        return FPQ_ERR_NULL;
    if (!aligned(x, 4) || !aligned(y, 4) || !aligned(w_prepared, 128) || !aligned(w_scale, 4) ||
        (bias && !aligned(bias, 4)))
        return FPQ_ERR_ALIGN;
    // one kernel where the geometry allows it (stride 1): the activations are quantized inside the
    // contraction's operand staging; otherwise quantize to codes first
    // (the library's own choice: the CTA-pair kernel for the shapes it measured faster on, else two kernels)
    if ((g_path_policy == FPQ_PATH_FUSED || g_path_policy == FPQ_PATH_AUTO) && is_e4m3_native(fx)) {
        s = conv2d_contract_impl(workspace, ws_bytes, w_prepared, w_scale, x_scale, fx, fw, bias, y, B, C, H, W, C_out,
                                 R, S, pad, stride, stream, 0, x, g_path_policy == FPQ_PATH_AUTO);
        if (s != FPQ_ERR_UNSUPPORTED)
            return s;
    }
    s = fpq_conv2d_quantize_input(x, x_scale, fx, fw, B, C, H, W, C_out, R, S, pad, stride, workspace, ws_bytes,
                                  stream);
    if (s != FPQ_OK)
        return s;
    return conv2d_contract_impl(workspace, ws_bytes, w_prepared, w_scale, x_scale, fx, fw, bias, y, B, C, H, W, C_out,
                                R, S, pad, stride, stream, 1, nullptr);
}

// ---- convolution over two concatenated input tensors, each with its own scale ----------------

static fpq_status split_shape(int C1, int C2)
{
    if (C1 < 1 || C2 < 1 || (int64_t)C1 + C2 > (1 << 20))
        return FPQ_ERR_SHAPE;
    return FPQ_OK;
}

size_t fpq_prepared_size_split(fpq_format fmt, int32_t N, int32_t C1, int32_t C2, int32_t R, int32_t S)
{
    QFormat q;
    fpq_layer_desc d = {FPQ_CONV2D, N, C1 + C2, R, S};
    if (!resolve_format(fmt, &q) || split_shape(C1, C2) != FPQ_OK || check_desc(&d) != FPQ_OK)
        return 0;
    size_t elems = (size_t)N * R * S * (size_t)(padded_c(C1) + padded_c(C2));
    return (q.four_bit && !weight_reencoded(fmt)) ? elems / 2 : elems;
}

fpq_status fpq_prepare_weight_split(const uint8_t* codes, fpq_format fmt, int32_t N, int32_t C1, int32_t C2,
                                    int32_t R, int32_t S, void* prepared, void* stream)
{
    QFormat q;
    if (!resolve_format(fmt, &q))
        return FPQ_ERR_FORMAT;
    fpq_status s = split_shape(C1, C2);
    if (s != FPQ_OK)
        return s;
    fpq_layer_desc d = {FPQ_CONV2D, N, C1 + C2, R, S};
    s = check_desc(&d);
    if (s != FPQ_OK)
        return s;
    if (!codes || !prepared)
        return FPQ_ERR_NULL;
    if (!aligned(prepared, 128))
        return FPQ_ERR_ALIGN;
    const WeightClass& wc = classify_weight(fmt);
    const bool re = wc.kind == W_ONE_TERM;
    return launch_prepare_weight(codes, N, C1 + C2, R * S, (int)(padded_c(C1) + padded_c(C2)), q.four_bit, C1,
                                 (int)padded_c(C1), re ? &wc.t1 : nullptr, nullptr, (uint8_t*)prepared,
                                 (cudaStream_t)stream) == cudaSuccess
               ? FPQ_OK
               : FPQ_ERR_CUDA;
}

static size_t split_row_bytes(int C1, int C2) { return (size_t)(padded_c(C1) + round_up(C2, 16)); }

size_t fpq_conv2d_split_workspace_size(int B, int C1, int C2, int H, int W, int C_out, int R, int S, int pad,
                                       int stride, fpq_format fx, fpq_format fw)
{
    int Ho, Wo;
    if (check_pair(fx, fw) != FPQ_OK || split_shape(C1, C2) != FPQ_OK ||
        conv_shape(B, C1 + C2, H, W, C_out, R, S, pad, stride, &Ho, &Wo) != FPQ_OK)
        return 0;
    return (size_t)B * (H + 2 * pad) * (W + 2 * pad) * split_row_bytes(C1, C2);
}

fpq_status fpq_conv2d_split(const float* x1, int C1, float x1_scale, const float* x2, int C2, float x2_scale,
                            const void* w_prepared, const float* w_scale, fpq_format fx, fpq_format fw,
                            const float* bias, float* y, int B, int H, int W, int C_out, int R, int S, int pad,
                            int stride, void* workspace, size_t ws_bytes, void* stream)
{
    if (bad_scale(x1_scale) || bad_scale(x2_scale))
        return FPQ_ERR_SCALE;
    fpq_status s = check_pair(fx, fw);
    if (s != FPQ_OK)
        return s;
    s = split_shape(C1, C2);
    if (s != FPQ_OK)
        return s;
    int Ho, Wo;
    s = conv_shape(B, C1 + C2, H, W, C_out, R, S, pad, stride, &Ho, &Wo);
    if (s != FPQ_OK)
        return s;
    if (B == 0 || C_out == 0)
        return FPQ_OK;
    if (B > 65535)
        return FPQ_ERR_SHAPE;
    const size_t row = split_row_bytes(C1, C2);
    if (!workspace || ws_bytes < (size_t)B * (H + 2 * pad) * (W + 2 * pad) * row)
        return FPQ_ERR_WORKSPACE;
    if (!x1 || !x2 || !w_prepared || !w_scale || !y)
        return FPQ_ERR_NULL;
    if (!aligned(workspace, 128) || !aligned(x1, 4) || !aligned(x2, 4) || !aligned(y, 4) || !aligned(w_prepared, 128) ||
        !aligned(w_scale, 4) || (bias && !aligned(bias, 4)))
        return FPQ_ERR_ALIGN;
    if (!status_word())
        return FPQ_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    const int C1p = (int)padded_c(C1);
    // each tensor is quantized with its own scale into its own channel range of the framed
    // channels-last codes; the concatenated FP32 tensor is never formed
    const int e5 = is_e5m2_native(fx) ? 1 : 0;
    if (launch_quantize_nchw_to_nhwc_e4m3(x1, B, C1, H, W, pad, C1p, (int)row, 0, x1_scale, (uint8_t*)workspace, st, e5) !=
            cudaSuccess ||
        launch_quantize_nchw_to_nhwc_e4m3(x2, B, C2, H, W, pad, (int)round_up(C2, 16), (int)row, C1p, x2_scale,
                                          (uint8_t*)workspace, st, e5) != cudaSuccess)
        return FPQ_ERR_CUDA;
    GemmProblem p{};
    p.conv = 1;
    p.after_stage1 = 1;
    p.w4 = is_e2m1(fw) ? 1 : 0;
    p.w_e5m2 = is_e5m2_native(fw) ? 1 : 0;
    p.a_e5m2 = is_e5m2_native(fx) ? 1 : 0;
    p.M = (int64_t)B * Ho * Wo;
    p.N = C_out;
    p.Cp = C1p + (int)padded_c(C2);
    p.Ca = (int)row;
    p.B = B;
    p.H = H;
    p.W = W;
    p.Ho = Ho;
    p.Wo = Wo;
    p.R = R;
    p.S = S;
    p.pad = pad;
    p.stride = stride;
    p.a_codes = (const uint8_t*)workspace;
    p.w_prepared = w_prepared;
    p.w_scale = w_scale;
    p.x_scale = x1_scale;
    p.x_scale2 = x2_scale;
    p.c_seg = C1p / 128;
    p.bias = bias;
    p.y = y;
    return launch_gemm(p, st);
}

}  // extern "C"

// ---- host-buffer forms: copy in, layer, copy out, pipelined over slices of the batch --------------
//
// The two copies of one slice cannot overlap, but the copy-in of slice i + 1, the layer on slice i
// and the copy-out of slice i - 1 can (PCIe carries both directions at once).  The pipeline needs a
// stream per direction and an event per hand-over: they are created once per device at the first
// host-form call and kept.

namespace fpq {

constexpr int HOST_SLICES = 8;

struct HostPipe {
    bool ready;
    cudaStream_t in, out;
    cudaEvent_t start, end, copied[HOST_SLICES], computed[HOST_SLICES];
};

static HostPipe* host_pipe()
{
    static std::mutex m;
    static HostPipe pipes[64] = {};
    std::lock_guard<std::mutex> lock(m);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64)
        return nullptr;
    HostPipe& p = pipes[dev];
    if (!p.ready) {
        bool ok = cudaStreamCreateWithFlags(&p.in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&p.out, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&p.end, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; ok && i < HOST_SLICES; ++i)
            ok = cudaEventCreateWithFlags(&p.copied[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&p.computed[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok)
            return nullptr;
        p.ready = true;
    }
    return &p;
}

// units = rows (linear) or images (conv); in_stride / out_stride = floats per unit; layer(u0, n) enqueues
// the layer on units [u0, u0 + n) of the device buffers on `st`.
template <typename Layer>
static fpq_status host_pipeline(const float* x_host, float* x_dev, float* y_dev, float* y_host, int64_t units,
                                int64_t in_stride, int64_t out_stride, cudaStream_t st, Layer layer)
{
    if (units == 0)
        return FPQ_OK;
    HostPipe* hp = host_pipe();
    if (!hp)
        return FPQ_ERR_CUDA;
    // slices only when the copies are long enough to be worth overlapping
    const int64_t bytes = 4 * units * (in_stride + out_stride);
    int64_t slices = bytes >= (8ll << 20) ? HOST_SLICES : 1;
    if (slices > units)
        slices = units;
    bool ok = cudaEventRecord(hp->start, st) == cudaSuccess && cudaStreamWaitEvent(hp->in, hp->start, 0) == cudaSuccess &&
              cudaStreamWaitEvent(hp->out, hp->start, 0) == cudaSuccess;
    for (int64_t i = 0; ok && i < slices; ++i) {
        const int64_t u0 = units * i / slices, n = units * (i + 1) / slices - u0;
        ok = cudaMemcpyAsync(x_dev + u0 * in_stride, x_host + u0 * in_stride, sizeof(float) * (size_t)(n * in_stride),
                             cudaMemcpyHostToDevice, hp->in) == cudaSuccess &&
             cudaEventRecord(hp->copied[i], hp->in) == cudaSuccess;
    }
    fpq_status s = ok ? FPQ_OK : FPQ_ERR_CUDA;
    for (int64_t i = 0; s == FPQ_OK && i < slices; ++i) {
        const int64_t u0 = units * i / slices, n = units * (i + 1) / slices - u0;
        if (cudaStreamWaitEvent(st, hp->copied[i], 0) != cudaSuccess) {
            s = FPQ_ERR_CUDA;
            break;
        }
        s = layer(u0, n);
        if (s != FPQ_OK)
            break;
        if (cudaEventRecord(hp->computed[i], st) != cudaSuccess || cudaStreamWaitEvent(hp->out, hp->computed[i], 0) != cudaSuccess ||
            cudaMemcpyAsync(y_host + u0 * out_stride, y_dev + u0 * out_stride, sizeof(float) * (size_t)(n * out_stride),
                            cudaMemcpyDeviceToHost, hp->out) != cudaSuccess)
            s = FPQ_ERR_CUDA;
    }
    // whatever happened, nothing of this call may still be in flight on the side streams afterwards
    const bool drained = cudaStreamSynchronize(hp->in) == cudaSuccess && cudaStreamSynchronize(hp->out) == cudaSuccess &&
                         cudaStreamSynchronize(st) == cudaSuccess;
    if (s != FPQ_OK)
        return s;
    return drained ? FPQ_OK : FPQ_ERR_CUDA;
}

}  // namespace fpq

extern "C" {

fpq_status fpq_linear_host(const float* x_host, float* x_dev, const void* w_prepared, const float* w_scale,
                           float x_scale, fpq_format fx, fpq_format fw, const float* bias, float* y_dev,
                           float* y_host, int64_t M, int64_t N, int64_t K, void* workspace, size_t ws_bytes,
                           void* stream)
{
    if (!x_host || !x_dev || !y_dev || !y_host)
        return FPQ_ERR_NULL;
    if (M < 0 || N < 0 || K < 0)
        return FPQ_ERR_SHAPE;
    // (row slices stay 16-byte aligned only if whole rows are: otherwise one slice)
    const bool sliceable = (K % 4 == 0) && (N % 4 == 0);
    auto layer = [&](int64_t m0, int64_t m) {
        return fpq_linear(x_dev + m0 * K, w_prepared, w_scale, x_scale, fx, fw, bias, y_dev + m0 * N, m, N, K, workspace,
                          ws_bytes, stream);
    };
    if (!sliceable) {
        cudaStream_t st = (cudaStream_t)stream;
        if (cudaMemcpyAsync(x_dev, x_host, sizeof(float) * (size_t)M * K, cudaMemcpyHostToDevice, st) != cudaSuccess)
            return FPQ_ERR_CUDA;
        fpq_status s = layer(0, M);
        if (s != FPQ_OK)
            return s;
        if (cudaMemcpyAsync(y_host, y_dev, sizeof(float) * (size_t)M * N, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return FPQ_ERR_CUDA;
        return cudaStreamSynchronize(st) == cudaSuccess ? FPQ_OK : FPQ_ERR_CUDA;
    }
    return host_pipeline(x_host, x_dev, y_dev, y_host, M, K, N, (cudaStream_t)stream, layer);
}

fpq_status fpq_conv2d_host(const float* x_host, float* x_dev, const void* w_prepared, const float* w_scale,
                           float x_scale, fpq_format fx, fpq_format fw, const float* bias, float* y_dev,
                           float* y_host, int B, int C, int H, int W, int C_out, int R, int S, int pad, int stride,
                           void* workspace, size_t ws_bytes, void* stream)
{
    if (!x_host || !x_dev || !y_dev || !y_host)
        return FPQ_ERR_NULL;
    int Ho, Wo;
    fpq_status s = conv_shape(B, C, H, W, C_out, R, S, pad, stride, &Ho, &Wo);
    if (s != FPQ_OK)
        return s;
    const int64_t in_stride = (int64_t)C * H * W, out_stride = (int64_t)C_out * Ho * Wo;
    auto layer = [&](int64_t b0, int64_t b) {
        return fpq_conv2d(x_dev + b0 * in_stride, w_prepared, w_scale, x_scale, fx, fw, bias, y_dev + b0 * out_stride, (int)b,
                          C, H, W, C_out, R, S, pad, stride, workspace, ws_bytes, stream);
    };
    return host_pipeline(x_host, x_dev, y_dev, y_host, B, in_stride, out_stride, (cudaStream_t)stream, layer);
}

fpq_status fpq_zero_census(const uint8_t* codes, int64_t n, fpq_format fmt, uint64_t* count, void* stream)
{
    QFormat q;
    if (!resolve_format(fmt, &q))
        return FPQ_ERR_FORMAT;
    if (n < 0)
        return FPQ_ERR_SHAPE;
    if (!count || (n > 0 && !codes))
        return FPQ_ERR_NULL;
    if (!aligned(count, 8))
        return FPQ_ERR_ALIGN;
    return launch_zero_census(codes, n, q.four_bit, (unsigned long long*)count, (cudaStream_t)stream) == cudaSuccess
               ? FPQ_OK
               : FPQ_ERR_CUDA;
}

size_t fpq_search_workspace_size(int32_t n_enc, int32_t n_clip)
{
    if (n_enc < 1 || n_enc > search_max_enc() || n_clip < 1 || n_clip > search_max_clip() ||
        n_enc * n_clip > search_max_cand())
        return 0;
    return search_workspace_bytes(n_enc, n_clip);
}

fpq_status fpq_search_format(const float* x, int64_t n, const fpq_format* enc_host, int32_t n_enc, const float* clip,
                             int32_t n_clip, double* mse, int32_t* best, void* workspace, size_t ws_bytes,
                             void* stream)
{
    if (n < 0 || n_enc < 1 || n_enc > search_max_enc() || n_clip < 1 || n_clip > search_max_clip() ||
        n_enc * n_clip > search_max_cand())
        return FPQ_ERR_SHAPE;
    if (!enc_host || !clip || !mse || !best || (n > 0 && !x))
        return FPQ_ERR_NULL;
    for (int i = 0; i < n_enc; ++i) {
        QFormat q;
        if (!resolve_format(enc_host[i], &q))
            return FPQ_ERR_FORMAT;
        if (enc_host[i].sat_mode != FPQ_SAT_PAPER)
            return FPQ_ERR_UNSUPPORTED;
    }
    if (!aligned(x, 4) || !aligned(clip, 4) || !aligned(mse, 8) || !aligned(best, 4) || !aligned(workspace, 8))
        return FPQ_ERR_ALIGN;
    if (!workspace || ws_bytes < search_workspace_bytes(n_enc, n_clip))
        return FPQ_ERR_WORKSPACE;
    return launch_search(x, n, enc_host, n_enc, clip, n_clip, mse, best, workspace, (cudaStream_t)stream);
}

fpq_status fpq_search_clip_candidates(float maxabs, int32_t count, float* clip_host)
{
    if (!clip_host)
        return FPQ_ERR_NULL;
    if (count < 1 || count > search_max_clip() || !(maxabs > 0.f) || !isfinite(maxabs))
        return FPQ_ERR_SHAPE;
    for (int j = 0; j < count; ++j)
        clip_host[j] = (float)((double)maxabs * (double)(j + 1) / (double)count);
    return FPQ_OK;
}

static bool round_learn_shape_ok(int64_t M, int64_t N, int64_t K)
{
    const int64_t lim = (int64_t)1 << 31;
    return M >= 1 && N >= 1 && K >= 1 && M < lim - 128 && N <= 65535 * 128 && K <= 65535 * 128 &&
           N * K < ((int64_t)1 << 40) && M * round_up(N, 4) < ((int64_t)1 << 40);
}

size_t fpq_round_learn_workspace_size(int64_t M, int64_t N, int64_t K)
{
    if (!round_learn_shape_ok(M, N, K))
        return 0;
    return round_learn_workspace_bytes(M, N, K);
}

fpq_status fpq_round_learn_step(const float* w, const float* scale, fpq_format fmt, float* alpha, const float* a,
                                int64_t M, int64_t N, int64_t K, float reg, float lr, float* grad, double* loss,
                                void* workspace, size_t ws_bytes, void* stream)
{
    QFormat q;
    if (!resolve_format(fmt, &q))
        return FPQ_ERR_FORMAT;
    if (!round_learn_shape_ok(M, N, K) || !isfinite(reg) || !isfinite(lr))
        return FPQ_ERR_SHAPE;
    if (!w || !scale || !alpha || !a || !grad || !loss)
        return FPQ_ERR_NULL;
    if (!aligned(w, 4) || !aligned(scale, 4) || !aligned(alpha, 4) || !aligned(a, 4) || !aligned(grad, 4) ||
        !aligned(loss, 8) || !aligned(workspace, 256))
        return FPQ_ERR_ALIGN;
    if (!workspace || ws_bytes < round_learn_workspace_bytes(M, N, K))
        return FPQ_ERR_WORKSPACE;
    return launch_round_learn(w, scale, q, alpha, a, M, N, K, reg, lr, grad, loss, workspace, (cudaStream_t)stream);
}

fpq_status fpq_round_learn_unfold(const float* x, int32_t B, int32_t C, int32_t H, int32_t W, int32_t R, int32_t S,
                                  int32_t pad, int32_t stride, float* rows, void* stream)
{
    if (B < 0 || C < 1 || H < 1 || W < 1 || R < 1 || S < 1 || pad < 0 || stride < 1 || R > 64 || S > 64)
        return FPQ_ERR_SHAPE;
    if (H + 2 * (int64_t)pad < R || W + 2 * (int64_t)pad < S)
        return FPQ_ERR_SHAPE;
    int Ho = (H + 2 * pad - R) / stride + 1, Wo = (W + 2 * pad - S) / stride + 1;
    int64_t K = (int64_t)C * R * S;
    if (K > ((int64_t)1 << 30) || (int64_t)B * Ho * Wo > ((int64_t)1 << 40) / K || (int64_t)B * C * H * W > ((int64_t)1 << 40))
        return FPQ_ERR_SHAPE;
    if (B == 0)
        return FPQ_OK;
    if (!x || !rows)
        return FPQ_ERR_NULL;
    if (!aligned(x, 4) || !aligned(rows, 4))
        return FPQ_ERR_ALIGN;
    return launch_unfold(x, B, C, H, W, R, S, pad, stride, Ho, Wo, rows, (cudaStream_t)stream);
}

fpq_status fpq_round_learn_harden(const float* alpha, int64_t N, int64_t K, uint8_t* rounding_bits, void* stream)
{
    if (N < 0 || K < 0 || (K > 0 && N > (((int64_t)1 << 40) / K)))
        return FPQ_ERR_SHAPE;
    if (N * K > 0 && (!alpha || !rounding_bits))
        return FPQ_ERR_NULL;
    if (!aligned(alpha, 4))
        return FPQ_ERR_ALIGN;
    return launch_round_harden(alpha, N, K, rounding_bits, (cudaStream_t)stream);
}

int32_t fpq_conv2d_route(int B, int C, int H, int W, int C_out, int R, int S, int pad, int stride, fpq_format fx,
                         fpq_format fw)
{
    if (general_pair(fx, fw) || two_term_pair(fx, fw) || act_terms_pair(fx, fw, nullptr)) {
        QFormat q;
        if (!resolve_format(fx, &q) || !resolve_format(fw, &q))
            return FPQ_ERR_FORMAT;
        return FPQ_ROUTE_OTHER;
    }
    fpq_status s = check_pair(fx, fw);
    if (s != FPQ_OK)
        return s;
    int Ho, Wo;
    s = conv_shape(B, C, H, W, C_out, R, S, pad, stride, &Ho, &Wo);
    if (s != FPQ_OK)
        return s;
    if (g_path_policy == FPQ_PATH_TWO_KERNELS || g_path_policy == FPQ_PATH_TWO_KERNELS_NARROW || B == 0 || C_out == 0 ||
        !is_e4m3_native(fx))
        return FPQ_ROUTE_TWO_KERNELS;
    GemmProblem p{};
    p.conv = 1;
    p.x = reinterpret_cast<const float*>((uintptr_t)256);      // never followed: the plans only look at its alignment
    p.C = C;
    p.w4 = is_e2m1(fw) ? 1 : 0;
    p.w_e5m2 = is_e5m2_native(fw) ? 1 : 0;
    p.M = (int64_t)B * Ho * Wo;
    p.N = C_out;
    p.Cp = (int)padded_c(C);
    p.Ca = (int)round_up(C, 16);
    p.B = B, p.H = H, p.W = W, p.Ho = Ho, p.Wo = Wo, p.R = R, p.S = S, p.pad = pad, p.stride = stride;
    if (pair_conv_applies(p) && (g_path_policy == FPQ_PATH_FUSED || pair_conv_preferred(p)))
        return FPQ_ROUTE_PAIR_FUSED;
    if (g_path_policy == FPQ_PATH_FUSED && stride == 1)
        return FPQ_ROUTE_FUSED;                                  // (the general fused form; it may still fall back)
    return FPQ_ROUTE_TWO_KERNELS;
}

fpq_status fpq_selftest_bounded_wait(int64_t limit_cycles, void* stream)
{
    if (limit_cycles < 1 || limit_cycles > 1000000000ll)
        return FPQ_ERR_SHAPE;
    int* sw = status_word();
    if (!sw)
        return FPQ_ERR_CUDA;
    return launch_bounded_wait_selftest(limit_cycles, sw, (cudaStream_t)stream) == cudaSuccess ? FPQ_OK : FPQ_ERR_CUDA;
}

fpq_status fpq_set_path_policy(int32_t policy)
{
    if (policy != FPQ_PATH_AUTO && policy != FPQ_PATH_FUSED && policy != FPQ_PATH_TWO_KERNELS &&
        policy != FPQ_PATH_TWO_KERNELS_NARROW)
        return FPQ_ERR_UNSUPPORTED;
    g_path_policy = policy;
    return FPQ_OK;
}

int32_t fpq_get_path_policy(void) { return g_path_policy; }

fpq_status fpq_read_status(void* stream)
{
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess)
        return FPQ_ERR_CUDA;
    int* sw = status_word();
    if (!sw)
        return FPQ_ERR_CUDA;
    int v = 0, zero = 0;
    if (cudaMemcpy(&v, sw, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
        return FPQ_ERR_CUDA;
    if (v != 0 && cudaMemcpy(sw, &zero, sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess)
        return FPQ_ERR_CUDA;
    // one bit per kind of event; the most serious one is reported
    if (v & STATUS_BIT_TIMEOUT)
        return FPQ_ERR_TIMEOUT;
    if (v & STATUS_BIT_NAN)
        return FPQ_ERR_NAN_INPUT;
    return FPQ_OK;
}

const char* fpq_status_string(fpq_status s)
{
    switch (s) {
    case FPQ_OK: return "ok";
    case FPQ_ERR_NULL: return "null pointer";
    case FPQ_ERR_FORMAT: return "invalid number format";
    case FPQ_ERR_SHAPE: return "invalid shape";
    case FPQ_ERR_ALIGN: return "misaligned pointer";
    case FPQ_ERR_UNSUPPORTED: return "unsupported operand formats or geometry";
    case FPQ_ERR_WORKSPACE: return "workspace missing or too small";
    case FPQ_ERR_CUDA: return "CUDA call failed";
    case FPQ_ERR_SCALE: return "activation scale is not a positive finite number";
    case FPQ_ERR_TIMEOUT: return "device-side wait timed out";
    case FPQ_ERR_NAN_INPUT: return "NaN input quantized to zero";
    case FPQ_ERR_TOO_LARGE: return "problem larger than the built-in scratch capacity";
    default: return "unknown status";
    }
}

}  // extern "C"
