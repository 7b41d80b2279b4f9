// Quantized layer for operand formats the tensor cores have no type for (E3M4, E2M5, E5M2, the paper's
// E4M3 with its code for 480, or any activation format other than native E4M3).  Same arithmetic model
// as the tensor-core path - operands are exact grid values, every product is exact in FP32 (at most
// 7 + 8 significant bits), sums are FP32 - carried out on FP32 values:
//   quantize_values_kernel   x -> value of q(x / scale) in code units, FP32 (Sec. IV-B rounding equation)
//   decode_prepared_kernel   prepared weight codes -> FP32 values, [N][C*R*S] in the boundary's order
//   unfold (convolutions)    input rows written out
//   contraction              rows x weights^T with y = acc * (scale_x * scale_w[n]) + bias[n] in its epilogue, on the
//                            tensor cores (grid values are TF32 numbers: one exact product per term); rows that are
//                            not a multiple of 4 floats: FP32 multiply-adds on the CUDA cores, then dequant_store_kernel
#include "fpq_kernels.h"

namespace fpq {

namespace {

// Value of one code (format equation of Sec. IV-B), exact in FP32.
__device__ __forceinline__ float decode_code(uint32_t code, const QFormat& f)
{
    uint32_t mag = code & ((1u << f.sign_shift) - 1u);
    uint32_t p = mag >> f.m, d = mag & ((1u << f.m) - 1u);
    int ex = (p ? (int)p : 1) - f.B - f.m;
    float v = __uint2float_rn(p ? (1u << f.m) + d : d) * __uint_as_float((uint32_t)(ex + 127) << 23);
    return ((code >> f.sign_shift) & 1u) ? -v : v;
}

__global__ void __launch_bounds__(256) quantize_values_kernel(const float* __restrict__ x, int64_t n, float scale,
                                                              QFormat f, float* __restrict__ v, int* __restrict__ status)
{
    const float r = __fdiv_rn(1.0f, scale);
    bool any_nan = false;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        bool nan = false;
        uint32_t code = quantize_rne_bits(__fmul_rn(__ldg(x + i), r), f, nan);
        any_nan |= nan;
        v[i] = decode_code(code, f);
    }
    if (any_nan)
        flag_status(status, FPQ_ERR_NAN_INPUT);
}

// prepared [N][RS][Cp] (one byte per code, or two codes per byte, even index in the low nibble) ->
// values [N][C*RS] with column c * RS + tap, the order of the boundary's [C][R][S] weights.
// two_term: a prepared row holds [first terms | second terms], Cp bytes each, and a weight is their sum (exact).
__global__ void __launch_bounds__(256) decode_prepared_kernel(const uint8_t* __restrict__ prepared, int64_t N, int C,
                                                              int RS, int Cp, QFormat f, int two_term, float w_mul,
                                                              float* __restrict__ wv)
{
    const int64_t K = (int64_t)C * RS, total = N * K;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        int64_t n = i / K;
        int k = (int)(i - n * K);
        int c = k / RS, tap = k - c * RS;
        if (two_term) {
            int64_t e1 = (n * RS + tap) * (2 * (int64_t)Cp) + c;
            wv[i] = (decode_code(__ldg(prepared + e1), f) + decode_code(__ldg(prepared + e1 + Cp), f)) * w_mul;
            continue;
        }
        int64_t e = (n * RS + tap) * Cp + c;
        uint32_t code;
        if (f.four_bit) {
            uint32_t b = __ldg(prepared + (e >> 1));
            code = (e & 1) ? (b >> 4) : (b & 0xfu);
        } else {
            code = __ldg(prepared + e);
        }
        wv[i] = decode_code(code, f);
    }
}

__global__ void __launch_bounds__(256) dequant_store_kernel(const float* __restrict__ acc, int64_t ld, int64_t M,
                                                            int64_t N, const float* __restrict__ w_scale, float x_scale,
                                                            const float* __restrict__ bias, int conv, int64_t HoWo,
                                                            float* __restrict__ y)
{
    const int64_t total = M * N;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        int64_t m, n;
        if (conv) {   // i runs over NCHW: (b, n, pixel)
            int64_t pix = i % HoWo, bn = i / HoWo;
            n = bn % N;
            m = (bn / N) * HoWo + pix;
        } else {
            m = i / N;
            n = i - m * N;
        }
        float s = x_scale * __ldg(w_scale + n);
        y[i] = fmaf(acc[m * ld + n], s, bias ? __ldg(bias + n) : 0.f);
    }
}

int grid_for(int64_t total)
{
    int64_t blocks = (total + 255) / 256;
    return (int)(blocks < 1 ? 1 : (blocks > 148 * 16 ? 148 * 16 : blocks));
}

struct Plan {
    int64_t n_x, N4;
    size_t off_xv, off_rows, off_wv, off_acc, bytes;
};

Plan make_plan(const GeneralLayer& g)
{
    Plan p;
    p.n_x = g.conv ? (int64_t)g.B * g.C * g.H * g.W : g.M * g.K;
    p.N4 = round_up(g.N, 4);
    size_t o = 0;
    p.off_xv = o;
    o += (size_t)round_up(p.n_x * 4, 256);
    p.off_rows = o;
    if (g.conv)
        o += (size_t)round_up(g.M * g.K * 4, 256);
    p.off_wv = o;
    o += (size_t)round_up(g.N * g.K * 4, 256);
    p.off_acc = o;
    o += (size_t)round_up(g.M * p.N4 * 4, 256);
    p.bytes = o;
    return p;
}

}  // namespace

size_t general_layer_workspace_bytes(const GeneralLayer& g) { return make_plan(g).bytes; }

fpq_status launch_general_layer(const GeneralLayer& g, void* workspace, cudaStream_t st)
{
    Plan p = make_plan(g);
    char* ws = (char*)workspace;
    float* xv = (float*)(ws + p.off_xv);
    float* rows = (float*)(ws + p.off_rows);
    float* wv = (float*)(ws + p.off_wv);
    float* acc = (float*)(ws + p.off_acc);
    int* status = status_word();
    if (!status)
        return FPQ_ERR_CUDA;
    quantize_values_kernel<<<grid_for(p.n_x), 256, 0, st>>>(g.x, p.n_x, g.x_scale, g.fx, xv, status);
    decode_prepared_kernel<<<grid_for(g.N * g.K), 256, 0, st>>>((const uint8_t*)g.w_prepared, g.N, g.C, g.R * g.S, g.Cp,
                                                               g.fw, g.w_two_term, g.w_mul, wv);
    const float* a = xv;
    if (g.conv) {
        fpq_status s = launch_unfold(xv, g.B, g.C, g.H, g.W, g.R, g.S, g.pad, g.stride, g.Ho, g.Wo, rows, st);
        if (s != FPQ_OK)
            return s;
        a = rows;
    }
    // Grid values of formats of up to 8 bits have at most 8 significant bits: they are TF32 numbers, their products
    // are exact in FP32, and one tensor-core product per term computes what the FP32 multiply-add computes (the sums
    // differ in the order and rounding of the FP32 additions only).  Rows that are not a multiple of 4 floats stay
    // on the CUDA cores.  The tensor-core kernel's epilogue dequantizes and adds the bias itself.
    if (tf32x3_applies(a, g.K, wv, g.K, g.M, g.N, g.K) && g.M <= (1 << 21) && g.N <= (1 << 21) &&
        (int64_t)g.Ho * g.Wo < (1 << 30)) {
        const fpq_status s = launch_tf32x3(a, g.K, wv, g.K, g.M, g.N, g.K, (int)((g.K + 31) / 32), 2, g.y, g.N, 0, nullptr, st,
                                           1, g.w_scale, g.x_scale, g.bias, g.conv ? g.Ho * g.Wo : 0);
        if (s != FPQ_ERR_UNSUPPORTED)
            return s;
    }
    fpq_status s = launch_sgemm_nt(a, g.K, wv, g.K, acc, p.N4, g.M, g.N, g.K, st);
    if (s != FPQ_OK)
        return s;
    dequant_store_kernel<<<grid_for(g.M * g.N), 256, 0, st>>>(acc, p.N4, g.M, g.N, g.w_scale, g.x_scale, g.bias, g.conv,
                                                             (int64_t)g.Ho * g.Wo, g.y);
    return cudaGetLastError() == cudaSuccess ? FPQ_OK : FPQ_ERR_CUDA;
}

}  // namespace fpq
